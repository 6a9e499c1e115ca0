// Self-test of the bounded device waits (library plumbing; the paper has no counterpart).
//
// Every barrier wait in the kernels is bounded: a wait that runs out flags the per-device status
// word, the kernel returns, and mgn_attn_check reports MGN_ERR_DEVICE_TIMEOUT.  No input makes a
// product kernel take that path, so this one-CTA kernel takes it on purpose: it waits, with a short
// poll limit, on a barrier that nothing ever arrives on.  The wait gives up by construction --
// nothing spins unbounded, traps or faults -- and the context stays usable.  Not on any product
// path; a build without MGN_BUILD_SELFTEST leaves it out.
#ifdef MGN_BUILD_SELFTEST
#include "../../include/mgn_attn.h"
#include "kernels.h"
#include "ptx.cuh"

namespace mgn {
namespace {

constexpr uint32_t kSelftestPolls = 1u << 10;

__global__ void __launch_bounds__(32)
wait_timeout_kernel(unsigned* status, unsigned* polled)
{
    __shared__ __align__(8) uint64_t bar_storage;
    const uint32_t bar = smem_u32(&bar_storage);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);          // one arrival expected; none will come
        fence_mbar_init();
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        const bool ok = mbar_wait_polls(bar, 0, status, kSelftestPolls);
        if (polled) *polled = ok ? 0u : 1u;   // 1: the wait gave up, as it must
    }
}

}  // namespace
}  // namespace mgn

extern "C" int mgn_selftest_wait_timeout(unsigned* gave_up, void* stream)
{
    unsigned* status = nullptr;
    if (int r = mgn::device_status_word(&status)) return r;
    mgn::wait_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status, gave_up);
    return cudaGetLastError() == cudaSuccess ? MGN_OK : MGN_ERR_CUDA;
}
#endif  // MGN_BUILD_SELFTEST
