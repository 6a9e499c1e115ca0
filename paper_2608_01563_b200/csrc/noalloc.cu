// mgn_attn_bwd_noalloc: attention backward for callers that cannot allocate device memory.
//
// The ordinary backward needs a caller-provided workspace (the per-row delta vector and, in
// fast mode, an f32 dQ accumulator).  Some callers have no way to provide one: code running
// where cudaMalloc is forbidden or would synchronise the device (inside a latency-critical
// serving loop, under a memory pool that owns the whole GPU, in a plug-in that is handed
// tensors but no allocator).  For them the workspace lives in a fixed array that is part of
// the library image itself: every GPU that loads the library reserves kNoAllocScratchBytes of
// its memory for it until the process exits.
#include <stdint.h>

#include <mutex>

#include "../../include/mgn_attn.h"

namespace {

constexpr size_t kNoAllocScratchBytes = MGN_NOALLOC_MAX_WORKSPACE_BYTES;

// Device scratch.  In host code this name is only a handle for cudaGetSymbolAddress: it is
// NOT a device address and must never be passed to a kernel or a memset directly.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices];   // device address of the array, per device, once resolved
std::mutex g_mu;

// Resolves the array's device address for the current device (first call per device only).
int scratch_for_current_device(void** out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MGN_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return MGN_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_scratch_ptr[dev] == nullptr) {
        void* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return MGN_ERR_CUDA;
        }
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return MGN_OK;
}

}  // namespace

extern "C" {

size_t mgn_attn_bwd_noalloc_max_workspace_bytes(void) { return kNoAllocScratchBytes; }

int mgn_attn_bwd_noalloc(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                         const float* lse, void* dq, void* dk, void* dv,
                         int B, int H, int S, int D, int causal, float scale, int mode, void* stream)
{
    // Size gate first: it needs no device and gives the caller a definite answer.
    const size_t need = mgn_attn_bwd_workspace_bytes(B, H, S, D, mode);
    if (need == 0) {
        // invalid or unsupported sizes: let the ordinary entry point name the exact error
        return mgn_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, reinterpret_cast<void*>(256), 0, B, H, S, D, causal,
                            scale, mode, stream);
    }
    if (need > kNoAllocScratchBytes) return MGN_ERR_WORKSPACE;
    void* scratch = nullptr;
    if (int r = scratch_for_current_device(&scratch)) return r;
    // Same kernels as mgn_attn_bwd, with the built-in array as their workspace.  Everything that
    // must start from zero (the dQ accumulation target) is cleared on `stream` by that path, and
    // delta is fully rewritten, so the previous call's leftovers in the array do not matter.
    return mgn_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, scratch, kNoAllocScratchBytes, B, H, S, D, causal, scale,
                        mode, stream);
}

}  // extern "C"
