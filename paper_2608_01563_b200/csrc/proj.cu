// Output projection around attention, fast mode (bf16 operands, tcgen05 products, f32 accumulation).
//
// The paper gives its matrix-product kernels prologues and epilogues that absorb the steps around
// them (Section 3.3, kernel archetypes) and finds that dispatch structure matters where kernels are
// small (Section 7.3).  The step after attention is the projection of the concatenated heads,
//     Y[b,s,:] = sum_h O[b,h,s,:] W[h*D:(h+1)*D, :],
// and two fusions fall out of writing that product here instead of calling a library GEMM:
//   FWD  reads O where attention left it ([B,H,S,D], heads separate): the operand tiles are fetched by
//        TMA from the head-major tensor, so no transposed / concatenated copy of O is ever made;
//   DO   the backward product dO = dY W^T writes dO straight into the [B,H,S,D] layout the attention
//        backward reads, and its epilogue also emits delta = rowsum(dO o O) -- the attention
//        backward's preprocess pass -- while the dO tile is still in registers.
// One CTA computes a 128 x 256 output tile: rows are 128 positions s of one batch element, columns
// are 256 output features (FWD) or 256 (head, d) columns = 256 / D whole heads (DO).  Warp 0 streams
// 64-wide contraction slices of both operands through a four-stage TMA ring, one lane of warp 1
// issues the products into a 256-column tensor-memory accumulator, warps 2-5 (one thread per row)
// read it out.
#include <cuda_bf16.h>

#include "kernels.h"
#include "umma.cuh"

namespace mgn {
namespace {

constexpr int kThreads = 192;
constexpr int TM = 128, TN = 256, TK = 64, kStages = 4;
constexpr int A_BYTES = TM * TK * 2;          // 16 KB
constexpr int B_BYTES = TN * TK * 2;          // 32 KB
constexpr int OFF_A = 0, OFF_B = kStages * A_BYTES, OFF_BAR = OFF_B + kStages * B_BYTES;
constexpr int PAYLOAD = OFF_BAR + 128;
constexpr int SMEM = PAYLOAD + 1024;
enum { B_FULL = 0, B_EMPTY = kStages, B_ACC = 2 * kStages, B_COUNT = 2 * kStages + 1 };

// DO = false: Y = O_concat W       A = O  (rank-3 map D x S x B*H),  B = W as MN-major operand (rows = k)
// DO = true : dO = dY W^T, delta   A = dY (rank-3 map E x S x B),    B = W as K-major operand (rows = n)
template <bool DO>
__global__ void __launch_bounds__(kThreads, 1)
proj_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ O, float* __restrict__ delta,
            int H, int S, int D, int E, unsigned* status)
{
    extern __shared__ uint8_t smem_raw[];
    if (*reinterpret_cast<volatile unsigned*>(status) != 0) return;   // an earlier wait on this device gave up
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sA = base + OFF_A, sB = base + OFF_B, bars = base + OFF_BAR;
    const uint32_t tmem_slot = bars + B_COUNT * 8;
    auto bar = [&](int i) { return bars + 8u * i; };
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = static_cast<int>(blockIdx.x) * TN, s0 = static_cast<int>(blockIdx.y) * TM, b = static_cast<int>(blockIdx.z);
    const int K = DO ? E : H * D, N = DO ? H * D : E;
    const int n_kt = (K + TK - 1) / TK;

    if (tid == 0) {
        for (int i = 0; i < B_COUNT; ++i) mbar_init(bar(i), 1);
        fence_mbar_init();
    }
    __syncwarp();
    if (warp == 0) tmem_alloc(tmem_slot, TN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = lds32u(tmem_slot);

    if (warp == 0 && lane == 0) {
        // ---------------------------------------------------------------- TMA producer
        for (int kt = 0; kt < n_kt; ++kt) {
            const int st = kt % kStages, k0 = kt * TK;
            if (kt >= kStages) mbar_wait(bar(B_EMPTY + st), ((kt / kStages) - 1) & 1, status);
            mbar_arrive_expect_tx(bar(B_FULL + st), A_BYTES + B_BYTES);
            if constexpr (DO) {
                tma_load_3d(sA + st * A_BYTES, &tmA, bar(B_FULL + st), k0, s0, b);
                tma_load_3d(sB + st * B_BYTES, &tmB, bar(B_FULL + st), k0, n0, 0);          // 256 rows n x 64 k
            } else {
                tma_load_3d(sA + st * A_BYTES, &tmA, bar(B_FULL + st), k0 % D, s0, b * H + k0 / D);
#pragma unroll
                for (int c = 0; c < TN / 64; ++c)                                             // four blocks of 64 k rows x 64 n
                    tma_load_3d(sB + st * B_BYTES + c * (TK * 128), &tmB, bar(B_FULL + st), n0 + 64 * c, k0, 0);
            }
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------------------------------------------------------- MMA issuer
        constexpr uint32_t idesc = umma_idesc_bf16(TM, TN, false, !DO);
        const uint64_t dA = umma_smem_desc(sA, 16, 1024);
        const uint64_t dB = DO ? umma_smem_desc(sB, 16, 1024) : umma_smem_desc(sB, TK * 128, 1024);
        for (int kt = 0; kt < n_kt; ++kt) {
            const int st = kt % kStages;
            mbar_wait(bar(B_FULL + st), (kt / kStages) & 1, status);
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < TK / 16; ++kk) {
                const uint64_t a = dA + static_cast<uint64_t>((st * A_BYTES + kk * 32) >> 4);
                const uint64_t bb = dB + static_cast<uint64_t>((st * B_BYTES + (DO ? kk * 32 : kk * 2048)) >> 4);
                umma_ss(tmem, a, bb, idesc, (kt > 0 || kk > 0) ? 1u : 0u);
            }
            umma_commit(bar(B_EMPTY + st));
        }
        umma_commit(bar(B_ACC));
    } else if (warp >= 2) {
        // ---------------------------------------------------------------- epilogue: one thread per row
        const int q4 = warp & 3, r = 32 * q4 + lane, s = s0 + r;
        const uint32_t tacc = tmem + (static_cast<uint32_t>(32 * q4) << 16);
        mbar_wait(bar(B_ACC), 0, status);
        tc_fence_after();
        float dl = 0.f;
#pragma unroll 1
        for (int c = 0; c < TN / 32; ++c) {
            uint32_t v[32];
            tmem_ld32(tacc + 32 * c, v);          // whole warp, whatever the row
            tmem_ld_wait();
            const int n = n0 + 32 * c;
            if (s >= S || n >= N) continue;
            uint32_t u[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) u[e] = pack_bf16(__uint_as_float(v[2 * e]), __uint_as_float(v[2 * e + 1]));
            if constexpr (DO) {
                const int h = n / D, d = n % D;
                const size_t row = ((static_cast<size_t>(b) * H + h) * S + s) * D + d;
                const uint4* orow = reinterpret_cast<const uint4*>(O + row);
                uint4* drow = reinterpret_cast<uint4*>(out + row);
#pragma unroll
                for (int p4 = 0; p4 < 4; ++p4) {
                    drow[p4] = make_uint4(u[4 * p4], u[4 * p4 + 1], u[4 * p4 + 2], u[4 * p4 + 3]);
                    const uint4 ov = orow[p4];
                    const uint32_t ow[4] = {ov.x, ov.y, ov.z, ov.w};
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        // delta from the bf16 values the attention backward will read
                        const uint32_t dv = u[4 * p4 + t];
                        dl = fmaf(__uint_as_float(dv << 16), __uint_as_float(ow[t] << 16), dl);
                        dl = fmaf(__uint_as_float(dv & 0xffff0000u), __uint_as_float(ow[t] & 0xffff0000u), dl);
                    }
                }
                if (d + 32 == D) {                // last chunk of this head
                    delta[(static_cast<size_t>(b) * H + h) * S + s] = dl;
                    dl = 0.f;
                }
            } else {
                uint4* yrow = reinterpret_cast<uint4*>(out + (static_cast<size_t>(b) * S + s) * E + n);
                const int valid = (E - n) / 8;    // 16-byte pieces inside the row (E is a multiple of 8)
#pragma unroll
                for (int p4 = 0; p4 < 4; ++p4)
                    if (p4 < valid) yrow[p4] = make_uint4(u[4 * p4], u[4 * p4 + 1], u[4 * p4 + 2], u[4 * p4 + 3]);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TN);
}

template <bool DO>
cudaError_t launch(const CUtensorMap& ta, const CUtensorMap& tb, void* out, const void* o, float* delta, int B, int H,
                   int S, int D, int E, unsigned* status, cudaStream_t st)
{
    auto kern = proj_kernel<DO>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
    if (e != cudaSuccess) return e;
    const int N = DO ? H * D : E;
    const dim3 grid((N + TN - 1) / TN, (S + TM - 1) / TM, B);
    kern<<<grid, kThreads, SMEM, st>>>(ta, tb, static_cast<__nv_bfloat16*>(out), static_cast<const __nv_bfloat16*>(o),
                                       delta, H, S, D, E, status);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_out_proj_fwd(const void* o, const void* w, void* y, int B, int H, int S, int D, int E,
                                unsigned* status, cudaStream_t st)
{
    CUtensorMap ta, tb;
    if (make_tmap_3d(&ta, o, 2, 1, B * H, S, D, 64, TM)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tb, w, 2, 1, 1, H * D, E, 64, TK)) return cudaErrorInvalidValue;
    return launch<false>(ta, tb, y, nullptr, nullptr, B, H, S, D, E, status, st);
}

cudaError_t launch_out_proj_bwd_data(const void* d_y, const void* w, const void* o, void* d_o, float* delta, int B,
                                     int H, int S, int D, int E, unsigned* status, cudaStream_t st)
{
    CUtensorMap ta, tb;
    if (make_tmap_3d(&ta, d_y, 2, 1, B, S, E, 64, TM)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tb, w, 2, 1, 1, H * D, E, 64, TN)) return cudaErrorInvalidValue;
    return launch<true>(ta, tb, d_o, o, delta, B, H, S, D, E, status, st);
}

}  // namespace mgn
