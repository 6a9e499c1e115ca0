// Fast-mode dQ as a separate pass: bf16 storage, tcgen05 tensor-core products with f32 accumulation
// in tensor memory (paper Section 3.3 lists "dQ" beside the "fused dK+dV" kernel; Section 7.3
// profiles them as FlashGradQ and FlashGradKV).  Part of the deterministic backward: no
// floating-point atomics, so results are bit-identical from run to run; S and dP are recomputed
// here, which makes seven matrix products per tile pair instead of the fused kernel's five.
//
// One CTA owns one 128-row query tile of one head, keeps its Q and dO tiles in shared memory and
// streams the 128-key blocks of K and V through a two-stage ring.  Per key block:
//   MMA  S  = Q K^T   -> tensor memory S        MMA  dP = dO V^T -> tensor memory P
//   compute (256 threads, two per query row, 64 key columns each):
//        P = exp2(S c - LSE), dS = P (dP - delta) -> bf16, written over S (the A operand of the next product)
//   MMA  dQ += dS K   (A from tensor memory, K as the MN-major shared-memory operand)
// The products of one block and the arithmetic of that block alternate (one buffer each for S and
// dP): this pass favours simplicity over overlap.  Epilogue: dQ * scale -> bf16 -> shared memory
// (the dead Q tile) -> TMA store.
// Warp roles (384 threads): warp 0 TMA producer, warp 1 MMA issuer, warps 4-11 compute.
#include <cuda_bf16.h>

#include "kernels.h"
#include "fast_items.cuh"
#include "umma.cuh"

namespace mgn {
namespace {

constexpr int kThreads = 384;
constexpr int BLK = 128;
constexpr float kLog2e = 1.4426950408889634f;

template <int D>
struct Cfg {
    static constexpr int NCH = D / 64;
    static constexpr int TILE_BYTES = BLK * D * 2;
    static constexpr int CHUNK_BYTES = BLK * 128;
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_DO = OFF_Q + TILE_BYTES;
    static constexpr int OFF_K = OFF_DO + TILE_BYTES;          // two stages
    static constexpr int OFF_V = OFF_K + 2 * TILE_BYTES;       // two stages
    static constexpr int OFF_BAR = OFF_V + 2 * TILE_BYTES;
    static constexpr int SMEM = OFF_BAR + 256 + 1024;
    static_assert(SMEM <= 232448, "shared memory budget");
    static constexpr uint32_t TM_S = 0, TM_P = 128, TM_DQ = 256, TM_COLS = 512;
};

enum { B_Q = 0, B_KFULL = 1, B_KEMPTY = 3, B_VFULL = 5, B_VEMPTY = 7, B_SPFULL = 9, B_DSFULL = 10, B_DQFULL = 11,
       B_COUNT = 12 };


template <int D>
__global__ void __launch_bounds__(kThreads, 1)
fast_dq_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmdO,
               const __grid_constant__ CUtensorMap tmdQ,
               const float* __restrict__ LSE, const float* __restrict__ DELTA,
               const Dims dm, int n_qt, int causal, float scale, unsigned* status)
{
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = base + C::OFF_Q, sdO = base + C::OFF_DO, sK = base + C::OFF_K, sV = base + C::OFF_V;
    const uint32_t bars = base + C::OFF_BAR;
    const uint32_t tmem_slot = bars + B_COUNT * 8;
    auto bar = [&](int i) { return bars + 8u * i; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (*reinterpret_cast<volatile unsigned*>(status) != 0) return;   // an earlier wait on this device gave up

    // Heaviest (last) query tiles first when causal.
    const int qt = n_qt - 1 - static_cast<int>(blockIdx.x) / dm.BH;
    const int bh = static_cast<int>(blockIdx.x) % dm.BH;
    const int bhk = (bh / dm.H) * (dm.H / dm.G) + (bh % dm.H) / dm.G;   // key/value head of this query head
    const int i0 = qt * BLK;
    const int n_kb_all = (dm.Sk + BLK - 1) / BLK;
    const int n_kb = causal ? min(n_kb_all, (min(i0 + BLK, dm.Sq) - 1 + dm.off) / BLK + 1) : n_kb_all;
    const float c2 = scale * kLog2e;

    if (tid == 0) {
        for (int i = 0; i < B_COUNT; ++i) mbar_init(bar(i), i == B_DSFULL ? 256u : 1u);
        fence_mbar_init();
    }
    __syncwarp();
    if (warp == 0) tmem_alloc(tmem_slot, C::TM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = lds32u(tmem_slot);

    if (warp < 4) {
        reg_dealloc<96>();
        if (warp == 0 && lane == 0) {
            // ------------------------------------------------------------------ TMA producer
            mbar_arrive_expect_tx(bar(B_Q), 2 * C::TILE_BYTES);
#pragma unroll
            for (int ch = 0; ch < C::NCH; ++ch) {
                tma_load_3d(sQ + ch * C::CHUNK_BYTES, &tmQ, bar(B_Q), ch * 64, i0, bh);
                tma_load_3d(sdO + ch * C::CHUNK_BYTES, &tmdO, bar(B_Q), ch * 64, i0, bh);
            }
            for (int n = 0; n < n_kb; ++n) {
                const int st = n & 1;
                const uint32_t ph = (n >> 1) & 1;
                mbar_wait(bar(B_KEMPTY + st), ph ^ 1, status);
                mbar_arrive_expect_tx(bar(B_KFULL + st), C::TILE_BYTES);
#pragma unroll
                for (int ch = 0; ch < C::NCH; ++ch)
                    tma_load_3d(sK + st * C::TILE_BYTES + ch * C::CHUNK_BYTES, &tmK, bar(B_KFULL + st), ch * 64, n * BLK, bhk);
                mbar_wait(bar(B_VEMPTY + st), ph ^ 1, status);
                mbar_arrive_expect_tx(bar(B_VFULL + st), C::TILE_BYTES);
#pragma unroll
                for (int ch = 0; ch < C::NCH; ++ch)
                    tma_load_3d(sV + st * C::TILE_BYTES + ch * C::CHUNK_BYTES, &tmV, bar(B_VFULL + st), ch * 64, n * BLK, bhk);
            }
        } else if (warp == 1 && lane == 0) {
            // ------------------------------------------------------------------ MMA issuer
            constexpr uint32_t idesc_s = umma_idesc_bf16(BLK, BLK, false, false);    // S, dP: both operands K-major
            constexpr uint32_t idesc_q = umma_idesc_bf16(BLK, D, false, true);       // dQ: A from tensor memory, B MN-major
            const uint64_t dQd = umma_smem_desc(sQ, 16, 1024), dOd = umma_smem_desc(sdO, 16, 1024);
            const uint64_t dK0 = umma_smem_desc(sK, 16, 1024), dV0 = umma_smem_desc(sV, 16, 1024);
            const uint64_t mK0 = umma_smem_desc(sK, C::CHUNK_BYTES, 1024);
            const uint32_t tS = tmem + C::TM_S, tP = tmem + C::TM_P, tDQ = tmem + C::TM_DQ;
            auto koff = [](int kk) { return static_cast<uint64_t>(((kk >> 2) * C::CHUNK_BYTES + (kk & 3) * 32) >> 4); };
            mbar_wait(bar(B_Q), 0, status);
            for (int n = 0; n < n_kb; ++n) {
                const int st = n & 1;
                const uint32_t ph = (n >> 1) & 1;
                const uint64_t stoff = static_cast<uint64_t>((st * C::TILE_BYTES) >> 4);
                // S(n): its region held dS(n-1), read by the dQ product issued just before (same thread: in order)
                mbar_wait(bar(B_KFULL + st), ph, status);
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) umma_ss(tS, dQd + koff(kk), dK0 + stoff + koff(kk), idesc_s, kk > 0);
                // dP(n): the compute warps finished reading dP(n-1) before they signalled dS(n-1)
                mbar_wait(bar(B_VFULL + st), ph, status);
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) umma_ss(tP, dOd + koff(kk), dV0 + stoff + koff(kk), idesc_s, kk > 0);
                umma_commit(bar(B_SPFULL));
                umma_commit(bar(B_VEMPTY + st));
                // dQ += dS(n) K(n)
                mbar_wait(bar(B_DSFULL), n & 1, status);
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < BLK / 16; ++kk)
                    umma_ts(tDQ, tS + (kk >> 2) * 64 + (kk & 3) * 8, mK0 + stoff + static_cast<uint64_t>((kk * 2048) >> 4),
                            idesc_q, (kk > 0 || n > 0) ? 1u : 0u);
                umma_commit(bar(B_KEMPTY + st));
            }
            umma_commit(bar(B_DQFULL));
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ compute warps
        reg_alloc<200>();
        const int h = (warp - 4) >> 2;                     // which 64 key columns of every block
        const int r = (tid - 128) & 127;                   // row within the tile = tensor-memory lane
        const uint32_t lane_base = static_cast<uint32_t>(r & ~31) << 16;
        const uint32_t tS = tmem + lane_base + C::TM_S + 64 * h, tP = tmem + lane_base + C::TM_P + 64 * h;
        const int i = i0 + r;
        const bool row_ok = i < dm.Sq;
        const float lse2 = row_ok ? LSE[static_cast<size_t>(bh) * dm.Sq + i] * kLog2e : INFINITY;   // P = 0 past the end
        const float dl = row_ok ? DELTA[static_cast<size_t>(bh) * dm.Sq + i] : 0.f;

        for (int n = 0; n < n_kb; ++n) {
            const int j0 = n * BLK + 64 * h;
            const bool masked = causal && (j0 + 63 > i0 + dm.off);
            const int jmax = i + dm.off - j0;              // causal: columns c <= jmax of this half are visible
            mbar_wait(bar(B_SPFULL), n & 1, status);
            tc_fence_after();
            uint32_t pk[32];
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t s[32], dp[32];
                tmem_ld32(tS + 32 * c, s);
                tmem_ld32(tP + 32 * c, dp);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    float p0 = ex2(fmaf(__uint_as_float(s[e]), c2, -lse2));
                    float p1 = ex2(fmaf(__uint_as_float(s[e + 1]), c2, -lse2));
                    if (masked) {
                        if (32 * c + e > jmax) p0 = 0.f;
                        if (32 * c + e + 1 > jmax) p1 = 0.f;
                    }
                    pk[16 * c + e / 2] = pack_bf16(p0 * (__uint_as_float(dp[e]) - dl), p1 * (__uint_as_float(dp[e + 1]) - dl));
                }
            }
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t u[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) u[e] = pk[16 * c + e];
                tmem_st16(tS + 16 * c, u);                 // dS of this half: packed columns [64h, 64h + 32)
            }
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(bar(B_DSFULL));
        }

        // ---- epilogue: dQ * scale -> bf16 -> shared memory (the Q tile is dead) -> TMA store
        mbar_wait(bar(B_DQFULL), 0, status);
        tc_fence_after();
        {
            const uint32_t tDQ = tmem + lane_base + C::TM_DQ + (D / 2) * h;
#pragma unroll
            for (int c = 0; c < D / 64; ++c) {
                uint32_t v[32];
                tmem_ld32(tDQ + 32 * c, v);
                tmem_ld_wait();
                uint32_t u[16];
#pragma unroll
                for (int e = 0; e < 16; ++e)
                    u[e] = pack_bf16(__uint_as_float(v[2 * e]) * scale, __uint_as_float(v[2 * e + 1]) * scale);
                const int col = (D / 2) * h + 32 * c;      // first output column of this chunk
                const uint32_t rowaddr = sQ + (col >> 6) * C::CHUNK_BYTES + r * 128;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int piece = ((col & 63) >> 3) + q;
                    sts128(rowaddr + ((piece ^ (r & 7)) << 4), u[4 * q], u[4 * q + 1], u[4 * q + 2], u[4 * q + 3]);
                }
            }
            fence_proxy_async_smem();
            named_bar_sync(1, 256);
            if (r == 0 && h == 0) {
#pragma unroll
                for (int ch = 0; ch < C::NCH; ++ch) tma_store_3d(&tmdQ, sQ + ch * C::CHUNK_BYTES, ch * 64, i0, bh);
                tma_store_commit_and_wait_read();
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, C::TM_COLS);
}

template <int D>
cudaError_t launch(const Problem& p, const void* q, const void* k, const void* v, const void* d_o,
                   const float* lse, const float* delta, void* dq, unsigned* status, cudaStream_t st)
{
    using C = Cfg<D>;
    CUtensorMap tq, tk, tv, tdo, tdq;
    if (make_tmap_3d(&tq, q, 2, 1, p.BH(), p.Sq, p.D, 64, BLK)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tdo, d_o, 2, 1, p.BH(), p.Sq, p.D, 64, BLK)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tk, k, 2, 1, p.BHkv(), p.Sk, p.D, 64, BLK)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tv, v, 2, 1, p.BHkv(), p.Sk, p.D, 64, BLK)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tdq, dq, 2, 1, p.BH(), p.Sq, p.D, 64, BLK)) return cudaErrorInvalidValue;
    auto kern = fast_dq_kernel<D>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
    if (e != cudaSuccess) return e;
    const int n_qt = (p.Sq + BLK - 1) / BLK;
    const long long blocks = static_cast<long long>(n_qt) * p.BH();
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    const Dims dm{p.Sq, p.Sk, p.BH(), p.H, p.group(), p.off()};
    kern<<<static_cast<unsigned>(blocks), kThreads, C::SMEM, st>>>(tq, tk, tv, tdo, tdq, lse, delta, dm, n_qt, p.causal,
                                                                   p.scale, status);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fast_dq(const Problem& p, const void* q, const void* k, const void* v, const void* d_o,
                           const float* lse, const float* delta, void* dq, unsigned* status, cudaStream_t st)
{
    switch (p.D) {
        case 32:  // the 64-wide build on zero-filled 32-element rows (see fast_fwd.cu)
        case 64:  return launch<64>(p, q, k, v, d_o, lse, delta, dq, status, st);
        case 128: return launch<128>(p, q, k, v, d_o, lse, delta, dq, status, st);
        default:  return cudaErrorNotSupported;
    }
}

}  // namespace mgn
