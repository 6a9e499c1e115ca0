// Strict-mode dQ as a separate pass (paper Section 3.3 lists "dQ" beside the "fused dK+dV"
// kernel; Section 7.3 profiles them as FlashGradQ and FlashGradKV).  This is the deterministic
// variant of the backward: no floating-point atomics anywhere, so results are bit-identical from
// run to run.  It costs two more matrix products than the fused single pass (S and dP are
// recomputed here): 7 instead of 5.
//
// One CTA owns BM query rows of one head, keeps their Q and dO tiles resident, and streams the
// BN-key tiles of K and V.  Per key tile:
//   A. S = Q K^T and dP = dO V^T in one fused loop over d; P = exp(S - LSE), dS = P o (dP - delta)
//      in registers; dS to shared memory (row-major [i][j]),
//   C. dQ += dS K (contraction over the keys of the tile), accumulated in registers over all tiles.
// Thread layout, tile layout in shared memory and the two phases are those of strict_bwd.cu.
#include "kernels.h"
#include "strict_tiles.cuh"

namespace mgn {
namespace {

constexpr float kLog2e = 1.4426950408889634f;

template <int D, int BM, int BN, int THREADS>
struct DqCfg {
    static constexpr int TR = THREADS / 16;  // row groups
    static constexpr int RM = BM / TR;   // query rows per thread
    static constexpr int RN = BN / 16;   // key columns per thread (phase A)
    static constexpr int DV = D / 16;    // d columns per thread (phase C)
    static constexpr int NCH = D / 32;
    static constexpr int PSTR = BN + 4;
    static constexpr int KV_BYTES = BN * D * 4;
    static constexpr int Q_BYTES = BM * D * 4;
    static constexpr int P_BYTES = BM * PSTR * 4;
    static constexpr int SMEM = 2 * KV_BYTES + 2 * Q_BYTES + P_BYTES + 64 + 1024;
};


template <int D, int BM, int BN, int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS == 128 ? 2 : 1)
strict_dq_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmdO,
                 const float* __restrict__ LSE, const float* __restrict__ DELTA, float* __restrict__ dQ,
                 int Sq, int Sk, int BH, int H, int G, int n_qt, int causal, float scale, unsigned* status)
{
    using C = DqCfg<D, BM, BN, THREADS>;
    constexpr int RM = C::RM, RN = C::RN, DV = C::DV, NCH = C::NCH, PSTR = C::PSTR, TR = C::TR;

    extern __shared__ uint8_t smem_raw[];
    if (*reinterpret_cast<volatile unsigned*>(status) != 0) return;   // an earlier wait on this device gave up
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = base;
    const uint32_t sdO = sQ + C::Q_BYTES;
    const uint32_t sK = sdO + C::Q_BYTES;
    const uint32_t sV = sK + C::KV_BYTES;
    const uint32_t sdS = sV + C::KV_BYTES;
    const uint32_t barQ = sdS + C::P_BYTES, barK = barQ + 8, barV = barQ + 16;

    const int tid = threadIdx.x;
    const int tr = 2 * (tid >> 5) + ((tid & 31) >> 4);   // 0..TR-1: row group
    const int tc = tid & 15;                             // 0..15: column group

    // Heaviest (last) query tiles first when causal.
    const int qt = n_qt - 1 - static_cast<int>(blockIdx.x) / BH;
    const int bh = static_cast<int>(blockIdx.x) % BH;
    const int bhk = (bh / H) * (H / G) + (bh % H) / G;   // key/value head of this query head
    const int coff = Sk - Sq;                            // causal: key j visible to query i iff j <= i + coff
    const int i0 = qt * BM;
    const int i_last = min(i0 + BM, Sq) - 1;
    const int n_kt = causal ? ((i_last + coff) / BN + 1) : ((Sk + BN - 1) / BN);
    const float c2 = scale * kLog2e;

    if (tid == 0) {
        mbar_init(barQ, 1);
        mbar_init(barK, 1);
        mbar_init(barV, 1);
        fence_mbar_init();
    }
    __syncthreads();
    if (tid == 0) {
        mbar_arrive_expect_tx(barQ, 2 * C::Q_BYTES);
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) {
            tma_load_3d(sQ + ch * BM * 128, &tmQ, barQ, ch * 32, i0, bh);
            tma_load_3d(sdO + ch * BM * 128, &tmdO, barQ, ch * 32, i0, bh);
        }
        mbar_arrive_expect_tx(barK, C::KV_BYTES);
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) tma_load_3d(sK + ch * BN * 128, &tmK, barK, ch * 32, 0, bhk);
        mbar_arrive_expect_tx(barV, C::KV_BYTES);
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) tma_load_3d(sV + ch * BN * 128, &tmV, barV, ch * 32, 0, bhk);
    }

    // row statistics of this thread's query rows (rows past Sq: P = 0 via lse = +inf)
    float lse2[RM], dl[RM];
#pragma unroll
    for (int x = 0; x < RM; ++x) {
        const int i = i0 + tr + TR * x;
        const bool ok = i < Sq;
        lse2[x] = ok ? LSE[static_cast<size_t>(bh) * Sq + i] * kLog2e : INFINITY;
        dl[x] = ok ? DELTA[static_cast<size_t>(bh) * Sq + i] : 0.f;
    }

    float dq[RM][DV];
#pragma unroll
    for (int x = 0; x < RM; ++x)
#pragma unroll
        for (int e = 0; e < DV; ++e) dq[x][e] = 0.f;

    mbar_wait(barQ, 0, status);

    for (int kt = 0; kt < n_kt; ++kt) {
        const uint32_t ph = kt & 1;
        const int j0 = kt * BN;
        mbar_wait(barK, ph, status);
        mbar_wait(barV, ph, status);

        // ---- A: S = Q K^T and dP = dO V^T, fused over d ---------------------------------------
        float s[RM][RN], dp[RM][RN];
#pragma unroll
        for (int x = 0; x < RM; ++x)
#pragma unroll
            for (int y = 0; y < RN; ++y) { s[x][y] = 0.f; dp[x][y] = 0.f; }
        {
            const int xq = tr & 7, xk = tc & 7;
#pragma unroll
            for (int pc = 0; pc < D / 4; ++pc) {
                const uint32_t oq = (pc >> 3) * (BM * 128) + tr * 128 + (((pc & 7) ^ xq) << 4);
                const uint32_t ok = (pc >> 3) * (BN * 128) + tc * 128 + (((pc & 7) ^ xk) << 4);
                float4 bk[RN], bv[RN];
#pragma unroll
                for (int y = 0; y < RN; ++y) {
                    bk[y] = lds128(sK + ok + y * 16 * 128);
                    bv[y] = lds128(sV + ok + y * 16 * 128);
                }
#pragma unroll
                for (int x = 0; x < RM; ++x) {
                    const float4 aq = lds128(sQ + oq + x * TR * 128);
                    const float4 ad = lds128(sdO + oq + x * TR * 128);
#pragma unroll
                    for (int y = 0; y < RN; ++y) {
                        s[x][y] = fmaf(aq.x, bk[y].x, s[x][y]);
                        s[x][y] = fmaf(aq.y, bk[y].y, s[x][y]);
                        s[x][y] = fmaf(aq.z, bk[y].z, s[x][y]);
                        s[x][y] = fmaf(aq.w, bk[y].w, s[x][y]);
                        dp[x][y] = fmaf(ad.x, bv[y].x, dp[x][y]);
                        dp[x][y] = fmaf(ad.y, bv[y].y, dp[x][y]);
                        dp[x][y] = fmaf(ad.z, bv[y].z, dp[x][y]);
                        dp[x][y] = fmaf(ad.w, bv[y].w, dp[x][y]);
                    }
                }
            }
        }
        __syncthreads();   // every warp is done with this V tile
        if (tid == 0 && kt + 1 < n_kt) {
            mbar_arrive_expect_tx(barV, C::KV_BYTES);
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) tma_load_3d(sV + ch * BN * 128, &tmV, barV, ch * 32, j0 + BN, bhk);
        }
        {
            const bool need_mask = (causal && (j0 + BN - 1 > i0 + coff)) || (j0 + BN > Sk);
#pragma unroll
            for (int x = 0; x < RM; ++x) {
                const int i = i0 + tr + TR * x;
                const uint32_t row = ((tr + TR * x) * PSTR + tc) * 4;
#pragma unroll
                for (int y = 0; y < RN; ++y) {
                    float p = ex2(fmaf(s[x][y], c2, -lse2[x]));
                    if (need_mask) {
                        const int j = j0 + tc + 16 * y;
                        if (j >= Sk || (causal && j > i + coff)) p = 0.f;
                    }
                    sts32(sdS + row + y * 64, p * (dp[x][y] - dl[x]));
                }
            }
        }
        __syncthreads();   // dS visible

        // ---- C: dQ += dS K : contraction over the keys of this tile ------------------------
#pragma unroll 2
        for (int j8 = 0; j8 < BN / 8; ++j8) {
            float4 d4[2][RM];
#pragma unroll
            for (int hlf = 0; hlf < 2; ++hlf)
#pragma unroll
                for (int x = 0; x < RM; ++x)
                    d4[hlf][x] = lds128(sdS + ((tr + TR * x) * PSTR + j8 * 8 + hlf * 4) * 4);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                float kv[DV];
                load_row_cols<D, BN>(sK, j8 * 8 + u, u, tc, kv);
#pragma unroll
                for (int x = 0; x < RM; ++x) {
                    const float dsv = f4_get(d4[u >> 2][x], u & 3);
#pragma unroll
                    for (int e = 0; e < DV; ++e) dq[x][e] = fmaf(dsv, kv[e], dq[x][e]);
                }
            }
        }
        __syncthreads();   // every warp is done with this K tile and with dS
        if (tid == 0 && kt + 1 < n_kt) {
            mbar_arrive_expect_tx(barK, C::KV_BYTES);
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) tma_load_3d(sK + ch * BN * 128, &tmK, barK, ch * 32, j0 + BN, bhk);
        }
    }

    // ---- epilogue: dQ = scale * accumulated rows, plain stores ---------------------------------
#pragma unroll
    for (int x = 0; x < RM; ++x) {
        const int i = i0 + tr + TR * x;
        if (i < Sq) {
            float* row = dQ + (static_cast<size_t>(bh) * Sq + i) * D;
            if constexpr (DV == 2) {
                *reinterpret_cast<float2*>(row + 2 * tc) = make_float2(dq[x][0] * scale, dq[x][1] * scale);
            } else {
#pragma unroll
                for (int e = 0; e < DV / 4; ++e)
                    *reinterpret_cast<float4*>(row + 4 * tc + 64 * e) =
                        make_float4(dq[x][4 * e] * scale, dq[x][4 * e + 1] * scale, dq[x][4 * e + 2] * scale,
                                    dq[x][4 * e + 3] * scale);
            }
        }
    }
}

template <int D, int BM, int BN, int THREADS>
cudaError_t launch(const Problem& p, const float* q, const float* k, const float* v, const float* d_o,
                   const float* lse, const float* delta, float* dq, unsigned* status, cudaStream_t st)
{
    using C = DqCfg<D, BM, BN, THREADS>;
    CUtensorMap tq, tk, tv, tdo;
    if (make_tmap_3d(&tq, q, 4, 0, p.BH(), p.Sq, D, 32, BM)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tdo, d_o, 4, 0, p.BH(), p.Sq, D, 32, BM)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tk, k, 4, 0, p.BHkv(), p.Sk, D, 32, BN)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tv, v, 4, 0, p.BHkv(), p.Sk, D, 32, BN)) return cudaErrorInvalidValue;
    auto kern = strict_dq_kernel<D, BM, BN, THREADS>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
    if (e != cudaSuccess) return e;
    const int n_qt = (p.Sq + BM - 1) / BM;
    const long long blocks = static_cast<long long>(n_qt) * p.BH();
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    kern<<<static_cast<unsigned>(blocks), THREADS, C::SMEM, st>>>(tq, tk, tv, tdo, lse, delta, dq, p.Sq, p.Sk, p.BH(),
                                                                   p.H, p.group(), n_qt, p.causal, p.scale, status);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_strict_dq(const Problem& p, const float* q, const float* k, const float* v, const float* d_o,
                             const float* lse, const float* delta, float* dq, unsigned* status, cudaStream_t st)
{
    switch (p.D) {
        case 32:  return launch<32, 64, 64, 128>(p, q, k, v, d_o, lse, delta, dq, status, st);
        case 64:  return launch<64, 64, 64, 128>(p, q, k, v, d_o, lse, delta, dq, status, st);
        case 128: return launch<128, 64, 64, 256>(p, q, k, v, d_o, lse, delta, dq, status, st);
        default:  return cudaErrorInvalidValue;
    }
}

}  // namespace mgn
