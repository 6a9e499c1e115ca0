// Strict-mode attention backward: f32 storage, f32 FFMA arithmetic (paper Section 3.3,
// "dQ, and fused dK+dV kernels"; Section 7.3 names them FlashGradQ and FlashGradKV).
//
// Single pass: one CTA (256 threads) keeps one BN-key tile of K and V resident, holds
// the dK and dV accumulators of that tile in registers, and walks over the BM-row query
// tiles.  For each (query tile, key tile) pair it
//   A. recomputes S = Q K^T and computes dP = dO V^T in one fused loop over d,
//      forms P = exp(S - LSE) and dS = P o (dP - delta) in registers, and writes P and dS
//      to shared memory (row-major [i][j]),
//   B. accumulates dV += P^T dO and dK += dS^T Q (contraction over query rows),
//   C. forms the partial dQ = dS K of this pair and adds it to global dQ with 128-bit
//      floating-point reductions (the "atomic accumulation" variant of the dQ kernel),
// so exactly the five counted matrix products are executed.  Tiles arrive by TMA in the
// swizzled layout described in strict_fwd.cu.  With grouped key/value heads the CTA walks over the
// query tiles of every query head of its group in turn (dK, dV sum over the group in registers);
// with separate query and key lengths the causal mask is aligned bottom-right.
#include "kernels.h"
#include "strict_tiles.cuh"

namespace mgn {
namespace {

constexpr float kLog2e = 1.4426950408889634f;

// THREADS/16 row groups x 16 column groups; 128-thread CTAs run two per SM so that one CTA's
// FFMA loops cover the other's barriers and exponentials.
template <int D, int BM, int BN, int THREADS>
struct BwdCfg {
    static constexpr int TR = THREADS / 16;  // row groups
    static constexpr int RM = BM / TR;   // query rows per thread (phases A, C)
    static constexpr int RN = BN / 16;   // key columns per thread (phase A)
    static constexpr int JN = BN / TR;   // key rows per thread (phase B), groups of 4 contiguous
    static constexpr int DV = D / 16;    // d columns per thread (phases B, C)
    static constexpr int NCH = D / 32;
    static constexpr int PSTR = (D == 128 && THREADS == 128) ? BN : BN + 4;   // no room for the pad beside 128-wide tiles with two CTAs per SM
    static constexpr int KV_BYTES = BN * D * 4;
    static constexpr int Q_BYTES = BM * D * 4;
    static constexpr int P_BYTES = BM * PSTR * 4;
    static constexpr int PAYLOAD = 2 * KV_BYTES + 2 * Q_BYTES + 2 * P_BYTES + 64;
    // Two 128-thread CTAs per SM must fit 2 x (SMEM + 1 KB reserved) into 228 KB; where that leaves less than
    // the 1023 bytes a worst-case alignment of the tile base could need, the kernel checks the slack it got.
    static constexpr int SLACK = (THREADS == 128 && PAYLOAD + 1024 > 115712) ? 115712 - PAYLOAD : 1024;
    static constexpr int SMEM = PAYLOAD + SLACK;
    static_assert(SLACK >= 0, "shared memory budget");
    static_assert(JN % 4 == 0, "key rows per thread come in float4 groups");
};


// GEN = false is the square multi-head case (Sk == Sq, one key/value head per query head): the
// offset, the group loop and the second length fold away at compile time.
// WITH_DQ = false leaves phase C (the dQ partial and its floating-point reductions) out: the fused
// dK+dV kernel of the deterministic backward, whose dQ comes from the separate pass in strict_dq.cu.
template <int D, int BM, int BN, int THREADS, bool GEN, bool WITH_DQ>
__global__ void __launch_bounds__(THREADS, THREADS == 128 ? 2 : 1)
strict_bwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmdO,
                  const float* __restrict__ LSE, const float* __restrict__ DELTA,
                  float* __restrict__ dQ, float* __restrict__ dK, float* __restrict__ dV,
                  int Sq, int Sk_, int BHkv, int H, int G_, int n_qt, int causal, float scale, unsigned* status)
{
    const int Sk = GEN ? Sk_ : Sq;
    const int G = GEN ? G_ : 1;
    using C = BwdCfg<D, BM, BN, THREADS>;
    constexpr int RM = C::RM, RN = C::RN, JN = C::JN, DV = C::DV, NCH = C::NCH, PSTR = C::PSTR, TR = C::TR;

    extern __shared__ uint8_t smem_raw[];
    if (*reinterpret_cast<volatile unsigned*>(status) != 0) return;   // an earlier wait on this device gave up
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sK = base;
    const uint32_t sV = sK + C::KV_BYTES;
    const uint32_t sQ = sV + C::KV_BYTES;
    const uint32_t sdO = sQ + C::Q_BYTES;
    const uint32_t sP = sdO + C::Q_BYTES;
    const uint32_t sdS = sP + C::P_BYTES;
    const uint32_t barKV = sdS + C::P_BYTES, barQ = barKV + 8;
    if (base + C::PAYLOAD > smem_u32(smem_raw) + C::SMEM) {      // alignment slack ran out
        if (threadIdx.x == 0) atomicMax(status, kStatusSmemLayout);
        return;
    }

    const int tid = threadIdx.x;
    const int tr = 2 * (tid >> 5) + ((tid & 31) >> 4);   // 0..15
    const int tc = tid & 15;                             // 0..15

    // Heaviest key tiles (lowest j0) first when causal.
    const int kt = static_cast<int>(blockIdx.x) / BHkv;
    const int bhk = static_cast<int>(blockIdx.x) % BHkv;          // (batch, key/value head)
    const int Hkv = H / G;
    const int bhq0 = GEN ? (bhk / Hkv) * H + (bhk % Hkv) * G : bhk;   // first query head of the group
    const int coff = GEN ? Sk - Sq : 0;                           // causal: key j visible to query i iff j <= i + coff
    const int j0 = kt * BN;
    const int qt0 = causal ? (max(j0 - coff, 0) / BM) : 0;         // first query tile that sees this key tile
    const int nq = n_qt - qt0;                                    // query tiles per head (>= 1)
    const int steps = G * nq;                                     // (query head of the group, query tile) pairs
    const float c2 = scale * kLog2e;

    if (tid == 0) {
        mbar_init(barKV, 1);
        mbar_init(barQ, 1);
        fence_mbar_init();
    }
    __syncthreads();
    if (tid == 0) {
        mbar_arrive_expect_tx(barKV, 2 * C::KV_BYTES);
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) {
            tma_load_3d(sK + ch * BN * 128, &tmK, barKV, ch * 32, j0, bhk);
            tma_load_3d(sV + ch * BN * 128, &tmV, barKV, ch * 32, j0, bhk);
        }
        mbar_arrive_expect_tx(barQ, 2 * C::Q_BYTES);
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) {
            tma_load_3d(sQ + ch * BM * 128, &tmQ, barQ, ch * 32, qt0 * BM, bhq0);
            tma_load_3d(sdO + ch * BM * 128, &tmdO, barQ, ch * 32, qt0 * BM, bhq0);
        }
    }

    // dK, dV accumulators as packed pairs of adjacent key rows: [a][e] = {key 2a, key 2a+1} of column e
    uint64_t dk[JN / 2][DV], dv[JN / 2][DV];
#pragma unroll
    for (int a = 0; a < JN / 2; ++a)
#pragma unroll
        for (int e = 0; e < DV; ++e) { dk[a][e] = f2_pack(0.f, 0.f); dv[a][e] = f2_pack(0.f, 0.f); }

    mbar_wait(barKV, 0, status);

    // Step counter: the general case counts (head, tile) pairs from 0; the square case counts
    // query tiles from qt0 as the loop always did (the two forms compile to different schedules).
    for (int t = GEN ? 0 : qt0; t < (GEN ? steps : n_qt); ++t) {
        const int bh = GEN ? bhq0 + t / nq : bhq0;    // query head
        const int i0 = (GEN ? qt0 + t % nq : t) * BM;
        const uint32_t ph = (GEN ? t : t - qt0) & 1;

        // row statistics of this thread's query rows (rows past S: P = 0 via lse = +inf)
        float lse2[RM], dl[RM];
#pragma unroll
        for (int x = 0; x < RM; ++x) {
            const int i = i0 + tr + TR * x;
            const bool ok = i < Sq;
            lse2[x] = ok ? LSE[static_cast<size_t>(bh) * Sq + i] * kLog2e : INFINITY;
            dl[x] = ok ? DELTA[static_cast<size_t>(bh) * Sq + i] : 0.f;
        }

        mbar_wait(barQ, ph, status);

        // ---- A: S = Q K^T and dP = dO V^T, fused over d ---------------------------------------
        float s[RM][RN], dp[RM][RN];
#pragma unroll
        for (int x = 0; x < RM; ++x)
#pragma unroll
            for (int y = 0; y < RN; ++y) { s[x][y] = 0.f; dp[x][y] = 0.f; }
        {
            const int xq = tr & 7, xk = tc & 7;
            // Unroll factors are set by the instruction cache: with the packed FMAs of phase B the top
            // stall of this kernel became instruction fetch (0.94 stalled warps per issue), and a fully
            // unrolled phase A alone is 70 KB of code.  Measured at D = 64 with 64-row tiles: 16 / 8 / 4 / 2 / 1
            // steps per iteration -> 0.808 / 0.760 / 0.731 / 0.724 / 0.723 ms on the GPT-2-small shape; at
            // D = 128 (one 256-thread CTA per SM, 64-row tiles) four steps were best (2.13 against 2.16 ms unrolled,
            // 2.23 with two); the 5-row micro-tile of the 40-row tiles prefers eight (0.300 against 0.310 ms with
            // two).  D = 128 now runs two 128-thread CTAs per SM with 32-row query tiles (1.94 ms; 1.92 with
            // eight steps here, one row group in phase B and two key groups in phase C per iteration).
            constexpr int kUnrollA = (D == 128) ? (GEN ? 4 : 8) : (RM == 5) ? 8 : 2;   // (the general-shape build at D = 128 spills one register with eight)
#pragma unroll kUnrollA
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
        __syncthreads();   // phase C of the previous pair has finished reading dS
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
                    const float ds = p * (dp[x][y] - dl[x]);
                    sts32(sP + row + y * 64, p);
                    sts32(sdS + row + y * 64, ds);
                }
            }
        }
        __syncthreads();   // P, dS visible

        // ---- B: dV += P^T dO, dK += dS^T Q : contraction over the query rows ---------------
        {
            // this thread's key rows: j = 4*tr + 64*g + u, g < JN/4, u < 4
            // two groups of eight query rows per iteration (and four groups of keys in phase C) run 1 % faster
            // with the 64-row tiles; the 40-row tiles lose 11 % that way and keep the rolled forms (measured)
                        constexpr int kUnrollB = (RM == 5 || D == 128) ? 1 : 2;
#pragma unroll kUnrollB
            for (int i8 = 0; i8 < BM; i8 += 8)
#pragma unroll
            for (int iu = 0; iu < 8; ++iu) {
                const int i = i8 + iu;
                // Two adjacent keys per packed FMA: the pairs of P and dS come as they are stored
                // (row-major, keys contiguous), dO and Q values are duplicated into both lanes.
                float dov[DV], qv[DV];
                load_row_cols<D, BM>(sdO, i, iu, tc, dov);
                load_row_cols<D, BM>(sQ, i, iu, tc, qv);
                uint64_t do2[DV], q2[DV];
#pragma unroll
                for (int e = 0; e < DV; ++e) { do2[e] = f2_pack(dov[e], dov[e]); q2[e] = f2_pack(qv[e], qv[e]); }
#pragma unroll
                for (int g = 0; g < JN / 4; ++g) {
                    const U64x2 p4 = lds128_pairs(sP + (i * PSTR + 4 * tr + 4 * TR * g) * 4);
                    const U64x2 d4 = lds128_pairs(sdS + (i * PSTR + 4 * tr + 4 * TR * g) * 4);
#pragma unroll
                    for (int e = 0; e < DV; ++e) {
                        dv[2 * g][e] = f2_fma(p4.lo, do2[e], dv[2 * g][e]);
                        dv[2 * g + 1][e] = f2_fma(p4.hi, do2[e], dv[2 * g + 1][e]);
                        dk[2 * g][e] = f2_fma(d4.lo, q2[e], dk[2 * g][e]);
                        dk[2 * g + 1][e] = f2_fma(d4.hi, q2[e], dk[2 * g + 1][e]);
                    }
                }
            }
        }
        __syncthreads();   // Q and dO tiles are free
        if (tid == 0 && t + 1 < (GEN ? steps : n_qt)) {
            const int bh1 = GEN ? bhq0 + (t + 1) / nq : bhq0, i1 = (GEN ? qt0 + (t + 1) % nq : t + 1) * BM;
            mbar_arrive_expect_tx(barQ, 2 * C::Q_BYTES);
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
                tma_load_3d(sQ + ch * BM * 128, &tmQ, barQ, ch * 32, i1, bh1);
                tma_load_3d(sdO + ch * BM * 128, &tmdO, barQ, ch * 32, i1, bh1);
            }
        }

        // ---- C: dQ partial = dS K : contraction over keys, reduced into global dQ ----------
        if constexpr (WITH_DQ) {
            float dq[RM][DV];
#pragma unroll
            for (int x = 0; x < RM; ++x)
#pragma unroll
                for (int e = 0; e < DV; ++e) dq[x][e] = 0.f;
                        constexpr int kUnrollC = 2;
#pragma unroll kUnrollC
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
#pragma unroll
            for (int x = 0; x < RM; ++x) {
                const int i = i0 + tr + TR * x;
                if (i < Sq) {
                    float* row = dQ + (static_cast<size_t>(bh) * Sq + i) * D;
                    if constexpr (DV == 2) {
                        red_add_v2(row + 2 * tc, dq[x][0] * scale, dq[x][1] * scale);
                    } else {
#pragma unroll
                        for (int e = 0; e < DV / 4; ++e)
                            red_add_v4(row + 4 * tc + 64 * e, dq[x][4 * e] * scale, dq[x][4 * e + 1] * scale,
                                       dq[x][4 * e + 2] * scale, dq[x][4 * e + 3] * scale);
                    }
                }
            }
        }
    }

    // ---- epilogue: dK (scaled) and dV of this key tile ----------------------------------------
#pragma unroll
    for (int g = 0; g < JN / 4; ++g)
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int j = j0 + 4 * tr + 4 * TR * g + u;
            float kx[DV], vx[DV];
#pragma unroll
            for (int e = 0; e < DV; ++e) {
                float lo, hi;
                f2_unpack(dk[2 * g + (u >> 1)][e], lo, hi);
                kx[e] = ((u & 1) ? hi : lo) * scale;
                f2_unpack(dv[2 * g + (u >> 1)][e], lo, hi);
                vx[e] = (u & 1) ? hi : lo;
            }
            if (j < Sk) {
                const size_t off = (static_cast<size_t>(bhk) * Sk + j) * D;
                if constexpr (DV == 2) {
                    *reinterpret_cast<float2*>(dK + off + 2 * tc) = make_float2(kx[0], kx[1]);
                    *reinterpret_cast<float2*>(dV + off + 2 * tc) = make_float2(vx[0], vx[1]);
                } else {
#pragma unroll
                    for (int e = 0; e < DV / 4; ++e) {
                        *reinterpret_cast<float4*>(dK + off + 4 * tc + 64 * e) =
                            make_float4(kx[4 * e], kx[4 * e + 1], kx[4 * e + 2], kx[4 * e + 3]);
                        *reinterpret_cast<float4*>(dV + off + 4 * tc + 64 * e) =
                            make_float4(vx[4 * e], vx[4 * e + 1], vx[4 * e + 2], vx[4 * e + 3]);
                    }
                }
            }
        }
}

template <int D, int BM, int BN, int THREADS, bool GEN, bool WITH_DQ>
cudaError_t launch_gen(const Problem& p, const float* q, const float* k, const float* v, const float* d_o,
                       const float* lse, const float* delta, float* dq, float* dk, float* dv, unsigned* status,
                       cudaStream_t st)
{
    using C = BwdCfg<D, BM, BN, THREADS>;
    CUtensorMap tq, tk, tv, tdo;
    if (make_tmap_3d(&tq, q, 4, 0, p.BH(), p.Sq, D, 32, BM)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tdo, d_o, 4, 0, p.BH(), p.Sq, D, 32, BM)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tk, k, 4, 0, p.BHkv(), p.Sk, D, 32, BN)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tv, v, 4, 0, p.BHkv(), p.Sk, D, 32, BN)) return cudaErrorInvalidValue;
    auto kern = strict_bwd_kernel<D, BM, BN, THREADS, GEN, WITH_DQ>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
    if (e != cudaSuccess) return e;
    const int n_qt = (p.Sq + BM - 1) / BM;
    const int n_kt = (p.Sk + BN - 1) / BN;
    const long long blocks = static_cast<long long>(n_kt) * p.BHkv();
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    kern<<<static_cast<unsigned>(blocks), THREADS, C::SMEM, st>>>(tq, tk, tv, tdo, lse, delta, dq, dk, dv, p.Sq, p.Sk,
                                                                   p.BHkv(), p.H, p.group(), n_qt, p.causal, p.scale,
                                                                   status);
    return cudaGetLastError();
}

template <int D, int BM, int BN, int THREADS>
cudaError_t launch(const Problem& p, const float* q, const float* k, const float* v, const float* d_o,
                   const float* lse, const float* delta, float* dq, float* dk, float* dv, unsigned* status,
                   cudaStream_t st)
{
    if (dq == nullptr)   // fused dK+dV only (deterministic backward): the general-shape build serves every shape
        return launch_gen<D, BM, BN, THREADS, true, false>(p, q, k, v, d_o, lse, delta, dq, dk, dv, status, st);
    return (p.Hkv != p.H || p.Sq != p.Sk)
               ? launch_gen<D, BM, BN, THREADS, true, true>(p, q, k, v, d_o, lse, delta, dq, dk, dv, status, st)
               : launch_gen<D, BM, BN, THREADS, false, true>(p, q, k, v, d_o, lse, delta, dq, dk, dv, status, st);
}

}  // namespace

cudaError_t launch_strict_bwd(const Problem& p, const float* q, const float* k, const float* v,
                              const float* d_o, const float* lse, const float* delta,
                              float* dq, float* dk, float* dv, unsigned* status, cudaStream_t st)
{
    int BM, BN;
    strict_bwd_tiles(p, &BM, &BN);
    switch (p.D) {
        case 32:  return launch<32, 64, 64, 128>(p, q, k, v, d_o, lse, delta, dq, dk, dv, status, st);
        case 64:
            if (BM == 40)   // short ragged sequences
                return launch<64, 40, 64, 128>(p, q, k, v, d_o, lse, delta, dq, dk, dv, status, st);
            return launch<64, 64, 64, 128>(p, q, k, v, d_o, lse, delta, dq, dk, dv, status, st);
        case 128: return launch<128, 32, 64, 128>(p, q, k, v, d_o, lse, delta, dq, dk, dv, status, st);
        default:  return cudaErrorInvalidValue;
    }
}

}  // namespace mgn
