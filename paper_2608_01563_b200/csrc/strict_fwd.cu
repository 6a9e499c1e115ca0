// Strict-mode attention forward: f32 storage, f32 FFMA arithmetic (paper Section 3.3,
// "tiled attention forward"; Section 4.2 strict arithmetic contract).
//
// One CTA (256 threads) owns BM query rows of one head and streams BN-key tiles of
// K and V through shared memory with TMA.  Scores live in registers (each thread an
// (BM/16)x(BN/16) micro-tile), the softmax is the online form (running row max in
// the log2 domain, thread-local partial row sums), P goes through shared memory
// once to become the A operand of O += P V.  Query head h reads key/value head h / G (grouped
// heads); queries and keys may differ in length, the causal mask then being aligned bottom-right.
//
// Shared-memory tile layout (as TMA writes it with the 128-byte swizzle): a tile of
// R rows x D floats is stored as D/32 chunks; chunk c holds, for every row, the 32
// floats [32c, 32c+32) in a 128-byte line, lines at 128-byte pitch, and the 16-byte
// piece p of row r sits at piece position p ^ (r & 7).  Rows that a warp reads in one
// instruction are consecutive modulo 8, so every 128-bit shared load is conflict free.
#include "kernels.h"
#include "ptx.cuh"

#include <type_traits>

namespace mgn {
namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// THREADS/16 row groups x 16 column groups.  128-thread CTAs fit two per SM (registers and shared
// memory), which decouples their barriers and softmax phases: one CTA's FFMA loop fills the
// issue slots the other leaves idle.
template <int D, int BM, int BN, int THREADS>
struct FwdCfg {
    static constexpr int TR = THREADS / 16;   // row groups
    static constexpr int RM = BM / TR;        // query rows per thread
    static constexpr int RN = BN / 16;    // key columns per thread
    static constexpr int DV = D / 16;     // output columns per thread
    static constexpr int NCH = D / 32;    // 128-byte chunks per row
    // P is stored key-major as pairs of query rows: for key column j, row group tr owns 32 bytes =
    // four (row 2q, row 2q+1) pairs of its own rows (pairs past RM are zero); 16-byte piece
    // c = 2 tr + h sits at piece position c ^ (j & 7).  A packed two-lane FMA then takes a pair as
    // one operand, and both the stores (one column per lane) and the loads (one row group per half
    // warp) are conflict free.
    static constexpr int RP = (RM + 1) / 2;   // row pairs per thread
    static constexpr int PROW = TR * 32;      // bytes per key column
    // Half-tile form of the two products (first BN/2 keys only): needs the half to be whole column groups
    // and a whole number of the P V loop's unrolled key groups (32 keys at most).
    static constexpr bool HALF_OK = (BN % 64 == 0);
    static constexpr int Q_BYTES = BM * D * 4;
    static constexpr int KV_BYTES = BN * D * 4;
    static constexpr int P_BYTES = BN * PROW;
    static_assert(RM <= 8, "a row group's pairs fill two 16-byte pieces");
    static constexpr int PAYLOAD = Q_BYTES + 2 * KV_BYTES + P_BYTES + 64;
    // Two 128-thread CTAs per SM must fit 2 x (SMEM + 1 KB reserved) into 228 KB, which leaves less
    // than the 1023 bytes a worst-case 1024-byte alignment of the tile base could need; the kernel
    // checks the slack it actually got and reports through the status word if it is short.
    static constexpr int SLACK = (THREADS == 128 && PAYLOAD + 1024 > 115712) ? 115712 - PAYLOAD : 1024;
    static constexpr int SMEM = PAYLOAD + SLACK;
    static_assert(SLACK >= 0, "shared memory budget");
};

// Byte offset of the 16-byte piece `piece` (0..D/4-1) of row `r` in a swizzled tile of R rows.
template <int R>
__device__ __forceinline__ uint32_t tile_off(int r, int piece) {
    return static_cast<uint32_t>((piece >> 3) * (R * 128) + r * 128 + (((piece & 7) ^ (r & 7)) << 4));
}

// GEN = false is the square multi-head case (Sk == Sq, one key/value head per query head): the
// offset, the group size and the second length fold away at compile time.
template <int D, int BM, int BN, int THREADS, bool GEN>
__global__ void __launch_bounds__(THREADS, THREADS == 128 ? 2 : 1)
strict_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, float* __restrict__ O, float* __restrict__ LSE,
                  int Sq, int Sk_, int BH, int H, int G_, int n_qt, int causal, float c2, unsigned* status)
{
    const int Sk = GEN ? Sk_ : Sq;
    const int G = GEN ? G_ : 1;
    using C = FwdCfg<D, BM, BN, THREADS>;
    constexpr int RM = C::RM, RN = C::RN, DV = C::DV, NCH = C::NCH, TR = C::TR, RP = C::RP, PROW = C::PROW;

    extern __shared__ uint8_t smem_raw[];
    if (*reinterpret_cast<volatile unsigned*>(status) != 0) return;   // an earlier wait on this device gave up
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = base;
    const uint32_t sK = sQ + C::Q_BYTES;
    const uint32_t sV = sK + C::KV_BYTES;
    const uint32_t sP = sV + C::KV_BYTES;
    const uint32_t barQ = sP + C::P_BYTES, barK = barQ + 8, barV = barQ + 16;
    if (base + C::PAYLOAD > smem_u32(smem_raw) + C::SMEM) {      // alignment slack ran out
        if (threadIdx.x == 0) atomicMax(status, kStatusSmemLayout);
        return;
    }

    const int tid = threadIdx.x;
    const int tr = 2 * (tid >> 5) + ((tid & 31) >> 4);   // 0..15: row group
    const int tc = tid & 15;                             // 0..15: column group

    // Heaviest (last) query tiles first when causal.
    const int qt = n_qt - 1 - static_cast<int>(blockIdx.x) / BH;
    const int bh = static_cast<int>(blockIdx.x) % BH;
    const int bhk = GEN ? (bh / H) * (H / G) + (bh % H) / G : bh;   // key/value head of this query head
    const int off = GEN ? Sk - Sq : 0;                   // causal: key j visible to query i iff j <= i + off
    const int i0 = qt * BM;
    const int i_last = min(i0 + BM, Sq) - 1;
    const int n_kt = causal ? ((i_last + off) / BN + 1) : ((Sk + BN - 1) / BN);

    if (tid == 0) {
        mbar_init(barQ, 1);
        mbar_init(barK, 1);
        mbar_init(barV, 1);
        fence_mbar_init();
    }
    __syncthreads();
    if (tid == 0) {
        mbar_arrive_expect_tx(barQ, C::Q_BYTES);
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) tma_load_3d(sQ + ch * BM * 128, &tmQ, barQ, ch * 32, i0, bh);
        mbar_arrive_expect_tx(barK, C::KV_BYTES);
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) tma_load_3d(sK + ch * BN * 128, &tmK, barK, ch * 32, 0, bhk);
        mbar_arrive_expect_tx(barV, C::KV_BYTES);
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) tma_load_3d(sV + ch * BN * 128, &tmV, barV, ch * 32, 0, bhk);
    }

    // O accumulators as packed pairs: o[q][e] = {row 2q, row 2q+1} of output column e
    uint64_t o[RP][DV];
    float m[RM], l[RM];
#pragma unroll
    for (int x = 0; x < RM; ++x) {
        m[x] = -INFINITY;
        l[x] = 0.f;
    }
#pragma unroll
    for (int q = 0; q < RP; ++q)
#pragma unroll
        for (int e = 0; e < DV; ++e) o[q][e] = f2_pack(0.f, 0.f);

    mbar_wait(barQ, 0, status);

    for (int kt = 0; kt < n_kt; ++kt) {
        const uint32_t ph = kt & 1;
        const int j0 = kt * BN;
        float s[RM][RN];
#pragma unroll
        for (int x = 0; x < RM; ++x)
#pragma unroll
            for (int y = 0; y < RN; ++y) s[x][y] = 0.f;

        // Keys of this tile that some row of the query tile can see.  When they fill at most the first half of
        // the tile (the last tile of every other query tile under a causal mask with BN = 2 BM; a ragged
        // tail), both products run over that half only; the scores of the other half stay 0 and are masked.
        const int k_vis = min(Sk, causal ? i_last + off + 1 : Sk) - j0;
        const bool half_tile = C::HALF_OK && k_vis <= BN / 2;

        mbar_wait(barK, ph, status);
        // ---- S = Q K^T : contraction along d, float4 pieces --------------------------------
        auto qk = [&](auto yn_tag) {
            constexpr int YN = decltype(yn_tag)::value;
            const uint32_t qa = sQ + tr * 128, ka = sK + tc * 128;
            const int xq = tr & 7, xk = tc & 7;
            // Unroll factors are set by the instruction cache (instruction fetch is this kernel's top stall,
            // 0.87 stalled warps per issue with the loops of both products unrolled far): measured on the
            // GPT-2-small shape, 8 contraction steps x 32 keys per iteration -> 0.363 ms, 4 x 32 -> 0.326,
            // 4 x 16 -> 0.328, 1 x 16 -> 0.324; the 5-row micro-tile of the 40-row tiles keeps 8 x 32 (0.135 against
            // 0.137-0.139 ms).  D = 128 (decoder sweep, S = 1024): one 256-thread CTA per SM with 128 x 64 tiles ran
            // 0.844 ms at 32 x 32 and 0.828 at 16 x 16; two 128-thread CTAs per SM with 64 x 64 tiles run 0.776 at
            // 16 x 16, 0.754 at 4 x 16 and 0.739 at 8 x 16, which is what D = 128 now uses.
            constexpr int kUnrollQK = (RM == 5 || D == 128) ? 8 : 4;
#pragma unroll kUnrollQK
            for (int pc = 0; pc < D / 4; ++pc) {
                const uint32_t oq = (pc >> 3) * (BM * 128) + (((pc & 7) ^ xq) << 4);
                const uint32_t ok = (pc >> 3) * (BN * 128) + (((pc & 7) ^ xk) << 4);
                float4 b[YN];
#pragma unroll
                for (int y = 0; y < YN; ++y) b[y] = lds128(ka + ok + y * 16 * 128);
#pragma unroll
                for (int x = 0; x < RM; ++x) {
                    const float4 a = lds128(qa + oq + x * TR * 128);
#pragma unroll
                    for (int y = 0; y < YN; ++y) {
                        s[x][y] = fmaf(a.x, b[y].x, s[x][y]);
                        s[x][y] = fmaf(a.y, b[y].y, s[x][y]);
                        s[x][y] = fmaf(a.z, b[y].z, s[x][y]);
                        s[x][y] = fmaf(a.w, b[y].w, s[x][y]);
                    }
                }
            }
        };
        if constexpr (C::HALF_OK) {
            if (half_tile) qk(std::integral_constant<int, RN / 2>{});
            else qk(std::integral_constant<int, RN>{});
        } else {
            qk(std::integral_constant<int, RN>{});
        }
        __syncthreads();   // every warp is done with this K tile (and with P of the previous tile)
        if (tid == 0 && kt + 1 < n_kt) {
            mbar_arrive_expect_tx(barK, C::KV_BYTES);
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) tma_load_3d(sK + ch * BN * 128, &tmK, barK, ch * 32, j0 + BN, bhk);
        }

        // ---- scale into the log2 domain, mask, online softmax ------------------------------
        const bool need_mask = (causal && (j0 + BN - 1 > i0 + off)) || (j0 + BN > Sk);
        float alpha[2 * RP];
#pragma unroll
        for (int x = 0; x < RM; ++x) {
            const int i = i0 + tr + TR * x;
            float mx = -INFINITY;
#pragma unroll
            for (int y = 0; y < RN; ++y) {
                float v = s[x][y] * c2;
                if (need_mask) {
                    const int j = j0 + tc + 16 * y;
                    if (j >= Sk || (causal && j > i + off)) v = -INFINITY;
                }
                s[x][y] = v;
                mx = fmaxf(mx, v);
            }
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
            const float m_new = fmaxf(m[x], mx);    // finite from the first tile on (key 0 is never masked)
            alpha[x] = ex2(m[x] - m_new);
            m[x] = m_new;
            float psum = 0.f;
#pragma unroll
            for (int y = 0; y < RN; ++y) {
                const float p = ex2(s[x][y] - m_new);
                psum += p;
                s[x][y] = p;
            }
            l[x] = fmaf(l[x], alpha[x], psum);
        }
        if constexpr (RM & 1) alpha[RM] = 1.f;
        // P: this thread's rows of key column j = tc + 16 y as row pairs, two 16-byte stores per column
#pragma unroll
        for (int y = 0; y < RN; ++y) {
            const uint32_t col = sP + (tc + 16 * y) * PROW;
            const int jx = tc & 7;                      // (tc + 16 y) & 7
            auto pv = [&](int x) { return x < RM ? s[x < RM ? x : 0][y] : 0.f; };
            sts128f(col + (((2 * tr) ^ jx) << 4), pv(0), pv(1), pv(2), pv(3));
            if constexpr (RM > 4) sts128f(col + (((2 * tr + 1) ^ jx) << 4), pv(4), pv(5), pv(6), pv(7));
        }
#pragma unroll
        for (int q = 0; q < RP; ++q) {
            const uint64_t a2 = f2_pack(alpha[2 * q], alpha[2 * q + 1]);
#pragma unroll
            for (int e = 0; e < DV; ++e) o[q][e] = f2_mul(o[q][e], a2);
        }
        __syncthreads();   // P visible
        mbar_wait(barV, ph, status);

        // ---- O += P V : contraction along keys, two query rows per packed FMA ------------------
        // Per key: V's columns of this thread are loaded once and duplicated into both lanes, the
        // row pairs of P come as they are stored; DV * RP packed FMAs follow.
        {
            const uint32_t pa = sP + ((2 * tr) << 4);
            constexpr int kUnrollPV = (D == 32) ? 8 : (D == 128) ? 16 : 32;
            static_assert(!C::HALF_OK || (BN / 2) % kUnrollPV == 0, "half a tile is whole unrolled groups");
            auto pv_key = [&](int j) {
                const int u = j & 7;
                float vv[DV];
                if constexpr (DV == 2) {
                    const float2 t = lds64(sV + j * 128 + ((((tc >> 1)) ^ u) << 4) + (tc & 1) * 8);
                    vv[0] = t.x; vv[1] = t.y;
                } else {
#pragma unroll
                    for (int e = 0; e < DV / 4; ++e) {
                        const int piece = tc + 16 * e;
                        const float4 t = lds128(sV + (piece >> 3) * (BN * 128) + j * 128 + (((piece & 7) ^ u) << 4));
                        vv[4 * e + 0] = t.x; vv[4 * e + 1] = t.y; vv[4 * e + 2] = t.z; vv[4 * e + 3] = t.w;
                    }
                }
                uint64_t vd[DV];
#pragma unroll
                for (int e = 0; e < DV; ++e) vd[e] = f2_pack(vv[e], vv[e]);
                // pieces 2 tr and 2 tr + 1 of column j: positions (2 tr) ^ u and that with bit 0 flipped
                const uint32_t pj = (pa + j * PROW) ^ static_cast<uint32_t>(u << 4);
                const U64x2 p01 = lds128_pairs(pj);
                uint64_t pp[4] = {p01.lo, p01.hi, 0ull, 0ull};
                if constexpr (RP > 2) {
                    const U64x2 p23 = lds128_pairs(pj ^ 16u);
                    pp[2] = p23.lo;
                    pp[3] = p23.hi;
                }
#pragma unroll
                for (int q = 0; q < RP; ++q)
#pragma unroll
                    for (int e = 0; e < DV; ++e) o[q][e] = f2_fma(pp[q], vd[e], o[q][e]);
            };
            if constexpr (C::HALF_OK) {          // run-time key count, a whole number of unrolled groups
                const int jn = half_tile ? BN / 2 : BN;
                for (int jb = 0; jb < jn; jb += kUnrollPV)
#pragma unroll
                    for (int jj = 0; jj < kUnrollPV; ++jj) pv_key(jb + jj);
            } else {
#pragma unroll kUnrollPV
                for (int j = 0; j < BN; ++j) pv_key(j);
            }
        }
        __syncthreads();   // every warp is done with this V tile and with P
        if (tid == 0 && kt + 1 < n_kt) {
            mbar_arrive_expect_tx(barV, C::KV_BYTES);
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) tma_load_3d(sV + ch * BN * 128, &tmV, barV, ch * 32, j0 + BN, bhk);
        }
    }

    // ---- epilogue: O / l, LSE = ln2 (m + log2 l) -----------------------------------------------
#pragma unroll
    for (int x = 0; x < RM; ++x) {
        float lt = l[x];
        lt += __shfl_xor_sync(0xffffffffu, lt, 1);
        lt += __shfl_xor_sync(0xffffffffu, lt, 2);
        lt += __shfl_xor_sync(0xffffffffu, lt, 4);
        lt += __shfl_xor_sync(0xffffffffu, lt, 8);
        const int i = i0 + tr + TR * x;
        float ox[DV];
#pragma unroll
        for (int e = 0; e < DV; ++e) {
            float lo, hi;
            f2_unpack(o[x >> 1][e], lo, hi);
            ox[e] = (x & 1) ? hi : lo;
        }
        if (i < Sq) {
            const float inv = 1.0f / lt;
            float* orow = O + (static_cast<size_t>(bh) * Sq + i) * D;
            if constexpr (DV == 2) {
                *reinterpret_cast<float2*>(orow + 2 * tc) = make_float2(ox[0] * inv, ox[1] * inv);
            } else {
#pragma unroll
                for (int e = 0; e < DV / 4; ++e)
                    *reinterpret_cast<float4*>(orow + 4 * tc + 64 * e) =
                        make_float4(ox[4 * e] * inv, ox[4 * e + 1] * inv, ox[4 * e + 2] * inv, ox[4 * e + 3] * inv);
            }
            if (tc == 0) LSE[static_cast<size_t>(bh) * Sq + i] = (m[x] + log2f(lt)) * kLn2;
        }
    }
}

template <int D, int BM, int BN, int THREADS, bool GEN>
cudaError_t launch_gen(const Problem& p, const float* q, const float* k, const float* v, float* o, float* lse,
                   unsigned* status, cudaStream_t st)
{
    using C = FwdCfg<D, BM, BN, THREADS>;
    CUtensorMap tq, tk, tv;
    if (make_tmap_3d(&tq, q, 4, 0, p.BH(), p.Sq, D, 32, BM)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tk, k, 4, 0, p.BHkv(), p.Sk, D, 32, BN)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tv, v, 4, 0, p.BHkv(), p.Sk, D, 32, BN)) return cudaErrorInvalidValue;
    auto kern = strict_fwd_kernel<D, BM, BN, THREADS, GEN>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
    if (e != cudaSuccess) return e;
    const int n_qt = (p.Sq + BM - 1) / BM;
    const long long blocks = static_cast<long long>(n_qt) * p.BH();
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    kern<<<static_cast<unsigned>(blocks), THREADS, C::SMEM, st>>>(tq, tk, tv, o, lse, p.Sq, p.Sk, p.BH(), p.H, p.group(), n_qt,
                                                                   p.causal,
                                                                   p.scale * kLog2e, status);
    return cudaGetLastError();
}

template <int D, int BM, int BN, int THREADS>
cudaError_t launch(const Problem& p, const float* q, const float* k, const float* v, float* o, float* lse,
                   unsigned* status, cudaStream_t st)
{
    return (p.Hkv != p.H || p.Sq != p.Sk) ? launch_gen<D, BM, BN, THREADS, true>(p, q, k, v, o, lse, status, st)
                                          : launch_gen<D, BM, BN, THREADS, false>(p, q, k, v, o, lse, status, st);
}

}  // namespace

cudaError_t launch_strict_fwd(const Problem& p, const float* q, const float* k, const float* v,
                              float* o, float* lse, unsigned* status, cudaStream_t st)
{
    int BM, BN;
    strict_fwd_tiles(p, &BM, &BN);
    switch (p.D) {
        case 32:  return launch<32, 64, 128, 128>(p, q, k, v, o, lse, status, st);
        case 64:
            if (BM == 40) return launch<64, 40, 112, 128>(p, q, k, v, o, lse, status, st);   // short ragged sequences
            return launch<64, 64, 128, 128>(p, q, k, v, o, lse, status, st);
        case 128: return launch<128, 64, 64, 128>(p, q, k, v, o, lse, status, st);
        default:  return cudaErrorInvalidValue;
    }
}

}  // namespace mgn
