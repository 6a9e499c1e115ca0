// Fast-mode attention forward for short key sequences (at most two 128-key blocks): the latency path.
//
// The paper's own attention shapes are small -- 197 vision-transformer tokens, sequence-128 and
// minimal-shape cells, 50 action tokens over 16 context tokens, 77-token text cross-attention
// (Section 4.1, workload table) -- and its profiles show dispatch structure mattering where kernels are
// small (Section 7.3).  The persistent kernel in fast_fwd.cu is built for long items: with one or two
// key blocks per item its fill, hand-offs and epilogue (about 5 us per item, one item at a time per SM)
// are all there is.  Here one small CTA owns one 128-row query tile of one head and up to four of them
// share an SM (two at D = 128), so the latencies of neighbouring tiles overlap:
//   warp 0, one lane   TMA loads (Q once; K and V per block, single buffers) and all tensor-core issue
//   warps 1-4          softmax, ONE THREAD PER ROW (tensor-memory lane): the row maximum, the running
//                      sum and the rescaling factor are thread-local, so the classic online softmax
//                      needs no exchange between threads and no speculation
// Tensor memory (256 columns): S [0,128), O [128,128+D).  P (bf16) overwrites S, keys 0-127 at S[0,64),
// each 16-column piece written over columns the thread has already read.  The output tile leaves through
// the Q buffer (dead after the last score product) and a TMA store.
#include "kernels.h"
#include "fast_items.cuh"
#include "umma.cuh"

namespace mgn {
namespace {

constexpr int kThreads = 160;
constexpr int BM = 128, BN = 128;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

template <int D>
struct Cfg {
    static constexpr int NCH = D / 64;
    static constexpr int TILE_BYTES = 128 * D * 2;
    static constexpr int CHUNK_BYTES = 128 * 128;
    static constexpr int OFF_Q = 0, OFF_K = TILE_BYTES, OFF_V = 2 * TILE_BYTES, OFF_BAR = 3 * TILE_BYTES;
    static constexpr int PAYLOAD = OFF_BAR + 64;
    static constexpr int SMEM = PAYLOAD + 1024;
    static constexpr uint32_t TM_S = 0, TM_O = 128, TM_COLS = 256;
};
enum { B_Q = 0, B_K = 1, B_V = 2, B_SFULL = 3, B_PFULL = 4, B_PVDONE = 5, B_COUNT = 6 };

template <int D, bool GEN>
__global__ void __launch_bounds__(kThreads, 2)
fast_fwd_small_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                      const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                      float* __restrict__ LSE, const Dims dm, int n_qt, int causal, float c2, unsigned* status)
{
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    if (*reinterpret_cast<volatile unsigned*>(status) != 0) return;   // an earlier wait on this device gave up
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = base + C::OFF_Q, sK = base + C::OFF_K, sV = base + C::OFF_V, bars = base + C::OFF_BAR;
    const uint32_t tmem_slot = bars + B_COUNT * 8;
    auto bar = [&](int i) { return bars + 8u * i; };
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    const int Sq = dm.Sq, Sk = GEN ? dm.Sk : dm.Sq, coff = GEN ? dm.off : 0;
    const int bh = static_cast<int>(blockIdx.x) / n_qt;
    const int row0 = (n_qt - 1 - static_cast<int>(blockIdx.x) % n_qt) * BM;       // last (heaviest) tiles of a head first
    const int bhk = GEN ? (bh / dm.H) * (dm.H / dm.G) + (bh % dm.H) / dm.G : bh;
    const int n_kb = (Sk + BN - 1) / BN;
    const int nb = causal ? min(n_kb, (min(row0 + BM, Sq) - 1 + coff) / BN + 1) : n_kb;   // key blocks this tile sees (>= 1)

    if (tid == 0) {
        for (int i = 0; i < B_COUNT; ++i) mbar_init(bar(i), i == B_PFULL ? 4 : 1);   // P: one arrival per softmax warp
        fence_mbar_init();
    }
    __syncwarp();
    if (warp == 0) tmem_alloc(tmem_slot, C::TM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = lds32u(tmem_slot);

    if (warp == 0) {
        if (lane == 0) {
            // ---------------------------------------------------------------- loads and tensor-core issue
            constexpr uint32_t idesc_s = umma_idesc_bf16(BM, BN, false, false);
            constexpr uint32_t idesc_o = umma_idesc_bf16(BM, D, false, true);
            const uint64_t qd = umma_smem_desc(sQ, 16, 1024), kd = umma_smem_desc(sK, 16, 1024);
            const uint64_t vd = umma_smem_desc(sV, C::CHUNK_BYTES, 1024);
            const uint32_t tS = tmem + C::TM_S, tO = tmem + C::TM_O;
            auto load_tile = [&](uint32_t dst, const CUtensorMap* map, int b, int r, int head) {
                mbar_arrive_expect_tx(bar(b), C::TILE_BYTES);
#pragma unroll
                for (int ch = 0; ch < C::NCH; ++ch) tma_load_3d(dst + ch * C::CHUNK_BYTES, map, bar(b), ch * 64, r, head);
            };
            auto issue_s = [&]() {
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint64_t off = static_cast<uint64_t>(((kk >> 2) * C::CHUNK_BYTES + (kk & 3) * 32) >> 4);
                    umma_ss(tS, qd + off, kd + off, idesc_s, kk > 0);
                }
                umma_commit(bar(B_SFULL));
            };
            load_tile(sQ, &tmQ, B_Q, row0, bh);
            load_tile(sK, &tmK, B_K, 0, bhk);
            load_tile(sV, &tmV, B_V, 0, bhk);
            mbar_wait(bar(B_Q), 0, status);
            mbar_wait(bar(B_K), 0, status);
            tc_fence_after();
            issue_s();
            for (int n = 0; n < nb; ++n) {
                if (n + 1 < nb) {                                   // K is free once the scores of block n are complete
                    mbar_wait(bar(B_SFULL), n & 1, status);
                    load_tile(sK, &tmK, B_K, (n + 1) * BN, bhk);
                }
                mbar_wait(bar(B_V), n & 1, status);
                mbar_wait(bar(B_PFULL), n & 1, status);
                tc_fence_after();
                // O (+)= P V, P from tensor memory (8 columns per 16 keys); only the 16-key steps that hold keys:
                // the softmax threads leave the 32-column pieces past the end of the sequence unwritten
                const int ksteps = (min(Sk - n * BN, BN) + 15) >> 4;
                for (int kk = 0; kk < ksteps; ++kk)
                    umma_ts(tO, tS + kk * 8, vd + static_cast<uint64_t>((kk * 2048) >> 4), idesc_o, (kk > 0 || n > 0) ? 1u : 0u);
                umma_commit(bar(B_PVDONE));
                if (n + 1 < nb) {
                    mbar_wait(bar(B_K), (n + 1) & 1, status);
                    tc_fence_after();
                    issue_s();                                      // overwrites P(n): in issue order behind the product that read it
                    mbar_wait(bar(B_PVDONE), n & 1, status);        // V is free
                    load_tile(sV, &tmV, B_V, (n + 1) * BN, bhk);
                }
            }
        }
        __syncwarp();
    } else {
        // -------------------------------------------------------------------- softmax, one thread per row
        const int q4 = warp & 3, r = 32 * q4 + lane, i = row0 + r;
        const uint32_t lane_base = static_cast<uint32_t>(32 * q4) << 16;
        const uint32_t tS = tmem + lane_base + C::TM_S, tO = tmem + lane_base + C::TM_O;
        float m = -INFINITY, l = 0.f;
        for (int n = 0; n < nb; ++n) {
            mbar_wait(bar(B_SFULL), n & 1, status);
            tc_fence_after();
            const int j0 = n * BN;
            const bool masked = (causal && (j0 + BN - 1 > row0 + coff)) || (j0 + BN > Sk);
            const int jmax = min(Sk - 1, causal ? i + coff : Sk - 1) - j0;     // columns c <= jmax of this block are visible
            const int nch = (min(Sk - j0, BN) + 31) >> 5;       // 32-column pieces that hold keys
            // pass 1: the row maximum of this block (thread-local: the whole row is this thread's)
            float mx = -INFINITY;
#pragma unroll 1
            for (int c = 0; c < nch; ++c) {
                uint32_t v[32];
                tmem_ld32(tS + 32 * c, v);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    if (!masked || 32 * c + e <= jmax) mx = fmaxf(mx, __uint_as_float(v[e]) * c2);
            }
            const float m_new = fmaxf(m, mx);                   // finite for every row that is stored (key 0 is visible)
            const float alpha = (m_new == -INFINITY) ? 1.0f : ex2(m - m_new);   // 0 in the first block of a row that sees a key
            if (n > 0 && __any_sync(0xffffffffu, alpha != 1.0f)) {
                // the scores of block n are complete, so the product that accumulated block n - 1 into O is too
#pragma unroll 1
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld32(tO + 32 * c, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) * alpha);
                    tmem_st32(tO + 32 * c, v);
                }
            }
            l *= alpha;
            m = m_new;
            // pass 2: p = exp2(s c2 - m), row sum, bf16 pack over the columns already read
            const float neg_m = (m_new == -INFINITY) ? 0.f : -m_new;          // rows past the end: nothing visible
            float ls0 = 0.f, ls1 = 0.f;
#pragma unroll 1
            for (int c = 0; c < nch; ++c) {
                uint32_t v[32];
                tmem_ld32(tS + 32 * c, v);
                tmem_ld_wait();
                uint32_t u[16];
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    float y0 = fmaf(__uint_as_float(v[e]), c2, neg_m), y1 = fmaf(__uint_as_float(v[e + 1]), c2, neg_m);
                    if (masked) {
                        if (32 * c + e > jmax) y0 = -INFINITY;
                        if (32 * c + e + 1 > jmax) y1 = -INFINITY;
                    }
                    const float p0 = ex2(y0), p1 = ex2(y1);
                    ls0 += p0;
                    ls1 += p1;
                    u[e / 2] = pack_bf16(p0, p1);
                }
                tmem_st16(tS + 16 * c, u);
            }
            l += ls0 + ls1;
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_PFULL));
        }

        // ---- epilogue: O / l -> bf16 -> the Q buffer (swizzled like the TMA box) -> TMA store; LSE
        mbar_wait(bar(B_PVDONE), (nb - 1) & 1, status);
        tc_fence_after();
        const float inv = l > 0.f ? 1.0f / l : 0.f;
        if (i < Sq) LSE[static_cast<size_t>(bh) * Sq + i] = (m + log2f(l)) * kLn2;
#pragma unroll 1
        for (int c = 0; c < D / 32; ++c) {
            uint32_t v[32];
            tmem_ld32(tO + 32 * c, v);
            tmem_ld_wait();
            uint32_t u[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) u[e] = pack_bf16(__uint_as_float(v[2 * e]) * inv, __uint_as_float(v[2 * e + 1]) * inv);
            const int col = 32 * c;
            const uint32_t rowaddr = sQ + (col >> 6) * C::CHUNK_BYTES + r * 128;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int piece = ((col & 63) >> 3) + q;
                sts128(rowaddr + ((piece ^ (r & 7)) << 4), u[4 * q], u[4 * q + 1], u[4 * q + 2], u[4 * q + 3]);
            }
        }
        fence_proxy_async_smem();
        named_bar_sync(1, 128);
        if (r == 0) {
#pragma unroll
            for (int ch = 0; ch < C::NCH; ++ch) tma_store_3d(&tmO, sQ + ch * C::CHUNK_BYTES, ch * 64, row0, bh);
            tma_store_commit_and_wait_read();
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, C::TM_COLS);
}

template <int D, bool GEN>
cudaError_t launch_gen(const Problem& p, const void* q, const void* k, const void* v, void* o, float* lse,
                       unsigned* status, cudaStream_t st)
{
    using C = Cfg<D>;
    CUtensorMap tq, tk, tv, to;
    if (make_tmap_3d(&tq, q, 2, 1, p.BH(), p.Sq, p.D, 64, 128)) return MGN_FAIL(cudaErrorInvalidValue, "tensor map q");
    if (make_tmap_3d(&tk, k, 2, 1, p.BHkv(), p.Sk, p.D, 64, 128)) return MGN_FAIL(cudaErrorInvalidValue, "tensor map k");
    if (make_tmap_3d(&tv, v, 2, 1, p.BHkv(), p.Sk, p.D, 64, 128)) return MGN_FAIL(cudaErrorInvalidValue, "tensor map v");
    if (make_tmap_3d(&to, o, 2, 1, p.BH(), p.Sq, p.D, 64, 128)) return MGN_FAIL(cudaErrorInvalidValue, "tensor map o");
    auto kern = fast_fwd_small_kernel<D, GEN>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
    if (e != cudaSuccess) return MGN_FAIL(e, "cudaFuncSetAttribute");
    const int n_qt = (p.Sq + BM - 1) / BM;
    const long long blocks = static_cast<long long>(n_qt) * p.BH();
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
    const Dims dm{p.Sq, p.Sk, p.BH(), p.H, p.group(), p.off()};
    kern<<<static_cast<unsigned>(blocks), kThreads, C::SMEM, st>>>(tq, tk, tv, to, lse, dm, n_qt, p.causal,
                                                                   p.scale * kLog2e, status);
    return MGN_FAIL(cudaGetLastError(), "small forward launch");
}

template <int D>
cudaError_t launch(const Problem& p, const void* q, const void* k, const void* v, void* o, float* lse,
                   unsigned* status, cudaStream_t st)
{
    return (p.Hkv != p.H || p.Sq != p.Sk) ? launch_gen<D, true>(p, q, k, v, o, lse, status, st)
                                          : launch_gen<D, false>(p, q, k, v, o, lse, status, st);
}

}  // namespace

cudaError_t launch_fast_fwd_small(const Problem& p, const void* q, const void* k, const void* v, void* o, float* lse,
                                  unsigned* status, cudaStream_t st)
{
    switch (p.D) {
        case 32:  // the 64-wide build on zero-filled 32-element rows (see fast_fwd.cu)
        case 64:  return launch<64>(p, q, k, v, o, lse, status, st);
        case 128: return launch<128>(p, q, k, v, o, lse, status, st);
        default:  return cudaErrorNotSupported;
    }
}

}  // namespace mgn
