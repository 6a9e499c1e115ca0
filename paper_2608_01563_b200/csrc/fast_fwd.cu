// Fast-mode attention forward: bf16 storage, tcgen05 tensor-core products with f32
// accumulation in tensor memory, f32 softmax statistics (paper Section 3.3 "tiled attention
// forward"; Section 4.2: the validated reduced-input path with f32 accumulation).
//
// Persistent kernel: one CTA per SM walks over work items (two 128-row query tiles of one head
// each -- one tile when there would be fewer items than SMs; two item orders, see make_item) and, per item, over 128-key blocks of that head's
// key/value head.  All barriers keep counting across items, so the producer prefetches the next
// item's Q/K/V and the issuers compute its first scores while the softmax warps are still writing
// the previous item's output: most of the per-item fill and drain is hidden instead of paid by
// every CTA.
// Warp roles (384 threads):
//   warp 0      TMA producer: Q tiles once, then K and V blocks through a 2-stage ring
//   warps 1, 2  MMA issuers, one per query tile: S_t = Q_t K^T (operands in shared memory) and
//               O_t += P_t V (P_t read from tensor memory, V as an MN-major shared-memory
//               operand).  One lane each; with two issuers the tensor core keeps working on one
//               tile while the other issuer sits in a barrier wait (a wait costs a few hundred
//               clocks even when it succeeds at once, and the issue queue is shallow)
//   warps 4-11  softmax: all 256 threads work on ONE query tile at a time, two threads per row
//               (64 key columns each), alternating between the two tiles.  A lone warp per
//               scheduler cannot keep the exp2 unit busy; two can, so a tile's softmax takes half
//               as long and the tensor core's S/PV products of the other tile hide it.
// Tensor memory (512 columns): S_0 [0,128), S_1 [128,256), O_0 [256,256+D), O_1 [256+D,256+2D).
// P_t (bf16) overwrites S_t: keys 0-63 at S_t[0,32), keys 64-127 at S_t[64,96) (each half in the
// columns its own threads have already read).  The softmax reference point of a row only moves
// (and O is rescaled in tensor memory) when a row outgrows it so far that a thread's partial sum of
// exponentials passes a limit (2^60; 2^12 with f16 probabilities), which is exact: any reference point works for a softmax as long as
// nothing overflows.  The two threads of a row agree on that through a barrier with an
// OR-reduction per block.
#include "kernels.h"
#include "fast_items.cuh"
#include "umma.cuh"

namespace mgn {
namespace {

constexpr int kThreads = 384;
constexpr int BM = 128;      // rows per query tile
constexpr int BN = 128;      // keys per block
constexpr int kStages = 2;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
// A thread's partial row sum (64 columns) above this limit moves the reference points.  Every p stays
// below the limit and the sums of a row below 2^13 times it, so nothing overflows.  With f16
// probabilities the limit is 2^12 (f16 ends at 65504).  With bf16 it is 2^60: bf16 and f32 share the
// exponent range, a softmax is exact for any reference point, and a low limit is expensive -- one row
// in 128 passing it makes the whole tile repeat the pass, which heavy-tailed scores (1 % of the
// inputs scaled by 8 in the decoder sweep) did in most key blocks: forward +50-60 % there.
constexpr float kGrowthLimitF16 = 4096.0f;
constexpr float kGrowthLimitBf16 = 1152921504606846976.0f;   // 2^60

template <int D>
struct Cfg {
    static constexpr int NCH = D / 64;                 // 128-byte chunks per row
    static constexpr int TILE_BYTES = 128 * D * 2;     // a 128-row tile of Q, K or V
    static constexpr int CHUNK_BYTES = 128 * 128;      // one 64-column chunk of a 128-row tile
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = OFF_Q + 2 * TILE_BYTES;
    static constexpr int OFF_V = OFF_K + kStages * TILE_BYTES;
    static constexpr int OFF_OST = OFF_V + kStages * TILE_BYTES;    // output staging, one tile
    static constexpr int OFF_XCHG = OFF_OST + TILE_BYTES;           // [2 halves][128 rows] f32 exchange
    static constexpr int OFF_BAR = OFF_XCHG + 2 * 128 * 4;
    static constexpr int SMEM = OFF_BAR + 256 + 1024;
    static_assert(SMEM <= 232448, "shared memory budget");
    static constexpr uint32_t TM_S = 0, TM_O = 256, TM_COLS = 512;
};

// barrier slots (8 bytes each)
enum { B_Q = 0, B_KFULL = 1, B_KEMPTY = 3, B_VFULL = 5, B_VEMPTY = 7, B_SFULL = 9, B_PFULL = 11, B_OFULL = 13,
       B_QEMPTY = 15, B_OEMPTY = 16, B_COUNT = 18 };

// Work item `it`: query-tile pair and head.  Order 0 (block-major): heaviest tiles of every head
// first, dealt in snake order -- balanced for any item count, but the CTAs running at one time touch
// every head.  Order 1 (head-major): the tile pairs of a head are consecutive, heaviest and lightest
// remaining in turn, and CTA c takes the item pairs c, c+G, ... -- the CTAs running at one time
// share the K, V of a few heads, which then stay in L2.  The launcher chooses (pick_schedule).
struct Item {
    int pair, bh, bhk, row0[2], nblk[2], n_max;
};
// GEN = false is the square multi-head case (Sk == Sq, G == 1): offsets and the head mapping fold away.
template <bool GEN>
__device__ __forceinline__ Item make_item(int it, const Dims& dm, int n_pairs, int tpi, int causal, int order) {
    const int BH = dm.BH;
    const int Sk = GEN ? dm.Sk : dm.Sq, off = GEN ? dm.off : 0;
    Item w;
    if (order == 0) {                          // block-major, heaviest (last) query tiles first
        w.pair = n_pairs - 1 - it / BH;
        w.bh = it % BH;
    } else {                                   // head-major, heaviest / lightest remaining tile pair in turn
        w.bh = it / n_pairs;
        const int j = it % n_pairs;
        w.pair = (j & 1) ? (j >> 1) : n_pairs - 1 - (j >> 1);
    }
    w.bhk = GEN ? (w.bh / dm.H) * (dm.H / dm.G) + (w.bh % dm.H) / dm.G : w.bh;
    const int n_kb = (Sk + BN - 1) / BN;
#pragma unroll
    for (int t = 0; t < 2; ++t) {
        w.row0[t] = (w.pair * tpi + t) * BM;          // tpi = tiles per item: 2, or 1 when items would be too few
        if (t >= tpi || w.row0[t] >= dm.Sq) w.nblk[t] = 0;
        else w.nblk[t] = causal ? min(n_kb, (min(w.row0[t] + BM, dm.Sq) - 1 + off) / BN + 1) : n_kb;
    }
    w.n_max = max(w.nblk[0], w.nblk[1]);
    return w;
}

// F16 = true is the forward of the accelerated policy (paper Section 4.2, table "Arithmetic
// permissions"): operands are IEEE f16 copies of f32 tensors, P is packed as f16, and O leaves as f32
// with plain stores (O32); otherwise operands and O are bf16 and O leaves through TMA (tmO).
template <int D, bool GEN, bool F16>
__global__ void __launch_bounds__(kThreads, 1)
fast_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                float* __restrict__ LSE, float* __restrict__ O32, const Dims dm, int n_pairs, int tpi, int causal, int order,
                float c2, unsigned* status)
{
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = base + C::OFF_Q, sK = base + C::OFF_K, sV = base + C::OFF_V;
    const uint32_t bars = base + C::OFF_BAR;
    const uint32_t tmem_slot = bars + B_COUNT * 8;
    auto bar = [&](int i) { return bars + 8u * i; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (*reinterpret_cast<volatile unsigned*>(status) != 0) return;   // an earlier wait on this device gave up

    const int n_items = n_pairs * dm.BH;
    const int Sq = dm.Sq, Sk = GEN ? dm.Sk : dm.Sq, coff = GEN ? dm.off : 0;
    const int G = static_cast<int>(gridDim.x), cta = static_cast<int>(blockIdx.x);
    const int n_tiers = 2 * ((n_items + 2 * G - 1) / (2 * G));   // upper bound on items per CTA in either order

    if (tid == 0) {
        for (int i = 0; i < B_COUNT; ++i) {
            uint32_t cnt = 1;
            if (i == B_PFULL || i == B_PFULL + 1 || i == B_OEMPTY || i == B_OEMPTY + 1) cnt = 256;
            if ((i >= B_KEMPTY && i < B_KEMPTY + 2) || (i >= B_VEMPTY && i < B_VEMPTY + 2) || i == B_QEMPTY) cnt = 2;
            mbar_init(bar(i), cnt);
        }
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
        {
            int g = 0;                                       // key blocks loaded so far (all items)
            for (int k = 0; k < n_tiers; ++k) {
                const int it = item_index(cta, k, G, n_items, order);
                if (it < 0) break;
                const Item w = make_item<GEN>(it, dm, n_pairs, tpi, causal, order);
                mbar_wait(bar(B_QEMPTY), (k & 1) ^ 1, status);   // both issuers are done with the previous Q tiles
                const int nq = (w.nblk[1] > 0) ? 2 : 1;
                mbar_arrive_expect_tx(bar(B_Q), nq * C::TILE_BYTES);
                for (int t = 0; t < nq; ++t)
#pragma unroll
                    for (int ch = 0; ch < C::NCH; ++ch)
                        tma_load_3d(sQ + t * C::TILE_BYTES + ch * C::CHUNK_BYTES, &tmQ, bar(B_Q), ch * 64, w.row0[t], w.bh);
                for (int n = 0; n < w.n_max; ++n, ++g) {
                    const int st = g & 1;
                    const uint32_t ph = (g >> 1) & 1;
                    mbar_wait(bar(B_KEMPTY + st), ph ^ 1, status);
                    mbar_arrive_expect_tx(bar(B_KFULL + st), C::TILE_BYTES);
#pragma unroll
                    for (int ch = 0; ch < C::NCH; ++ch)
                        tma_load_3d(sK + st * C::TILE_BYTES + ch * C::CHUNK_BYTES, &tmK, bar(B_KFULL + st), ch * 64, n * BN, w.bhk);
                    mbar_wait(bar(B_VEMPTY + st), ph ^ 1, status);
                    mbar_arrive_expect_tx(bar(B_VFULL + st), C::TILE_BYTES);
#pragma unroll
                    for (int ch = 0; ch < C::NCH; ++ch)
                        tma_load_3d(sV + st * C::TILE_BYTES + ch * C::CHUNK_BYTES, &tmV, bar(B_VFULL + st), ch * 64, n * BN, w.bhk);
                }
            }
        }
        } else if ((warp == 1 || warp == 2) && lane == 0) {
        // ------------------------------------------------------------------ MMA issuer of tile t
        {
            const int t = warp - 1;
            constexpr uint32_t idesc_s = F16 ? umma_idesc_f16(BM, BN, false, false) : umma_idesc_bf16(BM, BN, false, false);
            constexpr uint32_t idesc_o = F16 ? umma_idesc_f16(BM, D, false, true) : umma_idesc_bf16(BM, D, false, true);
            // Descriptors are built once; inside the loops only the start-address field moves (the
            // field holds address >> 4 and cannot carry out of its 14 bits within shared memory).
            const uint64_t qd = umma_smem_desc(sQ + t * C::TILE_BYTES, 16, 1024);
            const uint64_t dK0 = umma_smem_desc(sK, 16, 1024);
            const uint64_t dV0 = umma_smem_desc(sV, C::CHUNK_BYTES, 1024);
            const uint32_t tSd = tmem + C::TM_S + t * 128, tOd = tmem + C::TM_O + t * D;
            auto issue_s = [&](int st) {   // S_t = Q_t K(stage st)^T
                const uint64_t kd = dK0 + static_cast<uint64_t>((st * C::TILE_BYTES) >> 4);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint64_t off = static_cast<uint64_t>(((kk >> 2) * C::CHUNK_BYTES + (kk & 3) * 32) >> 4);
                    umma_ss(tSd, qd + off, kd + off, idesc_s, kk > 0);
                }
                umma_commit(bar(B_SFULL + t));
            };
            auto issue_o = [&](int st, uint32_t acc0) {   // O_t (+)= P_t V(stage st)
                const uint64_t vd = dV0 + static_cast<uint64_t>((st * C::TILE_BYTES) >> 4);
#pragma unroll
                for (int kk = 0; kk < BN / 16; ++kk)
                    umma_ts(tOd, tSd + (kk >> 2) * 64 + (kk & 3) * 8, vd + static_cast<uint64_t>((kk * 2048) >> 4), idesc_o,
                            kk > 0 ? 1u : acc0);
            };
            int g = 0;       // key blocks seen so far (all items): stage and phase of the K/V ring
            int cp = 0;      // P_t blocks consumed so far: phase of P_FULL[t]
            int co = 0;      // items in which this tile was active: phase of O_EMPTY[t]
            for (int k = 0; k < n_tiers; ++k) {
                const int it = item_index(cta, k, G, n_items, order);
                if (it < 0) break;
                const Item w = make_item<GEN>(it, dm, n_pairs, tpi, causal, order);
                const int nb = w.nblk[t];
                mbar_wait(bar(B_Q), k & 1, status);
                mbar_wait(bar(B_KFULL + (g & 1)), (g >> 1) & 1, status);
                tc_fence_after();
                if (nb > 0) issue_s(g & 1);
                umma_commit(bar(B_KEMPTY + (g & 1)));
                if (nb <= 1) umma_commit(bar(B_QEMPTY));          // no further S products of this item from this issuer
                if (nb > 0) mbar_wait(bar(B_OEMPTY + t), (co & 1) ^ 1, status);   // the last item's O_t has been read out
                for (int n = 0; n < w.n_max; ++n, ++g) {
                    const int st = g & 1;
                    // Every issuer waits for every block, also the ones its tile does not use: an
                    // issuer that ran ahead could release a ring slot twice in one phase.
                    mbar_wait(bar(B_VFULL + st), (g >> 1) & 1, status);
                    if (n < nb) {
                        mbar_wait(bar(B_PFULL + t), cp & 1, status);
                        ++cp;
                        tc_fence_after();
                        issue_o(st, n > 0);
                        if (n == nb - 1) umma_commit(bar(B_OFULL + t));
                    }
                    umma_commit(bar(B_VEMPTY + st));          // this issuer is done with V(n)
                    if (n + 1 < w.n_max) {
                        mbar_wait(bar(B_KFULL + (st ^ 1)), ((g + 1) >> 1) & 1, status);
                        if (n + 1 < nb) {
                            tc_fence_after();
                            issue_s(st ^ 1);
                            if (n + 2 == nb) umma_commit(bar(B_QEMPTY));   // that was this item's last S product
                        }
                        umma_commit(bar(B_KEMPTY + (st ^ 1)));   // ... and with K(n+1)
                    }
                }
                if (nb > 0) ++co;
            }
        }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ softmax + epilogue
        reg_alloc<200>();
        const int h = (warp - 4) >> 2;                     // which 64 key columns of every block
        const int r = (tid - 128) & 127;                   // row within the tile = tensor-memory lane
        const uint32_t lane_base = static_cast<uint32_t>(r & ~31) << 16;
        const uint32_t xchg = base + C::OFF_XCHG;
        const uint32_t my_x = xchg + (h * 128 + r) * 4, peer_x = xchg + ((h ^ 1) * 128 + r) * 4;
        const uint32_t ost = base + C::OFF_OST;
        int cs[2] = {0, 0};      // S_t blocks consumed so far (all items): phase of S_FULL[t]
        int co[2] = {0, 0};      // items in which tile t was active: phase of O_FULL[t]

        // barrier over the 256 softmax threads with an OR reduction of `pred`
        auto bar_or = [](bool pred) -> bool {
            uint32_t out;
            asm volatile(
                "{\n\t.reg .pred P, Q;\n\tsetp.ne.b32 P, %1, 0;\n\t"
                "barrier.cta.red.or.pred Q, 1, 256, P;\n\tselp.u32 %0, 1, 0, Q;\n\t}"
                : "=r"(out) : "r"(static_cast<uint32_t>(pred)) : "memory");
            return out != 0;
        };

        for (int k = 0; k < n_tiers; ++k) {
        const int it = item_index(cta, k, G, n_items, order);
        if (it < 0) break;
        const Item w = make_item<GEN>(it, dm, n_pairs, tpi, causal, order);
        const int bh = w.bh, n_max = w.n_max;
        const int row0[2] = {w.row0[0], w.row0[1]}, nblk[2] = {w.nblk[0], w.nblk[1]};
        float m_ref[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};

        for (int n = 0; n < n_max; ++n) {
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                if (n >= nblk[t]) continue;
                const uint32_t tS = tmem + lane_base + C::TM_S + t * 128 + 64 * h;   // this thread's 64 score columns
                const uint32_t tO = tmem + lane_base + C::TM_O + t * D + (D / 2) * h;
                const int i = row0[t] + r;
                mbar_wait(bar(B_SFULL + t), (cs[t] + n) & 1, status);
                tc_fence_after();
                const int j0 = n * BN + 64 * h;
                const bool masked = (causal && (j0 + 63 > row0[t] + coff)) || (j0 + 64 > Sk);
                const int jmax = min(Sk - 1, causal ? i + coff : Sk - 1) - j0;   // columns c <= jmax of this half are visible

                if (n == 0) {
                    // first block: the reference point is the row maximum of the scaled scores
                    float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t v[32];
                        tmem_ld32(tS + 32 * c, v);
                        tmem_ld_wait();
                        float x[32];
#pragma unroll
                        for (int e = 0; e < 32; ++e) x[e] = __uint_as_float(v[e]) * c2;
                        if (masked) {
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if (32 * c + e > jmax) x[e] = -INFINITY;
                        }
#pragma unroll
                        for (int e = 0; e < 32; e += 4) {
                            mx0 = fmaxf(mx0, x[e]);
                            mx1 = fmaxf(mx1, x[e + 1]);
                            mx2 = fmaxf(mx2, x[e + 2]);
                            mx3 = fmaxf(mx3, x[e + 3]);
                        }
                    }
                    const float mine = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
                    sts32(my_x, mine);
                    bar_or(false);
                    m_ref[t] = fmaxf(mine, lds32f(peer_x));      // finite: key 0 is visible to every row
                    bar_or(false);                                // exchange buffer may be reused
                }

                // One pass: y = s*c2 - m_ref, p = exp2(y), partial row sum, bf16 pack (kept in
                // registers); two columns per fma / add instruction.  A row that outgrew its reference
                // point shows in its partial sum (every p <= the sum): if any partial sum passes the
                // limit, the rows find their current maxima in a second look at S (still intact: P is
                // written over it only afterwards), move their reference points, rescale O and l, and
                // the pass is redone.  The common case pays no per-element maximum.
                uint32_t pk[32];
                float lsum = 0.f;
                for (int attempt = 0; attempt < 2; ++attempt) {
                    uint64_t la = f2_pack(0.f, 0.f), lb = la;
                    const float neg_m = -m_ref[t];
                    const uint64_t c2x2 = f2_pack(c2, c2), nm2 = f2_pack(neg_m, neg_m);
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t v[32];
                        tmem_ld32(tS + 32 * c, v);
                        tmem_ld_wait();
                        float y[32];
#pragma unroll
                        for (int e = 0; e < 32; e += 2)
                            f2_unpack(f2_fma(f2_pack(__uint_as_float(v[e]), __uint_as_float(v[e + 1])), c2x2, nm2), y[e], y[e + 1]);
                        if (masked) {
#pragma unroll
                            for (int e = 0; e < 32; ++e)
                                if (32 * c + e > jmax) y[e] = -INFINITY;
                        }
#pragma unroll
                        for (int e = 0; e < 32; e += 4) {
                            const float p0 = ex2(y[e]), p1 = ex2(y[e + 1]), p2 = ex2(y[e + 2]), p3 = ex2(y[e + 3]);
                            la = f2_add(la, f2_pack(p0, p1));
                            lb = f2_add(lb, f2_pack(p2, p3));
                            pk[16 * c + e / 2] = F16 ? pack_f16(p0, p1) : pack_bf16(p0, p1);
                            pk[16 * c + e / 2 + 1] = F16 ? pack_f16(p2, p3) : pack_bf16(p2, p3);
                        }
                    }
                    {
                        float a0, a1, a2, a3;
                        f2_unpack(la, a0, a1);
                        f2_unpack(lb, a2, a3);
                        lsum = (a0 + a1) + (a2 + a3);
                    }
                    if (attempt == 1) break;
                    if (!bar_or(!(lsum <= (F16 ? kGrowthLimitF16 : kGrowthLimitBf16)))) break;      // also true for an overflowed (inf / nan) sum
                    // some row grew: every row moves its reference point to its current maximum
                    float ymax = -INFINITY;
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t v[32];
                        tmem_ld32(tS + 32 * c, v);
                        tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (!masked || 32 * c + e <= jmax) ymax = fmaxf(ymax, fmaf(__uint_as_float(v[e]), c2, neg_m));
                    }
                    sts32(my_x, ymax);
                    bar_or(false);
                    const float ym = fmaxf(ymax, lds32f(peer_x));
                    const float m_new = fmaxf(m_ref[t], m_ref[t] + ym);
                    const float alpha = ex2(m_ref[t] - m_new);
                    m_ref[t] = m_new;
                    l[t] *= alpha;
#pragma unroll 1
                    for (int c = 0; c < D / 64; ++c) {
                        uint32_t v[32];
                        tmem_ld32(tO + 32 * c, v);
                        tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) * alpha);
                        tmem_st32(tO + 32 * c, v);
                    }
                    bar_or(false);                                // everyone has read the exchange buffer
                }
                l[t] += lsum;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t u[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) u[e] = pk[16 * c + e];
                    tmem_st16(tS + 16 * c, u);
                }
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(bar(B_PFULL + t));
            }
        }

        // ---- epilogue per tile: O / l -> bf16 -> shared (swizzled like the TMA box) -> TMA store; LSE
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            if (nblk[t] == 0) continue;
            const uint32_t tO = tmem + lane_base + C::TM_O + t * D + (D / 2) * h;
            const int i = row0[t] + r;
            sts32(my_x, l[t]);
            if (!F16 && r == 0 && h == 0) bulk_wait_group_read0();   // the previous store has finished reading the staging tile
            bar_or(false);
            const float lt = l[t] + lds32f(peer_x);
            mbar_wait(bar(B_OFULL + t), co[t] & 1, status);
            tc_fence_after();
            const float inv = 1.0f / lt;
            uint32_t v[D / 64][32];
#pragma unroll
            for (int c = 0; c < D / 64; ++c) tmem_ld32(tO + 32 * c, v[c]);
            tmem_ld_wait();
            tc_fence_before();
            mbar_arrive(bar(B_OEMPTY + t));                    // the next item may overwrite O_t
            if (h == 0 && i < Sq) LSE[static_cast<size_t>(bh) * Sq + i] = (m_ref[t] + log2f(lt)) * kLn2;
            if constexpr (F16) {
                // f32 output: this thread's D/2 contiguous columns of row i, 16-byte stores
                if (i < Sq) {
                    float* orow = O32 + (static_cast<size_t>(bh) * Sq + i) * D + (D / 2) * h;
#pragma unroll
                    for (int c = 0; c < D / 64; ++c)
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            *reinterpret_cast<float4*>(orow + 32 * c + 4 * e) =
                                make_float4(__uint_as_float(v[c][4 * e]) * inv, __uint_as_float(v[c][4 * e + 1]) * inv,
                                            __uint_as_float(v[c][4 * e + 2]) * inv, __uint_as_float(v[c][4 * e + 3]) * inv);
                }
                bar_or(false);                                 // exchange buffer may be reused
            } else {
#pragma unroll
                for (int c = 0; c < D / 64; ++c) {
                    uint32_t u[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                        u[e] = pack_bf16(__uint_as_float(v[c][2 * e]) * inv, __uint_as_float(v[c][2 * e + 1]) * inv);
                    const int col = (D / 2) * h + 32 * c;          // first output column of this chunk
                    const uint32_t rowaddr = ost + (col >> 6) * C::CHUNK_BYTES + r * 128;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int piece = ((col & 63) >> 3) + q;
                        sts128(rowaddr + ((piece ^ (r & 7)) << 4), u[4 * q], u[4 * q + 1], u[4 * q + 2], u[4 * q + 3]);
                    }
                }
                fence_proxy_async_smem();
                bar_or(false);
                if (r == 0 && h == 0) {
#pragma unroll
                    for (int ch = 0; ch < C::NCH; ++ch)
                        tma_store_3d(&tmO, ost + ch * C::CHUNK_BYTES, ch * 64, row0[t], bh);
                    bulk_commit_group();
                }
            }
            ++co[t];
        }
        cs[0] += nblk[0];
        cs[1] += nblk[1];
        }   // items
        if (!F16 && r == 0 && h == 0) bulk_wait_group_read0();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, C::TM_COLS);
}

template <int D, bool GEN, bool F16>
cudaError_t launch_gen(const Problem& p, const void* q, const void* k, const void* v, void* o, float* lse,
                       unsigned* status, cudaStream_t st)
{
    using C = Cfg<D>;
    CUtensorMap tq, tk, tv, to;
    if (make_tmap_3d(&tq, q, 2, 1, p.BH(), p.Sq, p.D, 64, 128)) return MGN_FAIL(cudaErrorInvalidValue, "tensor map q");
    if (make_tmap_3d(&tk, k, 2, 1, p.BHkv(), p.Sk, p.D, 64, 128)) return MGN_FAIL(cudaErrorInvalidValue, "tensor map k");
    if (make_tmap_3d(&tv, v, 2, 1, p.BHkv(), p.Sk, p.D, 64, 128)) return MGN_FAIL(cudaErrorInvalidValue, "tensor map v");
    // with f32 output the kernel stores O itself; the map then only has to be a valid one
    if (make_tmap_3d(&to, F16 ? q : o, 2, 1, p.BH(), p.Sq, p.D, 64, 128)) return MGN_FAIL(cudaErrorInvalidValue, "tensor map o");
    auto kern = fast_fwd_kernel<D, GEN, F16>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
    if (e != cudaSuccess) return MGN_FAIL(e, "cudaFuncSetAttribute");
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return cudaErrorInvalidValue;
    // An item is two query tiles of a head (their softmax and products interleave); with fewer such
    // items than SMs an item is one tile instead, so that twice as many SMs have work.
    const int n_tiles = (p.Sq + BM - 1) / BM;
    const int tpi = (static_cast<long long>((n_tiles + 1) / 2) * p.BH() < sms && n_tiles > 1) ? 1 : 2;
    const int n_pairs = (n_tiles + tpi - 1) / tpi;
    const long long items = static_cast<long long>(n_pairs) * p.BH();
    if (items > 0x7fffffffLL) return cudaErrorInvalidValue;
    const long long blocks = items < sms ? items : sms;       // persistent: one CTA per SM
    const Dims dm{p.Sq, p.Sk, p.BH(), p.H, p.group(), p.off()};
    // streamed per block and shared between the query tiles of a head: K, V
    const int order = pick_schedule(items, sms, static_cast<double>(p.BHkv()) * p.Sk * D * (2 + 2), dev);
    kern<<<static_cast<unsigned>(blocks), kThreads, C::SMEM, st>>>(tq, tk, tv, to, lse, F16 ? static_cast<float*>(o) : nullptr, dm,
                                                                   n_pairs, tpi, p.causal, order,
                                                                   p.scale * kLog2e, status);
    return MGN_FAIL(cudaGetLastError(), "forward launch");
}

template <int D>
cudaError_t launch(const Problem& p, const void* q, const void* k, const void* v, void* o, float* lse,
                   unsigned* status, cudaStream_t st)
{
    return (p.Hkv != p.H || p.Sq != p.Sk) ? launch_gen<D, true, false>(p, q, k, v, o, lse, status, st)
                                          : launch_gen<D, false, false>(p, q, k, v, o, lse, status, st);
}

// f32 -> IEEE f16, round to nearest even (HBM-bound, 8 elements per thread and step)
__global__ void __launch_bounds__(256)
to_f16_kernel(const float4* __restrict__ in, uint4* __restrict__ out, size_t n8)
{
    for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n8;
         i += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const float4 a = in[2 * i], b = in[2 * i + 1];
        out[i] = make_uint4(pack_f16(a.x, a.y), pack_f16(a.z, a.w), pack_f16(b.x, b.y), pack_f16(b.z, b.w));
    }
}

}  // namespace

cudaError_t launch_to_f16(const float* in, void* out, size_t n, cudaStream_t st)
{
    const size_t n8 = n / 8;   // callers pass multiples of D >= 32
    const unsigned blocks = static_cast<unsigned>(n8 / 256 + 1 < 148u * 16u ? n8 / 256 + 1 : 148u * 16u);
    to_f16_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const float4*>(in), static_cast<uint4*>(out), n8);
    return cudaGetLastError();
}

cudaError_t launch_fast_fwd_f16(const Problem& p, const void* q16, const void* k16, const void* v16, float* o,
                                float* lse, unsigned* status, cudaStream_t st)
{
    switch (p.D) {
        case 64:  return launch_gen<64, true, true>(p, q16, k16, v16, o, lse, status, st);
        case 128: return launch_gen<128, true, true>(p, q16, k16, v16, o, lse, status, st);
        default:  return cudaErrorNotSupported;
    }
}

cudaError_t launch_fast_fwd(const Problem& p, const void* q, const void* k, const void* v, void* o, float* lse,
                            unsigned* status, cudaStream_t st)
{
    if (fast_fwd_is_small(p)) return launch_fast_fwd_small(p, q, k, v, o, lse, status, st);
    switch (p.D) {
        // Head size 32 runs the 64-wide build: the tensor maps describe 32-element rows and a
        // 64-element box, so columns 32-63 of every operand tile are zero-filled on load (they add
        // nothing to the scores and give zero output columns) and clipped on store.
        case 32:
        case 64:  return launch<64>(p, q, k, v, o, lse, status, st);
        case 128: return launch<128>(p, q, k, v, o, lse, status, st);
        default:  return cudaErrorNotSupported;
    }
}

}  // namespace mgn
