// Fast-mode attention forward: bf16 storage, tcgen05 tensor-core products with f32
// accumulation in tensor memory, f32 softmax statistics (paper Section 3.3 "tiled attention
// forward"; Section 4.2: the validated reduced-input path with f32 accumulation).
//
// Persistent kernel: one CTA per SM walks over work items (one 128-row query tile of one head; two
// item orders, see make_item) and, per item, over 128-key blocks of that head's key/value head.
// The score tile is double-buffered in tensor memory and P has columns of its own, so the product
// S(n+2) = Q K(n+2)^T is issued as soon as the softmax warps have READ S(n): the scores of the next
// block are always waiting when a softmax pass ends, and neither product sits on the path between
// two passes.  All barriers and the block counter keep counting across items, so the first scores of
// the next item are computed, and its Q tile loaded, while the current item finishes, and the
// output of an item is written by a warpgroup of its own while the softmax warps start the next one.
// Warp roles (512 threads):
//   warps 0, 2    TMA producers: the Q tile of each item (two stages) and the K blocks; the V blocks (2-stage rings)
//   warps 1, 3    MMA issuers (one lane each): S(g) = Q K(g)^T (operands in shared memory), up to two blocks
//                 ahead; O += P(g) V(g) (P read from tensor memory, V as an MN-major shared-memory operand)
//   warps 4-11    softmax: two threads per row (64 key columns each), one block after the other
//   warps 12-15   epilogue: O / l -> bf16 -> shared memory -> TMA store (f32 build: plain stores), LSE
// Tensor memory (512 columns): S(even blocks) [0,128), S(odd) [128,256), P(even) [256,320),
// P(odd) [320,384), O [384,384+D).  The softmax reference point of a row only moves (and O is rescaled
// in tensor memory) when a row outgrows it so far that a thread's partial sum of exponentials passes
// a limit (2^60; 2^15 with f16 probabilities), which is exact: any reference point works for a
// softmax as long as nothing overflows.  The two threads of a row agree on that through a barrier
// with an OR-reduction per block.
#include "kernels.h"
#include "fast_items.cuh"
#include "umma.cuh"

namespace mgn {
namespace {

constexpr int kThreads = 512;
constexpr int BM = 128;      // rows per query tile
constexpr int BN = 128;      // keys per block
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
// A thread's partial row sum (64 columns) above this limit moves the reference points.  Every p stays
// below the limit and the sums of a row below 2^13 times it, so nothing overflows.  With f16
// probabilities the limit is 2^15 (f16 ends at 65504).  With bf16 it is 2^60: bf16 and f32 share the
// exponent range, a softmax is exact for any reference point, and a low limit is expensive -- one row
// in 128 passing it makes the whole tile repeat the pass, which heavy-tailed scores (1 % of the
// inputs scaled by 8 in the decoder sweep) did in most key blocks: forward +50-60 % there.
constexpr float kGrowthLimitF16 = 32768.0f;
// With f16 probabilities the reference point is set this far (log2 units) above the row maximum, so that a
// row has to outgrow its first maximum by a factor of 2^21 before its pass is repeated; the probabilities
// then start at 2^-6 and keep full f16 precision down to 2^-8 of the row maximum (subnormal below: an
// absolute step of 2^-18 of the maximum).
constexpr float kMarginF16 = 6.0f;
constexpr float kGrowthLimitBf16 = 1152921504606846976.0f;   // 2^60

// 2^x for two values on the FMA pipe instead of the special-function unit (16 results per clock
// and SM there, and a warp cannot issue anything else while it feeds that unit): x is clamped to
// [-127, 126], split as j + f with j = round(x) taken from the low mantissa bits of x + 1.5 * 2^23 and
// f in [-0.5, 0.5], 2^f by a cubic with constant term exactly 1 (maximum relative error 1.0e-4, a
// twentieth of the rounding step of the bf16 result), and j added to the exponent field.
// x = -127 (everything at or below it, -inf included) gives exactly +0.
// Every fourth pair of columns takes this path (long_context forward 0.1332 -> 0.1271 ms; every second
// pair: 0.1291).
constexpr int kPolyMask = 3;   // pairs q with (q & kPolyMask) == kPolyMask
__device__ __forceinline__ void ex2_poly_x2(float x0, float x1, float& p0, float& p1) {
    x0 = fminf(fmaxf(x0, -127.f), 126.f);
    x1 = fminf(fmaxf(x1, -127.f), 126.f);
    const uint64_t x = f2_pack(x0, x1);
    const uint64_t t = f2_add(x, f2_pack(12582912.f, 12582912.f));
    const uint64_t jf = f2_add(t, f2_pack(-12582912.f, -12582912.f));
    const uint64_t f = f2_fma(jf, f2_pack(-1.f, -1.f), x);
    uint64_t r = f2_fma(f, f2_pack(0.05500893f, 0.05500893f), f2_pack(0.24221095f, 0.24221095f));
    r = f2_fma(r, f, f2_pack(0.6932829f, 0.6932829f));
    r = f2_fma(r, f, f2_pack(1.f, 1.f));
    float r0, r1, t0, t1;
    f2_unpack(r, r0, r1);
    f2_unpack(t, t0, t1);
    p0 = __uint_as_float(__float_as_uint(r0) + (__float_as_uint(t0) << 23));
    p1 = __uint_as_float(__float_as_uint(r1) + (__float_as_uint(t1) << 23));
}

template <int D>
struct Cfg {
    static constexpr int NCH = D / 64;                 // 128-byte chunks per row
    static constexpr int TILE_BYTES = 128 * D * 2;     // a 128-row tile of Q, K or V
    static constexpr int CHUNK_BYTES = 128 * 128;      // one 64-column chunk of a 128-row tile
    static constexpr int OFF_Q = 0;                                 // two stages (item parity)
    static constexpr int OFF_K = OFF_Q + 2 * TILE_BYTES;            // two stages (block parity)
    static constexpr int OFF_V = OFF_K + 2 * TILE_BYTES;
    static constexpr int OFF_OST = OFF_V + 2 * TILE_BYTES;          // output staging, one tile
    static constexpr int OFF_XCHG = OFF_OST + TILE_BYTES;           // [2 halves][128 rows] f32 exchange; at item end: l of each half
    static constexpr int OFF_MREF = OFF_XCHG + 2 * 128 * 4;         // [128 rows] f32: reference point of each row at item end
    static constexpr int OFF_BAR = OFF_MREF + 128 * 4;
    static constexpr int SMEM = OFF_BAR + 256 + 1024;
    static_assert(SMEM <= 232448, "shared memory budget");
    static constexpr uint32_t TM_S = 0, TM_P = 256, TM_O = 384, TM_COLS = 512;
};

// barrier slots (8 bytes each); pairs are indexed by the parity of the item (Q) or of the block
//   S_GO[b]   (2 arrivals + bytes)   K(g) has landed AND the product P(g-2) V(g-2) has completed: S(g) may be
//                                    issued -- P(g-2) stored implies S(g-2) read, so the score buffer is free, and
//                                    by the time S(g) is visible its P buffer is free too
//   PV_GO[b]  (257 arrivals + bytes) V(g) has landed AND all 256 softmax threads have stored P(g)
// Every mbarrier operation of an issuing lane costs it 250-350 clocks while the tensor core streams
// operands from shared memory, hence one wait per product.
enum { B_QFULL = 0, B_QEMPTY = 2, B_KEMPTY = 4, B_VEMPTY = 6, B_SFULL = 8, B_SGO = 10, B_PVGO = 12, B_PVDONE = 14,
       B_OFULL = 16, B_OEMPTY = 17, B_STFULL = 18, B_STEMPTY = 19, B_COUNT = 20 };

// Work item `it`: query tile and head.  Order 0 (block-major): heaviest tiles of every head
// first, dealt in snake order -- balanced for any item count, but the CTAs running at one time touch
// every head.  Order 1 (head-major): the tiles of a head are consecutive, heaviest and lightest
// remaining in turn, and CTA c takes the item pairs c, c+G, ... -- the CTAs running at one time
// share the K, V of a few heads, which then stay in L2.  The launcher chooses (pick_schedule).
struct Item {
    int bh, bhk, row0, nblk;
};
// GEN = false is the square multi-head case (Sk == Sq, G == 1): offsets and the head mapping fold away.
template <bool GEN>
__device__ __forceinline__ Item make_item(int it, const Dims& dm, int n_tiles, int causal, int order) {
    const int BH = dm.BH;
    const int Sk = GEN ? dm.Sk : dm.Sq, off = GEN ? dm.off : 0;
    Item w;
    int tile;
    if (order == 0) {                          // block-major, heaviest (last) query tiles first
        tile = n_tiles - 1 - it / BH;
        w.bh = it % BH;
    } else {                                   // head-major, heaviest / lightest remaining tile in turn
        w.bh = it / n_tiles;
        const int j = it % n_tiles;
        tile = (j & 1) ? (j >> 1) : n_tiles - 1 - (j >> 1);
    }
    w.bhk = GEN ? (w.bh / dm.H) * (dm.H / dm.G) + (w.bh % dm.H) / dm.G : w.bh;
    const int n_kb = (Sk + BN - 1) / BN;
    w.row0 = tile * BM;
    w.nblk = causal ? min(n_kb, (min(w.row0 + BM, dm.Sq) - 1 + off) / BN + 1) : n_kb;
    return w;
}

// F16 = true is the forward of the accelerated policy (paper Section 4.2, table "Arithmetic
// permissions"): operands are IEEE f16 copies of f32 tensors, P is packed as f16, and O leaves as f32
// with plain stores (O32); otherwise operands and O are bf16 and O leaves through TMA (tmO).
template <int D, bool GEN, bool F16>
__global__ void __launch_bounds__(kThreads, 1)
fast_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                float* __restrict__ LSE, float* __restrict__ O32, const Dims dm, int n_tiles, int causal, int order,
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

    const int n_items = n_tiles * dm.BH;
    const int Sq = dm.Sq, Sk = GEN ? dm.Sk : dm.Sq, coff = GEN ? dm.off : 0;
    const int G = static_cast<int>(gridDim.x), cta = static_cast<int>(blockIdx.x);
    const int n_tiers = 2 * ((n_items + 2 * G - 1) / (2 * G));   // upper bound on items per CTA in either order

    if (tid == 0) {
        for (int i = 0; i < B_COUNT; ++i) {
            uint32_t cnt = 1;
            if (i == B_STFULL) cnt = 256;
            if (i == B_PVGO || i == B_PVGO + 1) cnt = 257;
            if (i == B_SGO || i == B_SGO + 1) cnt = 2;
            if (i == B_OEMPTY || i == B_STEMPTY) cnt = 128;
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
        reg_dealloc<72>();
        if (warp == 0 && lane == 0) {
        // ------------------------------------------------------------------ TMA producer
        {
            int g = 0;                                       // key blocks loaded so far (all items)
            for (int k = 0; k < n_tiers; ++k) {
                const int it = item_index(cta, k, G, n_items, order);
                if (it < 0) break;
                const Item w = make_item<GEN>(it, dm, n_tiles, causal, order);
                const int qs = k & 1;
                mbar_wait(bar(B_QEMPTY + qs), ((k >> 1) & 1) ^ 1, status);   // the last S product of item k - 2 is done
                mbar_arrive_expect_tx(bar(B_QFULL + qs), C::TILE_BYTES);
#pragma unroll
                for (int ch = 0; ch < C::NCH; ++ch)
                    tma_load_3d(sQ + qs * C::TILE_BYTES + ch * C::CHUNK_BYTES, &tmQ, bar(B_QFULL + qs), ch * 64, w.row0, w.bh);
                for (int n = 0; n < w.nblk; ++n, ++g) {
                    const int st = g & 1;
                    const uint32_t ph = (g >> 1) & 1;
                    mbar_wait(bar(B_KEMPTY + st), ph ^ 1, status);
                    mbar_arrive_expect_tx(bar(B_SGO + st), C::TILE_BYTES);
#pragma unroll
                    for (int ch = 0; ch < C::NCH; ++ch)
                        tma_load_3d(sK + st * C::TILE_BYTES + ch * C::CHUNK_BYTES, &tmK, bar(B_SGO + st), ch * 64, n * BN, w.bhk);
                }
            }
        }
        } else if (warp == 2 && lane == 0) {
        // ------------------------------------------------------------------ TMA producer of V
        // A thread of its own: K(g+2) is wanted half a block before P(g) exists, V(g+2) only once the
        // product with V(g) has completed; one thread loading both in turn would hold K back.
        {
            int g = 0;
            for (int k = 0; k < n_tiers; ++k) {
                const int it = item_index(cta, k, G, n_items, order);
                if (it < 0) break;
                const Item w = make_item<GEN>(it, dm, n_tiles, causal, order);
                for (int n = 0; n < w.nblk; ++n, ++g) {
                    const int st = g & 1;
                    mbar_wait(bar(B_VEMPTY + st), ((g >> 1) & 1) ^ 1, status);
                    mbar_arrive_expect_tx(bar(B_PVGO + st), C::TILE_BYTES);
#pragma unroll
                    for (int ch = 0; ch < C::NCH; ++ch)
                        tma_load_3d(sV + st * C::TILE_BYTES + ch * C::CHUNK_BYTES, &tmV, bar(B_PVGO + st), ch * 64, n * BN, w.bhk);
                }
            }
        }
        } else if ((warp == 1 || warp == 3) && lane == 0) {
        // ------------------------------------------------------------------ MMA issuers
        // Two lanes, each walking over this CTA's blocks (all items in sequence): warp 1 issues the score
        // products, which run up to two blocks ahead of the softmax warps, warp 3 the P V products.
        // Block g uses score buffer, P buffer and K/V stage g & 1.  While one lane sits in a wait the
        // other keeps the tensor core fed.
        {
            constexpr uint32_t idesc_s = F16 ? umma_idesc_f16(BM, BN, false, false) : umma_idesc_bf16(BM, BN, false, false);
            constexpr uint32_t idesc_o = F16 ? umma_idesc_f16(BM, D, false, true) : umma_idesc_bf16(BM, D, false, true);
            // Descriptors are built once; inside the loops only the start-address field moves (the
            // field holds address >> 4 and cannot carry out of its 14 bits within shared memory).
            int g = 0;
            if (warp == 1) {
                const uint64_t dQ0 = umma_smem_desc(sQ, 16, 1024);
                const uint64_t dK0 = umma_smem_desc(sK, 16, 1024);
                mbar_arrive(bar(B_SGO));         // blocks 0 and 1 have no product before them to wait for
                mbar_arrive(bar(B_SGO + 1));
                for (int k = 0; k < n_tiers; ++k) {
                    const int it = item_index(cta, k, G, n_items, order);
                    if (it < 0) break;
                    const int nblk = make_item<GEN>(it, dm, n_tiles, causal, order).nblk;
                    const int qs = k & 1;
                    const uint64_t qd = dQ0 + static_cast<uint64_t>((qs * C::TILE_BYTES) >> 4);
                    mbar_wait(bar(B_QFULL + qs), (k >> 1) & 1, status);
                    for (int n = 0; n < nblk; ++n, ++g) {
                        const int b = g & 1;
                        mbar_wait(bar(B_SGO + b), (g >> 1) & 1, status);
                        tc_fence_after();
                        const uint64_t kd = dK0 + static_cast<uint64_t>((b * C::TILE_BYTES) >> 4);
                        const uint32_t tS = tmem + C::TM_S + b * 128;
#pragma unroll
                        for (int kk = 0; kk < D / 16; ++kk) {
                            const uint64_t off = static_cast<uint64_t>(((kk >> 2) * C::CHUNK_BYTES + (kk & 3) * 32) >> 4);
                            umma_ss(tS, qd + off, kd + off, idesc_s, kk > 0);
                        }
                        umma_commit(bar(B_SFULL + b));
                        umma_commit(bar(B_KEMPTY + b));
                    }
                    umma_commit(bar(B_QEMPTY + qs));      // that was this item's last S product
                }
            } else {
                const uint64_t dV0 = umma_smem_desc(sV, C::CHUNK_BYTES, 1024);
                const uint32_t tO = tmem + C::TM_O;
                for (int k = 0; k < n_tiers; ++k) {
                    const int it = item_index(cta, k, G, n_items, order);
                    if (it < 0) break;
                    const int nblk = make_item<GEN>(it, dm, n_tiles, causal, order).nblk;
                    mbar_wait(bar(B_OEMPTY), (k & 1) ^ 1, status);   // the last item's O has been read out
                    for (int n = 0; n < nblk; ++n, ++g) {
                        const int b = g & 1;
                        mbar_wait(bar(B_PVGO + b), (g >> 1) & 1, status);
                        tc_fence_after();
                        const uint64_t vd = dV0 + static_cast<uint64_t>((b * C::TILE_BYTES) >> 4);
                        const uint32_t tP = tmem + C::TM_P + b * 64;
#pragma unroll
                        for (int kk = 0; kk < BN / 16; ++kk)
                            umma_ts(tO, tP + kk * 8, vd + static_cast<uint64_t>((kk * 2048) >> 4), idesc_o, (kk > 0 || n > 0) ? 1u : 0u);
                        umma_commit(bar(B_SGO + b));          // with K(g+2): S(g+2) may go
                        umma_commit(bar(B_VEMPTY + b));
                        umma_commit(bar(B_PVDONE + b));
                    }
                    umma_commit(bar(B_OFULL));
                }
            }
        }
        }
        __syncwarp();
    } else if (warp >= 12) {
        // ------------------------------------------------------------------ epilogue warpgroup
        // Per item: O / l -> bf16 -> shared (swizzled like the TMA box) -> TMA store; LSE.  The row sums
        // and reference points come from the softmax warps through shared memory.
        reg_dealloc<88>();
        const int r = tid - 384;                           // row within the tile = tensor-memory lane
        const uint32_t tOr = tmem + (static_cast<uint32_t>(r & ~31) << 16) + C::TM_O;
        const uint32_t xchg = base + C::OFF_XCHG, mref = base + C::OFF_MREF;
        const uint32_t ost = base + C::OFF_OST;
        for (int k = 0; k < n_tiers; ++k) {
            const int it = item_index(cta, k, G, n_items, order);
            if (it < 0) break;
            const Item w = make_item<GEN>(it, dm, n_tiles, causal, order);
            const int i = w.row0 + r;
            mbar_wait(bar(B_STFULL), k & 1, status);
            const float lt = lds32f(xchg + r * 4) + lds32f(xchg + (128 + r) * 4);
            const float mr = lds32f(mref + r * 4);
            mbar_arrive(bar(B_STEMPTY));                      // the softmax warps may use the exchange buffer again
            const float inv = 1.0f / lt;
            if (i < Sq) LSE[static_cast<size_t>(w.bh) * Sq + i] = (mr + log2f(lt)) * kLn2;
            if (!F16) {
                if (r == 0) bulk_wait_group_read0();          // the previous store has finished reading the staging tile
                named_bar_sync(5, 128);
            }
            mbar_wait(bar(B_OFULL), k & 1, status);
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t v[32];
                tmem_ld32(tOr + 32 * c, v);
                tmem_ld_wait();
                if (c == D / 32 - 1) {
                    tc_fence_before();
                    mbar_arrive(bar(B_OEMPTY));                // the next item may overwrite O
                }
                if constexpr (F16) {
                    // f32 output: 32 contiguous columns of row i, 16-byte stores
                    if (i < Sq) {
                        float* orow = O32 + (static_cast<size_t>(w.bh) * Sq + i) * D + 32 * c;
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            *reinterpret_cast<float4*>(orow + 4 * e) =
                                make_float4(__uint_as_float(v[4 * e]) * inv, __uint_as_float(v[4 * e + 1]) * inv,
                                            __uint_as_float(v[4 * e + 2]) * inv, __uint_as_float(v[4 * e + 3]) * inv);
                    }
                } else {
                    uint32_t u[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                        u[e] = pack_bf16(__uint_as_float(v[2 * e]) * inv, __uint_as_float(v[2 * e + 1]) * inv);
                    const int col = 32 * c;                        // first output column of this chunk
                    const uint32_t rowaddr = ost + (col >> 6) * C::CHUNK_BYTES + r * 128;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int piece = ((col & 63) >> 3) + q;
                        sts128(rowaddr + ((piece ^ (r & 7)) << 4), u[4 * q], u[4 * q + 1], u[4 * q + 2], u[4 * q + 3]);
                    }
                }
            }
            if (!F16) {
                fence_proxy_async_smem();
                named_bar_sync(5, 128);
                if (r == 0) {
#pragma unroll
                    for (int ch = 0; ch < C::NCH; ++ch)
                        tma_store_3d(&tmO, ost + ch * C::CHUNK_BYTES, ch * 64, w.row0, w.bh);
                    bulk_commit_group();
                }
            }
        }
        if (!F16 && r == 0) bulk_wait_group_read0();
    } else {
        // ------------------------------------------------------------------ softmax warps
        reg_alloc<176>();
        const int h = (warp - 4) >> 2;                     // which 64 key columns of every block
        const int r = (tid - 128) & 127;                   // row within the tile = tensor-memory lane
        const uint32_t lane_base = static_cast<uint32_t>(r & ~31) << 16;
        const uint32_t xchg = base + C::OFF_XCHG;
        const uint32_t my_x = xchg + (h * 128 + r) * 4, peer_x = xchg + ((h ^ 1) * 128 + r) * 4;
        const uint32_t tO = tmem + lane_base + C::TM_O + (D / 2) * h;
        int g = 0;               // blocks seen so far (all items): buffer and phase of S, P

        // Barrier with an OR reduction of `pred` over the two warps that share 32 rows (one per half of the
        // key columns).  Everything the two threads of a row have to agree on is local to these 64
        // threads, so a row that outgrows its reference point makes 32 rows repeat their pass, not 128.
        const uint32_t pair_id = 1 + ((warp - 4) & 3);
        auto bar_or = [pair_id](bool pred) -> bool {
            uint32_t out;
            asm volatile(
                "{\n\t.reg .pred P, Q;\n\tsetp.ne.b32 P, %1, 0;\n\t"
                "barrier.cta.red.or.pred Q, %2, 64, P;\n\tselp.u32 %0, 1, 0, Q;\n\t}"
                : "=r"(out) : "r"(static_cast<uint32_t>(pred)), "r"(pair_id) : "memory");
            return out != 0;
        };

        for (int k = 0; k < n_tiers; ++k) {
        const int it = item_index(cta, k, G, n_items, order);
        if (it < 0) break;
        const Item w = make_item<GEN>(it, dm, n_tiles, causal, order);
        const int i = w.row0 + r;
        float m_ref = -INFINITY, l = 0.f;
        // the exchange buffer carried the row sums of the last item to the epilogue warps
        if (k > 0) mbar_wait(bar(B_STEMPTY), (k - 1) & 1, status);

        for (int n = 0; n < w.nblk; ++n, ++g) {
            const int b = g & 1;
            const uint32_t ph = (g >> 1) & 1;
            const uint32_t tS = tmem + lane_base + C::TM_S + b * 128 + 64 * h;   // this thread's 64 score columns
            const uint32_t tP = tmem + lane_base + C::TM_P + b * 64 + 32 * h;    // ... and where their probabilities go
            mbar_wait(bar(B_SFULL + b), ph, status);
            tc_fence_after();
            const int j0 = n * BN + 64 * h;
            const bool masked = (causal && (j0 + 63 > w.row0 + coff)) || (j0 + 64 > Sk);
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
                m_ref = fmaxf(mine, lds32f(peer_x)) + (F16 ? kMarginF16 : 0.f);      // finite: key 0 is visible to every row
                bar_or(false);                                // exchange buffer may be reused
            }

            // One pass: y = s*c2 - m_ref, p = exp2(y), partial row sum, bf16 pack (kept in
            // registers); two columns per fma / add instruction.  A row that outgrew its reference
            // point shows in its partial sum (every p <= the sum): if any partial sum passes the
            // limit, the rows find their current maxima in a second look at S (still intact), move their
            // reference points, rescale O and l, and the pass is redone.  The common case pays no
            // per-element maximum.
            uint32_t pk[32];
            float lsum = 0.f;
            for (int attempt = 0; attempt < 2; ++attempt) {
                uint64_t la = f2_pack(0.f, 0.f), lb = la;
                const float neg_m = -m_ref;
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
                        float p0, p1, p2, p3;
                        if ((((e >> 1)) & kPolyMask) == kPolyMask) ex2_poly_x2(y[e], y[e + 1], p0, p1);
                        else { p0 = ex2(y[e]); p1 = ex2(y[e + 1]); }
                        if ((((e >> 1) + 1) & kPolyMask) == kPolyMask) ex2_poly_x2(y[e + 2], y[e + 3], p2, p3);
                        else { p2 = ex2(y[e + 2]); p3 = ex2(y[e + 3]); }
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
                const float m_new = fmaxf(m_ref, m_ref + ym + (F16 ? kMarginF16 : 0.f));
                const float alpha = ex2(m_ref - m_new);
                m_ref = m_new;
                l *= alpha;
                if (n > 0) {
                    // O holds the blocks up to n - 1 once the product P(g-1) V(g-1) has completed
                    mbar_wait(bar(B_PVDONE + (b ^ 1)), ((g - 1) >> 1) & 1, status);
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < D / 64; ++c) {
                        uint32_t v[32];
                        tmem_ld32(tO + 32 * c, v);
                        tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(__uint_as_float(v[e]) * alpha);
                        tmem_st32(tO + 32 * c, v);
                    }
                }
                bar_or(false);                                // everyone has read the exchange buffer
            }
            l += lsum;
            // P buffer g & 1 is free: S(g) was issued after the product P(g-2) V(g-2) had completed
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t u[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) u[e] = pk[16 * c + e];
                tmem_st16(tP + 16 * c, u);
            }
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(bar(B_PVGO + b));
        }

        // row sums (one per half) and reference points for the epilogue warps
        sts32(my_x, l);
        if (h == 0) sts32(base + C::OFF_MREF + r * 4, m_ref);
        mbar_arrive(bar(B_STFULL));
        }   // items
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
    const int n_tiles = (p.Sq + BM - 1) / BM;
    const long long items = static_cast<long long>(n_tiles) * p.BH();
    if (items > 0x7fffffffLL) return cudaErrorInvalidValue;
    const long long blocks = items < sms ? items : sms;       // persistent: one CTA per SM
    const Dims dm{p.Sq, p.Sk, p.BH(), p.H, p.group(), p.off()};
    // streamed per block and shared between the query tiles of a head: K, V
    const int order = pick_schedule(items, sms, static_cast<double>(p.BHkv()) * p.Sk * D * (2 + 2), dev);
    kern<<<static_cast<unsigned>(blocks), kThreads, C::SMEM, st>>>(tq, tk, tv, to, lse, F16 ? static_cast<float*>(o) : nullptr, dm,
                                                                   n_tiles, p.causal, order,
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
