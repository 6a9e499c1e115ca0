// Fast-mode attention backward: bf16 storage, tcgen05 tensor-core products with f32
// accumulation in tensor memory (paper Section 3.3 "dQ, and fused dK+dV kernels"; Section 7.3
// FlashGradKV / FlashGradQ; Section 4.2 for the reduced-input arithmetic contract).
//
// Single pass, persistent: one CTA per SM walks over work items (one 128-key block of one
// key/value head each; two item orders, see below).  Per item it keeps the K, V tiles resident in
// shared memory, holds the dK and dV accumulators of that block in tensor memory, and walks over
// (query head of the group, 128-row query block) pairs -- from the first block that sees the key block
// when causal.  Every barrier keeps counting across items (g = running pair count, k = running item
// count), so the producer and the issuers start the next item (loads, first S^T and dP^T) while the
// compute warps write out dK/dV.  All score-shaped tiles are computed TRANSPOSED (lanes = keys,
// columns = queries) so that P^T can feed dV = P^T dO straight from tensor memory.  Per pair:
//   MMA1  S^T  = K Q^T            -> X            MMA2  dP^T = V dO^T -> Y
//   compute (256 threads, one key lane x 64 query columns each):
//         P^T = exp2(S^T c - LSE) -> bf16 into X;  dS^T = P^T (dP^T - delta) -> bf16 into shared
//         memory, one buffer whose bytes are at once the K-major operand dS^T (rows = keys) and
//         the MN-major operand dS (rows = queries)
//   MMA4  dV  += P^T dO   (A from tensor memory)
//   MMA5  dK  += dS^T Q   (A from shared memory)
//   MMA6  dQp  = dS K  -> Y, then drained by a dedicated warpgroup: tensor memory -> registers ->
//         a 32 KB shared-memory staging area (f32, swizzled 32-column boxes) -> TMA reduce-add into
//         the f32 dQ accumulator in global memory (a later kernel scales and converts it to bf16).
//         Global f32 reduce-add runs at about 20 bytes per clock per SM on this part (3300 clocks
//         for one 64 KB partial), and issued from the load/store unit it stalls every shared-memory
//         access of the SM; so it goes through TMA and is waited for only by the drain warps.
// Two issuing threads share the tensor core.  Issuer A runs MMA4(n), MMA1(n+1) as soon as P^T(n)
// is in tensor memory (before dS(n) exists), so the next scores are ready when the compute warps
// come back for them; issuer B runs MMA6(n), MMA2(n+1), MMA5(n) once dS(n) is in shared memory
// (the dQ partial first so its drain starts early, dP^T of the next pair as soon as Y has been
// drained, then dK).  Y holds dP^T and then the dQ partial, and all 512 tensor-memory columns are
// taken at D = 128, so each pair runs the serial cycle  dS -> MMA6 -> drain -> MMA2 -> dS.
// Item epilogue: dK (scaled) and dV leave through bf16 registers, the idle dS buffer and coalesced
// 16-byte stores.
// Tensor memory: X [0,128)  Y [128,256)  dK [256,256+D)  dV [256+D,256+2D).
// Warp roles (512 threads): warp 0 TMA producer, warps 1-2 MMA issuers, warp 3 row statistics
// (LSE, delta staged two pairs ahead), warps 4-11 compute, warps 12-15 dQ drain; register budgets
// are rebalanced with setmaxnreg (104 / 128 / 128 / 152).
#include <cuda_bf16.h>

#include "kernels.h"
#include "fast_items.cuh"
#include "umma.cuh"

namespace mgn {
namespace {

constexpr int kThreads = 512;
constexpr int BLK = 128;     // keys per CTA block and query rows per step
constexpr float kLog2e = 1.4426950408889634f;

template <int D>
struct Cfg {
    static constexpr int NCH = D / 64;
    static constexpr int TILE_BYTES = BLK * D * 2;
    static constexpr int CHUNK_BYTES = BLK * 128;
    static constexpr int DS_BYTES = BLK * BLK * 2;
    static constexpr int OFF_K = 0;
    static constexpr int OFF_V = OFF_K + TILE_BYTES;
    static constexpr int OFF_Q = OFF_V + TILE_BYTES;           // two stages
    static constexpr int OFF_DO = OFF_Q + 2 * TILE_BYTES;
    static constexpr int OFF_DS = OFF_DO + TILE_BYTES;
    static constexpr int OFF_DQ = OFF_DS + DS_BYTES;           // dQ staging: 2 boxes of 128 rows x 32 f32
    static constexpr int OFF_STAT = OFF_DQ + 2 * CHUNK_BYTES;  // [2 stages][lse2 | delta][128] f32
    static constexpr int OFF_BAR = OFF_STAT + 2 * 2 * BLK * 4;
    static constexpr int PAYLOAD = OFF_BAR + 224;   // 25 barriers, the tensor-memory slot, four work-item slots
    // Aligning the tile base to 1024 bytes can cost up to 1023 bytes; only 864 are left under the
    // 227 KB per-block limit at D = 128.  The kernel checks the slack it actually got.
    static constexpr int SMEM = (PAYLOAD + 1024 <= 232448) ? PAYLOAD + 1024 : 232448;
    static_assert(SMEM <= 232448, "shared memory budget");
    static constexpr uint32_t TM_X = 0, TM_Y = 128, TM_DK = 256, TM_DV = 256 + D, TM_COLS = 512;
};

enum { B_KV = 0, B_QFULL = 1, B_QEMPTY = 3, B_DOFULL = 5, B_DOEMPTY = 6, B_SFULL = 7, B_DPFULL = 8,
       B_PDSFULL = 9, B_DQFULL = 10, B_DQEMPTY = 11, B_DVFULL = 12, B_DSEMPTY = 13, B_PFULL = 14, B_STATFULL = 15 /* two: one per buffer */,
       B_KVEMPTY = 17, B_DKVEMPTY = 18, B_PDSFULL1 = 19 /* dS of odd pairs; B_PDSFULL: even pairs */, B_DKFULL = 20,
       B_ITEM = 21 /* four: work-item slot k & 3 has been filled */, B_COUNT = 25 };

// Work items are (key block, head), handed out at run time: the producer thread of a CTA takes the
// next position of one global list with an atomic add on a counter in the workspace (cleared by the
// preprocess kernel) and publishes it to the other roles through a four-slot ring in shared memory.
// The list keeps both the load balance of a heaviest-first order and the L2 locality of a
// head-by-head order: heads are taken in groups of Hg whose tensors fit L2 (the f32 dQ accumulator,
// Q, dO, K, V of a group); a group's heavy half (its first key blocks, which see the most query
// blocks under a causal mask) is interleaved with the light half of the group before it, so that
// every stretch of the list holds the same mix of weights, the list starts with heavy items only and
// ends with the lightest ones.  Hg = all heads gives a plain heaviest-first list, Hg = 1 a
// head-by-head one.  Positions whose head does not exist (last group) are skipped.
__device__ __forceinline__ int pos_to_item(unsigned pos, int nb, int BHkv, int Hg) {
    const int nh = nb / 2, nl = nb - nh, ng = (BHkv + Hg - 1) / Hg;
    const unsigned first = static_cast<unsigned>(Hg) * nh, per = static_cast<unsigned>(Hg) * nb;
    int g, kb, c;
    if (pos < first) {                       // phase 0: heavy half of group 0
        g = 0; kb = static_cast<int>(pos) / Hg; c = static_cast<int>(pos) % Hg;
    } else {
        const unsigned q = pos - first;
        const int ph = 1 + static_cast<int>(q / per), rem = static_cast<int>(q % per);
        if (ph >= ng) {                      // last phase: light half of the last group
            if (ph > ng || rem >= Hg * nl) return -1;
            g = ng - 1; kb = nh + rem / Hg; c = rem % Hg;
        } else if (rem < nh * 2 * Hg) {      // rows of Hg heavy items of group ph, then Hg light items of group ph - 1
            const int r = rem / (2 * Hg);
            c = rem % (2 * Hg);
            if (c < Hg) { g = ph; kb = r; } else { g = ph - 1; kb = nh + r; c -= Hg; }
        } else {                             // odd number of blocks: the lightest block of group ph - 1
            g = ph - 1; kb = nb - 1; c = rem - nh * 2 * Hg;
        }
    }
    const int head = g * Hg + c;
    return head < BHkv ? kb * BHkv + head : -2;   // -2: no such head, take the next position
}
// An item is one key block of one key/value head; its pairs run over the query heads of the group
// and, for each, over the query blocks that see the key block.
// GEN = false is the square multi-head case (Sk == Sq, G == 1): the head mapping, the offset and the
// divisions by the number of query blocks fold away.
template <bool GEN>
struct Item {
    int kb, bhk, bhq0, j0, qb0, nq, N;
    __device__ __forceinline__ int bh(int n) const { return GEN ? bhq0 + n / nq : bhq0; }          // query head of pair n
    __device__ __forceinline__ int i0(int n) const { return (qb0 + (GEN ? n % nq : n)) * BLK; }   // first query row of pair n
};
template <bool GEN>
__device__ __forceinline__ Item<GEN> make_item(int it, const Dims& dm, int causal) {
    Item<GEN> w;
    const int Sk = GEN ? dm.Sk : dm.Sq, G = GEN ? dm.G : 1, off = GEN ? dm.off : 0;
    const int nqb = (dm.Sq + BLK - 1) / BLK;
    const int Hkv = dm.H / G, BHkv = dm.BH / G;
    w.kb = it / BHkv;                                     // pos_to_item's encoding
    w.bhk = it % BHkv;
    (void)Sk;
    w.bhq0 = GEN ? (w.bhk / Hkv) * dm.H + (w.bhk % Hkv) * G : w.bhk;
    w.j0 = w.kb * BLK;
    w.qb0 = causal ? max(w.j0 - off, 0) / BLK : 0;       // first query block with a row that sees key j0
    w.nq = nqb - w.qb0;                                   // query blocks visited per head (>= 1)
    w.N = G * w.nq;
    return w;
}

// WITH_DQ = false leaves the dQ partial product, its drain and the global reductions out: the fused
// dK+dV kernel of the deterministic backward, whose dQ comes from the separate pass in fast_dq.cu.
template <int D, bool GEN, bool WITH_DQ>
__global__ void __launch_bounds__(kThreads, 1)
fast_bwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmdO,
                const __grid_constant__ CUtensorMap tmdQ,
                const float* __restrict__ LSE, const float* __restrict__ DELTA,
                __nv_bfloat16* __restrict__ dK, __nv_bfloat16* __restrict__ dV,
                const Dims dm, int causal, int Hg, unsigned* __restrict__ sched, float scale, int Dg,
                __nv_bfloat16* __restrict__ dQ_direct, unsigned* status)
{
    // dQ_direct (non-null only when the problem has a single key block): every (query head, query block)
    // tile then receives exactly one partial, which is the final dQ -- it is scaled, rounded and stored
    // from registers, and no f32 accumulator, clearing pass or conversion pass is needed.
    // Dg: head size in global memory.  Dg = 32 runs the D = 64 build on operand tiles whose columns
    // 32-63 are zero-filled by the tensor maps; only the first 32 columns of dQ, dK, dV are written.
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sK = base + C::OFF_K, sV = base + C::OFF_V, sQ = base + C::OFF_Q, sdO = base + C::OFF_DO;
    const uint32_t sdS = base + C::OFF_DS, sStat = base + C::OFF_STAT, bars = base + C::OFF_BAR;
    const uint32_t tmem_slot = bars + B_COUNT * 8;
    auto bar = [&](int i) { return bars + 8u * i; };
    // dS(g) complete: one barrier per parity of g, so that a waiter two pairs behind cannot alias phases
    auto pds_bar = [&](int g) { return bars + 8u * ((g & 1) ? B_PDSFULL1 : B_PDSFULL); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (*reinterpret_cast<volatile unsigned*>(status) != 0) return;   // an earlier wait on this device gave up
    if (base + C::PAYLOAD > smem_u32(smem_raw) + C::SMEM) {           // alignment slack ran out
        if (tid == 0) atomicMax(status, kStatusSmemLayout);
        return;
    }

    const int Sq = dm.Sq, Sk = GEN ? dm.Sk : dm.Sq, coff = GEN ? dm.off : 0;
    const int n_kb = (Sk + BLK - 1) / BLK, BHkv = dm.BH / (GEN ? dm.G : 1);
    const unsigned n_pos = static_cast<unsigned>((BHkv + Hg - 1) / Hg) * Hg * n_kb;   // list positions, skipped ones included
    const uint32_t item_slot = tmem_slot + 16;
    // Work item k of this CTA (-1: none left).  The producer thread takes it from the global list and
    // publishes it; every other role reads it from slot k & 3.  A slot is rewritten four items later:
    // the producer loads item k only after both issuers have finished item k - 2, and by then every
    // role has read the slots up to k - 2.
    auto take_item = [&](int k) -> int {
        int it = -1;
        for (;;) {
            const unsigned pos = atomicAdd(sched, 1u);
            if (pos >= n_pos) break;
            it = pos_to_item(pos, n_kb, BHkv, Hg);
            if (it != -2) break;
        }
        if (it == -2) it = -1;
        asm volatile("st.shared.u32 [%0], %1;" ::"r"(item_slot + 4u * (k & 3)), "r"(it) : "memory");
        mbar_arrive(bar(B_ITEM + (k & 3)));
        return it;
    };
    auto read_item = [&](int k) -> int {
        if (!mbar_wait(bar(B_ITEM + (k & 3)), (k >> 2) & 1, status)) return -1;
        return static_cast<int>(lds32u(item_slot + 4u * (k & 3)));
    };
    const float c2 = scale * kLog2e;

    if (tid == 0) {
        for (int i = 0; i < B_COUNT; ++i) {
            uint32_t cnt = 1;
            if (i == B_PDSFULL || i == B_PDSFULL1 || i == B_PFULL || i == B_DKVEMPTY) cnt = 256;
            if (i == B_DQEMPTY) cnt = 128;
            if (i == B_STATFULL || i == B_STATFULL + 1) cnt = 32;
            if (i == B_KVEMPTY || i == B_DOEMPTY) cnt = 2;   // one arrival per issuer
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
    // Launched as a programmatic dependent of the preprocess kernel: everything above overlapped its
    // tail; delta, the cleared accumulator and the work-item counter are read only after this wait.
    pdl_launch_dependents();
    pdl_wait();

    if (warp < 4) {
        reg_dealloc<104>();
        if (warp == 0 && lane == 0) {
        // ------------------------------------------------------------------ TMA producer
        {
            int g = 0;                                          // pairs loaded so far (all items)
            for (int k = 0;; ++k) {
                const int it = take_item(k);
                if (it < 0) break;
                const Item<GEN> w = make_item<GEN>(it, dm, causal);
                mbar_wait(bar(B_KVEMPTY), (k & 1) ^ 1, status);  // both issuers are done with the previous K, V
                mbar_arrive_expect_tx(bar(B_KV), 2 * C::TILE_BYTES);
#pragma unroll
                for (int ch = 0; ch < C::NCH; ++ch) {
                    tma_load_3d(sK + ch * C::CHUNK_BYTES, &tmK, bar(B_KV), ch * 64, w.j0, w.bhk);
                    tma_load_3d(sV + ch * C::CHUNK_BYTES, &tmV, bar(B_KV), ch * 64, w.j0, w.bhk);
                }
                for (int n = 0; n < w.N; ++n, ++g) {
                    const int st = g & 1;
                    const int i0 = w.i0(n), bh = w.bh(n);
                    mbar_wait(bar(B_QEMPTY + st), ((g >> 1) & 1) ^ 1, status);
                    mbar_arrive_expect_tx(bar(B_QFULL + st), C::TILE_BYTES);
#pragma unroll
                    for (int ch = 0; ch < C::NCH; ++ch)
                        tma_load_3d(sQ + st * C::TILE_BYTES + ch * C::CHUNK_BYTES, &tmQ, bar(B_QFULL + st), ch * 64, i0, bh);
                    mbar_wait(bar(B_DOEMPTY), (g & 1) ^ 1, status);
                    mbar_arrive_expect_tx(bar(B_DOFULL), C::TILE_BYTES);
#pragma unroll
                    for (int ch = 0; ch < C::NCH; ++ch)
                        tma_load_3d(sdO + ch * C::CHUNK_BYTES, &tmdO, bar(B_DOFULL), ch * 64, i0, bh);
                }
            }
        }
        } else if ((warp == 1 || warp == 2) && lane == 0) {
        // ------------------------------------------------------------------ MMA issuers
        {
            constexpr uint32_t idesc_st = umma_idesc_bf16(BLK, BLK, false, false);   // S^T, dP^T
            constexpr uint32_t idesc_dv = umma_idesc_bf16(BLK, D, false, true);      // A tmem / K-major, B MN-major
            constexpr uint32_t idesc_dq = umma_idesc_bf16(BLK, D, true, true);       // A MN-major, B MN-major
            // Descriptors are built once; inside the loops only the start-address field moves (it
            // holds address >> 4 and cannot carry out of its 14 bits within shared memory).
            auto kmajor_off = [](int kk) { return static_cast<uint64_t>(((kk >> 2) * C::CHUNK_BYTES + (kk & 3) * 32) >> 4); };
            auto mn_off = [](int kk) { return static_cast<uint64_t>((kk * 2048) >> 4); };
            const uint32_t tXa = tmem + C::TM_X, tYa = tmem + C::TM_Y, tDK = tmem + C::TM_DK, tDV = tmem + C::TM_DV;
            if (warp == 1) {
                // ---- issuer A: dV += P^T dO (MMA4), then the next S^T = K Q^T (MMA1) into X
                const uint64_t kK = umma_smem_desc(sK, 16, 1024), kQ = umma_smem_desc(sQ, 16, 1024);
                const uint64_t mdO = umma_smem_desc(sdO, C::CHUNK_BYTES, 1024);
                auto mma1 = [&](int g) {
                    const uint64_t qd = kQ + static_cast<uint64_t>(((g & 1) * C::TILE_BYTES) >> 4);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) umma_ss(tXa, kK + kmajor_off(kk), qd + kmajor_off(kk), idesc_st, kk > 0);
                    umma_commit(bar(B_SFULL));
                };
                int g = 0;
                for (int k = 0;; ++k) {
                    const int it = read_item(k);
                    if (it < 0) break;
                    const Item<GEN> w = make_item<GEN>(it, dm, causal);
                    mbar_wait(bar(B_KV), k & 1, status);
                    mbar_wait(bar(B_QFULL + (g & 1)), (g >> 1) & 1, status);
                    tc_fence_after();
                    mma1(g);             // X: P^T of the previous item was read by its last MMA4 (same issuer)
                    for (int n = 0; n < w.N; ++n, ++g) {
                        // P^T(n) is complete as soon as the exponentials are done, well before dS(n):
                        // dV and the next scores are issued at that point, so S^T(n+1) is waiting when
                        // the compute warps finish dS(n).  The operand tile arrives long before P^T.
                        mbar_wait(bar(B_DOFULL), g & 1, status);
                        mbar_wait(bar(B_PFULL), g & 1, status);
                        if (n == 0) mbar_wait(bar(B_DKVEMPTY), (k & 1) ^ 1, status);   // last item's dV has been read out
                        tc_fence_after();
                        // P^T: queries 0-63 at X[0,32), queries 64-127 at X[64,96)
#pragma unroll
                        for (int kk = 0; kk < BLK / 16; ++kk)
                            umma_ts(tDV, tXa + (kk >> 2) * 64 + (kk & 3) * 8, mdO + mn_off(kk), idesc_dv,
                                    (kk > 0 || n > 0) ? 1u : 0u);
                        umma_commit(bar(B_DOEMPTY));
                        if (n + 1 < w.N) {
                            mbar_wait(bar(B_QFULL + ((g + 1) & 1)), ((g + 1) >> 1) & 1, status);
                            tc_fence_after();
                            mma1(g + 1);      // X is free once MMA4 has read P^T (same issuer: in order)
                        }
                    }
                    umma_commit(bar(B_DVFULL));
                    umma_commit(bar(B_KVEMPTY));      // this issuer's last product with K of this item is done
                }
            } else {
                // ---- issuer B: dQ partial (MMA6), dP^T of the next pair (MMA2), dK (MMA5)
                const uint64_t kV = umma_smem_desc(sV, 16, 1024), kdO = umma_smem_desc(sdO, 16, 1024);
                const uint64_t kdS = umma_smem_desc(sdS, 16, 1024), mdS = umma_smem_desc(sdS, C::CHUNK_BYTES, 1024);
                const uint64_t mK = umma_smem_desc(sK, C::CHUNK_BYTES, 1024), mQ = umma_smem_desc(sQ, C::CHUNK_BYTES, 1024);
                auto mma2 = [&]() {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) umma_ss(tYa, kV + kmajor_off(kk), kdO + kmajor_off(kk), idesc_st, kk > 0);
                    umma_commit(bar(B_DPFULL));
                    umma_commit(bar(B_DOEMPTY));     // with issuer A's arrival after dV: both readers of dO are done
                };
                int g = 0;
                for (int k = 0;; ++k) {
                    const int it = read_item(k);
                    if (it < 0) break;
                    const Item<GEN> w = make_item<GEN>(it, dm, causal);
                    mbar_wait(bar(B_KV), k & 1, status);
                    mbar_wait(bar(B_DOFULL), g & 1, status);
                    if (WITH_DQ && g > 0) mbar_wait(bar(B_DQEMPTY), (g - 1) & 1, status);   // Y: last item's final dQ partial drained
                    tc_fence_after();
                    mma2();
                    for (int n = 0; n < w.N; ++n, ++g) {
                        const uint64_t qm = mQ + static_cast<uint64_t>(((g & 1) * C::TILE_BYTES) >> 4);
                        mbar_wait(pds_bar(g), (g >> 1) & 1, status);
                        tc_fence_after();
                        if constexpr (WITH_DQ) {
#pragma unroll
                            for (int kk = 0; kk < BLK / 16; ++kk) umma_ss(tYa, mdS + mn_off(kk), mK + mn_off(kk), idesc_dq, kk > 0);
                            umma_commit(bar(B_DQFULL));
                        }
                        if (n + 1 < w.N) {
                            mbar_wait(bar(B_DOFULL), (g + 1) & 1, status);
                            if (WITH_DQ) mbar_wait(bar(B_DQEMPTY), g & 1, status);   // Y drained (else: dP^T(n) was consumed before dS(n) completed)
                            tc_fence_after();
                            mma2();
                        }
                        if (n == 0) mbar_wait(bar(B_DKVEMPTY), (k & 1) ^ 1, status);   // last item's dK has been read out
#pragma unroll
                        for (int kk = 0; kk < BLK / 16; ++kk)
                            umma_ss(tDK, kdS + kmajor_off(kk), qm + mn_off(kk), idesc_dv, (kk > 0 || n > 0) ? 1u : 0u);
                        umma_commit(bar(B_QEMPTY + (g & 1)));
                        umma_commit(bar(B_DSEMPTY));                             // dS(n) buffer may be rewritten
                    }
                    umma_commit(bar(B_DKFULL));
                    umma_commit(bar(B_KVEMPTY));
                }
            }
        }
        } else if (warp == 3) {
        // ------------------------------------------------------------------ row statistics
        // Stages the log2-domain LSE and delta of each query block in shared memory, two pairs
        // ahead of the compute warps (across item boundaries), so that they find them there
        // without global loads of their own.  Buffer g&1 may be rewritten once dS(g-2) is complete.
            int g = 0;
            for (int k = 0;; ++k) {
                const int it = read_item(k);
                if (it < 0) break;
                const Item<GEN> w = make_item<GEN>(it, dm, causal);
                for (int n = 0; n < w.N; ++n, ++g) {
                    if (g >= 2) mbar_wait(pds_bar(g), ((g - 2) >> 1) & 1, status);
                    const uint32_t buf = sStat + (g & 1) * (2 * BLK * 4);
                    const int i = w.i0(n) + 4 * lane;                  // rows i..i+3 of the query head
                    const size_t row0 = static_cast<size_t>(w.bh(n)) * Sq;
                    float l2[4], dl[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const bool ok = i + e < Sq;
                        l2[e] = ok ? -LSE[row0 + i + e] * kLog2e : -INFINITY;   // negated: added in the exponent
                        dl[e] = ok ? -DELTA[row0 + i + e] : 0.f;                  // negated: added to dP
                    }
                    sts128(buf + lane * 16, __float_as_uint(l2[0]), __float_as_uint(l2[1]), __float_as_uint(l2[2]),
                           __float_as_uint(l2[3]));
                    sts128(buf + BLK * 4 + lane * 16, __float_as_uint(dl[0]), __float_as_uint(dl[1]),
                           __float_as_uint(dl[2]), __float_as_uint(dl[3]));
                    mbar_arrive(bar(B_STATFULL + (g & 1)));
                }
            }
        }
        __syncwarp();
    } else if (warp >= 12) {
        // ------------------------------------------------------------------ dQ drain warps
        reg_alloc<152>();
        const int r = tid - 384;                           // query row of the block = tensor-memory lane
        const uint32_t tY = tmem + (static_cast<uint32_t>(r & ~31) << 16) + C::TM_Y;
        const uint32_t stage = base + C::OFF_DQ;
        int g = 0;
        for (int k = 0; WITH_DQ; ++k) {
        const int it = read_item(k);
        if (it < 0) break;
        const Item<GEN> w = make_item<GEN>(it, dm, causal);
        for (int n = 0; n < w.N; ++n, ++g) {
            const int i0 = w.i0(n), bh = w.bh(n);
            mbar_wait(bar(B_DQFULL), g & 1, status);
            tc_fence_after();
            uint32_t v[D / 32][32];
#pragma unroll
            for (int c = 0; c < D / 32; ++c) tmem_ld32(tY + 32 * c, v[c]);
            tmem_ld_wait();
            tc_fence_before();
            mbar_arrive(bar(B_DQEMPTY));                   // Y may be overwritten by dP^T of the next pair
            if (dQ_direct != nullptr) {
                if (i0 + r < Sq) {
                    __nv_bfloat16* row = dQ_direct + (static_cast<size_t>(bh) * Sq + i0 + r) * Dg;
#pragma unroll
                    for (int c = 0; c < D / 32; ++c)
                        if (32 * c < Dg) {
                            uint32_t u[16];
#pragma unroll
                            for (int e = 0; e < 16; ++e)
                                u[e] = pack_bf16(__uint_as_float(v[c][2 * e]) * scale, __uint_as_float(v[c][2 * e + 1]) * scale);
#pragma unroll
                            for (int q = 0; q < 4; ++q)
                                *reinterpret_cast<uint4*>(row + 32 * c + 8 * q) = make_uint4(u[4 * q], u[4 * q + 1], u[4 * q + 2], u[4 * q + 3]);
                        }
                }
                continue;
            }
#pragma unroll
            for (int round = 0; round < D / 64; ++round) {
                // the previous reduction must have finished reading the staging area
                if (r == 0) bulk_wait_group_read0();
                named_bar_sync(4, 128);
#pragma unroll
                for (int b = 0; b < 2; ++b)
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        sts128(stage + b * C::CHUNK_BYTES + r * 128 + ((q ^ (r & 7)) << 4), v[2 * round + b][4 * q],
                               v[2 * round + b][4 * q + 1], v[2 * round + b][4 * q + 2], v[2 * round + b][4 * q + 3]);
                fence_proxy_async_smem();
                named_bar_sync(4, 128);
                if (r == 0) {
                    tma_reduce_add_3d(&tmdQ, stage, 64 * round, i0, bh);
                    if (64 * round + 32 < Dg) tma_reduce_add_3d(&tmdQ, stage + C::CHUNK_BYTES, 64 * round + 32, i0, bh);
                    bulk_commit_group();
                }
            }
        }
        }
        if (WITH_DQ && r == 0) bulk_wait_group_read0();
    } else {
        // ------------------------------------------------------------------ compute warps
        reg_alloc<128>();
        const int half = (warp - 4) >> 2;                  // which 64 query columns
        const int r = (tid - 128) & 127;                   // key lane 0..127
        const uint32_t lane_base = static_cast<uint32_t>(r & ~31) << 16;
        const uint32_t tX = tmem + lane_base + C::TM_X, tY = tmem + lane_base + C::TM_Y;

        uint32_t pk[32];                                                     // P^T of the current pair, packed bf16

        // P^T = exp2(S^T c - lse) of pair n: bf16 into X (A operand of dV) and into pk (for dS)
        const uint64_t c2x2 = f2_pack(c2, c2);
        auto exp_phase = [&](const Item<GEN>& w, int n, int g) {
            // key lane r (key j0 + r) is visible to query column c (query i0 + c) iff r <= c + dlt
            const int dlt = w.i0(n) + coff - w.j0;
            const bool diag = causal && dlt < BLK - 1;
            const uint32_t statL = sStat + (g & 1) * (2 * BLK * 4);
            mbar_wait(bar(B_STATFULL + (g & 1)), (g >> 1) & 1, status);
            mbar_wait(bar(B_SFULL), g & 1, status);
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t v[32];
                tmem_ld32(tX + half * 64 + 32 * c, v);
                tmem_ld_wait();
                float p[32];
#pragma unroll
                for (int e4 = 0; e4 < 8; ++e4) {
                    // s c - lse in the log2 domain, two columns per instruction (the buffer holds -lse)
                    const float4 l4 = lds128(statL + (half * 64 + 32 * c + 4 * e4) * 4);
                    float y0, y1, y2, y3;
                    f2_unpack(f2_fma(f2_pack(__uint_as_float(v[4 * e4 + 0]), __uint_as_float(v[4 * e4 + 1])), c2x2,
                                     f2_pack(l4.x, l4.y)), y0, y1);
                    f2_unpack(f2_fma(f2_pack(__uint_as_float(v[4 * e4 + 2]), __uint_as_float(v[4 * e4 + 3])), c2x2,
                                     f2_pack(l4.z, l4.w)), y2, y3);
                    p[4 * e4 + 0] = ex2(y0);
                    p[4 * e4 + 1] = ex2(y1);
                    p[4 * e4 + 2] = ex2(y2);
                    p[4 * e4 + 3] = ex2(y3);
                }
                if (diag) {   // keep key j <= query i, i.e. lane r <= column
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        if (r > half * 64 + 32 * c + e + dlt) p[e] = 0.f;
                }
                uint32_t u[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    u[e] = pack_bf16(p[2 * e], p[2 * e + 1]);
                    pk[16 * c + e] = u[e];
                }
                tmem_st16(tX + half * 64 + 16 * c, u);
            }
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(bar(B_PFULL));
        };

        int g = 0;
        for (int k = 0;; ++k) {
        const int it = read_item(k);
        if (it < 0) break;
        const Item<GEN> w = make_item<GEN>(it, dm, causal);
        exp_phase(w, 0, g);

        for (int n = 0; n < w.N; ++n, ++g) {
            // dS^T = P^T (dP^T - delta) -> bf16 -> shared memory [key][query]
            const uint32_t statD = sStat + (g & 1) * (2 * BLK * 4) + BLK * 4;
            mbar_wait(bar(B_DPFULL), g & 1, status);
            if (g > 0) mbar_wait(bar(B_DSEMPTY), (g - 1) & 1, status);     // dK/dQ products of the last pair are done with dS
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t v[32];
                tmem_ld32(tY + half * 64 + 32 * c, v);
                tmem_ld_wait();
                uint32_t u[16];
#pragma unroll
                for (int e4 = 0; e4 < 8; ++e4) {
                    const float4 d4 = lds128(statD + (half * 64 + 32 * c + 4 * e4) * 4);
                    const uint32_t k0 = pk[16 * c + 2 * e4], k1 = pk[16 * c + 2 * e4 + 1];
                    // P (dP - delta), two columns per instruction (the buffer holds -delta)
                    float a0, a1, a2, a3;
                    f2_unpack(f2_mul(f2_pack(__uint_as_float(k0 << 16), __uint_as_float(k0 & 0xffff0000u)),
                                     f2_add(f2_pack(__uint_as_float(v[4 * e4 + 0]), __uint_as_float(v[4 * e4 + 1])),
                                            f2_pack(d4.x, d4.y))), a0, a1);
                    f2_unpack(f2_mul(f2_pack(__uint_as_float(k1 << 16), __uint_as_float(k1 & 0xffff0000u)),
                                     f2_add(f2_pack(__uint_as_float(v[4 * e4 + 2]), __uint_as_float(v[4 * e4 + 3])),
                                            f2_pack(d4.z, d4.w))), a2, a3);
                    u[2 * e4] = pack_bf16(a0, a1);
                    u[2 * e4 + 1] = pack_bf16(a2, a3);
                }
                const uint32_t rowaddr = sdS + half * C::CHUNK_BYTES + r * 128;
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    sts128(rowaddr + (((4 * c + q) ^ (r & 7)) << 4), u[4 * q], u[4 * q + 1], u[4 * q + 2], u[4 * q + 3]);
            }
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(pds_bar(g));

            // next pair's statistics and exponentials while the dQ/dK products of this pair run
            if (n + 1 < w.N) exp_phase(w, n + 1, g + 1);
        }

        // ---- item epilogue.  Each warpgroup writes D/2 columns of dV, then D/2 columns of dK (scaled):
        // tensor memory -> bf16 registers -> this warpgroup's half of the dS buffer (idle here) ->
        // coalesced 16-byte global stores.  Not a TMA store: it would queue behind the dQ reductions
        // of the last pairs in the copy engine.
        {
            constexpr int HC = D / 2;                      // columns per warpgroup and tensor
            constexpr int PCS = HC / 8;                    // 16-byte pieces per staged row
            const uint32_t stage = sdS + half * C::CHUNK_BYTES;
            auto swz = [](int piece, int row) { return D == 128 ? (piece ^ (row & 7)) : (piece ^ ((row >> 1) & 3)); };
            auto emit = [&](uint32_t tAcc, float mul, __nv_bfloat16* out, bool last) {
                uint32_t u[HC / 2];
#pragma unroll
                for (int c = 0; c < HC / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld32(tAcc + half * HC + 32 * c, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                        u[16 * c + e] = pack_bf16(__uint_as_float(v[2 * e]) * mul, __uint_as_float(v[2 * e + 1]) * mul);
                }
                if (last) {
                    tc_fence_before();
                    mbar_arrive(bar(B_DKVEMPTY));          // the next item may accumulate into dK, dV
                }
#pragma unroll
                for (int q = 0; q < PCS; ++q)
                    sts128(stage + r * (HC * 2) + (swz(q, r) << 4), u[4 * q], u[4 * q + 1], u[4 * q + 2], u[4 * q + 3]);
                named_bar_sync(2 + half, 128);
                out += (static_cast<size_t>(w.bhk) * Sk + w.j0) * Dg + half * HC;
                const bool cols_exist = half * HC < Dg;
                float4 val[PCS];
#pragma unroll
                for (int i = 0; i < PCS; ++i) {
                    const int idx = i * 128 + r, row = idx / PCS, piece = idx % PCS;   // a warp covers whole rows
                    val[i] = lds128(stage + row * (HC * 2) + (swz(piece, row) << 4));
                }
#pragma unroll
                for (int i = 0; i < PCS; ++i) {
                    const int idx = i * 128 + r, row = idx / PCS, piece = idx % PCS;
                    if (cols_exist && w.j0 + row < Sk)
                        *reinterpret_cast<float4*>(out + static_cast<size_t>(row) * Dg + piece * 8) = val[i];
                }
                named_bar_sync(2 + half, 128);             // the slab has been read: the buffer may be rewritten
            };
            // Both accumulators complete: then the last dK and dQ products have also finished reading
            // the dS buffer that the slabs are staged in.
            mbar_wait(bar(B_DVFULL), k & 1, status);
            mbar_wait(bar(B_DKFULL), k & 1, status);
            tc_fence_after();
            emit(tmem + lane_base + C::TM_DV, 1.0f, dV, false);
            emit(tmem + lane_base + C::TM_DK, scale, dK, true);
        }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, C::TM_COLS);
}

// dq = bf16(scale * dq_acc)
__global__ void __launch_bounds__(256)
dq_convert_kernel(const float4* __restrict__ acc, uint2* __restrict__ out, size_t n4, float scale)
{
    pdl_wait();   // programmatic dependent of the main kernel: resident early, reads after it has completed
    constexpr int UNR = 4;     // loads in flight per thread (one at a time ran at half the DRAM rate)
    const size_t step = static_cast<size_t>(gridDim.x) * blockDim.x;
    for (size_t i0 = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i0 < n4; i0 += UNR * step) {
        float4 a[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u)
            if (i0 + u * step < n4) a[u] = acc[i0 + u * step];
#pragma unroll
        for (int u = 0; u < UNR; ++u)
            if (i0 + u * step < n4) {
                uint2 o;
                o.x = pack_bf16(a[u].x * scale, a[u].y * scale);
                o.y = pack_bf16(a[u].z * scale, a[u].w * scale);
                out[i0 + u * step] = o;
            }
    }
}

template <int D, bool GEN, bool WITH_DQ>
cudaError_t launch_gen(const Problem& p, const void* q, const void* k, const void* v, const void* d_o,
                       const float* lse, const float* delta, float* dq_acc, void* dq, void* dk, void* dv,
                       unsigned* sched, unsigned* status, cudaStream_t st)
{
    using C = Cfg<D>;
    CUtensorMap tq, tk, tv, tdo, tdq;
    // without the dQ product the map is never used; it only has to be a valid one
    if (make_tmap_3d(&tdq, WITH_DQ ? static_cast<const void*>(dq_acc) : static_cast<const void*>(delta), 4, 0,
                     WITH_DQ ? p.BH() : 1, WITH_DQ ? p.Sq : 1, WITH_DQ ? p.D : 32, 32, WITH_DQ ? BLK : 1))
        return cudaErrorInvalidValue;
    if (make_tmap_3d(&tq, q, 2, 1, p.BH(), p.Sq, p.D, 64, BLK)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tk, k, 2, 1, p.BHkv(), p.Sk, p.D, 64, BLK)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tv, v, 2, 1, p.BHkv(), p.Sk, p.D, 64, BLK)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tdo, d_o, 2, 1, p.BH(), p.Sq, p.D, 64, BLK)) return cudaErrorInvalidValue;
    auto kern = fast_bwd_kernel<D, GEN, WITH_DQ>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
    if (e != cudaSuccess) return e;
    const int n_kb = (p.Sk + BLK - 1) / BLK;
    const long long items = static_cast<long long>(n_kb) * p.BHkv();
    if (items > 0x7fffffffLL) return cudaErrorInvalidValue;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return cudaErrorInvalidValue;
    const long long blocks = items < sms ? items : sms;       // persistent: one CTA per SM
    // Heads per group of the work-item list: what the items of a group share -- the f32 dQ accumulator,
    // Q and dO of its query heads, K and V -- should stay in L2 while two groups are in flight
    // (measured: half of L2 per group is the best size from 1024 to 8192 tokens).
    int l2 = 0;
    if (cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) != cudaSuccess || l2 <= 0) l2 = 64 << 20;
    const double per_head = static_cast<double>(p.group()) * p.Sq * D * (4 + 2 + 2) + static_cast<double>(p.Sk) * D * 4;
    long long hg = static_cast<long long>(0.5 * l2 / per_head);
    // ... but a group must hold enough items to keep every CTA busy through its phase of the list
    // (measured: 96 long items per group cost a grouped-head decoder shape 10 %)
    const long long hg_min = (3LL * sms / 2 + n_kb - 1) / n_kb;
    if (hg < hg_min) hg = hg_min;
    hg = hg < 1 ? 1 : hg > p.BHkv() ? p.BHkv() : hg;
    const long long n_groups = (p.BHkv() + hg - 1) / hg;
    hg = (p.BHkv() + n_groups - 1) / n_groups;       // equal groups: a short last group unbalances the end of the list
    if (g_forced_item_order == 0) hg = p.BHkv();      // one group: plain heaviest-first list
    if (g_forced_item_order == 1) hg = 1;             // head by head
    const int Hg = static_cast<int>(hg);
    const Dims dm{p.Sq, p.Sk, p.BH(), p.H, p.group(), p.off()};
    const bool direct = WITH_DQ && fast_bwd_writes_dq_directly(p);
    e = launch_pdl(kern, static_cast<unsigned>(blocks), kThreads, C::SMEM, st, tq, tk, tv, tdo, tdq, lse, delta,
                   static_cast<__nv_bfloat16*>(dk), static_cast<__nv_bfloat16*>(dv), dm, p.causal, Hg, sched, p.scale,
                   p.D, direct ? static_cast<__nv_bfloat16*>(dq) : nullptr, status);
    if (e != cudaSuccess || direct) return e;
    e = cudaGetLastError();
    if (e != cudaSuccess || !WITH_DQ) return e;
    const size_t n4 = static_cast<size_t>(p.BH()) * p.Sq * p.D / 4;
    const unsigned cblocks = static_cast<unsigned>(n4 / 256 + 1 < 148u * 16u ? n4 / 256 + 1 : 148u * 16u);
    return launch_pdl(dq_convert_kernel, cblocks, 256, 0, st, reinterpret_cast<const float4*>(dq_acc),
                      reinterpret_cast<uint2*>(dq), n4, p.scale);
}

template <int D>
cudaError_t launch(const Problem& p, const void* q, const void* k, const void* v, const void* d_o,
                   const float* lse, const float* delta, float* dq_acc, void* dq, void* dk, void* dv,
                   unsigned* sched, unsigned* status, cudaStream_t st)
{
    if (dq_acc == nullptr)   // fused dK+dV only (deterministic backward): the general-shape build serves every shape
        return launch_gen<D, true, false>(p, q, k, v, d_o, lse, delta, dq_acc, dq, dk, dv, sched, status, st);
    return (p.Hkv != p.H || p.Sq != p.Sk)
               ? launch_gen<D, true, true>(p, q, k, v, d_o, lse, delta, dq_acc, dq, dk, dv, sched, status, st)
               : launch_gen<D, false, true>(p, q, k, v, d_o, lse, delta, dq_acc, dq, dk, dv, sched, status, st);
}

}  // namespace

cudaError_t launch_fast_bwd(const Problem& p, const void* q, const void* k, const void* v, const void* d_o,
                            const float* lse, const float* delta, float* dq_acc, void* dq, void* dk, void* dv,
                            unsigned* sched, unsigned* status, cudaStream_t st)
{
    switch (p.D) {
        case 32:  // the 64-wide build on zero-filled 32-element rows (see fast_fwd.cu)
        case 64:  return launch<64>(p, q, k, v, d_o, lse, delta, dq_acc, dq, dk, dv, sched, status, st);
        case 128: return launch<128>(p, q, k, v, d_o, lse, delta, dq_acc, dq, dk, dv, sched, status, st);
        default:  return cudaErrorNotSupported;
    }
}

}  // namespace mgn
