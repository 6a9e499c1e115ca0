// The projections either side of attention, fast mode (bf16 operands, tcgen05 products, f32 accumulation).
//
// The paper gives its matrix-product kernels prologues and epilogues that absorb the steps around
// them (Section 3.3, kernel archetypes) and finds that dispatch structure matters where kernels are
// small (Section 7.3).  Four products are written here instead of calling a library GEMM, because each
// absorbs a layout change or a pass that would otherwise be a kernel of its own:
//   QKV  (Q | K | V) = X W^T with the rotary embedding applied to Q and K in the epilogue, written
//        straight into the [B,H,S,D] / [B,Hkv,S,D] layouts the attention kernels read;
//   FWD  Y = O_concat W_o reads O where attention left it ([B,H,S,D], heads separate): the operand tiles
//        are fetched by TMA from the head-major tensor, no concatenated copy of O is made;
//   DO   dO = dY W_o^T writes dO into the [B,H,S,D] layout the attention backward reads, and its
//        epilogue also emits delta = rowsum(dO o O) -- the attention backward's preprocess pass -- while
//        the dO tile is still in registers;
//   DW   dW_o = O_concat^T dY contracts over the positions, again reading O head-major (both operands
//        are fed to the tensor core with the non-contracted index contiguous);
//   DX   dX = (gQ | gK | gV)_concat W_qkv, the data gradient of the QKV projection: like FWD, but the
//        heads of the concatenated operand live in three tensors ([B,H,S,D] and two [B,Hkv,S,D]);
//   DWX  dW_qkv = (gQ | gK | gV)_concat^T X, its weight gradient: like DW with the same three tensors.
// The last two take the gradients with respect to the UNROTATED projection: the rotation depends on the
// position, i.e. on the row of the operand, and cannot be folded into either product; rope_bwd_kernel
// applies the opposite rotation to dQ and dK in place first (a streaming pass over those two tensors).
// Persistent: one CTA per SM walks over 128 x 256 output tiles (tile t, t + grid, ...; neighbouring tiles
// share their row block, so the CTAs running at one time share operand tiles in L2).  Warp 0 streams
// 64-wide contraction slices of both operands through a four-stage TMA ring that keeps running across
// tiles (a lane of warp 6 does the same for the other operand), one lane of warp 1 issues the products
// into one of two 256-column tensor-memory accumulators, warps 2-5 (one thread per accumulator row) read
// the other one out meanwhile.
#include <cuda_bf16.h>

#include "kernels.h"
#include "umma.cuh"

namespace mgn {
namespace {

constexpr int kThreads = 224;
constexpr int TM = 128, TN = 256, TK = 64, kStages = 4;
constexpr int A_BYTES = TM * TK * 2;          // 16 KB
constexpr int B_BYTES = TN * TK * 2;          // 32 KB
constexpr int OFF_A = 0, OFF_B = kStages * A_BYTES, OFF_BAR = OFF_B + kStages * B_BYTES;
constexpr int PAYLOAD = OFF_BAR + 128;
constexpr int SMEM = PAYLOAD + 1024;
enum { B_FULL = 0, B_EMPTY = kStages, B_ACCFULL = 2 * kStages, B_ACCEMPTY = 2 * kStages + 2, B_COUNT = 2 * kStages + 4 };
enum { V_FWD = 0, V_DO = 1, V_DW = 2, V_QKV = 3, V_DX = 4, V_DWX = 5 };

struct ProjArgs {
    __nv_bfloat16* out;          // FWD: y   DO: d_o   DW, DWX: d_w   QKV: q   DX: d_x
    __nv_bfloat16* out_k;        // QKV: k
    __nv_bfloat16* out_v;        // QKV: v
    const __nv_bfloat16* o;      // DO: attention output, for delta
    float* delta;                // DO
    const float* cos_t;          // QKV: [S, D/2]
    const float* sin_t;
    int B, H, Hkv, S, D, E;
};

__device__ __forceinline__ void store_row32(__nv_bfloat16* dst, const uint32_t (&u)[16], int pieces) {
#pragma unroll
    for (int p4 = 0; p4 < 4; ++p4)
        if (p4 < pieces) reinterpret_cast<uint4*>(dst)[p4] = make_uint4(u[4 * p4], u[4 * p4 + 1], u[4 * p4 + 2], u[4 * p4 + 3]);
}

// Epilogue of the plain products: row `row` of the output (global row index), 32 columns starting at n.
template <int V>
__device__ __forceinline__ void epilogue_plain(const ProjArgs& a, const uint32_t (&v)[32], int b, int row, int n, float& dl)
{
    uint32_t u[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) u[e] = pack_bf16(__uint_as_float(v[2 * e]), __uint_as_float(v[2 * e + 1]));
    if constexpr (V == V_DO) {
        const int h = n / a.D, d = n % a.D;
        const size_t off = ((static_cast<size_t>(b) * a.H + h) * a.S + row) * a.D + d;
        store_row32(a.out + off, u, 4);
        const uint4* orow = reinterpret_cast<const uint4*>(a.o + off);
#pragma unroll
        for (int p4 = 0; p4 < 4; ++p4) {
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
        if (d + 32 == a.D) {                  // last chunk of this head
            a.delta[(static_cast<size_t>(b) * a.H + h) * a.S + row] = dl;
            dl = 0.f;
        }
    } else {
        // FWD, DX: y[b, row, n..]   DW, DWX: d_w[row, n..]   (E is a multiple of 8: whole 16-byte pieces)
        const size_t r = (V == V_FWD || V == V_DX) ? static_cast<size_t>(b) * a.S + row : static_cast<size_t>(row);
        store_row32(a.out + r * a.E + n, u, (a.E - n) / 8);
    }
}

// Epilogue of the QKV product: one head (D accumulator columns of this thread's row) at a time --
// rotate the (d, d + D/2) pairs of query and key heads by the caller's angles, round, store.
template <int D>
__device__ __forceinline__ void epilogue_qkv_head(const ProjArgs& a, uint32_t tacc_head, int b, int s, int hh, bool row_ok)
{
    constexpr int NC = D / 32, HALF = D / 2;
    const bool live = row_ok && hh < a.H + 2 * a.Hkv;
    __nv_bfloat16* dst = nullptr;
    if (live) {
        if (hh < a.H) dst = a.out + ((static_cast<size_t>(b) * a.H + hh) * a.S + s) * D;
        else if (hh < a.H + a.Hkv) dst = a.out_k + ((static_cast<size_t>(b) * a.Hkv + (hh - a.H)) * a.S + s) * D;
        else dst = a.out_v + ((static_cast<size_t>(b) * a.Hkv + (hh - a.H - a.Hkv)) * a.S + s) * D;
    }
    const bool rotate = hh < a.H + a.Hkv;
    // 32 columns of the lower half and the 32 columns D/2 further on at a time: the pairs of the rotation
#pragma unroll 1
    for (int c = 0; c < NC / 2; ++c) {
        uint32_t lo[32], hi[32];
        tmem_ld32(tacc_head + 32 * c, lo);                 // whole warp, whatever the row
        tmem_ld32(tacc_head + 32 * (c + NC / 2), hi);
        tmem_ld_wait();
        if (!live) continue;
        if (rotate) {
            const float* ct = a.cos_t + static_cast<size_t>(s) * HALF + 32 * c;
            const float* st = a.sin_t + static_cast<size_t>(s) * HALF + 32 * c;
#pragma unroll
            for (int e4 = 0; e4 < 8; ++e4) {
                const float4 c4 = *reinterpret_cast<const float4*>(ct + 4 * e4);
                const float4 s4 = *reinterpret_cast<const float4*>(st + 4 * e4);
                const float cc[4] = {c4.x, c4.y, c4.z, c4.w}, ss[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const float l = __uint_as_float(lo[4 * e4 + t]), h = __uint_as_float(hi[4 * e4 + t]);
                    lo[4 * e4 + t] = __float_as_uint(l * cc[t] - h * ss[t]);
                    hi[4 * e4 + t] = __float_as_uint(h * cc[t] + l * ss[t]);
                }
            }
        }
        uint32_t u[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) u[e] = pack_bf16(__uint_as_float(lo[2 * e]), __uint_as_float(lo[2 * e + 1]));
        store_row32(dst + 32 * c, u, 4);
#pragma unroll
        for (int e = 0; e < 16; ++e) u[e] = pack_bf16(__uint_as_float(hi[2 * e]), __uint_as_float(hi[2 * e + 1]));
        store_row32(dst + 32 * (c + NC / 2), u, 4);
    }
}

template <int V>
__global__ void __launch_bounds__(kThreads, 1)
proj_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmA2,
            const __grid_constant__ CUtensorMap tmA3, const __grid_constant__ CUtensorMap tmB, const ProjArgs a,
            unsigned* status)
{
    extern __shared__ uint8_t smem_raw[];
    if (*reinterpret_cast<volatile unsigned*>(status) != 0) return;   // an earlier wait on this device gave up
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sA = base + OFF_A, sB = base + OFF_B, bars = base + OFF_BAR;
    const uint32_t tmem_slot = bars + B_COUNT * 8;
    auto bar = [&](int i) { return bars + 8u * i; };
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // tile t: TN output columns from n0; TM rows from r0 (positions s of batch element b, or for DW, DWX rows of d_w)
    const int HD = a.H * a.D, F = (a.H + 2 * a.Hkv) * a.D;             // features: of the heads of O; of query | key | value
    const int n_sc = (a.S + TK - 1) / TK;                              // DW, DWX: 64-position slices per batch element
    const int N = V == V_DO ? HD : V == V_QKV ? F : a.E;
    const int n_kt = V == V_FWD ? HD / TK : V == V_DX ? F / TK : (V == V_DW || V == V_DWX) ? a.B * n_sc : (a.E + TK - 1) / TK;
    const int rows = V == V_DW ? HD : V == V_DWX ? F : a.S;
    // DX, DWX: 64 consecutive features of the concatenation (query | key | value heads) starting at f lie in one
    // head of one of three tensors; `idx` is that head's index in its tensor for batch element bb.  Past the
    // last head the index runs off the value tensor, and the load returns zeros.
    auto head_of = [&](int f, int bb, int& idx) -> const CUtensorMap* {
        const int hh = f / a.D;
        if (hh < a.H) { idx = bb * a.H + hh; return &tmA; }
        if (hh < a.H + a.Hkv) { idx = bb * a.Hkv + hh - a.H; return &tmA2; }
        idx = hh < a.H + 2 * a.Hkv ? bb * a.Hkv + hh - a.H - a.Hkv : a.B * a.Hkv;
        return &tmA3;
    };

    const int tiles_n = (N + TN - 1) / TN, tiles_m = (rows + TM - 1) / TM;
    const int n_tiles = tiles_n * tiles_m * ((V == V_DW || V == V_DWX) ? 1 : a.B);
    const int t0 = static_cast<int>(blockIdx.x), dt = static_cast<int>(gridDim.x);
    auto tile_at = [&](int t, int& n0, int& r0, int& b) {
        n0 = (t % tiles_n) * TN;
        r0 = ((t / tiles_n) % tiles_m) * TM;
        b = t / (tiles_n * tiles_m);
    };

    if (tid == 0) {
        for (int i = 0; i < B_COUNT; ++i)
            mbar_init(bar(i), (i == B_ACCEMPTY || i == B_ACCEMPTY + 1) ? 128 : (i >= B_FULL && i < B_FULL + kStages) ? 2 : 1);
        fence_mbar_init();
    }
    __syncwarp();
    if (warp == 0) tmem_alloc(tmem_slot, 2 * TN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = lds32u(tmem_slot);

    if ((warp == 0 || warp == 6) && lane == 0) {
        // ---------------------------------------------------------------- TMA producers
        // Two lanes, one per operand (warp 0: A, warp 6: B).  A lane's turn per slice is a barrier wait (250-350
        // clocks while the tensor core streams operands from shared memory) plus up to six copy instructions,
        // and the products of a slice take 512 clocks: one lane for both operands was the limit of the
        // variants that fetch their operands in 64-wide blocks.
        const bool opA = warp == 0;
        int g = 0;                                     // slices loaded so far (all tiles): stage and phase of the ring
        for (int t = t0; t < n_tiles; t += dt) {
        int n0, r0, b;
        tile_at(t, n0, r0, b);
        int bb = 0, s0 = 0;                            // DW, DWX: batch element and first position of the slice
        for (int kt = 0; kt < n_kt; ++kt, ++g) {
            const int st = g % kStages, k0 = kt * TK;
            if (g >= kStages) mbar_wait(bar(B_EMPTY + st), ((g / kStages) - 1) & 1, status);
            mbar_arrive_expect_tx(bar(B_FULL + st), opA ? A_BYTES : B_BYTES);
            const uint32_t dA = sA + st * A_BYTES, dB = sB + st * B_BYTES, full = bar(B_FULL + st);
            if constexpr (V == V_DO || V == V_QKV) {
                if (opA) tma_load_3d(dA, &tmA, full, k0, r0, b);                         // 128 positions x 64 e
                else tma_load_3d(dB, &tmB, full, k0, n0, 0);                             // 256 rows n x 64 e
            } else if constexpr (V == V_FWD || V == V_DX) {
                if (opA) {
                    if constexpr (V == V_FWD) {
                        tma_load_3d(dA, &tmA, full, k0 % a.D, r0, b * a.H + k0 / a.D);   // 128 positions x 64 d of one head
                    } else {
                        int idx;
                        const CUtensorMap* m = head_of(k0, b, idx);
                        tma_load_3d(dA, m, full, k0 % a.D, r0, idx);
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < TN / 64; ++c)                                     // four blocks of 64 k rows x 64 n
                        tma_load_3d(dB + c * (TK * 128), &tmB, full, n0 + 64 * c, k0, 0);
                }
            } else {
                if (opA) {
#pragma unroll
                    for (int c = 0; c < TM / 64; ++c) {                                   // two blocks of 64 positions x 64 rows m
                        const int m = r0 + 64 * c;
                        if constexpr (V == V_DW) {
                            tma_load_3d(dA + c * (TK * 128), &tmA, full, m % a.D, s0, bb * a.H + m / a.D);
                        } else {
                            int idx;
                            const CUtensorMap* mp = head_of(m, bb, idx);
                            tma_load_3d(dA + c * (TK * 128), mp, full, m % a.D, s0, idx);
                        }
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < TN / 64; ++c)                                     // four blocks of 64 positions x 64 e
                        tma_load_3d(dB + c * (TK * 128), &tmB, full, n0 + 64 * c, s0, bb);
                }
                s0 += TK;                              // slices run over the positions of batch element 0, then 1, ...
                if (s0 >= n_sc * TK) { s0 = 0; ++bb; }
            }
        }
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------------------------------------------------------- MMA issuer
        constexpr bool A_MN = V == V_DW || V == V_DWX, B_MN = V == V_FWD || V == V_DW || V == V_DX || V == V_DWX;
        constexpr uint32_t idesc = umma_idesc_bf16(TM, TN, A_MN, B_MN);
        const uint64_t dA = A_MN ? umma_smem_desc(sA, TK * 128, 1024) : umma_smem_desc(sA, 16, 1024);
        const uint64_t dB = B_MN ? umma_smem_desc(sB, TK * 128, 1024) : umma_smem_desc(sB, 16, 1024);
        int g = 0, ti = 0;                             // slices and tiles so far
        for (int t = t0; t < n_tiles; t += dt, ++ti) {
            const int acc = ti & 1;
            mbar_wait(bar(B_ACCEMPTY + acc), ((ti >> 1) & 1) ^ 1, status);   // the tile two back has been read out
            tc_fence_after();
            for (int kt = 0; kt < n_kt; ++kt, ++g) {
                const int st = g % kStages;
                mbar_wait(bar(B_FULL + st), (g / kStages) & 1, status);
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < TK / 16; ++kk) {
                    const uint64_t da = dA + static_cast<uint64_t>((st * A_BYTES + (A_MN ? kk * 2048 : kk * 32)) >> 4);
                    const uint64_t db = dB + static_cast<uint64_t>((st * B_BYTES + (B_MN ? kk * 2048 : kk * 32)) >> 4);
                    umma_ss(tmem + acc * TN, da, db, idesc, (kt > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(bar(B_EMPTY + st));
            }
            umma_commit(bar(B_ACCFULL + acc));
        }
    } else if (warp >= 2 && warp < 6) {
        // ---------------------------------------------------------------- epilogue: one thread per row
        const int q4 = warp & 3, r = 32 * q4 + lane;
        int ti = 0;
        for (int t = t0; t < n_tiles; t += dt, ++ti) {
        int n0, r0, b;
        tile_at(t, n0, r0, b);
        const int row = r0 + r, acc = ti & 1;
        const uint32_t tacc = tmem + (static_cast<uint32_t>(32 * q4) << 16) + acc * TN;
        mbar_wait(bar(B_ACCFULL + acc), (ti >> 1) & 1, status);
        tc_fence_after();
        if constexpr (V == V_QKV) {
            if (a.D == 128) {
#pragma unroll 1
                for (int hh = 0; hh < TN / 128; ++hh) epilogue_qkv_head<128>(a, tacc + 128 * hh, b, row, n0 / 128 + hh, row < rows);
            } else {
#pragma unroll 1
                for (int hh = 0; hh < TN / 64; ++hh) epilogue_qkv_head<64>(a, tacc + 64 * hh, b, row, n0 / 64 + hh, row < rows);
            }
        } else {
            float dl = 0.f;
#pragma unroll 1
            for (int c = 0; c < TN / 32; ++c) {
                uint32_t v[32];
                tmem_ld32(tacc + 32 * c, v);          // whole warp, whatever the row
                tmem_ld_wait();
                const int n = n0 + 32 * c;
                if (row < rows && n < N) epilogue_plain<V>(a, v, b, row, n, dl);
            }
        }
        tc_fence_before();
        mbar_arrive(bar(B_ACCEMPTY + acc));             // this accumulator may be overwritten
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 2 * TN);
}

template <int V>
cudaError_t launch3(const CUtensorMap& ta, const CUtensorMap& ta2, const CUtensorMap& ta3, const CUtensorMap& tb,
                    const ProjArgs& a, unsigned* status, cudaStream_t st)
{
    auto kern = proj_kernel<V>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
    if (e != cudaSuccess) return e;
    const int F = (a.H + 2 * a.Hkv) * a.D;
    const int N = V == V_DO ? a.H * a.D : V == V_QKV ? F : a.E;
    const int rows = V == V_DW ? a.H * a.D : V == V_DWX ? F : a.S;
    const long long tiles = static_cast<long long>((N + TN - 1) / TN) * ((rows + TM - 1) / TM) *
                            ((V == V_DW || V == V_DWX) ? 1 : a.B);
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        sms <= 0 || tiles > 0x7fffffffLL)
        return cudaErrorInvalidValue;
    const unsigned grid = static_cast<unsigned>(tiles < sms ? tiles : sms);     // persistent: one CTA per SM
    kern<<<grid, kThreads, SMEM, st>>>(ta, ta2, ta3, tb, a, status);
    return cudaGetLastError();
}
template <int V>
cudaError_t launch(const CUtensorMap& ta, const CUtensorMap& tb, const ProjArgs& a, unsigned* status, cudaStream_t st)
{
    return launch3<V>(ta, ta, ta, tb, a, status, st);
}

// Rotation of the (d, d + D/2) pairs of every row of t [rows_bh * S, D] by the OPPOSITE of the angles in
// cos_t, sin_t [S, D/2], in place: the gradient of the rotary embedding.  Eight pairs per thread and step.
__global__ void __launch_bounds__(256)
rope_bwd_kernel(__nv_bfloat16* __restrict__ t, const float* __restrict__ cos_t, const float* __restrict__ sin_t,
                size_t n_rows, int S, int D)
{
    const int half = D / 2, per_row = half / 8;
    const size_t total = n_rows * per_row;
    for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const size_t row = i / per_row;
        const int d0 = static_cast<int>(i % per_row) * 8, s = static_cast<int>(row % S);
        uint4* plo = reinterpret_cast<uint4*>(t + row * D + d0);
        uint4* phi = reinterpret_cast<uint4*>(t + row * D + half + d0);
        const uint4 lo4 = *plo, hi4 = *phi;
        const float4 ca = *reinterpret_cast<const float4*>(cos_t + static_cast<size_t>(s) * half + d0);
        const float4 cb = *reinterpret_cast<const float4*>(cos_t + static_cast<size_t>(s) * half + d0 + 4);
        const float4 sa = *reinterpret_cast<const float4*>(sin_t + static_cast<size_t>(s) * half + d0);
        const float4 sb = *reinterpret_cast<const float4*>(sin_t + static_cast<size_t>(s) * half + d0 + 4);
        const float cc[8] = {ca.x, ca.y, ca.z, ca.w, cb.x, cb.y, cb.z, cb.w};
        const float ss[8] = {sa.x, sa.y, sa.z, sa.w, sb.x, sb.y, sb.z, sb.w};
        const uint32_t lw[4] = {lo4.x, lo4.y, lo4.z, lo4.w}, hw[4] = {hi4.x, hi4.y, hi4.z, hi4.w};
        uint32_t lo_out[4], hi_out[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float l0 = __uint_as_float(lw[j] << 16), l1 = __uint_as_float(lw[j] & 0xffff0000u);
            const float h0 = __uint_as_float(hw[j] << 16), h1 = __uint_as_float(hw[j] & 0xffff0000u);
            lo_out[j] = pack_bf16(l0 * cc[2 * j] + h0 * ss[2 * j], l1 * cc[2 * j + 1] + h1 * ss[2 * j + 1]);
            hi_out[j] = pack_bf16(h0 * cc[2 * j] - l0 * ss[2 * j], h1 * cc[2 * j + 1] - l1 * ss[2 * j + 1]);
        }
        *plo = make_uint4(lo_out[0], lo_out[1], lo_out[2], lo_out[3]);
        *phi = make_uint4(hi_out[0], hi_out[1], hi_out[2], hi_out[3]);
    }
}

}  // namespace

cudaError_t launch_out_proj_fwd(const void* o, const void* w, void* y, int B, int H, int S, int D, int E,
                                unsigned* status, cudaStream_t st)
{
    CUtensorMap ta, tb;
    if (make_tmap_3d(&ta, o, 2, 1, B * H, S, D, 64, TM)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tb, w, 2, 1, 1, H * D, E, 64, TK)) return cudaErrorInvalidValue;
    ProjArgs a{static_cast<__nv_bfloat16*>(y), nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, B, H, H, S, D, E};
    return launch<V_FWD>(ta, tb, a, status, st);
}

cudaError_t launch_out_proj_bwd_data(const void* d_y, const void* w, const void* o, void* d_o, float* delta, int B,
                                     int H, int S, int D, int E, unsigned* status, cudaStream_t st)
{
    CUtensorMap ta, tb;
    if (make_tmap_3d(&ta, d_y, 2, 1, B, S, E, 64, TM)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tb, w, 2, 1, 1, H * D, E, 64, TN)) return cudaErrorInvalidValue;
    ProjArgs a{static_cast<__nv_bfloat16*>(d_o), nullptr, nullptr, static_cast<const __nv_bfloat16*>(o), delta, nullptr,
               nullptr, B, H, H, S, D, E};
    return launch<V_DO>(ta, tb, a, status, st);
}

cudaError_t launch_out_proj_bwd_weight(const void* o, const void* d_y, void* d_w, int B, int H, int S, int D, int E,
                                       unsigned* status, cudaStream_t st)
{
    CUtensorMap ta, tb;
    if (make_tmap_3d(&ta, o, 2, 1, B * H, S, D, 64, TK)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tb, d_y, 2, 1, B, S, E, 64, TK)) return cudaErrorInvalidValue;
    ProjArgs a{static_cast<__nv_bfloat16*>(d_w), nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, B, H, H, S, D, E};
    return launch<V_DW>(ta, tb, a, status, st);
}

cudaError_t launch_qkv_rope(const void* x, const void* w, const float* cos_t, const float* sin_t, void* q, void* k,
                            void* v, int B, int S, int E, int H, int Hkv, int D, unsigned* status, cudaStream_t st)
{
    CUtensorMap ta, tb;
    if (make_tmap_3d(&ta, x, 2, 1, B, S, E, 64, TM)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tb, w, 2, 1, 1, (H + 2 * Hkv) * D, E, 64, TN)) return cudaErrorInvalidValue;
    ProjArgs a{static_cast<__nv_bfloat16*>(q), static_cast<__nv_bfloat16*>(k), static_cast<__nv_bfloat16*>(v), nullptr,
               nullptr, cos_t, sin_t, B, H, Hkv, S, D, E};
    return launch<V_QKV>(ta, tb, a, status, st);
}

cudaError_t launch_rope_bwd(void* dq, void* dk, const float* cos_t, const float* sin_t, int B, int H, int Hkv, int S,
                            int D, cudaStream_t st)
{
    void* ts[2] = {dq, dk};
    const int hs[2] = {H, Hkv};
    for (int i = 0; i < 2; ++i) {
        const size_t n_rows = static_cast<size_t>(B) * hs[i] * S, total = n_rows * (D / 16);
        const unsigned blocks = static_cast<unsigned>(total / 256 + 1 < 148u * 16u ? total / 256 + 1 : 148u * 16u);
        rope_bwd_kernel<<<blocks, 256, 0, st>>>(static_cast<__nv_bfloat16*>(ts[i]), cos_t, sin_t, n_rows, S, D);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_qkv_bwd_data(const void* gq, const void* gk, const void* gv, const void* w, void* dx, int B, int S,
                                int E, int H, int Hkv, int D, unsigned* status, cudaStream_t st)
{
    CUtensorMap ta, ta2, ta3, tb;
    if (make_tmap_3d(&ta, gq, 2, 1, B * H, S, D, 64, TM)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&ta2, gk, 2, 1, B * Hkv, S, D, 64, TM)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&ta3, gv, 2, 1, B * Hkv, S, D, 64, TM)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tb, w, 2, 1, 1, (H + 2 * Hkv) * D, E, 64, TK)) return cudaErrorInvalidValue;
    ProjArgs a{static_cast<__nv_bfloat16*>(dx), nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, B, H, Hkv, S, D, E};
    return launch3<V_DX>(ta, ta2, ta3, tb, a, status, st);
}

cudaError_t launch_qkv_bwd_weight(const void* gq, const void* gk, const void* gv, const void* x, void* dw, int B, int S,
                                  int E, int H, int Hkv, int D, unsigned* status, cudaStream_t st)
{
    CUtensorMap ta, ta2, ta3, tb;
    if (make_tmap_3d(&ta, gq, 2, 1, B * H, S, D, 64, TK)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&ta2, gk, 2, 1, B * Hkv, S, D, 64, TK)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&ta3, gv, 2, 1, B * Hkv, S, D, 64, TK)) return cudaErrorInvalidValue;
    if (make_tmap_3d(&tb, x, 2, 1, B, S, E, 64, TK)) return cudaErrorInvalidValue;
    ProjArgs a{static_cast<__nv_bfloat16*>(dw), nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, B, H, Hkv, S, D, E};
    return launch3<V_DWX>(ta, ta2, ta3, tb, a, status, st);
}

}  // namespace mgn
