// Internal launch interface between the C ABI (api.cu) and the kernel files.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>

#include <stdio.h>
#include <stdlib.h>

namespace mgn {

// Diagnostics, off unless the environment variable MGN_LOG is set: where a launch path gave up.
inline cudaError_t log_fail(cudaError_t e, const char* what, int line) {
    if (e != cudaSuccess && getenv("MGN_LOG")) fprintf(stderr, "mgn_attn: %s failed at line %d: %s\n", what, line, cudaGetErrorString(e));
    return e;
}
#define MGN_FAIL(e, what) ::mgn::log_fail((e), (what), __LINE__)

// q, o, d_o, dq: [B,H,Sq,D]; k, v, dk, dv: [B,Hkv,Sk,D]; query head h reads key/value head
// h / (H/Hkv).  With a causal mask key j is visible to query i iff j <= i + (Sk - Sq)
// (bottom-right aligned; the launchers are only given Sq <= Sk then).
struct Problem {
    int B, H, Hkv, Sq, Sk, D, causal;
    float scale;
    int BH() const { return B * H; }
    int BHkv() const { return B * Hkv; }
    int group() const { return H / Hkv; }
    int off() const { return Sk - Sq; }
};

// Tile pairs x tile area that a (BM-row query tile, BN-key tile) decomposition executes: the padded
// work that picks between tile shapes for short or ragged sequences.
inline double tiled_work(const Problem& p, int BM, int BN) {
    const int n_qt = (p.Sq + BM - 1) / BM, n_kt = (p.Sk + BN - 1) / BN;
    long long pairs = 0;
    for (int qt = 0; qt < n_qt; ++qt) {
        const int i_last = (qt * BM + BM < p.Sq ? qt * BM + BM : p.Sq) - 1;
        const int vis = p.causal ? (i_last + p.off()) / BN + 1 : n_kt;
        pairs += vis < n_kt ? vis : n_kt;
    }
    return static_cast<double>(pairs) * BM * BN;
}
// Tile shapes of the strict kernels (query rows x keys per CTA step).  Short sequences (both lengths
// <= 512) at D = 64 whose padded work under the default tiles exceeds that under the alternative by
// more than a seventh run with the alternative: 197 tokens execute 200 x 224 (forward) and
// 200 x 256 (backward) instead of 256 x 256.
inline bool prefer_alt_tiles(const Problem& p, int BM, int BN, int BM_alt, int BN_alt) {
    if (p.Sq > 512 || p.Sk > 512) return false;
    return tiled_work(p, BM_alt, BN_alt) * 8.0 < tiled_work(p, BM, BN) * 7.0;
}
inline void strict_fwd_tiles(const Problem& p, int* BM, int* BN) {
    *BM = 64;
    *BN = p.D == 128 ? 64 : 128;
    if (p.D == 64 && prefer_alt_tiles(p, 64, 128, 40, 112)) { *BM = 40; *BN = 112; }
}
inline void strict_bwd_tiles(const Problem& p, int* BM, int* BN) {
    *BM = p.D == 128 ? 32 : 64;
    *BN = 64;
    if (p.D == 64 && prefer_alt_tiles(p, 64, 64, 40, 64)) *BM = 40;
}

// Per-device set-up shared by every entry point: checks the architecture of the current device and
// returns the device address of its status word.  Returns an mgn_status code.
int device_status_word(unsigned** status);

// Launches `kern` as a programmatic dependent of the previous kernel on the stream (the kernel must
// call pdl_wait() before it reads that kernel's results).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t st,
                              Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// Tensor maps (host side).  rank-3 view (D, S, BH) of a dense [BH,S,D] tensor with
// a (box_d, box_rows, 1) box and the 128-byte swizzle.  Returns 0 on success.
int make_tmap_3d(CUtensorMap* out, const void* base, int elem_bytes, int is_bf16,
                 int BH, int S, int D, int box_d, int box_rows);

// Strict (f32 FFMA) kernels.
cudaError_t launch_strict_fwd(const Problem& p, const float* q, const float* k, const float* v,
                              float* o, float* lse, unsigned* status, cudaStream_t st);
cudaError_t launch_strict_bwd(const Problem& p, const float* q, const float* k, const float* v,
                              const float* d_o, const float* lse, const float* delta,
                              float* dq, float* dk, float* dv, unsigned* status, cudaStream_t st);

// Deterministic strict backward: launch_strict_bwd with dq == nullptr runs the fused dK+dV kernel
// without the dQ reductions, and this separate pass computes dQ with plain stores.
cudaError_t launch_strict_dq(const Problem& p, const float* q, const float* k, const float* v,
                             const float* d_o, const float* lse, const float* delta, float* dq,
                             unsigned* status, cudaStream_t st);

// delta_i = sum_d dO[i,d] O[i,d]  (f32 or bf16 inputs, f32 output), HBM-bound; also clears the
// f32 dQ accumulation target `zero` ([rows][D] floats) unless it is null.
// `counter` (one unsigned, may be null) is cleared too: the work-item counter of the fast backward.
cudaError_t launch_bwd_preprocess(const void* o, const void* d_o, float* delta, float* zero, unsigned* counter,
                                  size_t rows, int D, int is_bf16, cudaStream_t st);

// The clearing half of the preprocess pass alone (delta supplied by the caller): zeroes `n_floats`
// floats at `zero` (a multiple of four) and the work-item counter (may be null).
cudaError_t launch_bwd_clear(float* zero, size_t n_floats, unsigned* counter, cudaStream_t st);

// Output projection of the concatenated heads (fast mode, bf16): y [B,S,E] = concat_h(o [B,H,S,D]) w [H*D,E];
// and its data gradient d_o [B,H,S,D] = d_y w^T together with delta [B,H,S] = rowsum(d_o o o).
cudaError_t launch_out_proj_fwd(const void* o, const void* w, void* y, int B, int H, int S, int D, int E,
                                unsigned* status, cudaStream_t st);
cudaError_t launch_out_proj_bwd_data(const void* d_y, const void* w, const void* o, void* d_o, float* delta, int B,
                                     int H, int S, int D, int E, unsigned* status, cudaStream_t st);
// d_w [H*D,E] = concat_h(o)^T d_y, contracting over all B*S positions.
cudaError_t launch_out_proj_bwd_weight(const void* o, const void* d_y, void* d_w, int B, int H, int S, int D, int E,
                                       unsigned* status, cudaStream_t st);
// (q | k | v) = x [B,S,E] w^T, w [(H+2Hkv)*D, E] (query heads, key heads, value heads), rotary embedding
// (rotate-half pairing, angle tables cos_t, sin_t [S, D/2] f32) applied to q and k; q [B,H,S,D], k, v [B,Hkv,S,D].
cudaError_t launch_qkv_rope(const void* x, const void* w, const float* cos_t, const float* sin_t, void* q, void* k,
                            void* v, int B, int S, int E, int H, int Hkv, int D, unsigned* status, cudaStream_t st);
// Its backward.  launch_rope_bwd rotates dq [B,H,S,D] and dk [B,Hkv,S,D] in place by the opposite angles (the
// gradient with respect to the unrotated projection); then dx [B,S,E] = (gq | gk | gv)_concat w and
// dw [(H+2Hkv)*D, E] = (gq | gk | gv)_concat^T x, reading the three head-major tensors where they are.
cudaError_t launch_rope_bwd(void* dq, void* dk, const float* cos_t, const float* sin_t, int B, int H, int Hkv, int S,
                            int D, cudaStream_t st);
cudaError_t launch_qkv_bwd_data(const void* gq, const void* gk, const void* gv, const void* w, void* dx, int B, int S,
                                int E, int H, int Hkv, int D, unsigned* status, cudaStream_t st);
cudaError_t launch_qkv_bwd_weight(const void* gq, const void* gk, const void* gv, const void* x, void* dw, int B, int S,
                                  int E, int H, int Hkv, int D, unsigned* status, cudaStream_t st);

// Work-item order of the persistent fast kernels (see the kernels for the two orders).  Head-major
// order (1) is chosen when the data that the items of one head share (`shared_bytes`, over all
// heads) would not stay in L2 under block-major order, and there are enough item pairs per CTA
// for its static assignment to be balanced within 4 %.
extern int g_forced_item_order;   // -1: choose per call (set by mgn_attn_fast_item_order)
inline int pick_schedule(long long n_items, int sms, double shared_bytes, int device) {
    if (g_forced_item_order >= 0) return g_forced_item_order;
    int l2 = 0;
    if (cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, device) != cudaSuccess || l2 <= 0) return 0;
    const double x = static_cast<double>(n_items) / (2.0 * sms);
    if (x < 1.0) return 0;
    const double tiers = static_cast<double>((n_items + 2LL * sms - 1) / (2LL * sms));
    return (shared_bytes > 0.75 * l2 && tiers / x <= 1.04) ? 1 : 0;
}

// Fast (bf16 tcgen05) kernels.
cudaError_t launch_fast_fwd(const Problem& p, const void* q, const void* k, const void* v,
                            void* o, float* lse, unsigned* status, cudaStream_t st);
// The latency path of the forward: at most two 128-key blocks per head (Sk <= 256), one small CTA per
// 128-row query tile, several per SM.  launch_fast_fwd hands such problems to it.
inline bool fast_fwd_is_small(const Problem& p) { return p.Sk <= 256; }
cudaError_t launch_fast_fwd_small(const Problem& p, const void* q, const void* k, const void* v, void* o, float* lse,
                                  unsigned* status, cudaStream_t st);
// Forward of the accelerated policy: q16, k16, v16 are IEEE f16 copies (launch_to_f16) of f32
// tensors, tensor-core products with f32 accumulation, O and LSE stored as f32.
cudaError_t launch_to_f16(const float* in, void* out, size_t n, cudaStream_t st);
cudaError_t launch_fast_fwd_f16(const Problem& p, const void* q16, const void* k16, const void* v16, float* o,
                                float* lse, unsigned* status, cudaStream_t st);
// With a single 128-key block every dQ tile receives one partial: the fused kernel then stores dq itself
// and neither clears nor converts the f32 accumulator (which the caller need not clear either).
inline bool fast_bwd_writes_dq_directly(const Problem& p) { return p.Sk <= 128; }
cudaError_t launch_fast_bwd(const Problem& p, const void* q, const void* k, const void* v,
                            const void* d_o, const float* lse, const float* delta,
                            float* dq_acc, void* dq, void* dk, void* dv,
                            unsigned* sched, unsigned* status, cudaStream_t st);

// Deterministic fast backward: launch_fast_bwd with dq_acc == nullptr runs the fused dK+dV kernel
// without the dQ product and reductions (dq is not touched), and this separate pass computes dQ.
cudaError_t launch_fast_dq(const Problem& p, const void* q, const void* k, const void* v, const void* d_o,
                           const float* lse, const float* delta, void* dq, unsigned* status, cudaStream_t st);

}  // namespace mgn
