/*
 * mgn_attn.h -- C ABI of the B200 (sm_100a) scaled-dot-product attention library.
 *
 * The operations are the attention kernels the paper lists as one of its kernel
 * archetypes (Section 3.3: "tiled attention forward, dQ, and fused dK+dV kernels")
 * and profiles in Section 7.3 (FlashGradKV / FlashGradQ).  The two numerical modes
 * mirror the paper's arithmetic contracts (Section 4.2, Table "Arithmetic
 * permissions"): a strict f32 path and a validated reduced-input fast path with
 * f32 accumulation.
 *
 * Conventions shared by every entry point
 *   - All tensor pointers are DEVICE pointers on the current CUDA device.
 *   - q, k, v, o, d_o, dq, dk, dv are dense row-major [B,H,S,D], D innermost, no
 *     padding.  Element type: MGN_MODE_STRICT_F32 -> IEEE binary32,
 *     MGN_MODE_FAST_BF16 -> bfloat16.  lse is [B,H,S] binary32 in both modes.
 *   - Every tensor pointer must be 16-byte aligned.  D must be 32, 64 or 128 (in fast mode
 *     D = 32 runs as a zero-padded 64-wide problem: correct, at the cost of D = 64).
 *   - The caller owns every buffer.  The library allocates no device memory.
 *   - Calls only enqueue work on `stream` (a cudaStream_t passed as void*; NULL is
 *     the legacy default stream) and return without synchronising.  Inputs must
 *     stay valid, and outputs untouched, until the stream has passed the call.
 *   - Outputs need not be initialised.  Outputs must not alias inputs or each other.
 *   - Errors are reported by return code only (mgn_status); nothing aborts, and nothing is
 *     printed unless the environment variable MGN_LOG is set (then a launch path that
 *     gives up says on stderr where and with which CUDA error).  Argument errors are detected before any launch, in the
 *     order INVALID_ARG, UNSUPPORTED, MISALIGNED, WORKSPACE, ARCH.
 *   - Device status word.  Every wait inside a kernel is bounded; a wait that runs out
 *     sets one status word PER DEVICE (not per stream, not per call).  While that word is
 *     non-zero every later attention kernel of this library on that device -- forward,
 *     backward, dQ pass, on any stream -- returns at once WITHOUT WRITING ITS OUTPUTS (o, lse,
 *     dq, dk, dv of such calls are unwritten or partial), and the entry points still return
 *     MGN_OK (they only enqueue).  Only mgn_attn_check() reads and clears the word.  A
 *     caller that must know that its results are valid calls mgn_attn_check(stream)
 *     after the calls it cares about; MGN_OK from it means that no kernel of this library
 *     that has completed on the device so far gave up.  Because the word is shared, a time-out
 *     cannot be attributed to one call, and a check on one stream also clears a flag raised
 *     by another stream's kernel.
 *   - Threads.  Distinct host threads may call the attention entry points concurrently on
 *     distinct streams.  mgn_attn_profile_events() and mgn_attn_fast_item_order() change
 *     process-wide settings that those calls read without synchronisation: use them only
 *     while no other thread is inside the library.
 */
#ifndef MGN_ATTN_H
#define MGN_ATTN_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MGN_OK = 0,
    MGN_ERR_INVALID_ARG = 1,    /* null pointer, non-positive dim, causal not 0/1, non-finite scale, unknown mode */
    MGN_ERR_UNSUPPORTED = 2,    /* D not in {32,64,128}, or sizes beyond the index plan */
    MGN_ERR_MISALIGNED = 3,     /* a tensor pointer is not 16-byte aligned */
    MGN_ERR_WORKSPACE = 4,      /* workspace null or too small */
    MGN_ERR_CUDA = 5,           /* a CUDA runtime/driver call failed */
    MGN_ERR_ARCH = 6,           /* current device is not compute capability 10.x */
    MGN_ERR_DEVICE_TIMEOUT = 7  /* a bounded wait inside a kernel gave up (see mgn_attn_check) */
} mgn_status;

enum { MGN_MODE_STRICT_F32 = 0, MGN_MODE_FAST_BF16 = 1 };

/*
 * Attention forward (paper Section 3.3, "tiled attention forward").
 *   s_ij = scale * sum_d q[i,d] k[j,d];  causal != 0 keeps only j <= i;
 *   lse_i = log sum_j exp(s_ij)  (natural log, of the scaled and masked scores);
 *   o_i   = sum_j exp(s_ij - lse_i) v_j.
 * q,k,v: in.  o: out [B,H,S,D] (mode's element type).  lse: out [B,H,S] f32.
 * Strict mode computes in f32 FFMA; fast mode multiplies bf16 operands on the
 * tensor cores with f32 accumulation and f32 softmax statistics.
 * Range (fast mode): a row's running softmax reference may stay up to 2^60 below the
 * largest score seen so far, so the unnormalised sums reach 2^60 * S_k * max|v|; they
 * are f32.  Finite results need max|v| * S_k below about 2^60 (1e18), far beyond
 * any activation; inside that range o and lse do not depend on the lag.
 */
int mgn_attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
                 int B, int H, int S, int D, int causal, float scale, int mode, void* stream);

/*
 * Attention backward (paper Section 3.3 "dQ, and fused dK+dV kernels"; Section 7.3).
 * Given q,k,v, the forward's o and lse (of the same mode), and d_o = dLoss/do:
 *   delta_i = sum_d d_o[i,d] o[i,d];   p_ij = exp(s_ij - lse_i);
 *   dv_j = sum_i p_ij d_o_i;           dp_ij = sum_d d_o[i,d] v[j,d];
 *   ds_ij = p_ij (dp_ij - delta_i);
 *   dq_i = scale sum_j ds_ij k_j;      dk_j = scale sum_i ds_ij q_i.
 * dq, dk, dv: out.  workspace: device scratch of at least
 * mgn_attn_bwd_workspace_bytes(...) bytes, 256-byte aligned, contents ignored on
 * entry and undefined on exit; two calls that may overlap on the GPU need
 * distinct workspaces.  dq is accumulated with floating-point atomics, so its
 * low-order bits can differ from run to run; dk, dv, and the forward are
 * deterministic.
 */
int mgn_attn_bwd(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                 const float* lse, void* dq, void* dk, void* dv,
                 void* workspace, size_t workspace_bytes,
                 int B, int H, int S, int D, int causal, float scale, int mode, void* stream);

/* Bytes of workspace mgn_attn_bwd needs for these sizes; 0 if the arguments are invalid. */
size_t mgn_attn_bwd_workspace_bytes(int B, int H, int S, int D, int mode);

/*
 * Cross-attention and grouped key/value heads.  The paper's matched workloads (Section 4.1,
 * workload table) contain attention between sequences of different length (50 action tokens over
 * 16 context tokens; 77-token text cross-attention); it prints no formula for them, so these entry
 * points compute the textbook generalisation of the two above:
 *   q, o, d_o, dq : [B, H, S_q, D]      k, v, dk, dv : [B, H_kv, S_k, D]      lse : [B, H, S_q]
 *   H must be a multiple of H_kv; query head h reads key/value head h / (H / H_kv), and dk, dv of
 *   a key/value head sum the contributions of all its query heads;
 *   causal != 0 keeps key j for query i iff j <= i + (S_k - S_q): the mask is aligned to the
 *   bottom-right corner (the last query sees every key) and needs S_q <= S_k, else the call
 *   returns MGN_ERR_UNSUPPORTED (a query row without a visible key has no softmax).
 * Everything else -- element types per mode, alignment, ownership, stream semantics, error
 * order, dq accumulated with floating-point atomics -- is as for mgn_attn_fwd / mgn_attn_bwd,
 * which are these functions with H_kv = H and S_q = S_k = S.  H % H_kv != 0 is MGN_ERR_INVALID_ARG.
 * The workspace of mgn_attn_bwd_ext is mgn_attn_bwd_workspace_bytes(B, H, S_q, D, mode) bytes.
 */
int mgn_attn_fwd_ext(const void* q, const void* k, const void* v, void* o, float* lse,
                     int B, int H, int H_kv, int S_q, int S_k, int D, int causal, float scale, int mode,
                     void* stream);
int mgn_attn_bwd_ext(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                     const float* lse, void* dq, void* dk, void* dv,
                     void* workspace, size_t workspace_bytes,
                     int B, int H, int H_kv, int S_q, int S_k, int D, int causal, float scale, int mode,
                     void* stream);

/*
 * Forward of the paper's accelerated ("practical default") arithmetic policy (Section 4.2, table
 * "Arithmetic permissions"): persistent tensors stay f32; the forward attention inputs are rounded
 * locally to IEEE f16, multiplied on the tensor cores with f32 accumulation, and O and LSE are stored
 * as f32; the backward remains f32 -- call mgn_attn_bwd_ext (or mgn_attn_bwd_deterministic) with
 * MGN_MODE_STRICT_F32 on the same f32 tensors and this forward's o and lse.
 *   q [B,H,S_q,D], k, v [B,H_kv,S_k,D], o [B,H,S_q,D], lse [B,H,S_q]: all binary32, device pointers.
 *   D must be 64 or 128.  Shapes, grouping and the causal rule are those of mgn_attn_fwd_ext.
 *   workspace: device scratch of mgn_attn_fwd_accel_workspace_bytes(...) bytes (f16 copies of q, k
 *   and v), 256-byte aligned, contents ignored on entry and undefined on exit.
 * Inputs whose magnitude exceeds the f16 range (65504) become infinities; the softmax probabilities
 * are rounded to f16 before the second product, so entries below 6e-8 are dropped.
 * Errors as for mgn_attn_fwd_ext, plus MGN_ERR_WORKSPACE.
 */
size_t mgn_attn_fwd_accel_workspace_bytes(int B, int H, int H_kv, int S_q, int S_k, int D);
int mgn_attn_fwd_accel(const float* q, const float* k, const float* v, float* o, float* lse,
                       void* workspace, size_t workspace_bytes,
                       int B, int H, int H_kv, int S_q, int S_k, int D, int causal, float scale, void* stream);

/*
 * Deterministic backward (the "separate pass" form of the dQ kernel: paper Section 3.3 lists dQ
 * beside the fused dK+dV kernel, Section 7.3 profiles them separately).  Same arguments, shapes,
 * modes and results as mgn_attn_bwd_ext, but no floating-point atomics are used: the fused dK+dV
 * kernel runs without the dQ product and reductions, and a second kernel computes dQ with one CTA per
 * query tile, so dq, dk and dv are bit-identical from run to run.  It executes seven matrix products
 * per tile pair instead of five (S and dP are recomputed in the dQ pass).  The workspace holds only
 * delta, but must still be mgn_attn_bwd_workspace_bytes(B, H, S_q, D, mode) bytes.
 */
int mgn_attn_bwd_deterministic(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                               const float* lse, void* dq, void* dk, void* dv,
                               void* workspace, size_t workspace_bytes,
                               int B, int H, int H_kv, int S_q, int S_k, int D, int causal, float scale, int mode,
                               void* stream);

/*
 * The step after attention, fused with it at its two seams (paper Section 3.3: matrix-product
 * kernels with prologues and epilogues that absorb the neighbouring steps; Section 7.3: dispatch
 * structure matters where kernels are small).  The paper prints no formula; these are the textbook
 * output projection of the concatenated heads and its data gradient.  Fast mode only so far
 * (MGN_MODE_FAST_BF16: bf16 tensors, tensor-core products, f32 accumulation; strict mode returns
 * MGN_ERR_UNSUPPORTED), D in {64,128}, E a multiple of 8.  All pointers are device pointers, 16-byte
 * aligned; layouts dense row-major.
 *
 * mgn_out_proj_fwd:       y[b,s,e] = sum_{h,d} o[b,h,s,d] * w[h*D+d, e]
 *     o [B,H,S,D] as the attention forward wrote it (no concatenated copy is made), w [H*D, E],
 *     y [B,S,E] out.
 * mgn_out_proj_bwd_data:  d_o[b,h,s,d] = sum_e d_y[b,s,e] * w[h*D+d, e]      (into the [B,H,S,D] layout
 *                         delta[b,h,s] = sum_d d_o[b,h,s,d] * o[b,h,s,d]      the attention backward reads)
 *     d_y [B,S,E], w [H*D,E], o [B,H,S,D] in; d_o [B,H,S,D] (bf16) and delta [B,H,S] (f32) out.  delta is
 *     formed from the bf16-rounded d_o and is what mgn_attn_bwd's own first pass would compute from
 *     o and d_o; hand it to mgn_attn_bwd_given_delta.
 * mgn_out_proj_bwd_weight: d_w[h*D+d, e] = sum_{b,s} o[b,h,s,d] * d_y[b,s,e]
 *     o [B,H,S,D] read head-major again, d_y [B,S,E] in; d_w [H*D,E] (bf16) out.
 * mgn_qkv_rope_fwd:  the step before attention.  y[b,s,n] = sum_e x[b,s,e] * w[n,e] with
 *     w [(H + 2 H_kv) D, E]: rows of all query heads, then all key heads, then all value heads; query and
 *     key heads are rotated pairwise, columns d and d + D/2 ("rotate-half"), by the caller's angle tables
 *     cos_t, sin_t [S, D/2] (f32, device): out[d] = y[d] c - y[d+D/2] s, out[d+D/2] = y[d+D/2] c + y[d] s;
 *     value heads are copied.  q [B,H,S,D], k, v [B,H_kv,S,D] (bf16) out, in the layout the attention
 *     entry points read.  The rotation is done in f32 on the accumulators, before the one rounding to bf16.
 * The backward of that step, in three calls (fast mode, same limits):
 * mgn_rope_bwd_inplace:  rotates the pairs of dq [B,H,S,D] and dk [B,H_kv,S,D] (bf16, as the attention
 *     backward wrote them) IN PLACE by the opposite angles: g[d] = dq[d] c + dq[d+D/2] s,
 *     g[d+D/2] = dq[d+D/2] c - dq[d] s -- the gradient with respect to the unrotated projection.  A
 *     streaming pass: the rotation depends on the position, i.e. on the row of the operand, so it cannot be
 *     folded into the two products below.  The result is rounded to bf16 once more.
 * mgn_qkv_bwd_data:      dx[b,s,e] = sum_n g[b,s,n] * w[n,e], g the concatenation (query | key | value heads)
 *     of gq [B,H,S,D], gk, gv [B,H_kv,S,D] -- dq and dk after mgn_rope_bwd_inplace, and dv -- read where they
 *     are (no concatenated copy); w [(H + 2 H_kv) D, E]; dx [B,S,E] (bf16) out.
 * mgn_qkv_bwd_weight:    dw[n,e] = sum_{b,s} g[b,s,n] * x[b,s,e]; x [B,S,E] in; dw [(H + 2 H_kv) D, E] (bf16) out.
 * mgn_attn_bwd_given_delta: mgn_attn_bwd_ext without `o`, with a ready `delta` [B,H,S_q] (f32, read
 *     only): the pass over o and d_o is skipped.  Either mode.  Workspace as for mgn_attn_bwd_ext.
 * Errors as elsewhere: INVALID_ARG (null pointer, size <= 0, unknown mode), UNSUPPORTED, MISALIGNED,
 * WORKSPACE, ARCH, CUDA.
 */
int mgn_out_proj_fwd(const void* o, const void* w, void* y, int B, int H, int S, int D, int E, int mode, void* stream);
int mgn_out_proj_bwd_data(const void* d_y, const void* w, const void* o, void* d_o, float* delta,
                          int B, int H, int S, int D, int E, int mode, void* stream);
int mgn_out_proj_bwd_weight(const void* o, const void* d_y, void* d_w, int B, int H, int S, int D, int E, int mode,
                            void* stream);
int mgn_qkv_rope_fwd(const void* x, const void* w, const float* cos_t, const float* sin_t, void* q, void* k, void* v,
                     int B, int S, int E, int H, int H_kv, int D, int mode, void* stream);
int mgn_rope_bwd_inplace(void* dq, void* dk, const float* cos_t, const float* sin_t, int B, int H, int H_kv, int S,
                         int D, int mode, void* stream);
int mgn_qkv_bwd_data(const void* gq, const void* gk, const void* gv, const void* w, void* dx, int B, int S, int E, int H,
                     int H_kv, int D, int mode, void* stream);
int mgn_qkv_bwd_weight(const void* gq, const void* gk, const void* gv, const void* x, void* dw, int B, int S, int E,
                       int H, int H_kv, int D, int mode, void* stream);
int mgn_attn_bwd_given_delta(const void* q, const void* k, const void* v, const void* d_o, const float* lse,
                             const float* delta, void* dq, void* dk, void* dv,
                             void* workspace, size_t workspace_bytes,
                             int B, int H, int H_kv, int S_q, int S_k, int D, int causal, float scale, int mode,
                             void* stream);

/*
 * Synchronises `stream`, then reads and clears the device-side status word that
 * kernels set when one of their bounded waits (TMA / tensor-core completion
 * barriers) ran out.  Returns MGN_OK, MGN_ERR_DEVICE_TIMEOUT or MGN_ERR_CUDA.
 * The word belongs to the current device, not to `stream`: see "Device status word"
 * above.  After a MGN_ERR_DEVICE_TIMEOUT the outputs of every call since the last
 * MGN_OK check are to be treated as unwritten; the next call runs normally again.
 * (Library plumbing; the paper has no counterpart.)
 */
int mgn_attn_check(void* stream);

/*
 * Measurement hook (library plumbing; the paper has no counterpart).  While both
 * arguments are non-null cudaEvent_t handles, every later mgn_attn_fwd / mgn_attn_bwd
 * call records `before_main` on its stream immediately before its main kernel (the
 * forward kernel, or the fused dK/dV/dQ kernel) and `after_main` immediately after it,
 * so a benchmark can time that kernel alone inside a whole-call timed region.  Pass
 * two nulls to switch it off.  Process-wide state: meant for single-threaded
 * benchmarks only.  Returns MGN_OK, or MGN_ERR_INVALID_ARG if exactly one is null.
 */
int mgn_attn_profile_events(void* before_main, void* after_main);

/*
 * Tuning hook (library plumbing; the paper has no counterpart).  The fast-mode kernels are
 * persistent: each CTA walks a fixed list of work items (a block of keys or queries of one head).
 * Two item orders exist: 0, block-major (balanced for any size, but the CTAs running at one time
 * touch every head), and 1, head-major (the CTAs running at one time share a few heads, whose
 * tensors stay in L2; balanced only with many items per CTA).  By default (-1) each call picks the
 * order from the problem size; 0 or 1 forces it for all later fast-mode calls of the process.
 * Results are the same in either order up to the summation order of dq.  Returns MGN_OK, or
 * MGN_ERR_INVALID_ARG for any other value.
 */
int mgn_attn_fast_item_order(int order);

/*
 * Which tile shapes the strict-mode kernels run a problem with (host-only query; library plumbing,
 * the paper has no counterpart).  The strict kernels cover the score matrix with tiles of
 * fwd_bm x fwd_bn (forward) and bwd_bm x bwd_bn (backward) query rows x keys, and execute whole
 * tiles; for short sequences whose lengths are far from tile multiples (197 tokens of a vision
 * transformer, Section 4.1 workload table) a second shape with less padding is chosen.  Writes the
 * four sizes through host pointers out[0..3] = {fwd_bm, fwd_bn, bwd_bm, bwd_bn}.  Arguments as in
 * mgn_attn_fwd_ext.  Touches no device.  Returns MGN_OK, MGN_ERR_INVALID_ARG (out null, a size
 * <= 0, H % H_kv != 0, causal not 0/1) or MGN_ERR_UNSUPPORTED (D not in {32, 64, 128}; causal with
 * S_q > S_k).
 */
int mgn_attn_strict_tiles(int B, int H, int H_kv, int S_q, int S_k, int D, int causal, int* out);

/*
 * Backward for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this is a convenience of this library.)
 *
 * Who needs it: code that is handed tensors but may not call cudaMalloc -- a plug-in inside a
 * framework whose memory pool owns the whole GPU, a serving loop where an allocation would
 * synchronise the device, a caller that has only the pointers it was given.  mgn_attn_bwd asks
 * such a caller for a workspace it cannot produce; this entry point takes none.  The workspace
 * is a fixed MGN_NOALLOC_MAX_WORKSPACE_BYTES array inside the library image, so every GPU that
 * loads the library gives up that much memory until the process exits.
 *
 * Arguments, layouts, results and error codes are those of mgn_attn_bwd without `workspace`
 * and `workspace_bytes`.  Differences:
 *   - Sizes for which mgn_attn_bwd_workspace_bytes(B,H,S,D,mode) exceeds
 *     MGN_NOALLOC_MAX_WORKSPACE_BYTES are refused with MGN_ERR_WORKSPACE before anything is
 *     enqueued (strict mode needs 4 bytes per (b,h,s) row; fast mode 4*(D+1) bytes per row).
 *   - It calls no cudaMalloc, cudaFree or other allocating routine.
 *   - The first call on each device looks up the array's device address (a one-time, per-device
 *     set-up done with that device current); make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps whatever the last call left in it.
 *     Each call clears or overwrites everything it reads, so calls issued one after another on a
 *     stream are independent; calls that can overlap on the GPU (different streams, no ordering)
 *     race on the array and corrupt each other -- serialise them, or use mgn_attn_bwd with
 *     separate workspaces.
 */
#define MGN_NOALLOC_MAX_WORKSPACE_BYTES (8u << 20)
int mgn_attn_bwd_noalloc(const void* q, const void* k, const void* v, const void* o, const void* d_o,
                         const float* lse, void* dq, void* dk, void* dv,
                         int B, int H, int S, int D, int causal, float scale, int mode, void* stream);

/* The constant above, for callers that bind the library without the header. */
size_t mgn_attn_bwd_noalloc_max_workspace_bytes(void);

/*
 * Measures the FP32 FFMA peak of the current device with a register-only fused-multiply-add
 * loop on every SM (synchronous; a few milliseconds).  `scratch` is a device pointer to at least
 * one float (never written in practice), `tflops` a HOST pointer that receives the best of three
 * timed repetitions.  Measurement plumbing for the strict-mode roofline; the paper has no
 * counterpart.  Returns MGN_OK, MGN_ERR_INVALID_ARG or MGN_ERR_CUDA.
 */
int mgn_measure_fp32_ffma_tflops(float* scratch, double* tflops, void* stream);

/*
 * Self-test of the bounded waits (library plumbing; the paper has no counterpart; present only in
 * builds with MGN_BUILD_SELFTEST, which the in-tree build sets).  Enqueues a one-CTA kernel that
 * waits, with a limit of 1024 polls, on a barrier that nothing arrives on: the wait gives up, the
 * kernel sets the device status word and returns -- the path a product kernel would take if a
 * copy or a tensor-core completion never came.  Afterwards the device is in the state described
 * under "Device status word": kernels of this library skip their work until mgn_attn_check() has
 * returned MGN_ERR_DEVICE_TIMEOUT once.  `gave_up` is an optional DEVICE pointer that receives 1
 * if the wait ran out (0 if it did not).  Returns MGN_OK, MGN_ERR_ARCH or MGN_ERR_CUDA.
 */
int mgn_selftest_wait_timeout(unsigned* gave_up, void* stream);

/* Static string naming a status code. */
const char* mgn_status_string(int status);

/* Library version: major*10000 + minor*100 + patch. */
int mgn_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MGN_ATTN_H */
