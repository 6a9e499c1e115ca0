/*
 * attn_ref_ext.c -- CPU oracle for attention with separate query / key lengths and grouped
 * key/value heads (cross-attention, grouped-query attention).
 *
 * TEST INFRASTRUCTURE ONLY, like attn_ref.c: only the test-suite, the smoke check and the
 * benchmark's cpu-baseline / reference legs may call it; it shares nothing with the CUDA path.
 *
 * What it follows.  The paper's matched workloads (Section 4.1, workload table; Limitations
 * section) include attention whose queries and keys come from different sequences -- an action
 * expert attending from 50 action tokens to 16 vision-language tokens, and the 77-token text
 * cross-attention of a diffusion U-Net -- but the paper prints no formula for them; the definition
 * is the textbook one, written out one query row at a time:
 *
 *   q, o, d_o, dq : [B, H,    S_q, D]        k, v, dk, dv : [B, H_kv, S_k, D]
 *   H = G * H_kv; query head h reads key/value head h / G (integer division)
 *   visible keys of query row i:  all j < S_k,  or, if causal,  j <= i + (S_k - S_q)
 *     (the mask is aligned to the bottom-right corner: the last query sees every key;
 *      causal requires S_q <= S_k so that every row sees at least key 0)
 *   s_ij = scale * q_i . k_j ;  LSE_i = log sum_j exp(s_ij) ;  p_ij = exp(s_ij - LSE_i)
 *   o_i = sum_j p_ij v_j ;  delta_i = d_o_i . o_i ;  dp_ij = d_o_i . v_j
 *   ds_ij = p_ij (dp_ij - delta_i)
 *   dq_i = scale sum_j ds_ij k_j
 *   dk_j = scale sum_{h in group} sum_i ds_ij q_i ;  dv_j = sum_{h in group} sum_i p_ij d_o_i
 *
 * All arithmetic is IEEE binary64, two-pass softmax, no blocking, no fusion.  OpenMP runs over
 * (b, key/value head): each owns its dk, dv rows, so no two threads add into the same element.
 *
 * Parity pins (tests/test_oracle_ext_pins.py): equal to attn_ref.c when H_kv = H and S_q = S_k;
 * grouped heads equal ordinary heads on repeated K, V with dk, dv summed over the group (through
 * attn_ref.c); the causal case equals the last S_q rows of a square causal problem of length S_k
 * (through attn_ref.c); torch float64 dense evaluation with autograd; central finite differences.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* number of visible keys of query row i (keys 0 .. n-1) */
static int visible(int i, int Sq, int Sk, int causal)
{
    return causal ? i + (Sk - Sq) + 1 : Sk;
}

/* scores, LSE and probabilities of one query row into p[0..n); returns n */
static int row_probs_ext(const double *qi, const double *Kh, int n, int D, double scale,
                         double *p, double *lse_out)
{
    double m = -INFINITY;
    for (int j = 0; j < n; ++j) {
        const double *kj = Kh + (size_t)j * D;
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += qi[d] * kj[d];
        p[j] = scale * acc;
        if (p[j] > m) m = p[j];
    }
    double l = 0.0;
    for (int j = 0; j < n; ++j) l += exp(p[j] - m);
    const double lse = m + log(l);
    for (int j = 0; j < n; ++j) p[j] = exp(p[j] - lse);
    *lse_out = lse;
    return n;
}

/* Returns 0, or -1 if the shapes are outside the definition above. */
static int shapes_ok(int B, int H, int Hkv, int Sq, int Sk, int D, int causal)
{
    if (B <= 0 || H <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || D <= 0) return -1;
    if (H % Hkv != 0) return -1;
    if (causal && Sq > Sk) return -1;
    return 0;
}

int ref_attn_fwd_ext(const double *q, const double *k, const double *v, double *o, double *lse,
                     int B, int H, int Hkv, int Sq, int Sk, int D, int causal, double scale,
                     int nthreads)
{
    if (shapes_ok(B, H, Hkv, Sq, Sk, D, causal)) return -1;
    const int G = H / Hkv;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#endif
    (void)nthreads;
#pragma omp parallel
    {
        double *p = (double *)malloc(sizeof(double) * (size_t)Sk);
#pragma omp for schedule(dynamic, 1) collapse(2)
        for (int b = 0; b < B; ++b)
            for (int h = 0; h < H; ++h) {
                const size_t qoff = ((size_t)b * H + h) * (size_t)Sq * D;
                const size_t koff = ((size_t)b * Hkv + h / G) * (size_t)Sk * D;
                const double *Kh = k + koff, *Vh = v + koff;
                for (int i = 0; i < Sq; ++i) {
                    double *oi = o + qoff + (size_t)i * D;
                    const int n = row_probs_ext(q + qoff + (size_t)i * D, Kh, visible(i, Sq, Sk, causal), D,
                                                scale, p, &lse[((size_t)b * H + h) * Sq + i]);
                    for (int d = 0; d < D; ++d) oi[d] = 0.0;
                    for (int j = 0; j < n; ++j)
                        for (int d = 0; d < D; ++d) oi[d] += p[j] * Vh[(size_t)j * D + d];
                }
            }
        free(p);
    }
    return 0;
}

/* Backward.  Recomputes its own O and LSE (written to o_out / lse_out when not NULL). */
int ref_attn_bwd_ext(const double *q, const double *k, const double *v, const double *d_o,
                     double *o_out, double *lse_out, double *dq, double *dk, double *dv,
                     int B, int H, int Hkv, int Sq, int Sk, int D, int causal, double scale,
                     int nthreads)
{
    if (shapes_ok(B, H, Hkv, Sq, Sk, D, causal)) return -1;
    const int G = H / Hkv;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#endif
    (void)nthreads;
#pragma omp parallel
    {
        double *p = (double *)malloc(sizeof(double) * (size_t)Sk);
        double *oi = (double *)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 1) collapse(2)
        for (int b = 0; b < B; ++b)
            for (int hk = 0; hk < Hkv; ++hk) {
                const size_t koff = ((size_t)b * Hkv + hk) * (size_t)Sk * D;
                const double *Kh = k + koff, *Vh = v + koff;
                double *dKh = dk + koff, *dVh = dv + koff;
                for (size_t t = 0; t < (size_t)Sk * D; ++t) { dKh[t] = 0.0; dVh[t] = 0.0; }
                for (int h = hk * G; h < (hk + 1) * G; ++h) {        /* the query heads of this group */
                    const size_t qoff = ((size_t)b * H + h) * (size_t)Sq * D;
                    for (int i = 0; i < Sq; ++i) {
                        const double *qi = q + qoff + (size_t)i * D;
                        const double *doi = d_o + qoff + (size_t)i * D;
                        double *dqi = dq + qoff + (size_t)i * D;
                        double lse_i;
                        const int n = row_probs_ext(qi, Kh, visible(i, Sq, Sk, causal), D, scale, p, &lse_i);
                        for (int d = 0; d < D; ++d) oi[d] = 0.0;
                        for (int j = 0; j < n; ++j)
                            for (int d = 0; d < D; ++d) oi[d] += p[j] * Vh[(size_t)j * D + d];
                        if (o_out) memcpy(o_out + qoff + (size_t)i * D, oi, sizeof(double) * (size_t)D);
                        if (lse_out) lse_out[((size_t)b * H + h) * Sq + i] = lse_i;
                        double delta = 0.0;
                        for (int d = 0; d < D; ++d) delta += doi[d] * oi[d];
                        for (int d = 0; d < D; ++d) dqi[d] = 0.0;
                        for (int j = 0; j < n; ++j) {
                            const double *kj = Kh + (size_t)j * D, *vj = Vh + (size_t)j * D;
                            double dp = 0.0;
                            for (int d = 0; d < D; ++d) dp += doi[d] * vj[d];
                            const double ds = p[j] * (dp - delta);
                            for (int d = 0; d < D; ++d) {
                                dqi[d] += ds * kj[d];
                                dKh[(size_t)j * D + d] += ds * qi[d];
                                dVh[(size_t)j * D + d] += p[j] * doi[d];
                            }
                        }
                        for (int d = 0; d < D; ++d) dqi[d] *= scale;
                    }
                }
                for (size_t t = 0; t < (size_t)Sk * D; ++t) dKh[t] *= scale;
            }
        free(p);
        free(oi);
    }
    return 0;
}
