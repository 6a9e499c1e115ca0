/*
 * attn_ref.c -- CPU oracle for scaled-dot-product attention forward and backward.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, obviously-correct
 * statement of what the CUDA library must compute.  Only the test-suite, the
 * smoke check and the benchmark's cpu-baseline / reference legs may call it.
 * It shares no code, header, table or helper with the CUDA path.
 *
 * What it follows.  The paper names the kernels only ("tiled attention forward,
 * dQ, and fused dK+dV kernels", Section 3.3 kernel archetypes; the FlashGradKV /
 * FlashGradQ profile in Section 7.3).  A tiled ("flash") attention kernel reaches,
 * up to rounding order, the textbook result, so the oracle is that textbook
 * definition written out one query row at a time:
 *
 *   s_ij  = scale * sum_d Q[i,d] K[j,d]          for allowed j (all j<S, or j<=i if causal)
 *   m_i   = max_j s_ij ;  l_i = sum_j exp(s_ij - m_i) ;  LSE_i = m_i + log(l_i)
 *   p_ij  = exp(s_ij - LSE_i)                    (0 where masked)
 *   O_i   = sum_j p_ij V_j
 *   delta_i = sum_d dO[i,d] O[i,d]
 *   dP_ij = sum_d dO[i,d] V[j,d]
 *   dS_ij = p_ij (dP_ij - delta_i)
 *   dQ_i  = scale * sum_j dS_ij K_j
 *   dK_j  = scale * sum_i dS_ij Q_i
 *   dV_j  = sum_i p_ij dO_i
 *
 * All arithmetic is IEEE binary64, two-pass softmax (no online update), no
 * blocking, no fusion.  Tensors are dense row-major [B,H,S,D]; LSE is [B,H,S].
 * Heads are independent, so OpenMP parallelises over (b,h) and nothing else.
 *
 * Parity pins (tests/test_oracle_pins.py): central finite differences, closed
 * forms (identical keys, single key, identical V rows), softmax row sums,
 * sum_j dS_ij = 0, the dS-product swap identity, a hand-derived worked example,
 * a separately written dense-matrix evaluation, and torch's float64 CPU
 * attention with autograd as a third implementation.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static int allowed_count(int i, int S, int causal) { return causal ? (i + 1) : S; }

/* One query row: scores, LSE and probabilities into p[0..n). Returns n. */
static int row_probs(const double *Qh, const double *Kh, int i, int S, int D,
                     int causal, double scale, double *p, double *lse_out)
{
    const int n = allowed_count(i, S, causal);
    const double *qi = Qh + (size_t)i * D;
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

/* Forward: O [B,H,S,D], LSE [B,H,S]. */
void ref_attn_fwd(const double *q, const double *k, const double *v,
                  double *o, double *lse,
                  int B, int H, int S, int D, int causal, double scale, int nthreads)
{
    const long BH = (long)B * H;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#endif
    (void)nthreads;
#pragma omp parallel
    {
        double *p = (double *)malloc(sizeof(double) * (size_t)S);
#pragma omp for schedule(dynamic, 1)
        for (long bh = 0; bh < BH; ++bh) {
            const size_t off = (size_t)bh * S * D;
            const double *Qh = q + off, *Kh = k + off, *Vh = v + off;
            double *Oh = o + off, *Lh = lse + (size_t)bh * S;
            for (int i = 0; i < S; ++i) {
                const int n = row_probs(Qh, Kh, i, S, D, causal, scale, p, &Lh[i]);
                double *oi = Oh + (size_t)i * D;
                for (int d = 0; d < D; ++d) oi[d] = 0.0;
                for (int j = 0; j < n; ++j) {
                    const double *vj = Vh + (size_t)j * D;
                    for (int d = 0; d < D; ++d) oi[d] += p[j] * vj[d];
                }
            }
        }
        free(p);
    }
}

/* Backward.  Recomputes its own O and LSE in f64 (written to o_out / lse_out,
 * either may be NULL) so that nothing from another implementation enters. */
void ref_attn_bwd(const double *q, const double *k, const double *v, const double *d_o,
                  double *o_out, double *lse_out, double *dq, double *dk, double *dv,
                  int B, int H, int S, int D, int causal, double scale, int nthreads)
{
    const long BH = (long)B * H;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#endif
    (void)nthreads;
#pragma omp parallel
    {
        double *p = (double *)malloc(sizeof(double) * (size_t)S);
        double *oi = (double *)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 1)
        for (long bh = 0; bh < BH; ++bh) {
            const size_t off = (size_t)bh * S * D;
            const double *Qh = q + off, *Kh = k + off, *Vh = v + off, *dOh = d_o + off;
            double *dQh = dq + off, *dKh = dk + off, *dVh = dv + off;
            for (size_t t = 0; t < (size_t)S * D; ++t) { dKh[t] = 0.0; dVh[t] = 0.0; }
            for (int i = 0; i < S; ++i) {
                double lse_i;
                const int n = row_probs(Qh, Kh, i, S, D, causal, scale, p, &lse_i);
                const double *qi = Qh + (size_t)i * D;
                const double *doi = dOh + (size_t)i * D;
                /* O_i */
                for (int d = 0; d < D; ++d) oi[d] = 0.0;
                for (int j = 0; j < n; ++j) {
                    const double *vj = Vh + (size_t)j * D;
                    for (int d = 0; d < D; ++d) oi[d] += p[j] * vj[d];
                }
                if (o_out) memcpy(o_out + off + (size_t)i * D, oi, sizeof(double) * (size_t)D);
                if (lse_out) lse_out[(size_t)bh * S + i] = lse_i;
                /* delta_i */
                double delta = 0.0;
                for (int d = 0; d < D; ++d) delta += doi[d] * oi[d];
                double *dqi = dQh + (size_t)i * D;
                for (int d = 0; d < D; ++d) dqi[d] = 0.0;
                for (int j = 0; j < n; ++j) {
                    const double *kj = Kh + (size_t)j * D;
                    const double *vj = Vh + (size_t)j * D;
                    double *dkj = dKh + (size_t)j * D;
                    double *dvj = dVh + (size_t)j * D;
                    double dp = 0.0;
                    for (int d = 0; d < D; ++d) dp += doi[d] * vj[d];
                    const double ds = p[j] * (dp - delta);
                    for (int d = 0; d < D; ++d) {
                        dqi[d] += ds * kj[d];
                        dkj[d] += ds * qi[d];
                        dvj[d] += p[j] * doi[d];
                    }
                }
                for (int d = 0; d < D; ++d) dqi[d] *= scale;
            }
            for (size_t t = 0; t < (size_t)S * D; ++t) dKh[t] *= scale;
        }
        free(p);
        free(oi);
    }
}

/* One head, dense S x S matrices, for the pins: P, dP, dS (masked entries 0). */
void ref_attn_head_matrices(const double *q, const double *k, const double *v, const double *d_o,
                            double *P, double *dP, double *dS,
                            int S, int D, int causal, double scale)
{
    double *p = (double *)malloc(sizeof(double) * (size_t)S);
    double *oi = (double *)malloc(sizeof(double) * (size_t)D);
    for (int i = 0; i < S; ++i) {
        double lse_i;
        const int n = row_probs(q, k, i, S, D, causal, scale, p, &lse_i);
        const double *doi = d_o + (size_t)i * D;
        for (int d = 0; d < D; ++d) oi[d] = 0.0;
        for (int j = 0; j < n; ++j)
            for (int d = 0; d < D; ++d) oi[d] += p[j] * v[(size_t)j * D + d];
        double delta = 0.0;
        for (int d = 0; d < D; ++d) delta += doi[d] * oi[d];
        for (int j = 0; j < S; ++j) {
            const size_t ij = (size_t)i * S + j;
            if (j < n) {
                double dp = 0.0;
                for (int d = 0; d < D; ++d) dp += doi[d] * v[(size_t)j * D + d];
                P[ij] = p[j]; dP[ij] = dp; dS[ij] = p[j] * (dp - delta);
            } else {
                P[ij] = 0.0; dP[ij] = 0.0; dS[ij] = 0.0;
            }
        }
    }
    free(p);
    free(oi);
}

/* The two products of a given dS (one head): dQ = scale dS K, dK = scale dS^T Q. */
void ref_grads_from_ds(const double *dS, const double *q, const double *k,
                       double *dq, double *dk, int S, int D, double scale)
{
    for (size_t t = 0; t < (size_t)S * D; ++t) { dq[t] = 0.0; dk[t] = 0.0; }
    for (int i = 0; i < S; ++i)
        for (int j = 0; j < S; ++j) {
            const double ds = dS[(size_t)i * S + j];
            for (int d = 0; d < D; ++d) {
                dq[(size_t)i * D + d] += ds * k[(size_t)j * D + d];
                dk[(size_t)j * D + d] += ds * q[(size_t)i * D + d];
            }
        }
    for (size_t t = 0; t < (size_t)S * D; ++t) { dq[t] *= scale; dk[t] *= scale; }
}

int ref_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
