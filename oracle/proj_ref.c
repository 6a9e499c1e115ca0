/*
 * proj_ref.c -- CPU oracle for the output projection that follows attention, and its backward.
 *
 * TEST INFRASTRUCTURE ONLY (see attn_ref.c): plain, slow, IEEE binary64, shares nothing with the
 * CUDA path.
 *
 * What it follows.  The paper's kernel archetypes (Section 3.3) give its matrix-product kernels
 * prologues and epilogues that absorb the steps around them, and Section 7.3 finds that dispatch
 * structure matters where kernels are small.  The step after attention in every transformer block
 * is the output projection of the concatenated heads; the paper prints no formula for it, so this
 * is the textbook definition written out:
 *
 *   O  [B,H,S,D]  attention output, heads separate          W [H*D, E]  projection weight
 *   Y[b,s,e]        = sum_{h,d} O[b,h,s,d] * W[h*D+d, e]                       (forward)
 *   dO[b,h,s,d]     = sum_e  dY[b,s,e] * W[h*D+d, e]                           (backward, data)
 *   dW[h*D+d, e]    = sum_{b,s} O[b,h,s,d] * dY[b,s,e]                          (backward, weight)
 *   delta[b,h,s]    = sum_d dO[b,h,s,d] * O[b,h,s,d]      (the row statistic the attention backward
 *                                                          needs; it falls out of the dO producer)
 *
 * No blocking, no reordering; OpenMP over output rows only (no two threads add into one element).
 * Pins (tests/test_oracle_proj_pins.py): a hand-worked example, central finite differences of
 * L = sum Y o dY, torch float64 einsum + autograd, the identity weight (Y = concatenated heads),
 * linearity, and delta against the attention oracle's own delta identity.
 */
#include <stddef.h>
#ifdef _OPENMP
#include <omp.h>
#endif

void ref_out_proj_fwd(const double *O, const double *W, double *Y, int B, int H, int S, int D, int E)
{
    const long rows = (long)B * S;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        const int b = (int)(r / S), s = (int)(r % S);
        double *y = Y + (size_t)r * E;
        for (int e = 0; e < E; ++e) y[e] = 0.0;
        for (int h = 0; h < H; ++h) {
            const double *o = O + (((size_t)b * H + h) * S + s) * D;
            for (int d = 0; d < D; ++d) {
                const double *w = W + ((size_t)h * D + d) * E;
                for (int e = 0; e < E; ++e) y[e] += o[d] * w[e];
            }
        }
    }
}

/* dO and delta from dY; O is needed for delta only. */
void ref_out_proj_bwd_data(const double *dY, const double *W, const double *O, double *dO, double *delta,
                           int B, int H, int S, int D, int E)
{
    const long rows = (long)B * H * S;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        const int s = (int)(r % S), h = (int)((r / S) % H), b = (int)(r / ((long)S * H));
        const double *dy = dY + ((size_t)b * S + s) * E;
        double dl = 0.0;
        for (int d = 0; d < D; ++d) {
            const double *w = W + ((size_t)h * D + d) * E;
            double acc = 0.0;
            for (int e = 0; e < E; ++e) acc += dy[e] * w[e];
            dO[(size_t)r * D + d] = acc;
            dl += acc * O[(size_t)r * D + d];
        }
        delta[r] = dl;
    }
}

void ref_out_proj_bwd_weight(const double *O, const double *dY, double *dW, int B, int H, int S, int D, int E)
{
    const long rows = (long)H * D;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        const int h = (int)(r / D), d = (int)(r % D);
        double *dw = dW + (size_t)r * E;
        for (int e = 0; e < E; ++e) dw[e] = 0.0;
        for (int b = 0; b < B; ++b)
            for (int s = 0; s < S; ++s) {
                const double o = O[(((size_t)b * H + h) * S + s) * D + d];
                const double *dy = dY + ((size_t)b * S + s) * E;
                for (int e = 0; e < E; ++e) dw[e] += o * dy[e];
            }
    }
}
