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

/*
 * The step before attention: the fused query/key/value projection with rotary position embedding.
 * (Same sections of the paper: a matrix product whose epilogue absorbs the step that follows it.  The
 * paper prints no formula; this is the textbook definition, with the "rotate-half" pairing of
 * columns d and d + D/2 and the angle table supplied by the caller, so no convention about the
 * frequency base is baked in.)
 *
 *   X [B,S,E]   W [(H + 2 Hkv) D, E]  (rows: all query heads, then all key heads, then all value heads)
 *   y[b,s,n]  = sum_e X[b,s,e] * W[n,e]
 *   for query and key heads, with c = cos_t[s, d], sn = sin_t[s, d], d < D/2:
 *       out[d]       = y[d] * c - y[d + D/2] * sn
 *       out[d + D/2] = y[d + D/2] * c + y[d] * sn
 *   value heads are copied.  Q [B,H,S,D], K, V [B,Hkv,S,D].
 */
void ref_qkv_rope(const double *X, const double *W, const double *cos_t, const double *sin_t,
                  double *Q, double *K, double *V, int B, int S, int E, int H, int Hkv, int D)
{
    const int heads = H + 2 * Hkv, half = D / 2;
    const long rows = (long)B * S;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        const int b = (int)(r / S), s = (int)(r % S);
        const double *x = X + (size_t)r * E;
        for (int hh = 0; hh < heads; ++hh) {
            double y[1024];                                   /* D <= 1024 */
            for (int d = 0; d < D; ++d) {
                const double *w = W + ((size_t)hh * D + d) * E;
                double acc = 0.0;
                for (int e = 0; e < E; ++e) acc += x[e] * w[e];
                y[d] = acc;
            }
            double *out;
            int rope = 1;
            if (hh < H) out = Q + (((size_t)b * H + hh) * S + s) * D;
            else if (hh < H + Hkv) out = K + (((size_t)b * Hkv + (hh - H)) * S + s) * D;
            else { out = V + (((size_t)b * Hkv + (hh - H - Hkv)) * S + s) * D; rope = 0; }
            if (!rope) { for (int d = 0; d < D; ++d) out[d] = y[d]; continue; }
            for (int d = 0; d < half; ++d) {
                const double c = cos_t[(size_t)s * half + d], sn = sin_t[(size_t)s * half + d];
                out[d] = y[d] * c - y[d + half] * sn;
                out[d + half] = y[d + half] * c + y[d] * sn;
            }
        }
    }
}

/*
 * Backward of ref_qkv_rope (textbook reverse mode of the two steps it states, written out):
 *   the rotation of a (d, d + D/2) pair by the angle (c, sn) is linear with an orthogonal matrix, so the
 *   gradient with respect to the unrotated pair is the rotation by the opposite angle:
 *       gy[d]       =  g[d] * c + g[d + D/2] * sn
 *       gy[d + D/2] =  g[d + D/2] * c - g[d] * sn          (query and key heads; value heads: gy = g)
 *   then, with y[r, hh*D + d] = sum_e X[r, e] W[hh*D + d, e]:
 *       dX[r, e]        = sum_{hh,d} gy[r, hh, d] W[hh*D + d, e]
 *       dW[hh*D + d, e] = sum_r      gy[r, hh, d] X[r, e]
 * gQ [B,H,S,D], gK, gV [B,Hkv,S,D] are the gradients with respect to the ROTATED outputs.
 * GY (scratch and output) [B*S, (H+2Hkv)*D]: the gradient with respect to the unrotated projection.
 */
void ref_qkv_rope_bwd(const double *gQ, const double *gK, const double *gV, const double *X, const double *W,
                      const double *cos_t, const double *sin_t, double *GY, double *dX, double *dW,
                      int B, int S, int E, int H, int Hkv, int D)
{
    const int heads = H + 2 * Hkv, half = D / 2;
    const long rows = (long)B * S;
    const long F = (long)heads * D;
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        const int b = (int)(r / S), s = (int)(r % S);
        for (int hh = 0; hh < heads; ++hh) {
            const double *g;
            int rope = 1;
            if (hh < H) g = gQ + (((size_t)b * H + hh) * S + s) * D;
            else if (hh < H + Hkv) g = gK + (((size_t)b * Hkv + (hh - H)) * S + s) * D;
            else { g = gV + (((size_t)b * Hkv + (hh - H - Hkv)) * S + s) * D; rope = 0; }
            double *gy = GY + (size_t)r * F + (size_t)hh * D;
            if (!rope) { for (int d = 0; d < D; ++d) gy[d] = g[d]; continue; }
            for (int d = 0; d < half; ++d) {
                const double c = cos_t[(size_t)s * half + d], sn = sin_t[(size_t)s * half + d];
                gy[d] = g[d] * c + g[d + half] * sn;
                gy[d + half] = g[d + half] * c - g[d] * sn;
            }
        }
    }
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r)
        for (int e = 0; e < E; ++e) {
            double acc = 0.0;
            for (long f = 0; f < F; ++f) acc += GY[(size_t)r * F + f] * W[(size_t)f * E + e];
            dX[(size_t)r * E + e] = acc;
        }
#pragma omp parallel for schedule(static)
    for (long f = 0; f < F; ++f)
        for (int e = 0; e < E; ++e) {
            double acc = 0.0;
            for (long r = 0; r < rows; ++r) acc += GY[(size_t)r * F + f] * X[(size_t)r * E + e];
            dW[(size_t)f * E + e] = acc;
        }
}
