/*
 * CPU checker for backpropagation with pooling-compressed activations.
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, plain definition that the
 * CUDA library is compared against. It shares no code with the CUDA path and
 * must never be linked into, imported by or called from it.
 *
 * Everything is fp64 on logical NCHW arrays (row-major [N][C][H][W]).
 * Each function restates one passage of the paper's compression section
 * (Section 4, "Compressing Activation Maps") and its figure:
 *
 *   pool      Z = average pooling of the layer INPUT X with non-overlapping
 *             k x k blocks that start at index (0,0) (figure: mu_00 is the
 *             mean of X_00, X_01, X_10, X_11).
 *   inflate   the stored Z is expanded to X's shape again: every block
 *             mean stands for each element of its block.
 *   wgrad     the ordinary weight gradient, taken of the inflated tensor
 *             and the uncompressed output gradient: dL/dW ~ Z (*) dL/dY
 *             in the figure.
 *
 * Readings where the paper is silent (all listed in the design notes):
 *   - H or W not divisible by k: the last block row/column is partial and is
 *     averaged over its in-range elements only (ceil output size).
 *   - blocks are aligned to X itself, not to the zero-padded X; the
 *     convolution's zero padding is applied after inflation.
 *   - "(*)" is the ordinary convolution weight gradient (cross-correlation,
 *     dilation 1, one group); dW is overwritten, no extra scale.
 *
 * Parity pins: every function here is pinned by tests that do not call it to
 * produce their expected values (brute force in Python, closed forms,
 * invariants, the paper's Table 1 for the byte accounting).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

/* Section 4 / figure: Z[n,c,p,q] = mean of X over block (p,q). */
void oracle_pool(const double *x, int64_t N, int64_t C, int64_t H, int64_t W,
                 int64_t k, double *z)
{
    const int64_t Hp = ceil_div(H, k), Wp = ceil_div(W, k);
    #pragma omp parallel for schedule(static)
    for (int64_t nc = 0; nc < N * C; ++nc) {
        const double *xp = x + nc * H * W;
        double *zp = z + nc * Hp * Wp;
        for (int64_t p = 0; p < Hp; ++p) {
            for (int64_t q = 0; q < Wp; ++q) {
                double sum = 0.0;
                int64_t count = 0;
                for (int64_t h = p * k; h < (p + 1) * k && h < H; ++h) {
                    for (int64_t w = q * k; w < (q + 1) * k && w < W; ++w) {
                        sum += xp[h * W + w];
                        ++count;
                    }
                }
                zp[p * Wp + q] = sum / (double)count;
            }
        }
    }
}

/* Section 4: inflate Z back to X's dimensions; Xt[n,c,h,w] = Z[n,c,h/k,w/k]. */
void oracle_inflate(const double *z, int64_t N, int64_t C, int64_t H, int64_t W,
                    int64_t k, double *xt)
{
    const int64_t Hp = ceil_div(H, k), Wp = ceil_div(W, k);
    #pragma omp parallel for schedule(static)
    for (int64_t nc = 0; nc < N * C; ++nc) {
        const double *zp = z + nc * Hp * Wp;
        double *xp = xt + nc * H * W;
        for (int64_t h = 0; h < H; ++h)
            for (int64_t w = 0; w < W; ++w)
                xp[h * W + w] = zp[(h / k) * Wp + (w / k)];
    }
}

/* Element-wise max(a, 0): the ReLU that precedes a compressed conv input. */
void oracle_relu(const double *a, int64_t n, double *y)
{
    for (int64_t i = 0; i < n; ++i) y[i] = a[i] > 0.0 ? a[i] : 0.0;
}

/* One entry of the ordinary convolution weight gradient:
 * dW[co,ci,r,s] = sum_{n,ho,wo} dY[n,co,ho,wo] * Xpad[n,ci,ho*sh-ph+r, wo*sw-pw+s]
 * with Xpad = X inside [0,H)x[0,W) and 0 outside. */
static double wgrad_entry(const double *x, const double *dy,
                          int64_t N, int64_t Ci, int64_t Co, int64_t H, int64_t W,
                          int64_t Ho, int64_t Wo, int64_t sh, int64_t sw,
                          int64_t ph, int64_t pw,
                          int64_t co, int64_t ci, int64_t r, int64_t s)
{
    double acc = 0.0;
    for (int64_t n = 0; n < N; ++n) {
        const double *xp = x + (n * Ci + ci) * H * W;
        const double *gp = dy + (n * Co + co) * Ho * Wo;
        for (int64_t ho = 0; ho < Ho; ++ho) {
            const int64_t h = ho * sh - ph + r;
            if (h < 0 || h >= H) continue;
            for (int64_t wo = 0; wo < Wo; ++wo) {
                const int64_t w = wo * sw - pw + s;
                if (w < 0 || w >= W) continue;
                acc += gp[ho * Wo + wo] * xp[h * W + w];
            }
        }
    }
    return acc;
}

/* The ordinary weight gradient of a convolution layer (the "normal"
 * calculation the compression section refers to), dW as [Co][Ci][R][S]. */
void oracle_wgrad_dense(const double *x, const double *dy,
                        int64_t N, int64_t Ci, int64_t Co, int64_t H, int64_t W,
                        int64_t R, int64_t S, int64_t sh, int64_t sw,
                        int64_t ph, int64_t pw, double *dw)
{
    const int64_t Ho = (H + 2 * ph - R) / sh + 1;
    const int64_t Wo = (W + 2 * pw - S) / sw + 1;
    #pragma omp parallel for schedule(dynamic, 1)
    for (int64_t cc = 0; cc < Co * Ci; ++cc) {
        const int64_t co = cc / Ci, ci = cc % Ci;
        for (int64_t r = 0; r < R; ++r)
            for (int64_t s = 0; s < S; ++s)
                dw[((co * Ci + ci) * R + r) * S + s] =
                    wgrad_entry(x, dy, N, Ci, Co, H, W, Ho, Wo, sh, sw, ph, pw,
                                co, ci, r, s);
    }
}

/* Section 4, backward of a compressed layer: the stored Z is inflated to X's
 * shape and the ordinary weight gradient is taken of the result.
 * Returns 0, or -1 if the temporary cannot be allocated. */
int oracle_wgrad_compressed(const double *z, const double *dy,
                            int64_t N, int64_t Ci, int64_t Co, int64_t H, int64_t W,
                            int64_t R, int64_t S, int64_t sh, int64_t sw,
                            int64_t ph, int64_t pw, int64_t k, double *dw)
{
    double *xt = (double *)malloc(sizeof(double) * (size_t)(N * Ci * H * W));
    if (!xt) return -1;
    oracle_inflate(z, N, Ci, H, W, k, xt);
    oracle_wgrad_dense(xt, dy, N, Ci, Co, H, W, R, S, sh, sw, ph, pw, dw);
    free(xt);
    return 0;
}

/* Same definition, evaluated only at `count` chosen entries
 * idx[4*i..] = (co, ci, r, s); used where the full tensor would take the
 * CPU minutes. The inflated value is read through the index map h/k, w/k
 * instead of a materialised temporary; the sum and its order are the same. */
void oracle_wgrad_compressed_entries(const double *z, const double *dy,
                            int64_t N, int64_t Ci, int64_t Co, int64_t H, int64_t W,
                            int64_t R, int64_t S, int64_t sh, int64_t sw,
                            int64_t ph, int64_t pw, int64_t k,
                            const int64_t *idx, int64_t count, double *out)
{
    const int64_t Hp = ceil_div(H, k), Wp = ceil_div(W, k);
    const int64_t Ho = (H + 2 * ph - R) / sh + 1;
    const int64_t Wo = (W + 2 * pw - S) / sw + 1;
    (void)R; (void)S;
    #pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < count; ++i) {
        const int64_t co = idx[4 * i], ci = idx[4 * i + 1];
        const int64_t r = idx[4 * i + 2], s = idx[4 * i + 3];
        double acc = 0.0;
        for (int64_t n = 0; n < N; ++n) {
            const double *zp = z + (n * Ci + ci) * Hp * Wp;
            const double *gp = dy + (n * Co + co) * Ho * Wo;
            for (int64_t ho = 0; ho < Ho; ++ho) {
                const int64_t h = ho * sh - ph + r;
                if (h < 0 || h >= H) continue;
                for (int64_t wo = 0; wo < Wo; ++wo) {
                    const int64_t w = wo * sw - pw + s;
                    if (w < 0 || w >= W) continue;
                    acc += gp[ho * Wo + wo] * zp[(h / k) * Wp + (w / k)];
                }
            }
        }
        out[i] = acc;
    }
}

/* ---- Non-uniform pooling shapes (Section 6 names them as future work; the
 * definitions of Section 4 carry over with a k_h x k_w block in place of the
 * k x k one). Written out separately so that the square functions above stay
 * exactly as they are. ------------------------------------------------------ */

/* Z[n,c,p,q] = mean of X over rows [p*kh, min((p+1)*kh, H)) and columns
 * [q*kw, min((q+1)*kw, W)). */
void oracle_pool_rect(const double *x, int64_t N, int64_t C, int64_t H, int64_t W,
                      int64_t kh, int64_t kw, double *z)
{
    const int64_t Hp = ceil_div(H, kh), Wp = ceil_div(W, kw);
    #pragma omp parallel for schedule(static)
    for (int64_t nc = 0; nc < N * C; ++nc) {
        const double *xp = x + nc * H * W;
        double *zp = z + nc * Hp * Wp;
        for (int64_t p = 0; p < Hp; ++p) {
            for (int64_t q = 0; q < Wp; ++q) {
                double sum = 0.0;
                int64_t count = 0;
                for (int64_t h = p * kh; h < (p + 1) * kh && h < H; ++h) {
                    for (int64_t w = q * kw; w < (q + 1) * kw && w < W; ++w) {
                        sum += xp[h * W + w];
                        ++count;
                    }
                }
                zp[p * Wp + q] = sum / (double)count;
            }
        }
    }
}

/* Xt[n,c,h,w] = Z[n,c,h/kh,w/kw]. */
void oracle_inflate_rect(const double *z, int64_t N, int64_t C, int64_t H, int64_t W,
                         int64_t kh, int64_t kw, double *xt)
{
    const int64_t Hp = ceil_div(H, kh), Wp = ceil_div(W, kw);
    #pragma omp parallel for schedule(static)
    for (int64_t nc = 0; nc < N * C; ++nc) {
        const double *zp = z + nc * Hp * Wp;
        double *xp = xt + nc * H * W;
        for (int64_t h = 0; h < H; ++h)
            for (int64_t w = 0; w < W; ++w)
                xp[h * W + w] = zp[(h / kh) * Wp + (w / kw)];
    }
}

/* Inflate by (kh, kw), then the ordinary weight gradient. */
int oracle_wgrad_compressed_rect(const double *z, const double *dy,
                                 int64_t N, int64_t Ci, int64_t Co, int64_t H, int64_t W,
                                 int64_t R, int64_t S, int64_t sh, int64_t sw,
                                 int64_t ph, int64_t pw, int64_t kh, int64_t kw, double *dw)
{
    double *xt = (double *)malloc(sizeof(double) * (size_t)(N * Ci * H * W));
    if (!xt) return -1;
    oracle_inflate_rect(z, N, Ci, H, W, kh, kw, xt);
    oracle_wgrad_dense(xt, dy, N, Ci, Co, H, W, R, S, sh, sw, ph, pw, dw);
    free(xt);
    return 0;
}

/* The same sum at chosen entries idx[4*i..] = (co, ci, r, s), the inflated
 * value read through the index map h/kh, w/kw. */
void oracle_wgrad_compressed_rect_entries(const double *z, const double *dy,
                            int64_t N, int64_t Ci, int64_t Co, int64_t H, int64_t W,
                            int64_t R, int64_t S, int64_t sh, int64_t sw,
                            int64_t ph, int64_t pw, int64_t kh, int64_t kw,
                            const int64_t *idx, int64_t count, double *out)
{
    const int64_t Hp = ceil_div(H, kh), Wp = ceil_div(W, kw);
    const int64_t Ho = (H + 2 * ph - R) / sh + 1;
    const int64_t Wo = (W + 2 * pw - S) / sw + 1;
    (void)R; (void)S;
    #pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < count; ++i) {
        const int64_t co = idx[4 * i], ci = idx[4 * i + 1];
        const int64_t r = idx[4 * i + 2], s = idx[4 * i + 3];
        double acc = 0.0;
        for (int64_t n = 0; n < N; ++n) {
            const double *zp = z + (n * Ci + ci) * Hp * Wp;
            const double *gp = dy + (n * Co + co) * Ho * Wo;
            for (int64_t ho = 0; ho < Ho; ++ho) {
                const int64_t h = ho * sh - ph + r;
                if (h < 0 || h >= H) continue;
                for (int64_t wo = 0; wo < Wo; ++wo) {
                    const int64_t w = wo * sw - pw + s;
                    if (w < 0 || w >= W) continue;
                    acc += gp[ho * Wo + wo] * zp[(h / kh) * Wp + (w / kw)];
                }
            }
        }
        out[i] = acc;
    }
}

/* Number of OpenMP threads the loops above will use (for reporting). */
#ifdef _OPENMP
#include <omp.h>
int oracle_num_threads(void) { return omp_get_max_threads(); }
#else
int oracle_num_threads(void) { return 1; }
#endif
