/*
 * GDWS convolution forward: reference implementation for tests.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain CPU statement of what
 * a generalized depthwise-separable (GDWS) convolution computes, written from the
 * paper's definitions (arXiv 2110.14871).  It shares nothing with the CUDA
 * library: only tests, the smoke check and the CPU-baseline leg of the benchmark
 * may load it.
 *
 * Conventions (paper Section 3 notation; K is the filter size, M the number of
 * output channels, called D in the library's interface):
 *   - tensors are NCHW, row-major, double precision; callers upcast exactly;
 *   - the channel distribution vector g has C entries, G = sum_c g_c
 *     (Section 3.1, Definition);
 *   - intermediate channel i = off_c + j, off_c = sum_{c'<c} g_{c'}, j < g_c:
 *     the order of the non-zero rows of W_D (Property 2, Fig. 3), 0-based here;
 *   - depthwise weights  Kd[i][u][v]  (G x K x K, taps row-major),
 *     pointwise weights  P[d][i]      (M x G) = W_P (Property 1);
 *   - "convolving" is read as cross-correlation (no filter flip), zero padding,
 *     stride and padding applied by the GDW stage, which already produces the
 *     H' x W' maps (Section 3.1); the PW stage is 1x1, stride 1.
 *   - H' = floor((H + 2 pad - K) / stride) + 1, W' likewise.
 *   - bias (not in the paper; part of the library's interface) is added after
 *     the pointwise sum; NULL means zero.
 *
 * Every sum is accumulated in double, in the index order written below; there is
 * no blocking, fusion or reordering beyond the definitions.
 *
 * Pins (tests/test_oracle_pins.py): equality with a dense convolution whose
 * weights are W = W_P W_D (Property 1 + 2), reduction to a depthwise-separable
 * convolution for g = 1 (Section 3.1 "Relation to DWS"), g_c = K^2 delta filters
 * reproducing any dense convolution (Lemma 1), the MAC counts of Eq. 2 and Eq. 3,
 * the worked (3,2,4) example of Appendix B.2, the channel-duplication identity of
 * Appendix A.1 against library routines, and hand-written tiny cases.
 */
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* Output extent along one axis for input extent `in` (standard floor rule). */
int gdws_oracle_out_dim(int in, int k, int stride, int pad)
{
    int span = in + 2 * pad - k;
    if (span < 0) return 0;
    return span / stride + 1;
}

/* G = sum_c g_c; off has C+1 entries, off[c] = sum_{c'<c} g_{c'} (Property 2). */
int64_t gdws_oracle_offsets(int C, const int32_t *g, int64_t *off)
{
    int64_t s = 0;
    for (int c = 0; c < C; ++c) {
        off[c] = s;
        s += g[c];
    }
    off[C] = s;
    return s;
}

/* Eq. 2: MACs of a (C,K,M) standard convolution on one image. */
int64_t gdws_oracle_dense_macs(int Ho, int Wo, int C, int K, int M)
{
    return (int64_t)Ho * Wo * M * C * K * K;
}

/* Eq. 3: MACs of a (C,K,g,M) GDWS convolution on one image: H'W' G (K^2 + M). */
int64_t gdws_oracle_gdws_macs(int Ho, int Wo, int64_t G, int K, int M)
{
    return (int64_t)Ho * Wo * G * ((int64_t)K * K + M);
}

/* Number of weights of a GDWS layer: rows of W_D (G K^2) plus W_P (M G). */
int64_t gdws_oracle_gdws_params(int64_t G, int K, int M)
{
    return G * ((int64_t)K * K + M);
}

/*
 * GDW stage (Section 3.1): channel c of x is convolved with g_c K x K filters.
 *   z[n][i][ho][wo] = sum_{u,v} Kd[i][u][v] * xpad[n][c(i)][ho*s+u-p][wo*s+v-p]
 * Returns the number of multiply-accumulates performed, counting the taps that
 * fall on padding too (the paper's count, Eq. 3, ignores borders).
 */
int64_t gdws_oracle_gdw(int N, int C, int H, int W, int K, int stride, int pad,
                        const int32_t *g, const double *x, const double *Kd, double *z)
{
    const int Ho = gdws_oracle_out_dim(H, K, stride, pad);
    const int Wo = gdws_oracle_out_dim(W, K, stride, pad);
    int64_t *off = (int64_t *)malloc(sizeof(int64_t) * (size_t)(C + 1));
    const int64_t G = gdws_oracle_offsets(C, g, off);
    int64_t macs = 0;
#pragma omp parallel for collapse(2) reduction(+ : macs) schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int ho = 0; ho < Ho; ++ho) {
            for (int c = 0; c < C; ++c) {
                const double *xc = x + ((size_t)n * C + c) * H * W;
                for (int j = 0; j < g[c]; ++j) {
                    const int64_t i = off[c] + j;
                    const double *ker = Kd + (size_t)i * K * K;
                    double *zi = z + (((size_t)n * G + i) * Ho + ho) * Wo;
                    for (int wo = 0; wo < Wo; ++wo) {
                        double acc = 0.0;
                        for (int u = 0; u < K; ++u) {
                            const int hi = ho * stride + u - pad;
                            for (int v = 0; v < K; ++v) {
                                const int wi = wo * stride + v - pad;
                                double xv = 0.0;
                                if (hi >= 0 && hi < H && wi >= 0 && wi < W)
                                    xv = xc[(size_t)hi * W + wi];
                                acc += ker[u * K + v] * xv;
                                ++macs;
                            }
                        }
                        zi[wo] = acc;
                    }
                }
            }
        }
    }
    free(off);
    return macs;
}

/*
 * PW stage (Section 3.1): a (G,1,M) standard convolution, plus bias.
 *   y[n][d][ho][wo] = b[d] + sum_i P[d][i] * z[n][i][ho][wo]
 * relu != 0 applies max(.,0) afterwards (used only between chained layers).
 * Returns the MAC count.
 */
int64_t gdws_oracle_pw(int N, int64_t G, int Ho, int Wo, int M, const double *z,
                       const double *P, const double *bias, int relu, double *y)
{
    int64_t macs = 0;
#pragma omp parallel for collapse(2) reduction(+ : macs) schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int ho = 0; ho < Ho; ++ho) {
            for (int d = 0; d < M; ++d) {
                for (int wo = 0; wo < Wo; ++wo) {
                    double acc = 0.0;
                    for (int64_t i = 0; i < G; ++i) {
                        acc += P[(size_t)d * G + i] *
                               z[(((size_t)n * G + i) * Ho + ho) * Wo + wo];
                        ++macs;
                    }
                    acc += bias ? bias[d] : 0.0;
                    if (relu && acc < 0.0) acc = 0.0;
                    y[(((size_t)n * M + d) * Ho + ho) * Wo + wo] = acc;
                }
            }
        }
    }
    return macs;
}

/*
 * GDWS = PW after GDW, nothing in between (Property 1 needs the composition to
 * be linear).  z_out may be NULL; if not it receives the G intermediate maps.
 * Returns total MACs (GDW + PW), or -1 if scratch memory could not be had.
 */
int64_t gdws_oracle_forward(int N, int C, int H, int W, int M, int K, int stride, int pad,
                            const int32_t *g, const double *x, const double *Kd,
                            const double *P, const double *bias, int relu,
                            double *z_out, double *y)
{
    const int Ho = gdws_oracle_out_dim(H, K, stride, pad);
    const int Wo = gdws_oracle_out_dim(W, K, stride, pad);
    int64_t G = 0;
    for (int c = 0; c < C; ++c) G += g[c];
    double *z = z_out;
    if (!z) {
        z = (double *)malloc(sizeof(double) * (size_t)N * (size_t)G * Ho * Wo + 8);
        if (!z) return -1;
    }
    int64_t macs = gdws_oracle_gdw(N, C, H, W, K, stride, pad, g, x, Kd, z);
    macs += gdws_oracle_pw(N, G, Ho, Wo, M, z, P, bias, relu, y);
    if (!z_out) free(z);
    return macs;
}

/*
 * Standard (C,K,M) convolution, Eq. 1 written as direct loops:
 *   y[n][d][ho][wo] = b[d] + sum_{c,u,v} Wt[d][c][u][v] * xpad[n][c][ho*s+u-p][wo*s+v-p]
 * Returns the MAC count (Eq. 2 per image, padding taps included).
 */
int64_t gdws_oracle_dense_conv(int N, int C, int H, int W, int M, int K, int stride, int pad,
                               const double *x, const double *Wt, const double *bias,
                               double *y)
{
    const int Ho = gdws_oracle_out_dim(H, K, stride, pad);
    const int Wo = gdws_oracle_out_dim(W, K, stride, pad);
    int64_t macs = 0;
#pragma omp parallel for collapse(2) reduction(+ : macs) schedule(static)
    for (int n = 0; n < N; ++n) {
        for (int d = 0; d < M; ++d) {
            for (int ho = 0; ho < Ho; ++ho) {
                for (int wo = 0; wo < Wo; ++wo) {
                    double acc = 0.0;
                    for (int c = 0; c < C; ++c) {
                        for (int u = 0; u < K; ++u) {
                            const int hi = ho * stride + u - pad;
                            for (int v = 0; v < K; ++v) {
                                const int wi = wo * stride + v - pad;
                                double xv = 0.0;
                                if (hi >= 0 && hi < H && wi >= 0 && wi < W)
                                    xv = x[(((size_t)n * C + c) * H + hi) * W + wi];
                                acc += Wt[(((size_t)d * C + c) * K + u) * K + v] * xv;
                                ++macs;
                            }
                        }
                    }
                    acc += bias ? bias[d] : 0.0;
                    y[(((size_t)n * M + d) * Ho + ho) * Wo + wo] = acc;
                }
            }
        }
    }
    return macs;
}

/*
 * W_D as the full G x (C K^2) matrix of Property 2: sub-matrix c (columns
 * c K^2 .. (c+1) K^2 - 1) is zero except rows off_c .. off_c + g_c - 1, which hold
 * the g_c filters of channel c, taps vectorised row-major.
 */
void gdws_oracle_wd_matrix(int C, int K, const int32_t *g, const double *Kd, double *WD)
{
    const int K2 = K * K;
    int64_t G = 0;
    for (int c = 0; c < C; ++c) G += g[c];
    memset(WD, 0, sizeof(double) * (size_t)G * C * K2);
    int64_t i = 0;
    for (int c = 0; c < C; ++c)
        for (int j = 0; j < g[c]; ++j, ++i)
            for (int t = 0; t < K2; ++t)
                WD[(size_t)i * C * K2 + (size_t)c * K2 + t] = Kd[(size_t)i * K2 + t];
}

/*
 * Equivalent standard convolution (Property 1, W = W_P W_D, with the block
 * structure of Property 2 / the proof of Lemma 1):
 *   Wt[d][c][u][v] = sum_{j<g_c} P[d][off_c + j] * Kd[off_c + j][u][v]
 */
void gdws_oracle_reconstruct_dense(int C, int M, int K, const int32_t *g, const double *Kd,
                                   const double *P, double *Wt)
{
    const int K2 = K * K;
    int64_t G = 0;
    for (int c = 0; c < C; ++c) G += g[c];
    int64_t off = 0;
    for (int c = 0; c < C; ++c) {
        for (int d = 0; d < M; ++d) {
            for (int t = 0; t < K2; ++t) {
                double acc = 0.0;
                for (int j = 0; j < g[c]; ++j)
                    acc += P[(size_t)d * G + off + j] * Kd[(size_t)(off + j) * K2 + t];
                Wt[((size_t)d * C + c) * K2 + t] = acc;
            }
        }
        off += g[c];
    }
}
