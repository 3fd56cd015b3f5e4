/*
 * Oracle primitives: direct-loop convolution, its two adjoints, and 2-D max pooling,
 * all in double precision on NCHW tensors.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is part of the CPU oracle that the CUDA
 * path is checked against.  Nothing in the product library links, imports or
 * calls it, and it shares no code with the CUDA sources.
 *
 * The convolution is the plain cross-correlation that the residual functions
 * of the paper are built from (Section 2.2, Eq. 2: c_k(x) = Conv_kxk(a(x))),
 * written out as its definition, with zero padding and no bias:
 *
 *   out[n,co,i,j] = sum_{ci,kh,kw} w[co,ci,kh,kw] * a[n,ci, i*s+kh-p, j*s+kw-p]
 *
 * dgrad and wgrad are the exact adjoints of that sum with respect to a and w
 * (the "ordinary backprop" Jacobian products of Algorithm 1).
 *
 * Loop order puts the output column innermost so that the compiler can
 * vectorise; every output element still receives its terms one tap at a time
 * in (ci, kh, kw) order.  There is no blocking, no im2col, no FFT.
 */
#include <stddef.h>
#include <string.h>
#include <math.h>

#define IDX4(n, c, h, w, C, H, W) ((((size_t)(n) * (C) + (c)) * (H) + (h)) * (W) + (w))

static int out_size(int in, int k, int s, int p) { return (in + 2 * p - k) / s + 1; }

/* valid output column range [j0, j1) for which x = j*s + kw - p lies in [0, W) */
static void col_range(int W, int Wo, int s, int off, int *j0, int *j1)
{
    int lo = 0, hi = Wo;
    while (lo < hi && lo * s + off < 0) lo++;
    while (hi > lo && (hi - 1) * s + off >= W) hi--;
    *j0 = lo; *j1 = hi;
}

void oracle_conv_fwd(const double *a, const double *w, double *out,
                     int N, int Ci, int H, int W, int Co, int k, int s, int p)
{
    const int Ho = out_size(H, k, s, p), Wo = out_size(W, k, s, p);
    #pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; n++)
        for (int co = 0; co < Co; co++) {
            double *o = out + IDX4(n, co, 0, 0, Co, Ho, Wo);
            memset(o, 0, sizeof(double) * (size_t)Ho * Wo);
            for (int ci = 0; ci < Ci; ci++)
                for (int kh = 0; kh < k; kh++)
                    for (int kw = 0; kw < k; kw++) {
                        const double wv = w[IDX4(co, ci, kh, kw, Ci, k, k)];
                        int j0, j1;
                        col_range(W, Wo, s, kw - p, &j0, &j1);
                        for (int i = 0; i < Ho; i++) {
                            const int y = i * s + kh - p;
                            if (y < 0 || y >= H) continue;
                            const double *arow = a + IDX4(n, ci, y, 0, Ci, H, W) + (kw - p);
                            double *orow = o + (size_t)i * Wo;
                            for (int j = j0; j < j1; j++) orow[j] += wv * arow[j * s];
                        }
                    }
        }
}

/* da[n,ci,y,x] = sum over (co,kh,kw,i,j) with i*s+kh-p == y, j*s+kw-p == x of w[co,ci,kh,kw] * dout[n,co,i,j] */
void oracle_conv_dgrad(const double *dout, const double *w, double *da,
                       int N, int Ci, int H, int W, int Co, int k, int s, int p)
{
    const int Ho = out_size(H, k, s, p), Wo = out_size(W, k, s, p);
    #pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; n++)
        for (int ci = 0; ci < Ci; ci++) {
            double *d = da + IDX4(n, ci, 0, 0, Ci, H, W);
            memset(d, 0, sizeof(double) * (size_t)H * W);
            for (int co = 0; co < Co; co++)
                for (int kh = 0; kh < k; kh++)
                    for (int kw = 0; kw < k; kw++) {
                        const double wv = w[IDX4(co, ci, kh, kw, Ci, k, k)];
                        int j0, j1;
                        col_range(W, Wo, s, kw - p, &j0, &j1);
                        for (int i = 0; i < Ho; i++) {
                            const int y = i * s + kh - p;
                            if (y < 0 || y >= H) continue;
                            const double *grow = dout + IDX4(n, co, i, 0, Co, Ho, Wo);
                            double *drow = d + (size_t)y * W + (kw - p);
                            for (int j = j0; j < j1; j++) drow[j * s] += wv * grow[j];
                        }
                    }
        }
}

/* dw[co,ci,kh,kw] = sum_{n,i,j} dout[n,co,i,j] * a[n,ci,i*s+kh-p,j*s+kw-p] */
void oracle_conv_wgrad(const double *dout, const double *a, double *dw,
                       int N, int Ci, int H, int W, int Co, int k, int s, int p)
{
    const int Ho = out_size(H, k, s, p), Wo = out_size(W, k, s, p);
    #pragma omp parallel for collapse(2) schedule(static)
    for (int co = 0; co < Co; co++)
        for (int ci = 0; ci < Ci; ci++)
            for (int kh = 0; kh < k; kh++)
                for (int kw = 0; kw < k; kw++) {
                    int j0, j1;
                    col_range(W, Wo, s, kw - p, &j0, &j1);
                    double acc = 0.0;
                    for (int n = 0; n < N; n++)
                        for (int i = 0; i < Ho; i++) {
                            const int y = i * s + kh - p;
                            if (y < 0 || y >= H) continue;
                            const double *grow = dout + IDX4(n, co, i, 0, Co, Ho, Wo);
                            const double *arow = a + IDX4(n, ci, y, 0, Ci, H, W) + (kw - p);
                            for (int j = j0; j < j1; j++) acc += grow[j] * arow[j * s];
                        }
                    dw[IDX4(co, ci, kh, kw, Ci, k, k)] = acc;
                }
}

/* max pooling k x k, stride s, padding p (padding counts as -inf); idx records the
 * flat (y*W+x) position of the first maximum met in (kh,kw) row-major scan. */
void oracle_maxpool_fwd(const double *a, double *out, int *idx,
                        int N, int C, int H, int W, int k, int s, int p)
{
    const int Ho = out_size(H, k, s, p), Wo = out_size(W, k, s, p);
    #pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; n++)
        for (int c = 0; c < C; c++)
            for (int i = 0; i < Ho; i++)
                for (int j = 0; j < Wo; j++) {
                    double best = -INFINITY; int bi = -1;
                    for (int kh = 0; kh < k; kh++)
                        for (int kw = 0; kw < k; kw++) {
                            const int y = i * s + kh - p, x = j * s + kw - p;
                            if (y < 0 || y >= H || x < 0 || x >= W) continue;
                            const double v = a[IDX4(n, c, y, x, C, H, W)];
                            if (v > best) { best = v; bi = y * W + x; }
                        }
                    out[IDX4(n, c, i, j, C, Ho, Wo)] = best;
                    idx[IDX4(n, c, i, j, C, Ho, Wo)] = bi;
                }
}

void oracle_maxpool_bwd(const double *dout, const int *idx, double *da,
                        int N, int C, int H, int W, int Ho, int Wo)
{
    #pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; n++)
        for (int c = 0; c < C; c++) {
            double *d = da + IDX4(n, c, 0, 0, C, H, W);
            memset(d, 0, sizeof(double) * (size_t)H * W);
            for (int i = 0; i < Ho; i++)
                for (int j = 0; j < Wo; j++) {
                    const size_t o = IDX4(n, c, i, j, C, Ho, Wo);
                    if (idx[o] >= 0) d[idx[o]] += dout[o];
                }
        }
}
