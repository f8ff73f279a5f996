/*
 * CPU oracle of the Conv2d workload (paper, Evaluation, Table 2: Conv2d, N=8, C=64,
 * 56x56, F=128, 3x3, FP16).  TEST INFRASTRUCTURE ONLY: nothing in the product links,
 * loads or calls this file.
 *
 * The plain definition of a 2-D cross-correlation (the operation deep-learning
 * libraries call convolution), channels-last:
 *
 *   y[n][p][q][f] = sum over r < R, s < S, c < C of
 *                   x[n][p*stride_h + r - pad_h][q*stride_w + s - pad_w][c] * w[f][r][s][c]
 *
 * with terms whose input coordinate falls outside [0,H) x [0,W) equal to zero.  The
 * operands arrive already decoded to fp64 (every fp16 value is exact in fp64), products
 * and sums are fp64, summed in ascending (r, s, c).  absy receives the same sum over
 * |x| |w| (the scale of the error bound).  No blocking, no reordering, no im2col.
 */
#include <math.h>
#include <stdint.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_conv2d(int64_t N, int64_t H, int64_t W, int64_t C, int64_t F, int64_t R, int64_t S, int64_t pad_h,
                  int64_t pad_w, int64_t stride_h, int64_t stride_w, const double* x, const double* w, double* y,
                  double* absy, int nthreads)
{
    if (N < 0 || H < 0 || W < 0 || C < 0 || F < 0 || R < 1 || S < 1 || stride_h < 1 || stride_w < 1 || pad_h < 0 ||
        pad_w < 0)
        return 1;
    if (H + 2 * pad_h < R || W + 2 * pad_w < S) return 2;
    const int64_t P = (H + 2 * pad_h - R) / stride_h + 1;
    const int64_t Q = (W + 2 * pad_w - S) / stride_w + 1;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#endif
    const int64_t rows = N * P;
#pragma omp parallel for schedule(static)
    for (int64_t np = 0; np < rows; ++np) {
        const int64_t n = np / P, p = np % P;
        for (int64_t q = 0; q < Q; ++q) {
            for (int64_t f = 0; f < F; ++f) {
                double acc = 0.0, sab = 0.0;
                for (int64_t r = 0; r < R; ++r) {
                    const int64_t h = p * stride_h + r - pad_h;
                    if (h < 0 || h >= H) continue;
                    for (int64_t s = 0; s < S; ++s) {
                        const int64_t ww = q * stride_w + s - pad_w;
                        if (ww < 0 || ww >= W) continue;
                        const double* xp = x + ((n * H + h) * W + ww) * C;
                        const double* wp = w + ((f * R + r) * S + s) * C;
                        for (int64_t c = 0; c < C; ++c) {
                            acc += xp[c] * wp[c];
                            sab += fabs(xp[c]) * fabs(wp[c]);
                        }
                    }
                }
                y[((n * P + p) * Q + q) * F + f] = acc;
                if (absy) absy[((n * P + p) * Q + q) * F + f] = sab;
            }
        }
    }
    return 0;
}
