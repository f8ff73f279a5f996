/*
 * CPU oracle for the dense bf16 GEMM  C = A.B  with exact products and fp64
 * accumulation.  TEST INFRASTRUCTURE ONLY: nothing in the product path may
 * call, link or import this file; it shares no code with the CUDA kernels.
 *
 * What it computes is the plain definition of the matrix product that every
 * lineage rung (the paper's naive kernel K_0 up to the expert kernel K_n,
 * Method section, "lineage L = (K_0, tau_1, ..., K_n)") must reproduce:
 *
 *     C_ref[i][j] = sum_{k=0}^{K-1} double(A[i][k]) * double(B[k][j])
 *     S[i][j]     = sum_{k=0}^{K-1} |A[i][k]| * |B[k][j]|
 *
 * with k ascending for every element.  bf16 -> double is exact, and the
 * product of two bf16 values (8-bit significands) is exact in double, so the
 * only rounding is the fp64 running sum.  S is the magnitude sum the
 * tolerance K * 2^-23 * S_ij is built from.  The paper's GEMM workload is
 * "GEMM, M=N=K=4096, BF16" (Evaluation, Table 2); it fixes no tolerance, so
 * the fp64 definition is the reference.
 *
 * Layouts: A is row-major M x K with leading dimension lda (elements).
 * B is K x N, either row-major (b_col_major = 0, element (k,j) at
 * B[k*ldb + j]) or column-major (b_col_major = 1, element (k,j) at
 * B[j*ldb + k]).  C and S are row-major fp64 with leading dimension ldc and
 * are indexed by the ABSOLUTE row i (the slab [row_begin,row_end) only limits
 * which rows are computed).  S may be NULL.
 *
 * Loop orders: for row-major B the loops run i, k, j over a fp64 row of C;
 * for column-major B they run i, j, k.  Either way each C[i][j] receives its
 * K terms one at a time in ascending k, which is the definition above; there
 * is no blocking, no partial sums, no reassociation.
 *
 * Returns 0 on success, 1 on invalid arguments.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* bf16 is the top 16 bits of an IEEE-754 binary32. */
static inline double bf16_to_double(uint16_t h)
{
    uint32_t w = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

int oracle_gemm_bf16(int64_t M, int64_t N, int64_t K,
                     const uint16_t *A, int64_t lda,
                     const uint16_t *B, int64_t ldb, int b_col_major,
                     double *C, double *S, int64_t ldc,
                     int64_t row_begin, int64_t row_end, int nthreads)
{
    if (M < 0 || N < 0 || K < 0) return 1;
    if (row_begin < 0 || row_end > M || row_begin > row_end) return 1;
    if (M == 0 || N == 0) return 0;
    if (!C || ldc < N) return 1;
    if (K > 0) {
        if (!A || !B || lda < K) return 1;
        if (b_col_major ? (ldb < K) : (ldb < N)) return 1;
    }
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#else
    (void)nthreads;
#endif

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = row_begin; i < row_end; ++i) {
        double *c = C + i * ldc;
        double *s = S ? S + i * ldc : NULL;
        for (int64_t j = 0; j < N; ++j) c[j] = 0.0;
        if (s) for (int64_t j = 0; j < N; ++j) s[j] = 0.0;

        if (!b_col_major) {
            for (int64_t k = 0; k < K; ++k) {
                const double a = bf16_to_double(A[i * lda + k]);
                const double abs_a = fabs(a);
                const uint16_t *brow = B + k * ldb;
                for (int64_t j = 0; j < N; ++j) {
                    const double b = bf16_to_double(brow[j]);
                    c[j] += a * b;
                }
                if (s) {
                    for (int64_t j = 0; j < N; ++j) {
                        const double b = bf16_to_double(brow[j]);
                        s[j] += abs_a * fabs(b);
                    }
                }
            }
        } else {
            for (int64_t j = 0; j < N; ++j) {
                const uint16_t *bcol = B + j * ldb;
                double acc = 0.0, mag = 0.0;
                for (int64_t k = 0; k < K; ++k) {
                    const double a = bf16_to_double(A[i * lda + k]);
                    const double b = bf16_to_double(bcol[k]);
                    acc += a * b;
                    mag += fabs(a) * fabs(b);
                }
                c[j] = acc;
                if (s) s[j] = mag;
            }
        }
    }
    return 0;
}

/*
 * Round a double to bf16 with round-to-nearest-even, the rounding the GPU
 * epilogue applies to an fp32 accumulator (cvt.rn.bf16.f32).  The value is
 * first rounded to fp32 (the accumulator type), then to bf16; on the
 * integer-valued test inputs the fp32 step is exact, so there is no double
 * rounding there.  NaN maps to the canonical quiet NaN 0x7FC0.
 */
uint16_t oracle_round_to_bf16(double x)
{
    float f = (float)x;
    uint32_t w;
    memcpy(&w, &f, sizeof w);
    if ((w & 0x7F800000u) == 0x7F800000u && (w & 0x007FFFFFu))
        return 0x7FC0;
    const uint32_t lsb = (w >> 16) & 1u;
    w += 0x7FFFu + lsb;
    return (uint16_t)(w >> 16);
}

void oracle_round_to_bf16_array(const double *x, uint16_t *out, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) out[i] = oracle_round_to_bf16(x[i]);
}
