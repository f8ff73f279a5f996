// Rung 1 - "tile / sm_stage" (paper, Table 1; precondition: loops over the
// output).  A 128 x 128 block tile of C per CTA; A and B k-slabs of depth 16 are
// staged in shared memory as fp32 (converted from bf16 on the way in) and each
// of the 256 threads keeps an 8 x 8 register tile.  Loads are scalar and masked
// element by element, so every M/N/K tail and every alignment is handled the
// same way; nothing is vectorized or overlapped yet.
#include "common.cuh"

namespace klin {
namespace {

constexpr int BM = 128, BN = 128, BK = 16, TM = 8, TN = 8, NT = 256;

template <bool BCOL>
__global__ void __launch_bounds__(NT) r1_tiled_kernel(GemmArgs g, int tiles_m, int tiles_n)
{
    __shared__ float As[BK][BM + 1];
    __shared__ float Bs[BK][BN + 1];
    if (blockIdx.x == 0 && threadIdx.x == 0) g.status[1] = kIdTiled;

    int tm, tn;
    raster_tile(blockIdx.x, tiles_m, tiles_n, tm, tn);
    const int m0 = tm * BM, n0 = tn * BN;
    const int t = threadIdx.x;
    const int tx = t % 16, ty = t / 16;

    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < g.K; k0 += BK) {
        // A slab: 128 rows x 16 k, one element per thread per step, k fastest.
#pragma unroll
        for (int e = t; e < BM * BK; e += NT) {
            const int k = e % BK, m = e / BK;
            const int64_t gm = m0 + m;
            const int gk = k0 + k;
            As[k][m] = (gm < g.M && gk < g.K) ? bf16_bits_to_float(g.A[gm * g.lda + gk]) : 0.f;
        }
        if (BCOL) {
#pragma unroll
            for (int e = t; e < BN * BK; e += NT) {
                const int k = e % BK, n = e / BK;
                const int64_t gn = n0 + n;
                const int gk = k0 + k;
                Bs[k][n] = (gn < g.N && gk < g.K) ? bf16_bits_to_float(g.B[gn * g.ldb + gk]) : 0.f;
            }
        } else {
#pragma unroll
            for (int e = t; e < BN * BK; e += NT) {
                const int n = e % BN, k = e / BN;
                const int64_t gn = n0 + n;
                const int64_t gk = k0 + k;
                Bs[k][n] = (gn < g.N && gk < g.K) ? bf16_bits_to_float(g.B[gk * g.ldb + gn]) : 0.f;
            }
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            float a[TM], b[TN];
#pragma unroll
            for (int i = 0; i < TM; ++i) a[i] = As[k][ty * TM + i];
#pragma unroll
            for (int j = 0; j < TN; ++j) b[j] = Bs[k][tx * TN + j];
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int64_t gm = m0 + ty * TM + i;
        if (gm >= g.M) continue;
#pragma unroll
        for (int j = 0; j < TN; ++j) {
            const int64_t gn = n0 + tx * TN + j;
            if (gn < g.N) store_c(g.C, g.c_bf16, gm * g.ldc + gn, acc[i][j] + bias_at(g, gn));
        }
    }
}

}  // namespace

cudaError_t launch_r1_tiled(const GemmArgs& g, cudaStream_t stream, int* kernel_id)
{
    const int64_t tiles_m = (g.M + BM - 1) / BM, tiles_n = (g.N + BN - 1) / BN;
    if (tiles_m * tiles_n > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    const unsigned grid = static_cast<unsigned>(tiles_m * tiles_n);
    if (g.b_col)
        r1_tiled_kernel<true><<<grid, NT, 0, stream>>>(g, (int)tiles_m, (int)tiles_n);
    else
        r1_tiled_kernel<false><<<grid, NT, 0, stream>>>(g, (int)tiles_m, (int)tiles_n);
    *kernel_id = kIdTiled;
    return cudaGetLastError();
}

}  // namespace klin
