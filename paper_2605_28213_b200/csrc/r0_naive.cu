// Rung 0 - the naive kernel K_0 of the lineage (paper, Method: the lineage
// starts from a naive kernel): one thread per element of C, a K-loop straight
// over global memory, bounds-checked.  No staging, no vector access.
#include "common.cuh"

namespace klin {
namespace {

constexpr int kBx = 32, kBy = 8;

__global__ void __launch_bounds__(kBx* kBy) r0_naive_kernel(GemmArgs g, int tiles_n, int64_t tiles)
{
    if (blockIdx.x == 0 && threadIdx.x == 0 && threadIdx.y == 0) g.status[1] = kIdNaive;
    for (int64_t t = blockIdx.x; t < tiles; t += gridDim.x) {
        const int64_t i = (t / tiles_n) * kBy + threadIdx.y;
        const int64_t j = (t % tiles_n) * kBx + threadIdx.x;
        if (i >= g.M || j >= g.N) continue;
        const uint16_t* a = g.A + i * g.lda;
        float acc = 0.f;
        if (g.b_col) {
            const uint16_t* b = g.B + j * g.ldb;
            for (int k = 0; k < g.K; ++k) acc = fmaf(bf16_bits_to_float(a[k]), bf16_bits_to_float(b[k]), acc);
        } else {
            const uint16_t* b = g.B + j;
            for (int k = 0; k < g.K; ++k)
                acc = fmaf(bf16_bits_to_float(a[k]), bf16_bits_to_float(b[static_cast<int64_t>(k) * g.ldb]), acc);
        }
        store_c(g.C, g.c_bf16, i * g.ldc + j, acc + bias_at(g, j));
    }
}

__global__ void zero_fill_kernel(GemmArgs g)
{
    if (blockIdx.x == 0 && threadIdx.x == 0) g.status[1] = kIdZeroFill;
    const int64_t total = static_cast<int64_t>(g.M) * g.N;
    for (int64_t e = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; e < total;
         e += static_cast<int64_t>(gridDim.x) * blockDim.x)
        store_c(g.C, g.c_bf16, (e / g.N) * g.ldc + (e % g.N), 0.f + bias_at(g, e % g.N));
}

}  // namespace

cudaError_t launch_r0_naive(const GemmArgs& g, cudaStream_t stream, int* kernel_id)
{
    const int tiles_n = (g.N + kBx - 1) / kBx;
    const int64_t tiles = static_cast<int64_t>((g.M + kBy - 1) / kBy) * tiles_n;
    const unsigned grid = static_cast<unsigned>(tiles < 0x7FFFFFFFll ? tiles : 0x7FFFFFFFll);
    r0_naive_kernel<<<grid, dim3(kBx, kBy), 0, stream>>>(g, tiles_n, tiles);
    *kernel_id = kIdNaive;
    return cudaGetLastError();
}

// K == 0: the empty sum.  C <- 0.
cudaError_t launch_zero_fill(const GemmArgs& g, cudaStream_t stream, int* kernel_id)
{
    const int64_t total = static_cast<int64_t>(g.M) * g.N;
    const int64_t blocks = (total + 255) / 256;
    zero_fill_kernel<<<static_cast<unsigned>(blocks < 65536 ? blocks : 65536), 256, 0, stream>>>(g);
    *kernel_id = kIdZeroFill;
    return cudaGetLastError();
}

}  // namespace klin
