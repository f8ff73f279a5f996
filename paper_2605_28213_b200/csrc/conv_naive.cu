// Direct Conv2d, the naive rung of the convolution workload (paper, Evaluation, Table 2: Conv2d;
// Method: a lineage starts from a naive kernel K_0): one thread per output value
// y[n][p][q][f], a loop over the filter taps and channels in ascending (r, s, c) with fp32
// fused multiply-adds, zero padding by skipping taps outside the image.  Channels-last x
// (N, H, W, C) and w (F, R, S, C) in fp16; y (N, P, Q, F) in fp16 or fp32.
#include "common.cuh"

namespace klin {
namespace {

__global__ void __launch_bounds__(256) conv2d_naive_kernel(GemmArgs g, ConvGeom cv)
{
    const int64_t total = static_cast<int64_t>(g.M) * g.N;
    if (blockIdx.x == 0 && threadIdx.x == 0) g.status[1] = kIdConvNaive;
    const __half* x = reinterpret_cast<const __half*>(g.A);
    const __half* w = reinterpret_cast<const __half*>(g.B);
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int f = static_cast<int>(i % g.N);
        const int m = static_cast<int>(i / g.N);
        const int q = m % cv.Q, t = m / cv.Q;
        const int p = t % cv.P, n = t / cv.P;
        float acc = 0.f;
        for (int r = 0; r < cv.R; ++r) {
            const int h = p * cv.stride_h + r - cv.pad_h;
            if (h < 0 || h >= cv.H) continue;
            for (int s = 0; s < cv.S; ++s) {
                const int ww = q * cv.stride_w + s - cv.pad_w;
                if (ww < 0 || ww >= cv.W) continue;
                const __half* xp = x + ((static_cast<int64_t>(n) * cv.H + h) * cv.W + ww) * cv.C;
                const __half* wp = w + ((static_cast<int64_t>(f) * cv.R + r) * cv.S + s) * cv.C;
                for (int c = 0; c < cv.C; ++c) acc = fmaf(__half2float(xp[c]), __half2float(wp[c]), acc);
            }
        }
        if (g.c_bf16)   // 2-byte output: fp16 for this workload
            reinterpret_cast<__half*>(g.C)[static_cast<int64_t>(m) * g.ldc + f] = __float2half_rn(acc);
        else
            static_cast<float*>(g.C)[static_cast<int64_t>(m) * g.ldc + f] = acc;
    }
}

}  // namespace

cudaError_t launch_conv2d_naive(const GemmArgs& g, const ConvGeom& geom, cudaStream_t stream, int* kernel_id)
{
    const int64_t total = static_cast<int64_t>(g.M) * g.N;
    const int64_t blocks = (total + 255) / 256;
    *kernel_id = kIdConvNaive;
    conv2d_naive_kernel<<<static_cast<unsigned>(blocks < 148 * 16 ? blocks : 148 * 16), 256, 0, stream>>>(g, geom);
    return cudaGetLastError();
}

}  // namespace klin
