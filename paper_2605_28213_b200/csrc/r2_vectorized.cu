// Rung 2 - "vectorize_global" (paper, Table 1; precondition: 128-bit aligned
// access; Introduction: a wide load needs aligned addresses and a handled
// tail).  Same 128 x 128 x 16 tiling as rung 1, but
//   * A and B move in 16-byte groups of 8 bf16 whenever the operand's base
//     and leading dimension are 16-byte aligned (checked per call, per operand);
//     a group that crosses the M/N/K edge is loaded element by element under a
//     mask; an unaligned operand takes the masked scalar route for every group;
//   * shared memory is read with 128-bit loads (register tile = 2 x 2 blocks of
//     4 x 4, which keeps those loads free of bank conflicts);
//   * C leaves in 16-byte (fp32) or 8-byte (bf16) groups of 4 columns when C's
//     base and leading dimension allow it, element by element otherwise.
#include "common.cuh"

namespace klin {
namespace {

constexpr int BM = 128, BN = 128, BK = 16, NT = 256;
constexpr int LDS_A = BM + 4, LDS_B = BN + 4;   // keeps rows 16-byte aligned

// 8 consecutive bf16 starting at p; `valid` elements (0..8) are in range.
__device__ __forceinline__ void load8(const uint16_t* p, int valid, bool vec, float (&out)[8])
{
    if (vec && valid >= 8) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
        out[0] = bf16_lo(v.x); out[1] = bf16_hi(v.x);
        out[2] = bf16_lo(v.y); out[3] = bf16_hi(v.y);
        out[4] = bf16_lo(v.z); out[5] = bf16_hi(v.z);
        out[6] = bf16_lo(v.w); out[7] = bf16_hi(v.w);
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) out[e] = (e < valid) ? bf16_bits_to_float(p[e]) : 0.f;
    }
}

template <bool BCOL>
__global__ void __launch_bounds__(NT, 2)
r2_vectorized_kernel(GemmArgs g, int tiles_m, int tiles_n, int a_vec, int b_vec, int c_vec, int kid)
{
    __shared__ __align__(16) float As[BK][LDS_A];
    __shared__ __align__(16) float Bs[BK][LDS_B];
    if (blockIdx.x == 0 && threadIdx.x == 0) g.status[1] = kid;

    int tm, tn;
    raster_tile(blockIdx.x, tiles_m, tiles_n, tm, tn);
    const int m0 = tm * BM, n0 = tn * BN;
    const int t = threadIdx.x;
    const int tx = t % 16, ty = t / 16;

    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < g.K; k0 += BK) {
        float va[8], vb[8];
        {   // A: row t/2, k-group (t%2)*8
            const int m = t >> 1, kg = (t & 1) * 8;
            const int64_t gm = m0 + m;
            const int gk = k0 + kg;
            const int valid = (gm < g.M) ? min(8, max(0, g.K - gk)) : 0;
            load8(g.A + gm * g.lda + gk, valid, a_vec, va);
#pragma unroll
            for (int e = 0; e < 8; ++e) As[kg + e][m] = va[e];
        }
        if (BCOL) {   // B column-major: column t/2, k-group (t%2)*8
            const int n = t >> 1, kg = (t & 1) * 8;
            const int64_t gn = n0 + n;
            const int gk = k0 + kg;
            const int valid = (gn < g.N) ? min(8, max(0, g.K - gk)) : 0;
            load8(g.B + gn * g.ldb + gk, valid, b_vec, vb);
#pragma unroll
            for (int e = 0; e < 8; ++e) Bs[kg + e][n] = vb[e];
        } else {      // B row-major: k-row t/16, n-group (t%16)*8
            const int k = t >> 4, ng = (t & 15) * 8;
            const int64_t gk = k0 + k;
            const int gn = n0 + ng;
            const int valid = (gk < g.K) ? min(8, max(0, g.N - gn)) : 0;
            load8(g.B + gk * g.ldb + gn, valid, b_vec, vb);
            *reinterpret_cast<float4*>(&Bs[k][ng]) = make_float4(vb[0], vb[1], vb[2], vb[3]);
            *reinterpret_cast<float4*>(&Bs[k][ng + 4]) = make_float4(vb[4], vb[5], vb[6], vb[7]);
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const float4 a0 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 a1 = *reinterpret_cast<const float4*>(&As[k][64 + ty * 4]);
            const float4 b0 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float4 b1 = *reinterpret_cast<const float4*>(&Bs[k][64 + tx * 4]);
            const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int64_t gm = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
        if (gm >= g.M) continue;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int gn = n0 + h * 64 + tx * 4;
            float v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) v[j] = acc[i][h * 4 + j] + (gn + j < g.N ? bias_at(g, gn + j) : 0.f);
            if (c_vec && gn + 4 <= g.N) {
                if (g.c_bf16) {
                    uint2 w = make_uint2(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]));
                    *reinterpret_cast<uint2*>(static_cast<uint16_t*>(g.C) + gm * g.ldc + gn) = w;
                } else {
                    *reinterpret_cast<float4*>(static_cast<float*>(g.C) + gm * g.ldc + gn) =
                        make_float4(v[0], v[1], v[2], v[3]);
                }
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (gn + j < g.N) store_c(g.C, g.c_bf16, gm * g.ldc + gn + j, v[j]);
            }
        }
    }
}

}  // namespace

cudaError_t launch_r2_vectorized(const GemmArgs& g, cudaStream_t stream, int* kernel_id)
{
    const int64_t tiles_m = (g.M + BM - 1) / BM, tiles_n = (g.N + BN - 1) / BN;
    if (tiles_m * tiles_n > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    const unsigned grid = static_cast<unsigned>(tiles_m * tiles_n);
    // Preconditions of the 128-bit paths, per operand.
    const int a_vec = (reinterpret_cast<uintptr_t>(g.A) % 16 == 0) && (g.lda % 8 == 0);
    const int b_vec = (reinterpret_cast<uintptr_t>(g.B) % 16 == 0) && (g.ldb % 8 == 0);
    const int c_vec = g.c_bf16 ? ((reinterpret_cast<uintptr_t>(g.C) % 8 == 0) && (g.ldc % 4 == 0))
                               : ((reinterpret_cast<uintptr_t>(g.C) % 16 == 0) && (g.ldc % 4 == 0));
    const int kid = kIdVectorized + a_vec + 2 * b_vec + 4 * c_vec;
    if (g.b_col)
        r2_vectorized_kernel<true><<<grid, NT, 0, stream>>>(g, (int)tiles_m, (int)tiles_n, a_vec, b_vec, c_vec, kid);
    else
        r2_vectorized_kernel<false><<<grid, NT, 0, stream>>>(g, (int)tiles_m, (int)tiles_n, a_vec, b_vec, c_vec, kid);
    *kernel_id = kid;
    return cudaGetLastError();
}

}  // namespace klin
