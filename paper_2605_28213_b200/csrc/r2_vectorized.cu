// Rung 2 - "vectorize_global" (paper, Table 1; precondition: 128-bit aligned
// access; Introduction: a wide load needs aligned addresses and a handled
// tail).  Same T x T tiling as rung 1 (T = 128, 64 or 32 by the same rule), k-slabs of 16, 32 or 64, but
//   * A and B move in 16-byte groups of 8 bf16 whenever the operand's base
//     and leading dimension are 16-byte aligned (checked per call, per operand);
//     a group that crosses the M/N/K edge is loaded element by element under a
//     mask; an unaligned operand takes the masked scalar route for every group;
//   * shared memory is read with 128-bit loads (register tile = 2 x 2 blocks of
//     4 x 4 for the 128 tile, one 4 x 4 block for the 64 tile - both free of bank
//     conflicts - and 64-bit loads of a 2 x 2 tile for the 32 tile);
//   * C leaves in 16-byte (fp32) or 8-byte (bf16) groups of 4 columns when C's
//     base and leading dimension allow it, element by element otherwise.
#include "common.cuh"

namespace klin {
namespace {

constexpr int NT = 256;

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

template <bool BCOL, int T>
__global__ void __launch_bounds__(NT, 2)
r2_vectorized_kernel(GemmArgs g, int tiles_m, int tiles_n, int a_vec, int b_vec, int c_vec, int kid)
{
    // T x T block tile (128, 64 or 32: the largest that still gives every SM a CTA), register tile TT x TT.
    // The k-slab is as deep as it takes for every thread to move exactly one 16-byte group of A and one of B
    // (16 for the 128 tile, 32 and 64 for the smaller ones): a small tile synchronises less often.
    constexpr int TT = T / 16;
    constexpr int BK = 8 * NT / T;
    constexpr int LDS = T + 4;                 // keeps rows 16-byte aligned
    __shared__ __align__(16) float As[BK][LDS];
    __shared__ __align__(16) float Bs[BK][LDS];
    if (blockIdx.x == 0 && threadIdx.x == 0) g.status[1] = kid;

    int tm, tn;
    raster_tile(blockIdx.x, tiles_m, tiles_n, tm, tn);
    const int m0 = tm * T, n0 = tn * T;
    const int t = threadIdx.x;
    const int tx = t % 16, ty = t / 16;
    // Row / column of register-tile index i: two blocks of four 64 apart for the 128 tile (128-bit shared-memory
    // reads without bank conflicts), one block of TT otherwise.
    auto row_of = [&](int i) { return TT == 8 ? (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4)) : ty * TT + i; };
    auto col_of = [&](int j) { return TT == 8 ? (j < 4 ? tx * 4 + j : 64 + tx * 4 + (j - 4)) : tx * TT + j; };

    float acc[TT][TT];
#pragma unroll
    for (int i = 0; i < TT; ++i)
#pragma unroll
        for (int j = 0; j < TT; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < g.K; k0 += BK) {
        float va[8], vb[8];
        {   // A: row t / (BK/8), k-group (t % (BK/8)) * 8
            const int m = t / (BK / 8), kg = (t % (BK / 8)) * 8;
            const int64_t gm = m0 + m;
            const int gk = k0 + kg;
            const int valid = (gm < g.M) ? min(8, max(0, g.K - gk)) : 0;
            load8(g.A + gm * g.lda + gk, valid, a_vec, va);
#pragma unroll
            for (int e = 0; e < 8; ++e) As[kg + e][m] = va[e];
        }
        if (BCOL) {   // B column-major: column t / (BK/8), k-group (t % (BK/8)) * 8
            const int n = t / (BK / 8), kg = (t % (BK / 8)) * 8;
            const int64_t gn = n0 + n;
            const int gk = k0 + kg;
            const int valid = (gn < g.N) ? min(8, max(0, g.K - gk)) : 0;
            load8(g.B + gn * g.ldb + gk, valid, b_vec, vb);
#pragma unroll
            for (int e = 0; e < 8; ++e) Bs[kg + e][n] = vb[e];
        } else {      // B row-major: k-row t / (T/8), n-group (t % (T/8)) * 8
            const int k = t / (T / 8), ng = (t % (T / 8)) * 8;
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
            float a[TT], b[TT];
            if constexpr (TT == 2) {
                const float2 a0 = *reinterpret_cast<const float2*>(&As[k][ty * 2]);
                const float2 b0 = *reinterpret_cast<const float2*>(&Bs[k][tx * 2]);
                a[0] = a0.x; a[1] = a0.y;
                b[0] = b0.x; b[1] = b0.y;
            } else {
#pragma unroll
                for (int h = 0; h < TT / 4; ++h) {
                    const float4 av = *reinterpret_cast<const float4*>(&As[k][h * 64 + ty * 4]);
                    const float4 bv = *reinterpret_cast<const float4*>(&Bs[k][h * 64 + tx * 4]);
                    a[h * 4] = av.x; a[h * 4 + 1] = av.y; a[h * 4 + 2] = av.z; a[h * 4 + 3] = av.w;
                    b[h * 4] = bv.x; b[h * 4 + 1] = bv.y; b[h * 4 + 2] = bv.z; b[h * 4 + 3] = bv.w;
                }
            }
#pragma unroll
            for (int i = 0; i < TT; ++i)
#pragma unroll
                for (int j = 0; j < TT; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }

#pragma unroll
    for (int i = 0; i < TT; ++i) {
        const int64_t gm = m0 + row_of(i);
        if (gm >= g.M) continue;
        if constexpr (TT == 2) {
#pragma unroll
            for (int j = 0; j < TT; ++j) {
                const int gn = n0 + col_of(j);
                if (gn < g.N) store_c(g.C, g.c_bf16, gm * g.ldc + gn, acc[i][j] + bias_at(g, gn));
            }
        } else {
#pragma unroll
        for (int h = 0; h < TT / 4; ++h) {
            const int gn = n0 + col_of(h * 4);
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
}

template <int T>
cudaError_t launch_tile(const GemmArgs& g, int a_vec, int b_vec, int c_vec, int kid, cudaStream_t stream)
{
    const int64_t tiles_m = (g.M + T - 1) / T, tiles_n = (g.N + T - 1) / T;
    if (tiles_m * tiles_n > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    const unsigned grid = static_cast<unsigned>(tiles_m * tiles_n);
    if (g.b_col)
        r2_vectorized_kernel<true, T><<<grid, NT, 0, stream>>>(g, (int)tiles_m, (int)tiles_n, a_vec, b_vec, c_vec, kid);
    else
        r2_vectorized_kernel<false, T><<<grid, NT, 0, stream>>>(g, (int)tiles_m, (int)tiles_n, a_vec, b_vec, c_vec, kid);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_r2_vectorized(const GemmArgs& g, cudaStream_t stream, int* kernel_id)
{
    // Preconditions of the 128-bit paths, per operand.
    const int a_vec = (reinterpret_cast<uintptr_t>(g.A) % 16 == 0) && (g.lda % 8 == 0);
    const int b_vec = (reinterpret_cast<uintptr_t>(g.B) % 16 == 0) && (g.ldb % 8 == 0);
    const int c_vec = g.c_bf16 ? ((reinterpret_cast<uintptr_t>(g.C) % 8 == 0) && (g.ldc % 4 == 0))
                               : ((reinterpret_cast<uintptr_t>(g.C) % 16 == 0) && (g.ldc % 4 == 0));
    const int kid = kIdVectorized + a_vec + 2 * b_vec + 4 * c_vec;
    *kernel_id = kid;
    switch (staged_tile_edge(g)) {
        case 128: return launch_tile<128>(g, a_vec, b_vec, c_vec, kid, stream);
        case 64: return launch_tile<64>(g, a_vec, b_vec, c_vec, kid, stream);
        default: return launch_tile<32>(g, a_vec, b_vec, c_vec, kid, stream);
    }
}

}  // namespace klin
