// Rung 1 - "tile / sm_stage" (paper, Table 1; precondition: loops over the
// output).  A T x T block tile of C per CTA (T = 128, 64 or 32); A and B k-slabs
// of depth 16 or 32 are staged in shared memory as fp32 (converted from bf16 on the way
// in) and each of the 256 threads keeps a (T/16) x (T/16) register tile.  Loads
// are scalar and masked element by element, so every M/N/K tail and every
// alignment is handled the same way; nothing is vectorized or overlapped yet.
//
// Two CTAs share an SM (the register tile is capped at 128 registers per thread for it): one CTA's slab fill overlaps
// the other's arithmetic, which is all the overlap this rung has (8192^3: 20.3 -> 29.5 TFLOP/s at the time).
//
// In the 128 tile a thread's rows and columns come in groups of four consecutive ones (rows 4 ty + i and 64 + 4 ty + i,
// columns likewise with tx): one 16-byte shared-memory read fetches a group, 4 reads per 64 FMAs instead of 16 scalar
// ones (the 16 threads of a half warp read 256 consecutive bytes of a row of B and all the same 16 bytes of A), and
// a half warp's stores to C cover 64 consecutive elements: 8192^3 29.5 -> 37.6 TFLOP/s, 4096^3 34.1 -> 38.0.  (With
// columns tx * 8 + j - eight consecutive ones - the reads of B were four-way bank conflicts and the rung ran at a
// quarter of the fp32 pipe.)  The 64 and 32 tiles keep rows ty + 16 i and columns tx + 16 j, read word by word.
//
// The tile is the largest of the three that still gives every SM a CTA: a
// 256^3 product is 4 tiles of 128 x 128 but 64 of 32 x 32, and a rung that
// stages through shared memory should not be slower than the naive kernel just
// because most of the GPU has nothing to do.
#include "common.cuh"

namespace klin {
namespace {

constexpr int NT = 256;

template <bool BCOL, int T>
__global__ void __launch_bounds__(NT, 2) r1_tiled_kernel(GemmArgs g, int tiles_m, int tiles_n)
{
    constexpr int TT = T / 16;                 // register tile edge
    // k-slab depth: 16 for the 128 tile; 32 for the smaller ones, which synchronise twice per slab for a quarter or a
    // sixteenth of the arithmetic (measured: 16 x 8192 x 8192 535 -> 426 us, 1000 x 1001 x 999 105 -> 99 us; at 128
    // the deeper slab was slower, 8192^3 29.5 -> 27.3 TFLOP/s)
    constexpr int BK = T == 128 ? 16 : 32;
    // a warp covers 16 k of 2 rows: 2 mod 32 spreads them over 32 banks; 32 k of one row with the deeper slab: 1 mod 32
    // 128 tile: rows stay 16-byte aligned for the register tile's vector reads; smaller tiles: a warp's fill covers 32 k
    // of one row, 1 mod 32 spreads them over the banks
    constexpr int PITCH = T == 128 ? T + 4 : T + 1;
    // fill loops: eight loads in flight push the 128 tile past its 128 registers (spills); the smaller tiles want them all
    constexpr int FILL_UNROLL = T == 128 ? 4 : 8;
    // a thread's rows (columns) come in groups of V consecutive ones: 4 for the 128 tile (vector reads), else single
    // rows ty + 16 i and columns tx + 16 j read word by word (the smaller tiles stay as plain as the rung's name)
    constexpr int V = T == 128 ? 4 : 1;
    __shared__ __align__(16) float As[BK][PITCH];
    __shared__ __align__(16) float Bs[BK][PITCH];
    if (blockIdx.x == 0 && threadIdx.x == 0) g.status[1] = kIdTiled;

    int tm, tn;
    raster_tile(blockIdx.x, tiles_m, tiles_n, tm, tn);
    const int m0 = tm * T, n0 = tn * T;
    const int t = threadIdx.x;
    const int tx = t % 16, ty = t / 16;

    float acc[TT][TT];
#pragma unroll
    for (int i = 0; i < TT; ++i)
#pragma unroll
        for (int j = 0; j < TT; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < g.K; k0 += BK) {
        // A slab: T rows x 16 k, one element per thread per step, k fastest.
#pragma unroll FILL_UNROLL
        for (int e = t; e < T * BK; e += NT) {
            const int k = e % BK, m = e / BK;
            const int64_t gm = m0 + m;
            const int gk = k0 + k;
            As[k][m] = (gm < g.M && gk < g.K) ? bf16_bits_to_float(g.A[gm * g.lda + gk]) : 0.f;
        }
        if (BCOL) {
#pragma unroll FILL_UNROLL
            for (int e = t; e < T * BK; e += NT) {
                const int k = e % BK, n = e / BK;
                const int64_t gn = n0 + n;
                const int gk = k0 + k;
                Bs[k][n] = (gn < g.N && gk < g.K) ? bf16_bits_to_float(g.B[gn * g.ldb + gk]) : 0.f;
            }
        } else {
#pragma unroll FILL_UNROLL
            for (int e = t; e < T * BK; e += NT) {
                const int n = e % T, k = e / T;
                const int64_t gn = n0 + n;
                const int64_t gk = k0 + k;
                Bs[k][n] = (gn < g.N && gk < g.K) ? bf16_bits_to_float(g.B[gk * g.ldb + gn]) : 0.f;
            }
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            float a[TT], b[TT];
#pragma unroll
            for (int i = 0; i < TT; i += V) {
                const float* pa = &As[k][(i / V) * 16 * V + ty * V];
                const float* pb = &Bs[k][(i / V) * 16 * V + tx * V];
                if (V == 4) {
                    *reinterpret_cast<float4*>(&a[i]) = *reinterpret_cast<const float4*>(pa);
                    *reinterpret_cast<float4*>(&b[i]) = *reinterpret_cast<const float4*>(pb);
                } else {
                    a[i] = *pa;
                    b[i] = *pb;
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
        const int64_t gm = m0 + (i / V) * 16 * V + ty * V + (i % V);
        if (gm >= g.M) continue;
#pragma unroll
        for (int j = 0; j < TT; ++j) {
            const int64_t gn = n0 + (j / V) * 16 * V + tx * V + (j % V);
            if (gn < g.N) store_c(g.C, g.c_bf16, gm * g.ldc + gn, acc[i][j] + bias_at(g, gn));
        }
    }
}

template <int T>
cudaError_t launch_tile(const GemmArgs& g, cudaStream_t stream)
{
    const int64_t tiles_m = (g.M + T - 1) / T, tiles_n = (g.N + T - 1) / T;
    if (tiles_m * tiles_n > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    const unsigned grid = static_cast<unsigned>(tiles_m * tiles_n);
    if (g.b_col)
        r1_tiled_kernel<true, T><<<grid, NT, 0, stream>>>(g, (int)tiles_m, (int)tiles_n);
    else
        r1_tiled_kernel<false, T><<<grid, NT, 0, stream>>>(g, (int)tiles_m, (int)tiles_n);
    return cudaGetLastError();
}

}  // namespace

// Edge of the square block tile the staged rungs (1 to 3) use for a problem: the largest of 128 / 64 / 32
// whose grid still has a CTA for every SM, else 32.
int staged_tile_edge(const GemmArgs& g)
{
    int sms = 148;
    int dev = 0;
    static int cached_sms[64] = {};
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) {
        if (cached_sms[dev] == 0 &&
            cudaDeviceGetAttribute(&cached_sms[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            cudaGetLastError();
            cached_sms[dev] = 148;
        }
        sms = cached_sms[dev];
    } else {
        cudaGetLastError();
    }
    for (int t : {128, 64}) {
        const int64_t tiles = static_cast<int64_t>((g.M + t - 1) / t) * ((g.N + t - 1) / t);
        if (tiles >= sms) return t;
    }
    return 32;
}

cudaError_t launch_r1_tiled(const GemmArgs& g, cudaStream_t stream, int* kernel_id)
{
    *kernel_id = kIdTiled;
    switch (staged_tile_edge(g)) {
        case 128: return launch_tile<128>(g, stream);
        case 64: return launch_tile<64>(g, stream);
        default: return launch_tile<32>(g, stream);
    }
}

}  // namespace klin
