// Rung 3.5 - the legacy warp-level tensor-core path: "ldmatrix.swizzle" and
// "mma (m16n8k16)" (paper, Table 1; preconditions: the tile fits the mma shape,
// fragments come from swizzled shared memory).  It sits between the CUDA-core
// pipeline of rung 3 and the tcgen05 rung: the same 4-stage TMA / mbarrier ring
// (T x T x 32 tiles of raw bf16; T = 128, or 64 when 128 x 128 tiles would leave SMs
// without a CTA), but the multiply is
// mma.sync.aligned.m16n8k16 on fragments fetched with ldmatrix from shared
// memory laid out with TMA's swizzle patterns (64-byte swizzle for K-contiguous
// operands, 128-byte swizzle for the N-contiguous row-major B, read with
// ldmatrix.trans).  8 warps as 2 x 4, each a (T/2) x (T/4) warp tile (4 x 4 or 2 x 2 mma
// tiles, fp32 accumulators in registers).  On sm_100a this path compiles and runs but
// cannot reach tcgen05 throughput: it is kept as the lineage's intermediate step.
// Operands that break TMA's alignment rules take the producer-thread path of
// rung 3 (masked scalar loads written into the same swizzled layout).
#include "common.cuh"
#include "ptx.cuh"
#include <cstring>

namespace klin {
namespace {

constexpr int BK = 32, STAGES = 4, NT = 256;
constexpr int smem_bytes(int T) { return STAGES * (2 * T * BK * 2) + 1024 /*alignment slack*/ + 128 /*barriers*/; }

// Byte offsets of a 16-byte chunk (8 bf16) inside a stage.
//   K-contiguous operand (A; column-major B): [row][32 k], 64-byte rows, chunk index XORed
//   with (row >> 1) & 3 - the pattern TMA's 64-byte swizzle produces.
//   row-major B: two blocks of [32 k][64 n], 128-byte rows, chunk index XORed with k & 7
//   (TMA's 128-byte swizzle).
__device__ __forceinline__ int kmajor_chunk_off(int row, int kchunk) { return row * 64 + ((kchunk ^ ((row >> 1) & 3)) << 4); }
__device__ __forceinline__ int brow_chunk_off(int k, int nchunk)
{
    return (nchunk >> 3) * 4096 + k * 128 + (((nchunk & 7) ^ (k & 7)) << 4);
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// D (fp32, 16x8) += A (bf16, 16x16, row) * B (bf16, 16x8, col)
__device__ __forceinline__ void mma_m16n8k16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 gather8(const uint16_t* p, int valid)
{
    uint16_t v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = (e < valid) ? p[e] : uint16_t(0);
    uint4 r;
    r.x = v[0] | (uint32_t(v[1]) << 16);
    r.y = v[2] | (uint32_t(v[3]) << 16);
    r.z = v[4] | (uint32_t(v[5]) << 16);
    r.w = v[6] | (uint32_t(v[7]) << 16);
    return r;
}

template <bool BCOL, bool TMA, int T>
__global__ void __launch_bounds__(NT)
r35_mma_sync_kernel(GemmArgs g, const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                    int tiles_m, int tiles_n, int c_vec, int kid)
{
    constexpr int BM = T, BN = T;
    constexpr int kABytes = BM * BK * 2, kBBytes = BN * BK * 2, kStageBytes = kABytes + kBBytes;
    constexpr int MI = T / 32;                         // m16 tiles per warp (warp tile T/2 rows)
    constexpr int NJJ = T / 64;                        // pairs of n8 tiles per warp (warp tile T/4 columns)
    constexpr int kChunks = T * BK / 8;                // 16-byte chunks of one operand block
    constexpr int kPer = (kChunks + NT - 1) / NT;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * kStageBytes);
    uint64_t* empty = full + STAGES;
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(empty + STAGES);

    const int t = threadIdx.x;
    const int warp = t >> 5, lane = t & 31;
    const int wm = (warp >> 2) * (T / 2), wn = (warp & 3) * (T / 4);   // origin of the warp tile inside the block tile
    if (blockIdx.x == 0 && t == 0) g.status[1] = kid;

    int tm, tn;
    raster_tile(blockIdx.x, tiles_m, tiles_n, tm, tn);
    const int m0 = tm * BM, n0 = tn * BN;
    const int nkb = (g.K + BK - 1) / BK;

    if (t == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(&full[s], TMA ? 1 : NT);
            ptx::mbar_init(&empty[s], NT / 32);
        }
        abort_flag[0] = 0;
        abort_flag[1] = 0;   // a word that stays 0, for waits that must not be cut short
        ptx::fence_barrier_init();
        if (TMA) {
            ptx::prefetch_tensormap(&map_a);
            ptx::prefetch_tensormap(&map_b);
        }
    }
    __syncthreads();

    bool ok = true;
    int issued = 0;   // thread 0, TMA path: k-blocks whose loads were issued

    auto issue_tma = [&](int kb) {
        const int s = kb % STAGES;
        uint8_t* sa = smem + s * kStageBytes;
        ptx::mbar_arrive_expect_tx(&full[s], kStageBytes);
        ptx::tma_load_2d(sa, &map_a, kb * BK, m0, &full[s]);
        if (BCOL) {
            ptx::tma_load_2d(sa + kABytes, &map_b, kb * BK, n0, &full[s]);
        } else {
            ptx::tma_load_2d(sa + kABytes, &map_b, n0, kb * BK, &full[s]);
            if (BN > 64) ptx::tma_load_2d(sa + kABytes + 4096, &map_b, n0 + 64, kb * BK, &full[s]);
        }
        issued = kb + 1;
    };

    // Producer-thread path: up to kPer 16-byte chunks of A and of B per thread and stage.
    uint4 pre[2 * kPer];
    auto fetch_regs = [&](int kb) {
        const int k0 = kb * BK;
#pragma unroll
        for (int q = 0; q < kPer; ++q) {
            const int c = t + NT * q;
            if (c >= kChunks) break;
            {                                  // A: row c/4, k-chunk c%4
                const int r = c >> 2, kc = c & 3;
                const int64_t gm = m0 + r;
                const int gk = k0 + kc * 8;
                const int valid = (gm < g.M) ? min(8, max(0, g.K - gk)) : 0;
                pre[q] = gather8(g.A + gm * g.lda + gk, valid);
            }
            if (BCOL) {                        // B column-major: column c/4, k-chunk c%4
                const int n = c >> 2, kc = c & 3;
                const int64_t gn = n0 + n;
                const int gk = k0 + kc * 8;
                const int valid = (gn < g.N) ? min(8, max(0, g.K - gk)) : 0;
                pre[kPer + q] = gather8(g.B + gn * g.ldb + gk, valid);
            } else {                           // B row-major: k-row c / (T/8), n-chunk c % (T/8)
                const int k = c / (BN / 8), nc = c % (BN / 8);
                const int64_t gk = k0 + k;
                const int gn = n0 + nc * 8;
                const int valid = (gk < g.K) ? min(8, max(0, g.N - gn)) : 0;
                pre[kPer + q] = gather8(g.B + gk * g.ldb + gn, valid);
            }
        }
    };
    auto store_regs = [&](int kb) {
        uint8_t* sa = smem + (kb % STAGES) * kStageBytes;
        uint8_t* sb = sa + kABytes;
#pragma unroll
        for (int q = 0; q < kPer; ++q) {
            const int c = t + NT * q;
            if (c >= kChunks) break;
            *reinterpret_cast<uint4*>(sa + kmajor_chunk_off(c >> 2, c & 3)) = pre[q];
            if (BCOL)
                *reinterpret_cast<uint4*>(sb + kmajor_chunk_off(c >> 2, c & 3)) = pre[kPer + q];
            else
                *reinterpret_cast<uint4*>(sb + brow_chunk_off(c / (BN / 8), c % (BN / 8))) = pre[kPer + q];
        }
        ptx::mbar_arrive(&full[kb % STAGES]);
    };

    // Prologue: fill the first STAGES-1 stages.
    if (TMA) {
        if (t == 0)
            for (int kb = 0; kb < STAGES - 1 && kb < nkb; ++kb) issue_tma(kb);
    } else {
        for (int kb = 0; kb < STAGES - 1 && kb < nkb; ++kb) {
            fetch_regs(kb);
            store_regs(kb);
        }
    }

    float acc[MI][2 * NJJ][4];   // [m16 tile][n8 tile][fragment register]
#pragma unroll
    for (int i = 0; i < MI; ++i)
#pragma unroll
        for (int j = 0; j < 2 * NJJ; ++j)
#pragma unroll
            for (int r = 0; r < 4; ++r) acc[i][j][r] = 0.f;

    for (int kb = 0; kb < nkb && ok; ++kb) {
        const int s = kb % STAGES;
        const int nk = kb + STAGES - 1;            // k-block to fetch now
        const bool more = nk < nkb;
        const int ns = nk % STAGES, nf = nk / STAGES;
        if (more) {
            if (TMA) {
                if (t == 0) {
                    if (nf > 0 && !ptx::mbar_wait(&empty[ns], (nf - 1) & 1, abort_flag)) {
                        report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x300u | ns);
                        *abort_flag = 1;
                    } else {
                        issue_tma(nk);
                    }
                }
            } else {
                fetch_regs(nk);
            }
        }
        if (!ptx::mbar_wait(&full[s], (kb / STAGES) & 1, abort_flag)) {
            report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x310u | s);
            *abort_flag = 1;
            ok = false;
            break;
        }

        const uint32_t sa = ptx::smem_u32(smem + s * kStageBytes);
        const uint32_t sb = sa + kABytes;
#pragma unroll
        for (int k16 = 0; k16 < BK / 16; ++k16) {
            uint32_t af[MI][4], bf[NJJ][4];
            // A fragments: lanes 0-15 address rows 0-15 at k chunk 2*k16, lanes 16-31 the same rows at the next chunk
#pragma unroll
            for (int i = 0; i < MI; ++i)
                ldmatrix_x4(sa + kmajor_chunk_off(wm + i * 16 + (lane & 15), k16 * 2 + (lane >> 4)), af[i]);
            // B fragments, two n8 tiles per ldmatrix.x4: registers {b0, b1} of tile 2*jj, then of tile 2*jj+1
#pragma unroll
            for (int jj = 0; jj < NJJ; ++jj) {
                if (BCOL) {
                    const int n = wn + jj * 16 + ((lane >> 4) << 3) + (lane & 7);
                    ldmatrix_x4(sb + kmajor_chunk_off(n, k16 * 2 + ((lane >> 3) & 1)), bf[jj]);
                } else {
                    const int k = k16 * 16 + (((lane >> 3) & 1) << 3) + (lane & 7);
                    ldmatrix_x4_trans(sb + brow_chunk_off(k, ((wn + jj * 16) >> 3) + (lane >> 4)), bf[jj]);
                }
            }
#pragma unroll
            for (int i = 0; i < MI; ++i)
#pragma unroll
                for (int j = 0; j < 2 * NJJ; ++j)
                    mma_m16n8k16(acc[i][j], af[i], bf[j >> 1][(j & 1) * 2], bf[j >> 1][(j & 1) * 2 + 1]);
        }
        __syncwarp();
        if ((t & 31) == 0) ptx::mbar_arrive(&empty[s]);

        if (!TMA && more) {
            if (nf > 0 && !ptx::mbar_wait(&empty[ns], (nf - 1) & 1, abort_flag)) {
                report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x320u | ns);
                *abort_flag = 1;
                ok = false;
                break;
            }
            store_regs(nk);
        }
    }

    if (*abort_flag) ok = false;
    if (!ok) {
        // Give-up path: let loads already issued land before the CTA's shared
        // memory is released (bounded), then leave without writing C.
        if (TMA && t == 0) {
            for (int j = max(0, issued - STAGES); j < issued; ++j)
                ptx::mbar_wait(&full[j % STAGES], (j / STAGES) & 1, abort_flag + 1 /* never set */);
        }
        return;
    }

    // Epilogue: fragment register r of tile (i, j) is C[wm + 16 i + lane/4 + 8 (r/2)][wn + 8 j + 2 (lane%4) + r%2].
#pragma unroll
    for (int i = 0; i < MI; ++i)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int64_t gm = m0 + wm + i * 16 + (lane >> 2) + h * 8;
            if (gm >= g.M) continue;
#pragma unroll
            for (int j = 0; j < 2 * NJJ; ++j) {
                const int gn = n0 + wn + j * 8 + (lane & 3) * 2;
                const float v0 = acc[i][j][h * 2] + (gn < g.N ? bias_at(g, gn) : 0.f);
                const float v1 = acc[i][j][h * 2 + 1] + (gn + 1 < g.N ? bias_at(g, gn + 1) : 0.f);
                if (g.c_bf16) {
                    uint16_t* d = static_cast<uint16_t*>(g.C) + gm * g.ldc + gn;
                    if (gn + 1 < g.N && (reinterpret_cast<uintptr_t>(d) & 3) == 0) {
                        *reinterpret_cast<uint32_t*>(d) = pack_bf16x2(v0, v1);
                    } else {
                        if (gn < g.N) d[0] = float_to_bf16_bits(v0);
                        if (gn + 1 < g.N) d[1] = float_to_bf16_bits(v1);
                    }
                } else {
                    float* d = static_cast<float*>(g.C) + gm * g.ldc + gn;
                    if (gn + 1 < g.N && (reinterpret_cast<uintptr_t>(d) & 7) == 0) {
                        *reinterpret_cast<float2*>(d) = make_float2(v0, v1);
                    } else {
                        if (gn < g.N) d[0] = v0;
                        if (gn + 1 < g.N) d[1] = v1;
                    }
                }
            }
        }
}

template <bool BCOL, bool TMA, int T>
cudaError_t launch(const GemmArgs& g, const CUtensorMap& ma, const CUtensorMap& mb, int tiles_m, int tiles_n, int c_vec,
                   int kid, int device, cudaStream_t stream)
{
    auto kern = r35_mma_sync_kernel<BCOL, TMA, T>;
    static bool attr_set[64] = {};   // per instantiation and device
    if (device < 0 || device >= 64 || !attr_set[device]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(T));
        if (e != cudaSuccess) return e;
        if (device >= 0 && device < 64) attr_set[device] = true;
    }
    kern<<<static_cast<unsigned>(tiles_m) * tiles_n, NT, smem_bytes(T), stream>>>(g, ma, mb, tiles_m, tiles_n, c_vec, kid);
    return cudaGetLastError();
}

// TMA's rules for a 2-D bf16 operand: 16-byte aligned base, row pitch a
// multiple of 16 bytes and below 2^40.
bool tma_ok35(const void* base, int64_t ld_elems)
{
    return reinterpret_cast<uintptr_t>(base) % 16 == 0 && (ld_elems * 2) % 16 == 0 && ld_elems * 2 < (1ll << 40);
}

template <int T>
cudaError_t launch_tile(const GemmArgs& g, RunContext& ctx, cudaStream_t stream, int* kernel_id)
{
    const int64_t tiles_m = (g.M + T - 1) / T, tiles_n = (g.N + T - 1) / T;
    if (tiles_m * tiles_n > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    const bool tma = ctx.encode_tiled && tma_ok35(g.A, g.lda) && tma_ok35(g.B, g.ldb);
    const int c_vec = (reinterpret_cast<uintptr_t>(g.C) % 16 == 0) && (g.ldc % (g.c_bf16 ? 8 : 4) == 0);
    CUtensorMap ma, mb;
    memset(&ma, 0, sizeof ma);
    memset(&mb, 0, sizeof mb);
    if (tma) {
        bool ok = encode_map_2d(ctx, &ma, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.A, g.K, g.M, g.lda * 2, BK, T,
                                CU_TENSOR_MAP_SWIZZLE_64B);
        if (g.b_col)
            ok = ok && encode_map_2d(ctx, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B, g.K, g.N, g.ldb * 2, BK, T,
                                     CU_TENSOR_MAP_SWIZZLE_64B);
        else
            ok = ok && encode_map_2d(ctx, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B, g.N, g.K, g.ldb * 2, 64, BK,
                                     CU_TENSOR_MAP_SWIZZLE_128B);
        if (!ok) return cudaErrorInvalidValue;
    }
    const int kid = kIdMmaSync + (tma ? 0 : 1);
    *kernel_id = kid;
    const int tmi = static_cast<int>(tiles_m), tni = static_cast<int>(tiles_n);
    if (g.b_col)
        return tma ? launch<true, true, T>(g, ma, mb, tmi, tni, c_vec, kid, ctx.device, stream)
                   : launch<true, false, T>(g, ma, mb, tmi, tni, c_vec, kid, ctx.device, stream);
    return tma ? launch<false, true, T>(g, ma, mb, tmi, tni, c_vec, kid, ctx.device, stream)
               : launch<false, false, T>(g, ma, mb, tmi, tni, c_vec, kid, ctx.device, stream);
}

}  // namespace

cudaError_t launch_r35_mma_sync(const GemmArgs& g, RunContext& ctx, cudaStream_t stream, int* kernel_id)
{
    // 64 x 64 tiles when 128 x 128 tiles would leave SMs without a CTA (the rule of the staged rungs)
    return staged_tile_edge(g) == 128 ? launch_tile<128>(g, ctx, stream, kernel_id)
                                      : launch_tile<64>(g, ctx, stream, kernel_id);
}

}  // namespace klin
