// Rung 3 - "cp.async + pipeline" / "tma_load" (paper, Table 1; preconditions:
// data movement is shared-memory staged, the TMA descriptor is encoded;
// Introduction: a pipeline presupposes that data movement is staged).
//
// T x T x 32 tiles (T = 128, 64 or 32: the largest whose grid still gives every SM a CTA,
// as in rungs 1 and 2), a ring of 4 shared-memory stages holding RAW bf16, a
// full/empty mbarrier pair per stage with phase parity.  Loads for k-block
// kb+3 are in flight while k-block kb is multiplied (fp32 FMA on CUDA cores,
// bf16 -> fp32 widening when a value is read from shared memory).  With no
// global loads or shared-memory stores left in the issue stream, the multiply
// uses sm_100's packed fma.rn.f32x2 (two independent fp32 FMAs per instruction,
// same rounding as scalar fmaf), which leaves issue slots for the widening.
//
//   TMA path (A, B 16-byte aligned with 16-byte-multiple row pitch): one
//   thread issues cp.async.bulk.tensor loads that complete on the stage's
//   "full" barrier by byte count; out-of-range rows/columns/k are zero-filled
//   by the hardware, so tails cost nothing.
//   Producer-thread path (TMA's alignment rules fail): all threads fetch the
//   next stage with masked scalar loads into registers before the multiply and
//   store it into the same ring afterwards, arriving on the same barriers.
//
// No warp is dedicated to loading yet; that split is rung 4's.
#include "common.cuh"
#include "ptx.cuh"
#include <cstring>

namespace klin {
namespace {

constexpr int BK = 32, STAGES = 4, NT = 256;
// Shared memory of a T x T tile: STAGES x (A block + B block of T x 32 bf16 each), alignment slack, barriers.
constexpr int smem_bytes(int T) { return STAGES * (2 * T * BK * 2) + 1024 + 128; }

// Byte offset of B element group inside a stage's B block.
//   row-major   B: [k][128 n] dense, 256-byte rows
//   column-major B: [n][32 k], 64-byte rows, 16-byte chunk index XORed with
//   (n >> 1) & 3 - the pattern TMA's 64-byte swizzle produces.
__device__ __forceinline__ int b_col_chunk_off(int n, int kchunk) { return n * 64 + ((kchunk ^ ((n >> 1) & 3)) << 4); }

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
r3_pipelined_kernel(GemmArgs g, const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                    int tiles_m, int tiles_n, int c_vec, int kid)
{
    constexpr int BM = T, BN = T;
    constexpr int TT = T / 16;                         // register tile edge: rows ty + 16 i, TT columns per thread
    constexpr int kABytes = BM * BK * 2, kBBytes = BN * BK * 2, kStageBytes = kABytes + kBBytes;
    constexpr int kChunks = T * BK / 8;                // 16-byte chunks of one operand block
    constexpr int kPer = (kChunks + NT - 1) / NT;      // chunks of each operand a thread moves on the producer-thread path
    constexpr int kBRow = BN * 2;                      // bytes of one k-row of a row-major B block
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * kStageBytes);
    uint64_t* empty = full + STAGES;
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(empty + STAGES);

    const int t = threadIdx.x;
    const int tx = t % 16, ty = t / 16;
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
        if (BCOL)
            ptx::tma_load_2d(sa + kABytes, &map_b, kb * BK, n0, &full[s]);
        else
            ptx::tma_load_2d(sa + kABytes, &map_b, n0, kb * BK, &full[s]);
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
            *reinterpret_cast<uint4*>(sa + (c >> 2) * 64 + (c & 3) * 16) = pre[q];
            if (BCOL)
                *reinterpret_cast<uint4*>(sb + b_col_chunk_off(c >> 2, c & 3)) = pre[kPer + q];
            else
                *reinterpret_cast<uint4*>(sb + (c / (BN / 8)) * kBRow + (c % (BN / 8)) * 16) = pre[kPer + q];
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

    float2 acc2[TT][TT / 2];   // acc2[i][jp] = accumulators of columns 2*jp and 2*jp+1 of row i
#pragma unroll
    for (int i = 0; i < TT; ++i)
#pragma unroll
        for (int jp = 0; jp < TT / 2; ++jp) acc2[i][jp] = make_float2(0.f, 0.f);

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

        const uint8_t* sa = smem + s * kStageBytes;
        const uint8_t* sb = sa + kABytes;
#pragma unroll
        for (int kk = 0; kk < BK / 8; ++kk) {
            uint32_t aw[TT][4];
#pragma unroll
            for (int i = 0; i < TT; ++i) {
                const uint4 v = *reinterpret_cast<const uint4*>(sa + (ty + 16 * i) * 64 + kk * 16);
                aw[i][0] = v.x; aw[i][1] = v.y; aw[i][2] = v.z; aw[i][3] = v.w;
            }
            if (BCOL) {
                uint32_t bw[TT][4];
#pragma unroll
                for (int j = 0; j < TT; ++j) {
                    const uint4 v = *reinterpret_cast<const uint4*>(sb + b_col_chunk_off(tx + 16 * j, kk));
                    bw[j][0] = v.x; bw[j][1] = v.y; bw[j][2] = v.z; bw[j][3] = v.w;
                }
#pragma unroll
                for (int k8 = 0; k8 < 8; ++k8) {
                    float2 b2[TT / 2];
#pragma unroll
                    for (int jp = 0; jp < TT / 2; ++jp) {
                        b2[jp].x = (k8 & 1) ? bf16_hi(bw[2 * jp][k8 >> 1]) : bf16_lo(bw[2 * jp][k8 >> 1]);
                        b2[jp].y = (k8 & 1) ? bf16_hi(bw[2 * jp + 1][k8 >> 1]) : bf16_lo(bw[2 * jp + 1][k8 >> 1]);
                    }
#pragma unroll
                    for (int i = 0; i < TT; ++i) {
                        const float a = (k8 & 1) ? bf16_hi(aw[i][k8 >> 1]) : bf16_lo(aw[i][k8 >> 1]);
                        const float2 a2 = make_float2(a, a);
#pragma unroll
                        for (int jp = 0; jp < TT / 2; ++jp) acc2[i][jp] = __ffma2_rn(a2, b2[jp], acc2[i][jp]);
                    }
                }
            } else {
#pragma unroll
                for (int k8 = 0; k8 < 8; ++k8) {
                    // this thread's TT consecutive columns of k-row kk * 8 + k8: 16, 8 or 4 bytes
                    uint32_t w[TT / 2];
                    const uint8_t* src = sb + (kk * 8 + k8) * kBRow + tx * (TT * 2);
                    if constexpr (TT == 8) {
                        const uint4 v = *reinterpret_cast<const uint4*>(src);
                        w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
                    } else if constexpr (TT == 4) {
                        const uint2 v = *reinterpret_cast<const uint2*>(src);
                        w[0] = v.x; w[1] = v.y;
                    } else {
                        w[0] = *reinterpret_cast<const uint32_t*>(src);
                    }
                    float2 b2[TT / 2];
#pragma unroll
                    for (int jp = 0; jp < TT / 2; ++jp) b2[jp] = make_float2(bf16_lo(w[jp]), bf16_hi(w[jp]));
#pragma unroll
                    for (int i = 0; i < TT; ++i) {
                        const float a = (k8 & 1) ? bf16_hi(aw[i][k8 >> 1]) : bf16_lo(aw[i][k8 >> 1]);
                        const float2 a2 = make_float2(a, a);
#pragma unroll
                        for (int jp = 0; jp < TT / 2; ++jp) acc2[i][jp] = __ffma2_rn(a2, b2[jp], acc2[i][jp]);
                    }
                }
            }
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

    // Epilogue: rows ty + 16 i; columns tx * TT + j (row-major B) or tx + 16 j.
    float acc[TT][TT];
#pragma unroll
    for (int i = 0; i < TT; ++i)
#pragma unroll
        for (int jp = 0; jp < TT / 2; ++jp) {
            acc[i][2 * jp] = acc2[i][jp].x;
            acc[i][2 * jp + 1] = acc2[i][jp].y;
        }
    if (g.bias) {   // AddMM: the bias of each of this thread's columns
#pragma unroll
        for (int j = 0; j < TT; ++j) {
            const int gn = n0 + (BCOL ? tx + 16 * j : tx * TT + j);
            const float b = gn < g.N ? bias_at(g, gn) : 0.f;
#pragma unroll
            for (int i = 0; i < TT; ++i) acc[i][j] += b;
        }
    }
#pragma unroll
    for (int i = 0; i < TT; ++i) {
        const int64_t gm = m0 + ty + 16 * i;
        if (gm >= g.M) continue;
        if (BCOL) {
#pragma unroll
            for (int j = 0; j < TT; ++j) {
                const int gn = n0 + tx + 16 * j;
                if (gn < g.N) store_c(g.C, g.c_bf16, gm * g.ldc + gn, acc[i][j]);
            }
        } else {
            const int gn = n0 + tx * TT;
            bool done = false;
            if constexpr (TT == 8) {
                if (c_vec && gn + 8 <= g.N) {
                    if (g.c_bf16) {
                        uint4 w = make_uint4(pack_bf16x2(acc[i][0], acc[i][1]), pack_bf16x2(acc[i][2], acc[i][3]),
                                             pack_bf16x2(acc[i][4], acc[i][5]), pack_bf16x2(acc[i][6], acc[i][7]));
                        *reinterpret_cast<uint4*>(static_cast<uint16_t*>(g.C) + gm * g.ldc + gn) = w;
                    } else {
                        float* p = static_cast<float*>(g.C) + gm * g.ldc + gn;
                        *reinterpret_cast<float4*>(p) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
                        *reinterpret_cast<float4*>(p + 4) = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
                    }
                    done = true;
                }
            } else if constexpr (TT == 4) {
                if (c_vec && gn + 4 <= g.N) {      // (C 16-byte aligned, pitch a multiple of 16 bytes: 4 columns are 8 / 16 bytes)
                    if (g.c_bf16)
                        *reinterpret_cast<uint2*>(static_cast<uint16_t*>(g.C) + gm * g.ldc + gn) =
                            make_uint2(pack_bf16x2(acc[i][0], acc[i][1]), pack_bf16x2(acc[i][2], acc[i][3]));
                    else
                        *reinterpret_cast<float4*>(static_cast<float*>(g.C) + gm * g.ldc + gn) =
                            make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
                    done = true;
                }
            }
            if (!done) {
#pragma unroll
                for (int j = 0; j < TT; ++j)
                    if (gn + j < g.N) store_c(g.C, g.c_bf16, gm * g.ldc + gn + j, acc[i][j]);
            }
        }
    }
}

template <bool BCOL, bool TMA, int T>
cudaError_t launch(const GemmArgs& g, const CUtensorMap& ma, const CUtensorMap& mb, int tiles_m, int tiles_n, int c_vec,
                   int kid, int device, cudaStream_t stream)
{
    auto kern = r3_pipelined_kernel<BCOL, TMA, T>;
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
bool tma_ok(const void* base, int64_t ld_elems)
{
    return reinterpret_cast<uintptr_t>(base) % 16 == 0 && (ld_elems * 2) % 16 == 0 && ld_elems * 2 < (1ll << 40);
}

template <int T>
cudaError_t launch_tile(const GemmArgs& g, RunContext& ctx, cudaStream_t stream, int* kernel_id)
{
    const int64_t tiles_m = (g.M + T - 1) / T, tiles_n = (g.N + T - 1) / T;
    if (tiles_m * tiles_n > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    const bool tma = ctx.encode_tiled && tma_ok(g.A, g.lda) && tma_ok(g.B, g.ldb);
    const int c_vec = (reinterpret_cast<uintptr_t>(g.C) % 16 == 0) && (g.ldc % (g.c_bf16 ? 8 : 4) == 0);
    CUtensorMap ma, mb;
    memset(&ma, 0, sizeof ma);
    memset(&mb, 0, sizeof mb);
    if (tma) {
        bool ok = encode_map_2d(ctx, &ma, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.A, g.K, g.M, g.lda * 2, BK, T,
                                CU_TENSOR_MAP_SWIZZLE_NONE);
        if (g.b_col)
            ok = ok && encode_map_2d(ctx, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B, g.K, g.N, g.ldb * 2, BK, T,
                                     CU_TENSOR_MAP_SWIZZLE_64B);
        else
            ok = ok && encode_map_2d(ctx, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B, g.N, g.K, g.ldb * 2, T, BK,
                                     CU_TENSOR_MAP_SWIZZLE_NONE);
        if (!ok) return cudaErrorInvalidValue;
    }
    const int kid = kIdPipelined + (tma ? 0 : 1);
    *kernel_id = kid;
    const int tmi = static_cast<int>(tiles_m), tni = static_cast<int>(tiles_n);
    if (g.b_col)
        return tma ? launch<true, true, T>(g, ma, mb, tmi, tni, c_vec, kid, ctx.device, stream)
                   : launch<true, false, T>(g, ma, mb, tmi, tni, c_vec, kid, ctx.device, stream);
    return tma ? launch<false, true, T>(g, ma, mb, tmi, tni, c_vec, kid, ctx.device, stream)
               : launch<false, false, T>(g, ma, mb, tmi, tni, c_vec, kid, ctx.device, stream);
}

}  // namespace

cudaError_t launch_r3_pipelined(const GemmArgs& g, RunContext& ctx, cudaStream_t stream, int* kernel_id)
{
    switch (staged_tile_edge(g)) {
        case 128: return launch_tile<128>(g, ctx, stream, kernel_id);
        case 64: return launch_tile<64>(g, ctx, stream, kernel_id);
        default: return launch_tile<32>(g, ctx, stream, kernel_id);
    }
}

}  // namespace klin
