// Shared declarations of the GEMM lineage kernels: the argument block every
// rung receives, device-side status codes, bf16 helpers and the tile raster.
#pragma once
#include <cstdint>
#include <cuda.h>          // CUtensorMap and its enums only; libcuda is never linked
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

namespace klin {

// Problem description handed to every rung.  A is row-major M x K; B is K x N,
// row-major (b_col == 0: element (k,j) at B[k*ldb + j]) or column-major
// (b_col == 1: element (k,j) at B[j*ldb + k]); C is row-major M x N, fp32 or
// bf16.  Leading dimensions are in elements.  status points at the handle's
// device status block: status[0] = first device-side error code (0 = none),
// status[1] = id of the kernel that ran last, status[2..3] = error detail.
struct GemmArgs {
    int M, N, K;
    const uint16_t* A;
    int64_t lda;
    const uint16_t* B;
    int64_t ldb;
    void* C;
    int64_t ldc;
    int b_col;
    int c_bf16;
    unsigned* status;
    const uint16_t* bias;   // optional: N bf16 values added to every row of A.B (AddMM); nullptr = plain GEMM
    int f16 = 0;            // 1: operands are fp16 and a 2-byte C is fp16 (Conv2d as implicit GEMM); 0: bf16
};

// Device-side error codes written to status[0].
enum DeviceError : unsigned {
    kDevOk = 0,
    kDevBarrierTimeout = 1,   // a bounded mbarrier wait gave up
};

// Kernel ids written to status[1] and reported by klineage_gemm_last_kernel_id().
enum KernelId : int {
    kIdNaive = 0,
    kIdTiled = 100,
    kIdVectorized = 200,      // + 1 (A vector loads) + 2 (B vector loads) + 4 (C vector stores)
    kIdPipelined = 300,       // + 1 when the producer-thread path replaces TMA
    kIdTcgen05 = 400,         // + 1 generic-proxy producer, + 2 direct epilogue, + 4 split-K, + 8 skinny (swapped operands), + 16 cluster reduce, + 32 CTA pair,
                              // + 64 unaligned operands repacked into the workspace first, + 128 last wave of pair tiles streamed along K
    kIdMmaSync = 500,         // rung 3.5 (mma.sync); + 1 when the producer-thread path replaces TMA
    kIdConvNaive = 600,       // direct convolution, one thread per output
    kIdConvTcgen05 = 700,     // implicit GEMM on the tcgen05 rung, patches by TMA; + 4 patches gathered by producer threads,
                              // + 1 gathered element by element (C % 8 != 0 or unaligned x), + 2 direct epilogue
                              // 708: transposed orientation (F <= 128: filters as the 128-row operand, two patch tiles per unit)
    kIdZeroFill = 900,
};

__device__ __forceinline__ float bf16_bits_to_float(uint16_t h)
{
    return __uint_as_float(static_cast<uint32_t>(h) << 16);
}
// Low / high half of a packed pair of bf16 values.
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ uint16_t float_to_bf16_bits(float f)
{
    return __bfloat16_as_ushort(__float2bfloat16_rn(f));
}
// Two floats -> packed bf16x2 (lo in bits 0..15), round to nearest even.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    // one packed conversion instruction (cvt.rn.bf16x2.f32) instead of two scalar ones and a merge
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// Two floats -> packed 16-bit pair in the output type (bf16 or fp16), round to nearest even.
__device__ __forceinline__ uint32_t pack_out2(float lo, float hi, int f16)
{
    if (f16) {
        const __half2 h = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<const uint32_t*>(&h);
    }
    return pack_bf16x2(lo, hi);
}

// Geometry of a channels-last Conv2d run as an implicit GEMM (paper, Evaluation, Table 2: Conv2d):
// x (N, H, W, C), w (F, R, S, C), y (N, P, Q, F); GEMM row m = (n, p, q), column f, k = (r, s, c).
struct ConvGeom {
    int H, W, C, P, Q, R, S;
    int pad_h, pad_w, stride_h, stride_w;
};

// The bias of column `col` (0 when the call has none); col must be < N.
__device__ __forceinline__ float bias_at(const GemmArgs& g, int64_t col)
{
    return g.bias ? bf16_bits_to_float(__ldg(g.bias + col)) : 0.f;
}

__device__ __forceinline__ void store_c(void* C, int c_bf16, int64_t idx, float v)
{
    if (c_bf16)
        static_cast<uint16_t*>(C)[idx] = float_to_bf16_bits(v);
    else
        static_cast<float*>(C)[idx] = v;
}

__device__ __forceinline__ void report_error(unsigned* status, unsigned code, unsigned d0, unsigned d1)
{
    if (atomicCAS(&status[0], 0u, code) == 0u) {
        status[2] = d0;
        status[3] = d1;
    }
}

// Tile raster shared by the tiled rungs: linear tile index -> (tile_m, tile_n),
// walking groups of kGroupM tile-rows column by column so that the tiles in
// flight together share A row-panels and B column-panels in L2.
constexpr int kGroupM = 8;
__host__ __device__ __forceinline__ void raster_tile(int64_t t, int tiles_m, int tiles_n, int& tm, int& tn,
                                                     int group_m = kGroupM)
{
    if (tiles_m == 1) {   // one tile-row (the skinny orientation): no arithmetic on the critical path of short kernels
        tm = 0;
        tn = static_cast<int>(t);
        return;
    }
    const int64_t per_group = static_cast<int64_t>(group_m) * tiles_n;
    if (t < 0x7FFFFFFFll && per_group < 0x7FFFFFFFll) {
        // the common case in 32-bit arithmetic: a 64-bit division costs hundreds of cycles on the
        // critical path of short kernels
        const uint32_t t32 = static_cast<uint32_t>(t), pg = static_cast<uint32_t>(per_group);
        const uint32_t g = t32 / pg;
        const int first_m = static_cast<int>(g) * group_m;
        const uint32_t rows = static_cast<uint32_t>((tiles_m - first_m < group_m) ? (tiles_m - first_m) : group_m);
        const uint32_t r = t32 - g * pg;
        tm = first_m + static_cast<int>(r % rows);
        tn = static_cast<int>(r / rows);
        return;
    }
    const int g = static_cast<int>(t / per_group);
    const int first_m = g * group_m;
    const int rows = (tiles_m - first_m < group_m) ? (tiles_m - first_m) : group_m;
    const int64_t r = t - static_cast<int64_t>(g) * per_group;
    tm = first_m + static_cast<int>(r % rows);
    tn = static_cast<int>(r / rows);
}

// Per-rung launchers (defined one per translation unit).  Each enqueues its
// kernel(s) on `stream`, returns the launch error and reports the kernel id.
typedef CUresult (*TensorMapEncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                           const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                           CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                           CUtensorMapFloatOOBfill);

// Launch plan of the tcgen05 rung: the knobs its schedule leaves open.  Zero in a field
// lets the rung's own heuristic decide; the autotuner times candidate plans and pins the
// fastest per shape (paper, Table 1: `templatize` / `autotune` transitions).
struct R4Plan {
    int kernel = 0;      // 0 auto, 1 single-CTA kernel, 2 CTA-pair kernel
    int splits = 0;      // 0 auto, 1 no K split, n > 1 K splits
    int split_via = 0;   // with splits > 1: 0 auto, 1 global workspace, 2 cluster (distributed shared memory);
                         // pair kernel (splits == 1): 0 auto, 1 whole tiles only, 3 stream the last wave along K
    int group_m = 0;     // 0 auto, else tile-rows per raster group
    int half_tail = 0;   // 0 auto, 1 cut the last wave into half tiles, 2 never
    int tile_n = 0;      // 0 auto, else columns per output tile (pair kernel: a multiple of 64, at most 256;
                         // single-CTA kernel: 64, 128 or 256)
    int tail_n = 0;      // pair kernel: 0 auto, tile_n = uniform tiles, else the width of the narrow tiles that
                         // follow the wide ones in every tile row and balance the last wave
    int stages = 0;      // 0 auto, else depth of the operand ring (pair kernel: 3 = 256-row tiles, two k-blocks per stage)
};

// Host-side state of a handle that the TMA rungs need.
struct RunContext {
    int device = 0;
    int sm_count = 0;
    int cc_major = 0, cc_minor = 0;
    int max_smem_optin = 0;
    TensorMapEncodeTiledFn encode_tiled = nullptr;   // from cudaGetDriverEntryPoint
    void* workspace = nullptr;                       // split-K partial sums (fp32)
    size_t workspace_bytes = 0;
    unsigned* sk_flags = nullptr;                    // streamed last wave of the pair kernel: one flag per (pair, CTA,
                                                     // epilogue warp), holding the epoch of the launch that wrote it
    unsigned sk_epoch = 0;                           // bumped by every launch that streams its last wave
    unsigned* tile_counters = nullptr;               // split-K arrival counters, zero between calls
    int n_tile_counters = 0;
    unsigned flags = 0;
    bool allow_repack = true;   // rung 4 may copy unaligned operands into the workspace (needs scratch)
    int kid_flags = 0;          // added to the kernel id a rung-4 launch reports (64 = operands repacked)
    R4Plan plan;                // pinned plan of this call's shape (all zero = heuristics)
};

// Encodes a 2-D tiled tensor map (dims/strides innermost first; stride of the
// outer dimension in bytes).  Returns false when the driver rejects it.
bool encode_map_2d(const RunContext& ctx, CUtensorMap* map, CUtensorMapDataType dt, const void* base, uint64_t dim0,
                   uint64_t dim1, uint64_t stride1_bytes, uint32_t box0, uint32_t box1, CUtensorMapSwizzle swz);

// The same with a third, outermost dimension (the batch index of a batched GEMM): box 1 along it.
bool encode_map_3d(const RunContext& ctx, CUtensorMap* map, CUtensorMapDataType dt, const void* base, uint64_t dim0,
                   uint64_t dim1, uint64_t dim2, uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t box0,
                   uint32_t box1, CUtensorMapSwizzle swz);

// Several problems in one launch of the tcgen05 rung (paper, Appendix D: BMM and GroupedGEMM are
// held-out members of the GEMM family).
//   batched: `batch` problems of one shape, operand b at base + b * stride (elements); the tensor
//            maps get the batch as a third dimension, the tile schedule runs over batch x tiles.
//   grouped: problems of different shapes; one table entry per group in device memory holds
//            the group's tensor maps, sizes and its first tile in the launch-wide schedule.
struct BatchArgs {
    int batch = 1;
    int64_t stride_a = 0, stride_b = 0, stride_c = 0;   // elements
};
struct alignas(128) GroupEntry {
    CUtensorMap map_a, map_b, map_c;    // 3 x 128 bytes
    void* C;
    int64_t ldc;
    int M, N, K, nkb;
    int tiles_m, tiles_n;               // in tiles of the kernel that runs the table
    int tile_start;                     // first tile of this group in the launch-wide schedule
    int epi_tma;                        // this group's C can take the TMA-store epilogue
};
// One problem, several destinations (MODE 3): the epilogue writes every output block to each of
// `n_dst` C matrices - the fused all-gather of an N-partitioned multi-GPU GEMM, where the
// destinations are the column slice of this rank in every rank's C (peer memory, plain stores
// or TMA stores; never a load).
struct alignas(128) DstEntry {
    CUtensorMap map_c;
    void* C;
    int64_t ldc;
};
constexpr int kMaxDst = 16;
constexpr int kMaxGroups = 256;         // groups per launch (the schedule's prefix sums live in shared memory)

// 4-D tiled map of a channels-last image tensor (dims innermost first: C, W, H, N), box c_box x w_box x h_box x 1,
// elements of `elt` bytes.
bool encode_map_nhwc(const RunContext& ctx, CUtensorMap* map, CUtensorMapDataType dt, const void* base, uint64_t C,
                     uint64_t W, uint64_t H, uint64_t N, uint32_t c_box, uint32_t w_box, uint32_t h_box, int elt,
                     CUtensorMapSwizzle swz);

// Edge of the square block tile the staged rungs (1, 2, 3) use for a problem: the largest of 128 / 64 / 32 whose
// grid still has a CTA for every SM of the current device, else 32.
int staged_tile_edge(const GemmArgs& g);
cudaError_t launch_r0_naive(const GemmArgs& g, cudaStream_t stream, int* kernel_id);
cudaError_t launch_r1_tiled(const GemmArgs& g, cudaStream_t stream, int* kernel_id);
cudaError_t launch_r2_vectorized(const GemmArgs& g, cudaStream_t stream, int* kernel_id);
cudaError_t launch_r3_pipelined(const GemmArgs& g, RunContext& ctx, cudaStream_t stream, int* kernel_id);
cudaError_t launch_r4_tcgen05(const GemmArgs& g, RunContext& ctx, cudaStream_t stream, int* kernel_id);
cudaError_t launch_r35_mma_sync(const GemmArgs& g, RunContext& ctx, cudaStream_t stream, int* kernel_id);
cudaError_t launch_zero_fill(const GemmArgs& g, cudaStream_t stream, int* kernel_id);
// CTA-pair (cta_group::2) form of rung 4 and the test of its preconditions.
bool r4_pair_applicable(const GemmArgs& g, const RunContext& ctx);
// The same estimate for a batched or grouped launch, on its tile counts (128 x 256 / 256 x 256 / 512 x 256) and longest K.
bool r4_pair_faster_multi(int64_t tiles128, int64_t tiles256, int64_t tiles512, int64_t nkb, const RunContext& ctx);
// One wave of 128 x 128 tiles whose columns are at least 8 points fuller than those of 256-column tiles (N = 1064: 0.92
// against 0.83): the single-CTA kernel then runs its 128-column tiles, and the pair kernel's 256-column forms stand back.
bool r4_narrow_tiles_fill_better(int64_t M, int64_t N, int sm_count);
// Whether an unpinned single-destination launch takes the pair kernel's k-paired 256-row tiles.
bool r4_pair_k_paired_auto(const GemmArgs& g, const RunContext& ctx);
// Hard preconditions of the CTA-pair kernel only (operands TMA-loadable), without the size heuristic.
bool r4_pair_possible(const GemmArgs& g, const RunContext& ctx);
// Whether the pair kernel can stream this problem's last wave along K (enough k-blocks per piece, workspace for the
// partial tiles, every pair of the grid resident).
bool r4_pair_stream_k_possible(const GemmArgs& g, const RunContext& ctx);
// True when `plan` can run this problem on the tcgen05 rung (the launcher refuses it otherwise).
bool r4_plan_valid(const GemmArgs& g, const RunContext& ctx, const R4Plan& plan);
// Candidate plans of a problem, the all-zero heuristic plan first; returns how many were written.
int r4_enumerate_plans(const GemmArgs& g, const RunContext& ctx, R4Plan* out, int cap);
cudaError_t launch_r4_tcgen05_pair(const GemmArgs& g, RunContext& ctx, cudaStream_t stream, int* kernel_id);
// Batched form on the CTA-pair kernel: one launch over batch x tiles.  `possible` tests the
// preconditions (operands and batch strides TMA-loadable); shapes it refuses run batch by batch.
bool r4_pair_batched_possible(const GemmArgs& g, const BatchArgs& b, const RunContext& ctx);
cudaError_t launch_r4_pair_batched(const GemmArgs& g, const BatchArgs& b, RunContext& ctx, cudaStream_t stream,
                                   int* kernel_id);
// The same two forms on the single-CTA kernel (128 x 256 tiles, double-buffered accumulator: the
// better choice for short K, where the pair kernel's epilogue is exposed, and for small problems).
bool r4_single_batched_possible(const GemmArgs& g, const BatchArgs& b, const RunContext& ctx);
cudaError_t launch_r4_single_batched(const GemmArgs& g, const BatchArgs& b, RunContext& ctx, cudaStream_t stream,
                                     int* kernel_id);
bool r4_single_grouped_possible(const GemmArgs* groups, int n, const RunContext& ctx);
cudaError_t launch_r4_single_grouped(const GemmArgs* groups, int n, RunContext& ctx, cudaStream_t stream,
                                     int* kernel_id);
// Conv2d as an implicit GEMM on the single-CTA kernel (generic-proxy producers gather the patches).
// g: M = N*P*Q, N = F, K = R*S*C, A = x, B = w (column-major, ldb = K), C = y (ldc = F), f16 = 1.
cudaError_t launch_r4_conv2d(const GemmArgs& g, const ConvGeom& geom, RunContext& ctx, cudaStream_t stream,
                             int* kernel_id);
// Direct convolution, one thread per output value (the naive rung of the same operation).
cudaError_t launch_conv2d_naive(const GemmArgs& g, const ConvGeom& geom, cudaStream_t stream, int* kernel_id);
// Multi-destination form (either kernel, chosen as for a plain call): dst[i] = (C pointer, pitch).
bool r4_multi_dst_possible(const GemmArgs& g, const RunContext& ctx);
cudaError_t launch_r4_multi_dst(const GemmArgs& g, void* const* C, const int64_t* ldc, int n_dst, RunContext& ctx,
                                cudaStream_t stream, int* kernel_id);
cudaError_t launch_r4_pair_multi_dst(const GemmArgs& g, void* const* C, const int64_t* ldc, int n_dst, RunContext& ctx,
                                     cudaStream_t stream, int* kernel_id);
// Grouped form: `groups` host descriptions (A, B, C, sizes, pitches in GemmArgs form; all with the
// handle's B layout and C dtype).  The table is built in the handle's workspace on `stream`.
bool r4_pair_grouped_possible(const GemmArgs* groups, int n, const RunContext& ctx);
cudaError_t launch_r4_pair_grouped(const GemmArgs* groups, int n, RunContext& ctx, cudaStream_t stream, int* kernel_id);


// Timeline stamps for tuning (compiled in only with -DKLIN_TRACE; the shipped library carries none of it).
// A translation unit that stamps defines KLIN_TRACE_BUF as its own static __device__ array of
// kTraceSlots x (CTAs) 64-bit words; slot s of CTA b receives the SM's cycle counter.
#ifdef KLIN_TRACE
constexpr int kTraceSlots = 64, kTraceCtas = 160;
#define KLIN_T(slot)                                                                                  \
    do {                                                                                              \
        if ((slot) >= 0 && (slot) < klin::kTraceSlots && blockIdx.x < klin::kTraceCtas)               \
            KLIN_TRACE_BUF[blockIdx.x * klin::kTraceSlots + (slot)] = static_cast<unsigned long long>(clock64()); \
    } while (0)
#else
#define KLIN_T(slot) ((void)0)
#endif

}  // namespace klin
