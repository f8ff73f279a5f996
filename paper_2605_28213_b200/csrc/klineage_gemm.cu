// Host runtime and C ABI of the GEMM lineage: handle, argument validation,
// alignment classification, tensor-map encoding, rung dispatch, status block.
// No rung ever substitutes for another, and nothing here computes on the CPU.
#include "../../include/klineage_gemm.h"
#include "common.cuh"

#include <array>
#include <cstdio>
#include <cstring>
#include <map>
#include <new>

using namespace klin;

// Key of a pinned plan: the shape and the alignment class of the three operands (the class
// decides which sub-paths of the tcgen05 rung can run, so a plan tuned for one does not
// carry over to another).
typedef std::array<int64_t, 4> PlanKey;

struct klineage_gemm_s {
    RunContext ctx;
    int b_layout = 0;
    int c_dtype = 0;
    unsigned* status = nullptr;   // device: 4 words (error, kernel id, detail0, detail1)
    int last_kernel_id = -1;
    int last_launches = 0;             // GEMM kernels the last run call enqueued
    std::map<PlanKey, R4Plan> plans;   // pinned by klineage_gemm_set_plan / klineage_gemm_autotune
    unsigned give_up_block = 0, give_up_where = 0;   // detail of the last device-side give-up that was read
    bool forcing = false;              // autotune in progress: run `forced` whatever is pinned
    R4Plan forced;
    // klineage_gemm_run_host: copy streams and events, created by its first call
    static constexpr int kMaxSlabs = 16;
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_out = nullptr, ev_in[kMaxSlabs] = {}, ev_done[kMaxSlabs] = {};
    bool pipe_ready = false;
};

namespace klin {

bool encode_map_2d(const RunContext& ctx, CUtensorMap* map, CUtensorMapDataType dt, const void* base, uint64_t dim0,
                   uint64_t dim1, uint64_t stride1_bytes, uint32_t box0, uint32_t box1, CUtensorMapSwizzle swz)
{
    if (!ctx.encode_tiled) return false;
    const cuuint64_t dims[2] = {dim0, dim1};
    const cuuint64_t strides[1] = {stride1_bytes};
    const cuuint32_t box[2] = {box0, box1};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = ctx.encode_tiled(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr,
                                        CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool encode_map_3d(const RunContext& ctx, CUtensorMap* map, CUtensorMapDataType dt, const void* base, uint64_t dim0,
                   uint64_t dim1, uint64_t dim2, uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t box0,
                   uint32_t box1, CUtensorMapSwizzle swz)
{
    if (!ctx.encode_tiled) return false;
    const cuuint64_t dims[3] = {dim0, dim1, dim2};
    const cuuint64_t strides[2] = {stride1_bytes, stride2_bytes};
    const cuuint32_t box[3] = {box0, box1, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = ctx.encode_tiled(map, dt, 3, const_cast<void*>(base), dims, strides, box, estr,
                                        CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool encode_map_nhwc(const RunContext& ctx, CUtensorMap* map, CUtensorMapDataType dt, const void* base, uint64_t C,
                     uint64_t W, uint64_t H, uint64_t N, uint32_t c_box, uint32_t w_box, uint32_t h_box, int elt,
                     CUtensorMapSwizzle swz)
{
    if (!ctx.encode_tiled) return false;
    const cuuint64_t e = static_cast<cuuint64_t>(elt);
    const cuuint64_t dims[4] = {C, W, H, N};
    const cuuint64_t strides[3] = {C * e, W * C * e, H * W * C * e};
    const cuuint32_t box[4] = {c_box, w_box, h_box, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = ctx.encode_tiled(map, dt, 4, const_cast<void*>(base), dims, strides, box, estr,
                                        CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

}  // namespace klin

namespace {

constexpr size_t kDefaultWorkspace = 64u << 20;
constexpr int kTileCounters = 4096;

// Restores the caller's current device on scope exit.
struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        ok = (prev == dev) || (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard()
    {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

bool aligned16(const void* base, int64_t ld, int elt)
{
    return reinterpret_cast<uintptr_t>(base) % 16 == 0 && (ld * elt) % 16 == 0;
}

PlanKey plan_key(const klineage_gemm_s* h, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda, const void* B,
                 int64_t ldb, const void* C, int64_t ldc)
{
    const int celt = h->c_dtype == KLINEAGE_C_BF16 ? 2 : 4;
    const int64_t cls = (aligned16(A, lda, 2) ? 1 : 0) | (aligned16(B, ldb, 2) ? 2 : 0) | (aligned16(C, ldc, celt) ? 4 : 0);
    return PlanKey{M, N, K, cls};
}

GemmArgs make_args(const klineage_gemm_s* h, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda, const void* B,
                   int64_t ldb, const void* bias, void* C, int64_t ldc)
{
    GemmArgs g;
    g.M = static_cast<int>(M);
    g.N = static_cast<int>(N);
    g.K = static_cast<int>(K);
    g.A = static_cast<const uint16_t*>(A);
    g.lda = lda;
    g.B = static_cast<const uint16_t*>(B);
    g.ldb = ldb;
    g.C = C;
    g.ldc = ldc;
    g.b_col = h->b_layout == KLINEAGE_B_COL_MAJOR ? 1 : 0;
    g.c_bf16 = h->c_dtype == KLINEAGE_C_BF16 ? 1 : 0;
    g.status = h->status;
    g.bias = static_cast<const uint16_t*>(bias);
    return g;
}

klineage_gemm_plan_t to_public(const R4Plan& p)
{
    klineage_gemm_plan_t o;
    o.kernel = p.kernel;
    o.splits = p.splits;
    o.split_via = p.split_via;
    o.group_m = p.group_m;
    o.half_tail = p.half_tail;
    o.tile_n = p.tile_n;
    o.tail_n = p.tail_n;
    o.stages = p.stages;
    return o;
}

R4Plan from_public(const klineage_gemm_plan_t& p)
{
    R4Plan o;
    o.kernel = p.kernel;
    o.splits = p.splits;
    o.split_via = p.split_via;
    o.group_m = p.group_m;
    o.half_tail = p.half_tail;
    o.tile_n = p.tile_n;
    o.tail_n = p.tail_n;
    o.stages = p.stages;
    return o;
}

bool ranges_overlap(const void* a, size_t a_bytes, const void* b, size_t b_bytes)
{
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + b_bytes && b0 < a0 + a_bytes;
}

// Device copies of host operands (klineage_gemm_run_host): pitches rounded up to 8 elements (16 bytes for bf16, 32 for
// fp32), every matrix at a 256-byte offset of the caller's scratch.
struct HostLayout {
    int64_t lda2, ldb2, ldc2, b_rows, b_cols;
    size_t off_a, off_b, off_c, total;
};

HostLayout host_layout(int b_layout, int c_dtype, int64_t M, int64_t N, int64_t K)
{
    HostLayout L;
    const bool bcol = b_layout == KLINEAGE_B_COL_MAJOR;
    const size_t celt = c_dtype == KLINEAGE_C_BF16 ? 2 : 4;
    auto up8 = [](int64_t v) { return v > 0 ? (v + 7) & ~int64_t(7) : int64_t(8); };
    auto up256 = [](size_t v) { return (v + 255) & ~size_t(255); };
    L.b_rows = bcol ? N : K;
    L.b_cols = bcol ? K : N;
    L.lda2 = up8(K);
    L.ldb2 = up8(L.b_cols);
    L.ldc2 = up8(N);
    L.off_a = 0;
    L.off_b = up256(static_cast<size_t>(M) * L.lda2 * 2);
    L.off_c = L.off_b + up256(static_cast<size_t>(L.b_rows) * L.ldb2 * 2);
    L.total = L.off_c + up256(static_cast<size_t>(M) * L.ldc2 * celt);
    return L;
}

// A pitched copy; one linear copy when both sides are dense (the copy engines then see a single long transfer).
cudaError_t copy_rows(void* dst, size_t dpitch, const void* src, size_t spitch, size_t width, size_t rows,
                      cudaMemcpyKind kind, cudaStream_t s)
{
    if (rows == 0 || width == 0) return cudaSuccess;
    if (dpitch == width && spitch == width) return cudaMemcpyAsync(dst, src, width * rows, kind, s);
    return cudaMemcpy2DAsync(dst, dpitch, src, spitch, width, rows, kind, s);
}

void release_host_pipe(klineage_gemm_s* h)
{
    if (h->copy_in) cudaStreamDestroy(h->copy_in);
    if (h->copy_out) cudaStreamDestroy(h->copy_out);
    if (h->ev_start) cudaEventDestroy(h->ev_start);
    if (h->ev_out) cudaEventDestroy(h->ev_out);
    for (int i = 0; i < klineage_gemm_s::kMaxSlabs; ++i) {
        if (h->ev_in[i]) cudaEventDestroy(h->ev_in[i]);
        if (h->ev_done[i]) cudaEventDestroy(h->ev_done[i]);
        h->ev_in[i] = h->ev_done[i] = nullptr;
    }
    h->copy_in = h->copy_out = nullptr;
    h->ev_start = h->ev_out = nullptr;
    h->pipe_ready = false;
}

// Streams that do not synchronise with the legacy default stream: every ordering is an explicit event.
bool ensure_host_pipe(klineage_gemm_s* h)
{
    if (h->pipe_ready) return true;
    bool ok = cudaStreamCreateWithFlags(&h->copy_in, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&h->copy_out, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&h->ev_start, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&h->ev_out, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < klineage_gemm_s::kMaxSlabs; ++i) {
        ok = cudaEventCreateWithFlags(&h->ev_in[i], cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&h->ev_done[i], cudaEventDisableTiming) == cudaSuccess;
    }
    if (!ok) {
        cudaGetLastError();
        release_host_pipe(h);
        return false;
    }
    h->pipe_ready = true;
    return true;
}

}  // namespace

extern "C" {

klineage_status_t klineage_gemm_create(klineage_gemm_t* out, const klineage_gemm_config_t* cfg)
{
    if (!out) return KLINEAGE_ERR_INVALID_ARG;
    *out = nullptr;
    if (!cfg) return KLINEAGE_ERR_INVALID_ARG;
    if (cfg->b_layout != KLINEAGE_B_ROW_MAJOR && cfg->b_layout != KLINEAGE_B_COL_MAJOR) return KLINEAGE_ERR_INVALID_ARG;
    if (cfg->c_dtype != KLINEAGE_C_F32 && cfg->c_dtype != KLINEAGE_C_BF16 && cfg->c_dtype != KLINEAGE_C_F16)
        return KLINEAGE_ERR_INVALID_ARG;
    if (cfg->flags & ~(KLINEAGE_FLAG_STATIC_B | KLINEAGE_FLAG_TEST_GIVE_UP)) return KLINEAGE_ERR_INVALID_ARG;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || cfg->device < 0 || cfg->device >= ndev) {
        cudaGetLastError();
        return KLINEAGE_ERR_INVALID_ARG;
    }
    DeviceGuard guard(cfg->device);
    if (!guard.ok) return KLINEAGE_ERR_INVALID_ARG;

    klineage_gemm_s* h = new (std::nothrow) klineage_gemm_s();
    if (!h) return KLINEAGE_ERR_ALLOC;
    h->b_layout = cfg->b_layout;
    h->c_dtype = cfg->c_dtype;
    RunContext& c = h->ctx;
    c.device = cfg->device;
    c.flags = cfg->flags;
    cudaDeviceGetAttribute(&c.sm_count, cudaDevAttrMultiProcessorCount, c.device);
    cudaDeviceGetAttribute(&c.cc_major, cudaDevAttrComputeCapabilityMajor, c.device);
    cudaDeviceGetAttribute(&c.cc_minor, cudaDevAttrComputeCapabilityMinor, c.device);
    cudaDeviceGetAttribute(&c.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, c.device);

    // cuTensorMapEncodeTiled comes from the driver at run time, so the library
    // has no link-time dependency on libcuda.
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
        c.encode_tiled = reinterpret_cast<TensorMapEncodeTiledFn>(fn);
    else
        cudaGetLastError();

    c.workspace_bytes = cfg->workspace_bytes ? cfg->workspace_bytes : kDefaultWorkspace;
    c.n_tile_counters = kTileCounters;
    bool ok = cudaMalloc(&c.workspace, c.workspace_bytes) == cudaSuccess;
    ok = ok && cudaMalloc(reinterpret_cast<void**>(&c.tile_counters), sizeof(unsigned) * kTileCounters) == cudaSuccess;
    ok = ok && cudaMalloc(reinterpret_cast<void**>(&h->status), 4 * sizeof(unsigned)) == cudaSuccess;
    const size_t n_sk_flags = static_cast<size_t>(c.sm_count > 0 ? c.sm_count : 1) * 8;     // (SMs / 2 pairs) x 2 CTAs x 8 warps
    ok = ok && cudaMalloc(reinterpret_cast<void**>(&c.sk_flags), n_sk_flags * sizeof(unsigned)) == cudaSuccess;
    ok = ok && cudaMemset(c.sk_flags, 0, n_sk_flags * sizeof(unsigned)) == cudaSuccess;
    ok = ok && cudaMemset(c.tile_counters, 0, sizeof(unsigned) * kTileCounters) == cudaSuccess;
    ok = ok && cudaMemset(h->status, 0, 4 * sizeof(unsigned)) == cudaSuccess;
    ok = ok && cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        klineage_gemm_destroy(h);
        return KLINEAGE_ERR_ALLOC;
    }
    *out = h;
    return KLINEAGE_OK;
}

klineage_status_t klineage_gemm_destroy(klineage_gemm_t h)
{
    if (!h) return KLINEAGE_OK;
    {
        DeviceGuard guard(h->ctx.device);
        if (h->ctx.workspace) cudaFree(h->ctx.workspace);
        if (h->ctx.tile_counters) cudaFree(h->ctx.tile_counters);
        if (h->ctx.sk_flags) cudaFree(h->ctx.sk_flags);
        if (h->status) cudaFree(h->status);
        release_host_pipe(h);
    }
    delete h;
    return KLINEAGE_OK;
}

klineage_status_t klineage_gemm_check_args(int b_layout, int c_dtype, int64_t M, int64_t N, int64_t K, const void* A,
                                           int64_t lda, const void* B, int64_t ldb, const void* C, int64_t ldc,
                                           int variant)
{
    if (b_layout != KLINEAGE_B_ROW_MAJOR && b_layout != KLINEAGE_B_COL_MAJOR) return KLINEAGE_ERR_INVALID_ARG;
    if (c_dtype != KLINEAGE_C_F32 && c_dtype != KLINEAGE_C_BF16) return KLINEAGE_ERR_INVALID_ARG;
    if (variant < KLINEAGE_NAIVE || variant > KLINEAGE_MMA_SYNC) return KLINEAGE_ERR_BAD_VARIANT;
    const int64_t lim = int64_t(1) << 31;
    if (M < 0 || N < 0 || K < 0 || M >= lim || N >= lim || K >= lim) return KLINEAGE_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return KLINEAGE_OK;
    const bool bcol = b_layout == KLINEAGE_B_COL_MAJOR;
    const size_t celt = c_dtype == KLINEAGE_C_BF16 ? 2 : 4;
    if (!C || ldc < N) return KLINEAGE_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(C) % celt) return KLINEAGE_ERR_INVALID_ARG;
    if (K > 0) {
        if (!A || !B) return KLINEAGE_ERR_INVALID_ARG;
        if (lda < K || ldb < (bcol ? K : N)) return KLINEAGE_ERR_INVALID_ARG;
        if (reinterpret_cast<uintptr_t>(A) % 2 || reinterpret_cast<uintptr_t>(B) % 2) return KLINEAGE_ERR_INVALID_ARG;
        const size_t a_bytes = (size_t(M - 1) * lda + K) * 2;
        const size_t b_bytes = (size_t((bcol ? N : K) - 1) * ldb + (bcol ? K : N)) * 2;
        const size_t c_bytes = (size_t(M - 1) * ldc + N) * celt;
        if (ranges_overlap(A, a_bytes, C, c_bytes) || ranges_overlap(B, b_bytes, C, c_bytes))
            return KLINEAGE_ERR_INVALID_ARG;
    }
    return KLINEAGE_OK;
}

}  // extern "C"

// Shared body of klineage_gemm_run (bias == nullptr) and klineage_gemm_run_addmm.
static klineage_status_t run_impl(klineage_gemm_t h, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                  const void* B, int64_t ldb, const void* bias, void* C, int64_t ldc, int variant,
                                  void* stream)
{
    if (!h) return KLINEAGE_ERR_INVALID_ARG;
    const klineage_status_t chk = klineage_gemm_check_args(h->b_layout, h->c_dtype, M, N, K, A, lda, B, ldb, C, ldc, variant);
    if (chk != KLINEAGE_OK) return chk;
    if (M == 0 || N == 0) {
        h->last_kernel_id = -1;
        return KLINEAGE_OK;
    }
    const bool bcol = h->b_layout == KLINEAGE_B_COL_MAJOR;
    if ((variant == KLINEAGE_PIPELINED || variant == KLINEAGE_TCGEN05 || variant == KLINEAGE_MMA_SYNC) &&
        h->ctx.cc_major != 10)
        return KLINEAGE_ERR_UNSUPPORTED_DEVICE;

    DeviceGuard guard(h->ctx.device);
    if (!guard.ok) return KLINEAGE_ERR_LAUNCH;

    const GemmArgs g = make_args(h, M, N, K, A, lda, B, ldb, bias, C, ldc);
    (void)bcol;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int kid = -1;
    cudaError_t e;
    if (K == 0) {
        e = launch_zero_fill(g, s, &kid);
    } else {
        switch (variant) {
            case KLINEAGE_NAIVE: e = launch_r0_naive(g, s, &kid); break;
            case KLINEAGE_TILED: e = launch_r1_tiled(g, s, &kid); break;
            case KLINEAGE_VECTORIZED: e = launch_r2_vectorized(g, s, &kid); break;
            case KLINEAGE_PIPELINED: e = launch_r3_pipelined(g, h->ctx, s, &kid); break;
            case KLINEAGE_MMA_SYNC: e = launch_r35_mma_sync(g, h->ctx, s, &kid); break;
            default: {
                // the plan pinned for this shape and alignment class, else the rung's heuristics
                h->ctx.plan = R4Plan();
                if (h->forcing) {
                    h->ctx.plan = h->forced;
                } else if (!h->plans.empty()) {
                    const auto it = h->plans.find(plan_key(h, M, N, K, A, lda, B, ldb, C, ldc));
                    if (it != h->plans.end()) h->ctx.plan = it->second;
                }
                e = launch_r4_tcgen05(g, h->ctx, s, &kid);
                break;
            }
        }
    }
    if (e != cudaSuccess) {
        cudaGetLastError();
        return KLINEAGE_ERR_LAUNCH;
    }
    h->last_kernel_id = kid;
    h->last_launches += 1;
    return KLINEAGE_OK;
}

extern "C" {

int klineage_gemm_last_launch_count(klineage_gemm_t h) { return h ? h->last_launches : 0; }

klineage_status_t klineage_gemm_run(klineage_gemm_t h, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                    const void* B, int64_t ldb, void* C, int64_t ldc, int variant, void* stream)
{
    if (h) h->last_launches = 0;
    return run_impl(h, M, N, K, A, lda, B, ldb, nullptr, C, ldc, variant, stream);
}

size_t klineage_gemm_host_scratch_bytes(int b_layout, int c_dtype, int64_t M, int64_t N, int64_t K)
{
    if (b_layout != KLINEAGE_B_ROW_MAJOR && b_layout != KLINEAGE_B_COL_MAJOR) return 0;
    if (c_dtype != KLINEAGE_C_F32 && c_dtype != KLINEAGE_C_BF16) return 0;
    const int64_t lim = int64_t(1) << 31;
    if (M <= 0 || N <= 0 || K < 0 || M >= lim || N >= lim || K >= lim) return 0;
    return host_layout(b_layout, c_dtype, M, N, K).total;
}

klineage_status_t klineage_gemm_run_host(klineage_gemm_t h, int64_t M, int64_t N, int64_t K, const void* A_host,
                                         int64_t lda, const void* B_host, int64_t ldb, void* C_host, int64_t ldc,
                                         void* scratch_device, size_t scratch_bytes, int variant, void* stream)
{
    if (!h) return KLINEAGE_ERR_INVALID_ARG;
    h->last_launches = 0;
    // shapes, pitches, element alignment and overlap follow the rules of the device call
    const klineage_status_t chk =
        klineage_gemm_check_args(h->b_layout, h->c_dtype, M, N, K, A_host, lda, B_host, ldb, C_host, ldc, variant);
    if (chk != KLINEAGE_OK) return chk;
    if (M == 0 || N == 0) {
        h->last_kernel_id = -1;
        return KLINEAGE_OK;
    }
    if ((variant == KLINEAGE_PIPELINED || variant == KLINEAGE_TCGEN05 || variant == KLINEAGE_MMA_SYNC) &&
        h->ctx.cc_major != 10)
        return KLINEAGE_ERR_UNSUPPORTED_DEVICE;
    const HostLayout L = host_layout(h->b_layout, h->c_dtype, M, N, K);
    if (!scratch_device || reinterpret_cast<uintptr_t>(scratch_device) % 256 || scratch_bytes < L.total)
        return KLINEAGE_ERR_INVALID_ARG;

    DeviceGuard guard(h->ctx.device);
    if (!guard.ok) return KLINEAGE_ERR_LAUNCH;
    if (!ensure_host_pipe(h)) return KLINEAGE_ERR_ALLOC;

    const size_t celt = h->c_dtype == KLINEAGE_C_BF16 ? 2 : 4;
    uint8_t* base = static_cast<uint8_t*>(scratch_device);
    uint8_t *dA = base + L.off_a, *dB = base + L.off_b, *dC = base + L.off_c;
    const uint8_t* hA = static_cast<const uint8_t*>(A_host);
    uint8_t* hC = static_cast<uint8_t*>(C_host);
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    // row slabs: multiples of 128 rows, about 512 rows each, at most kMaxSlabs
    int64_t n_slabs = (M + 511) / 512;
    if (n_slabs > klineage_gemm_s::kMaxSlabs) n_slabs = klineage_gemm_s::kMaxSlabs;
    const int64_t slab = ((M + n_slabs - 1) / n_slabs + 127) / 128 * 128;
    n_slabs = (M + slab - 1) / slab;

    bool ok = cudaEventRecord(h->ev_start, s) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(h->copy_in, h->ev_start, 0) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(h->copy_out, h->ev_start, 0) == cudaSuccess;
    if (ok && K > 0)
        ok = copy_rows(dB, static_cast<size_t>(L.ldb2) * 2, B_host, static_cast<size_t>(ldb) * 2,
                       static_cast<size_t>(L.b_cols) * 2, static_cast<size_t>(L.b_rows), cudaMemcpyHostToDevice,
                       h->copy_in) == cudaSuccess;
    klineage_status_t st = KLINEAGE_OK;
    int launches = 0;
    for (int64_t i = 0; ok && i < n_slabs; ++i) {
        const int64_t r0 = i * slab, rows = (M - r0 < slab) ? M - r0 : slab;
        uint8_t* dA_i = dA + static_cast<size_t>(r0) * L.lda2 * 2;
        uint8_t* dC_i = dC + static_cast<size_t>(r0) * L.ldc2 * celt;
        if (K > 0)
            ok = copy_rows(dA_i, static_cast<size_t>(L.lda2) * 2, hA + static_cast<size_t>(r0) * lda * 2,
                           static_cast<size_t>(lda) * 2, static_cast<size_t>(K) * 2, static_cast<size_t>(rows),
                           cudaMemcpyHostToDevice, h->copy_in) == cudaSuccess;
        ok = ok && cudaEventRecord(h->ev_in[i], h->copy_in) == cudaSuccess;
        ok = ok && cudaStreamWaitEvent(s, h->ev_in[i], 0) == cudaSuccess;
        if (!ok) break;
        st = run_impl(h, rows, N, K, dA_i, L.lda2, dB, L.ldb2, nullptr, dC_i, L.ldc2, variant, stream);
        if (st != KLINEAGE_OK) break;
        launches = h->last_launches;
        ok = cudaEventRecord(h->ev_done[i], s) == cudaSuccess;
        ok = ok && cudaStreamWaitEvent(h->copy_out, h->ev_done[i], 0) == cudaSuccess;
        ok = ok && copy_rows(hC + static_cast<size_t>(r0) * ldc * celt, static_cast<size_t>(ldc) * celt, dC_i,
                             static_cast<size_t>(L.ldc2) * celt, static_cast<size_t>(N) * celt,
                             static_cast<size_t>(rows), cudaMemcpyDeviceToHost, h->copy_out) == cudaSuccess;
    }
    // whatever happened, `stream` continues only after both copy streams have drained what was enqueued
    const bool j1 = cudaEventRecord(h->ev_out, h->copy_out) == cudaSuccess && cudaStreamWaitEvent(s, h->ev_out, 0) == cudaSuccess;
    const bool j2 = cudaEventRecord(h->ev_start, h->copy_in) == cudaSuccess && cudaStreamWaitEvent(s, h->ev_start, 0) == cudaSuccess;
    h->last_launches = launches;
    if (st != KLINEAGE_OK) return st;
    if (!ok || !j1 || !j2) {
        cudaGetLastError();
        return KLINEAGE_ERR_LAUNCH;
    }
    return KLINEAGE_OK;
}

klineage_status_t klineage_gemm_run_addmm(klineage_gemm_t h, int64_t M, int64_t N, int64_t K, const void* A,
                                          int64_t lda, const void* B, int64_t ldb, const void* bias, void* C,
                                          int64_t ldc, int variant, void* stream)
{
    if (!h) return KLINEAGE_ERR_INVALID_ARG;
    h->last_launches = 0;
    if (M > 0 && N > 0) {
        if (!bias || reinterpret_cast<uintptr_t>(bias) % 2) return KLINEAGE_ERR_INVALID_ARG;
        if (C && N > 0 && M > 0 && ldc >= N) {
            const size_t celt = h->c_dtype == KLINEAGE_C_BF16 ? 2 : 4;
            const size_t c_bytes = (size_t(M - 1) * ldc + N) * celt;
            if (ranges_overlap(bias, size_t(N) * 2, C, c_bytes)) return KLINEAGE_ERR_INVALID_ARG;
        }
    }
    return run_impl(h, M, N, K, A, lda, B, ldb, bias, C, ldc, variant, stream);
}

// ------------------------------------------------------------------ batched and grouped GEMM
klineage_status_t klineage_gemm_run_batched(klineage_gemm_t h, int64_t batch, int64_t M, int64_t N, int64_t K,
                                            const void* A, int64_t lda, int64_t stride_a, const void* B, int64_t ldb,
                                            int64_t stride_b, void* C, int64_t ldc, int64_t stride_c, int variant,
                                            void* stream)
{
    if (!h || batch < 0 || batch > 65535) return KLINEAGE_ERR_INVALID_ARG;
    h->last_launches = 0;
    const klineage_status_t chk = klineage_gemm_check_args(h->b_layout, h->c_dtype, M, N, K, A, lda, B, ldb, C, ldc, variant);
    if (chk != KLINEAGE_OK) return chk;
    if (batch == 0 || M == 0 || N == 0) {
        h->last_kernel_id = -1;
        return KLINEAGE_OK;
    }
    const bool bcol = h->b_layout == KLINEAGE_B_COL_MAJOR;
    const size_t celt = h->c_dtype == KLINEAGE_C_BF16 ? 2 : 4;
    if (stride_a < 0 || stride_b < 0 || stride_c < 0) return KLINEAGE_ERR_INVALID_ARG;
    // the C matrices of different batches must not overlap; A and B may be shared (stride 0)
    const int64_t c_extent = (M - 1) * ldc + N;
    if (batch > 1 && stride_c < c_extent) return KLINEAGE_ERR_INVALID_ARG;
    if (K > 0) {
        const size_t a_bytes = (size_t(batch - 1) * stride_a + size_t(M - 1) * lda + K) * 2;
        const size_t b_bytes = (size_t(batch - 1) * stride_b + size_t((bcol ? N : K) - 1) * ldb + (bcol ? K : N)) * 2;
        const size_t c_bytes = (size_t(batch - 1) * stride_c + size_t(c_extent)) * celt;
        if (ranges_overlap(A, a_bytes, C, c_bytes) || ranges_overlap(B, b_bytes, C, c_bytes)) return KLINEAGE_ERR_INVALID_ARG;
    }
    const uint8_t* a8 = static_cast<const uint8_t*>(A);
    const uint8_t* b8 = static_cast<const uint8_t*>(B);
    uint8_t* c8 = static_cast<uint8_t*>(C);
    if (variant == KLINEAGE_TCGEN05 && K > 0 && h->ctx.cc_major == 10) {
        // one launch over batch x tiles on the CTA-pair kernel when the batch maps onto 3-D tensor maps
        const GemmArgs g = make_args(h, M, N, K, A, lda, B, ldb, nullptr, C, ldc);
        BatchArgs ba;
        ba.batch = static_cast<int>(batch);
        ba.stride_a = stride_a;
        ba.stride_b = stride_b;
        ba.stride_c = stride_c;
        // The CTA-pair kernel (512 x 256 or 256 x 256 tiles) or the single-CTA kernel (128 x 256 tiles), whichever the
        // cycle estimate of the two schedules favours over the whole batch.  A plan pinned for the per-problem shape
        // decides the kernel when it names one.
        const int half_sm = h->ctx.sm_count / 2;
        const int64_t pair_tiles = ((M + 511) / 512) * ((N + 255) / 256) * batch;
        const int64_t single_tiles = ((M + 127) / 128) * ((N + 255) / 256) * batch;
        const bool pair_ok = M > 256 && pair_tiles >= half_sm && r4_pair_batched_possible(g, ba, h->ctx);
        const bool single_ok = M > 64 && single_tiles >= half_sm && r4_single_batched_possible(g, ba, h->ctx);
        int want = 0;   // 1 single-CTA kernel, 2 pair kernel
        R4Plan pinned;
        const auto it = h->plans.find(plan_key(h, M, N, K, A, lda, B, ldb, C, ldc));
        if (it != h->plans.end()) pinned = it->second;
        if (pinned.kernel == 2 && pair_ok)
            want = 2;
        else if (pinned.kernel == 1 && single_ok)
            want = 1;
        else if (pair_ok && r4_pair_faster_multi(single_tiles, ((M + 255) / 256) * ((N + 255) / 256) * batch, pair_tiles, (K + 63) / 64, h->ctx))
            want = 2;
        else if (single_ok)
            want = 1;
        else if (pair_ok)
            want = 2;
        if (want != 0) {
            DeviceGuard guard(h->ctx.device);
            if (!guard.ok) return KLINEAGE_ERR_LAUNCH;
            h->ctx.plan = R4Plan();
            h->ctx.plan.group_m = pinned.group_m;
            if (want == 2 && pinned.kernel == 2) {      // the plan also says which tiles: stages 3 = 256 rows, two k-blocks per stage
                h->ctx.plan.kernel = 2;
                h->ctx.plan.stages = pinned.stages;
            }
            int kid = -1;
            const cudaError_t e = want == 2 ? launch_r4_pair_batched(g, ba, h->ctx, static_cast<cudaStream_t>(stream), &kid)
                                            : launch_r4_single_batched(g, ba, h->ctx, static_cast<cudaStream_t>(stream), &kid);
            if (e != cudaSuccess) {
                cudaGetLastError();
                return KLINEAGE_ERR_LAUNCH;
            }
            h->last_kernel_id = kid;
            h->last_launches = 1;
            return KLINEAGE_OK;
        }
    }
    // every other case: the rung's ordinary path, one launch per batch
    for (int64_t b = 0; b < batch; ++b) {
        const klineage_status_t st = run_impl(h, M, N, K, a8 ? a8 + b * stride_a * 2 : nullptr, lda,
                                              b8 ? b8 + b * stride_b * 2 : nullptr, ldb, nullptr,
                                              c8 + b * stride_c * celt, ldc, variant, stream);
        if (st != KLINEAGE_OK) return st;
    }
    return KLINEAGE_OK;
}

klineage_status_t klineage_gemm_run_grouped(klineage_gemm_t h, int groups, const int64_t* M, const int64_t* N,
                                            const int64_t* K, const void* const* A, const int64_t* lda,
                                            const void* const* B, const int64_t* ldb, void* const* C, const int64_t* ldc,
                                            int variant, void* stream)
{
    if (!h || groups < 0) return KLINEAGE_ERR_INVALID_ARG;
    h->last_launches = 0;
    if (groups == 0) {
        h->last_kernel_id = -1;
        return KLINEAGE_OK;
    }
    if (!M || !N || !K || !A || !lda || !B || !ldb || !C || !ldc) return KLINEAGE_ERR_INVALID_ARG;
    const bool bcol = h->b_layout == KLINEAGE_B_COL_MAJOR;
    const size_t celt = h->c_dtype == KLINEAGE_C_BF16 ? 2 : 4;
    // validate everything before anything is launched
    for (int i = 0; i < groups; ++i) {
        const klineage_status_t chk =
            klineage_gemm_check_args(h->b_layout, h->c_dtype, M[i], N[i], K[i], A[i], lda[i], B[i], ldb[i], C[i], ldc[i], variant);
        if (chk != KLINEAGE_OK) return chk;
    }
    // no group's C may overlap another group's C or any group's A or B
    for (int i = 0; i < groups; ++i) {
        if (M[i] == 0 || N[i] == 0) continue;
        const size_t ci = (size_t(M[i] - 1) * ldc[i] + N[i]) * celt;
        for (int j = 0; j < groups; ++j) {
            if (M[j] == 0 || N[j] == 0) continue;
            if (j != i && ranges_overlap(C[i], ci, C[j], (size_t(M[j] - 1) * ldc[j] + N[j]) * celt)) return KLINEAGE_ERR_INVALID_ARG;
            if (K[j] == 0) continue;
            const size_t aj = (size_t(M[j] - 1) * lda[j] + K[j]) * 2;
            const size_t bj = (size_t((bcol ? N[j] : K[j]) - 1) * ldb[j] + (bcol ? K[j] : N[j])) * 2;
            if (ranges_overlap(C[i], ci, A[j], aj) || ranges_overlap(C[i], ci, B[j], bj)) return KLINEAGE_ERR_INVALID_ARG;
        }
    }
    h->last_kernel_id = -1;
    if (variant == KLINEAGE_TCGEN05 && h->ctx.cc_major == 10) {
        // one launch over the tiles of all groups when every non-empty group suits the CTA-pair kernel
        GemmArgs* ga = new (std::nothrow) GemmArgs[groups];
        if (!ga) return KLINEAGE_ERR_ALLOC;
        int n = 0, first = -1;
        bool launchable = true, all_tall = true;
        int64_t k_max = 0;
        int64_t pair_tiles = 0, kp_tiles = 0, single_tiles = 0, rows = 0, rows_by_256 = 0;
        for (int i = 0; i < groups; ++i) {
            if (M[i] == 0 || N[i] == 0) continue;
            if (K[i] == 0) {            // a zero-fill group: leave the whole call to the ordinary path
                launchable = false;
                break;
            }
            if (first < 0) first = i;
            ga[n++] = make_args(h, M[i], N[i], K[i], A[i], lda[i], B[i], ldb[i], nullptr, C[i], ldc[i]);
            // (a pair tile with at most 256 live rows issues half of its MMAs: rows count in steps of 256)
            rows += M[i];
            rows_by_256 += (M[i] + 255) / 256 * 256;
            all_tall = all_tall && M[i] > 256;
            k_max = K[i] > k_max ? K[i] : k_max;
            pair_tiles += ((M[i] + 511) / 512) * ((N[i] + 255) / 256);
            kp_tiles += ((M[i] + 255) / 256) * ((N[i] + 255) / 256);
            single_tiles += ((M[i] + 127) / 128) * ((N[i] + 255) / 256);
        }
        launchable = launchable && n >= 1 && n <= kMaxGroups;
        // kernel choice as for the batched call; a plan pinned for the first group's shape may name it
        const int half_sm = h->ctx.sm_count / 2;
        // by default the pair kernel when every group has more than 256 rows, or - ragged groups - when rounding every
        // group up to 256 rows adds at most a quarter (a pinned plan may ask for it whatever the groups' heights)
        all_tall = all_tall || rows_by_256 * 4 <= rows * 5;
        const bool pair_ok = launchable && pair_tiles >= half_sm && r4_pair_grouped_possible(ga, n, h->ctx);
        const bool single_ok = launchable && single_tiles >= half_sm && r4_single_grouped_possible(ga, n, h->ctx);
        R4Plan pinned;
        if (first >= 0) {
            const auto it = h->plans.find(plan_key(h, M[first], N[first], K[first], A[first], lda[first], B[first],
                                                   ldb[first], C[first], ldc[first]));
            if (it != h->plans.end()) pinned = it->second;
        }
        int want = 0;
        if (pinned.kernel == 2 && pair_ok)
            want = 2;
        else if (pinned.kernel == 1 && single_ok)
            want = 1;
        else if (pair_ok && all_tall && r4_pair_faster_multi(single_tiles, kp_tiles, pair_tiles, (k_max + 63) / 64, h->ctx))
            want = 2;
        else if (single_ok)
            want = 1;
        else if (pair_ok)
            want = 2;
        if (want != 0) {
            DeviceGuard guard(h->ctx.device);
            klineage_status_t st = guard.ok ? KLINEAGE_OK : KLINEAGE_ERR_LAUNCH;
            int kid = -1;
            h->ctx.plan = R4Plan();
            h->ctx.plan.group_m = pinned.group_m;
            if (want == 2 && pinned.kernel == 2) {      // the plan also says which tiles: stages 3 = 256 rows, two k-blocks per stage
                h->ctx.plan.kernel = 2;
                h->ctx.plan.stages = pinned.stages;
            }
            if (st == KLINEAGE_OK) {
                const cudaError_t e = want == 2 ? launch_r4_pair_grouped(ga, n, h->ctx, static_cast<cudaStream_t>(stream), &kid)
                                                : launch_r4_single_grouped(ga, n, h->ctx, static_cast<cudaStream_t>(stream), &kid);
                if (e != cudaSuccess) {
                    cudaGetLastError();
                    st = KLINEAGE_ERR_LAUNCH;
                }
            }
            delete[] ga;
            if (st == KLINEAGE_OK) {
                h->last_kernel_id = kid;
                h->last_launches = 1;
            }
            return st;
        }
        delete[] ga;
    }
    // every other case: the rung's ordinary path, one launch per group
    for (int i = 0; i < groups; ++i) {
        const klineage_status_t st = run_impl(h, M[i], N[i], K[i], A[i], lda[i], B[i], ldb[i], nullptr, C[i], ldc[i], variant, stream);
        if (st != KLINEAGE_OK) return st;
    }
    return KLINEAGE_OK;
}

// ------------------------------------------------------------------ one product, several destinations
klineage_status_t klineage_gemm_run_multi_dst(klineage_gemm_t h, int64_t M, int64_t N, int64_t K, const void* A,
                                              int64_t lda, const void* B, int64_t ldb, int n_dst, void* const* C,
                                              const int64_t* ldc, int variant, void* stream)
{
    if (!h || n_dst < 1 || n_dst > kMaxDst || !C || !ldc) return KLINEAGE_ERR_INVALID_ARG;
    h->last_launches = 0;
    const size_t celt = h->c_dtype == KLINEAGE_C_BF16 ? 2 : 4;
    for (int d = 0; d < n_dst; ++d) {
        const klineage_status_t chk =
            klineage_gemm_check_args(h->b_layout, h->c_dtype, M, N, K, A, lda, B, ldb, C[d], ldc[d], variant);
        if (chk != KLINEAGE_OK) return chk;
    }
    if (M == 0 || N == 0) {
        h->last_kernel_id = -1;
        return KLINEAGE_OK;
    }
    for (int d = 0; d < n_dst; ++d)
        for (int e = d + 1; e < n_dst; ++e)
            if (ranges_overlap(C[d], (size_t(M - 1) * ldc[d] + N) * celt, C[e], (size_t(M - 1) * ldc[e] + N) * celt))
                return KLINEAGE_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (variant == KLINEAGE_TCGEN05 && K > 0 && h->ctx.cc_major == 10) {
        const GemmArgs g = make_args(h, M, N, K, A, lda, B, ldb, nullptr, C[0], ldc[0]);
        h->ctx.plan = R4Plan();
        const auto it = h->plans.find(plan_key(h, M, N, K, A, lda, B, ldb, C[0], ldc[0]));
        if (it != h->plans.end()) h->ctx.plan = it->second;
        if (r4_multi_dst_possible(g, h->ctx)) {
            // one launch: the epilogue stores every output block to each destination
            DeviceGuard guard(h->ctx.device);
            if (!guard.ok) return KLINEAGE_ERR_LAUNCH;
            int kid = -1;
            if (launch_r4_multi_dst(g, C, ldc, n_dst, h->ctx, s, &kid) != cudaSuccess) {
                cudaGetLastError();
                return KLINEAGE_ERR_LAUNCH;
            }
            h->last_kernel_id = kid;
            h->last_launches = 1;
            return KLINEAGE_OK;
        }
    }
    // every other case: the rung's ordinary path into the first destination, then strided copies
    // of that result to the others on the same stream
    const klineage_status_t st = run_impl(h, M, N, K, A, lda, B, ldb, nullptr, C[0], ldc[0], variant, stream);
    if (st != KLINEAGE_OK) return st;
    DeviceGuard guard(h->ctx.device);
    for (int d = 1; d < n_dst; ++d) {
        if (cudaMemcpy2DAsync(C[d], size_t(ldc[d]) * celt, C[0], size_t(ldc[0]) * celt, size_t(N) * celt, size_t(M),
                              cudaMemcpyDefault, s) != cudaSuccess) {
            cudaGetLastError();
            return KLINEAGE_ERR_LAUNCH;
        }
    }
    return KLINEAGE_OK;
}

// ------------------------------------------------------------------ Conv2d
klineage_status_t klineage_conv2d_check_args(int y_dtype, int64_t N, int64_t H, int64_t W, int64_t C, int64_t F,
                                             int64_t R, int64_t S, int64_t pad_h, int64_t pad_w, int64_t stride_h,
                                             int64_t stride_w, const void* x, const void* w, const void* y, int variant)
{
    if (y_dtype != KLINEAGE_C_F32 && y_dtype != KLINEAGE_C_F16) return KLINEAGE_ERR_INVALID_ARG;
    if (variant != KLINEAGE_NAIVE && variant != KLINEAGE_TCGEN05) return KLINEAGE_ERR_BAD_VARIANT;
    const int64_t lim = int64_t(1) << 20;
    if (N < 0 || H < 0 || W < 0 || C < 0 || F < 0 || N >= lim || H >= lim || W >= lim || C >= lim || F >= lim)
        return KLINEAGE_ERR_INVALID_ARG;
    if (R < 1 || S < 1 || R > 64 || S > 64 || stride_h < 1 || stride_w < 1 || stride_h > 64 || stride_w > 64 ||
        pad_h < 0 || pad_w < 0 || pad_h > 64 || pad_w > 64)
        return KLINEAGE_ERR_INVALID_ARG;
    if (H + 2 * pad_h < R || W + 2 * pad_w < S) return KLINEAGE_ERR_INVALID_ARG;     // no output pixel
    const int64_t P = (H + 2 * pad_h - R) / stride_h + 1, Q = (W + 2 * pad_w - S) / stride_w + 1;
    const int64_t M = N * P * Q, K = R * S * C;
    if (M >= (int64_t(1) << 31) || K >= (int64_t(1) << 31)) return KLINEAGE_ERR_INVALID_ARG;
    if (M == 0 || F == 0) return KLINEAGE_OK;
    const size_t yelt = y_dtype == KLINEAGE_C_F16 ? 2 : 4;
    if (!y || reinterpret_cast<uintptr_t>(y) % yelt) return KLINEAGE_ERR_INVALID_ARG;
    if (K > 0) {
        if (!x || !w || reinterpret_cast<uintptr_t>(x) % 2 || reinterpret_cast<uintptr_t>(w) % 2) return KLINEAGE_ERR_INVALID_ARG;
        const size_t xb = size_t(N) * H * W * C * 2, wb = size_t(F) * K * 2, yb = size_t(M) * F * yelt;
        if (ranges_overlap(x, xb, y, yb) || ranges_overlap(w, wb, y, yb)) return KLINEAGE_ERR_INVALID_ARG;
    }
    return KLINEAGE_OK;
}

klineage_status_t klineage_conv2d_run(klineage_gemm_t h, int64_t N, int64_t H, int64_t W, int64_t C, int64_t F,
                                      int64_t R, int64_t S, int64_t pad_h, int64_t pad_w, int64_t stride_h,
                                      int64_t stride_w, const void* x, const void* w, void* y, int variant, void* stream)
{
    if (!h) return KLINEAGE_ERR_INVALID_ARG;
    h->last_launches = 0;
    const klineage_status_t chk = klineage_conv2d_check_args(h->c_dtype, N, H, W, C, F, R, S, pad_h, pad_w, stride_h,
                                                             stride_w, x, w, y, variant);
    if (chk != KLINEAGE_OK) return chk;
    ConvGeom cv;
    cv.H = static_cast<int>(H);
    cv.W = static_cast<int>(W);
    cv.C = static_cast<int>(C);
    cv.R = static_cast<int>(R);
    cv.S = static_cast<int>(S);
    cv.pad_h = static_cast<int>(pad_h);
    cv.pad_w = static_cast<int>(pad_w);
    cv.stride_h = static_cast<int>(stride_h);
    cv.stride_w = static_cast<int>(stride_w);
    cv.P = static_cast<int>((H + 2 * pad_h - R) / stride_h + 1);
    cv.Q = static_cast<int>((W + 2 * pad_w - S) / stride_w + 1);
    const int64_t M = N * cv.P * cv.Q, K = R * S * C;
    if (M == 0 || F == 0) {
        h->last_kernel_id = -1;
        return KLINEAGE_OK;
    }
    if (variant == KLINEAGE_TCGEN05 && h->ctx.cc_major != 10) return KLINEAGE_ERR_UNSUPPORTED_DEVICE;
    DeviceGuard guard(h->ctx.device);
    if (!guard.ok) return KLINEAGE_ERR_LAUNCH;
    // the implicit GEMM: rows = output pixels, columns = filters, k = (r, s, c); the weights are its
    // column-major B with pitch K, y its row-major C with pitch F
    GemmArgs g;
    g.M = static_cast<int>(M);
    g.N = static_cast<int>(F);
    g.K = static_cast<int>(K);
    g.A = static_cast<const uint16_t*>(x);
    g.lda = K;
    g.B = static_cast<const uint16_t*>(w);
    g.ldb = K;
    g.C = y;
    g.ldc = F;
    g.b_col = 1;
    g.c_bf16 = h->c_dtype == KLINEAGE_C_F16 ? 1 : 0;     // "2-byte C"; f16 selects the rounding
    g.status = h->status;
    g.bias = nullptr;
    g.f16 = 1;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int kid = -1;
    cudaError_t e;
    if (K == 0)
        e = launch_zero_fill(g, s, &kid);
    else if (variant == KLINEAGE_NAIVE)
        e = launch_conv2d_naive(g, cv, s, &kid);
    else
        e = launch_r4_conv2d(g, cv, h->ctx, s, &kid);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return KLINEAGE_ERR_LAUNCH;
    }
    h->last_kernel_id = kid;
    h->last_launches = 1;
    return KLINEAGE_OK;
}

// ------------------------------------------------------------------ launch plans and the autotuner
klineage_status_t klineage_gemm_plan_candidates(klineage_gemm_t h, int64_t M, int64_t N, int64_t K, const void* A,
                                                int64_t lda, const void* B, int64_t ldb, const void* C, int64_t ldc,
                                                klineage_gemm_plan_t* out, int cap, int* count)
{
    if (!h || !count || cap < 0 || (cap > 0 && !out)) return KLINEAGE_ERR_INVALID_ARG;
    const klineage_status_t chk =
        klineage_gemm_check_args(h->b_layout, h->c_dtype, M, N, K, A, lda, B, ldb, C, ldc, KLINEAGE_TCGEN05);
    if (chk != KLINEAGE_OK) return chk;
    const GemmArgs g = make_args(h, M, N, K, A, lda, B, ldb, nullptr, const_cast<void*>(C), ldc);
    DeviceGuard guard(h->ctx.device);      // (the planner may ask the runtime how many clusters the device holds)
    R4Plan tmp[KLINEAGE_MAX_PLANS];
    const int n = r4_enumerate_plans(g, h->ctx, tmp, KLINEAGE_MAX_PLANS);
    *count = n;
    for (int i = 0; i < n && i < cap; ++i) out[i] = to_public(tmp[i]);
    return KLINEAGE_OK;
}

klineage_status_t klineage_gemm_set_plan(klineage_gemm_t h, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                         const void* B, int64_t ldb, const void* C, int64_t ldc,
                                         const klineage_gemm_plan_t* plan)
{
    if (!h) return KLINEAGE_ERR_INVALID_ARG;
    const klineage_status_t chk =
        klineage_gemm_check_args(h->b_layout, h->c_dtype, M, N, K, A, lda, B, ldb, C, ldc, KLINEAGE_TCGEN05);
    if (chk != KLINEAGE_OK) return chk;
    const PlanKey key = plan_key(h, M, N, K, A, lda, B, ldb, C, ldc);
    if (!plan) {
        h->plans.erase(key);
        return KLINEAGE_OK;
    }
    const R4Plan pl = from_public(*plan);
    const GemmArgs g = make_args(h, M, N, K, A, lda, B, ldb, nullptr, const_cast<void*>(C), ldc);
    DeviceGuard guard(h->ctx.device);
    if (!r4_plan_valid(g, h->ctx, pl)) return KLINEAGE_ERR_INVALID_ARG;
    h->plans[key] = pl;
    return KLINEAGE_OK;
}

klineage_status_t klineage_gemm_get_plan(klineage_gemm_t h, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                         const void* B, int64_t ldb, const void* C, int64_t ldc,
                                         klineage_gemm_plan_t* plan_out, int* pinned_out)
{
    if (!h || !plan_out) return KLINEAGE_ERR_INVALID_ARG;
    const auto it = h->plans.find(plan_key(h, M, N, K, A, lda, B, ldb, C, ldc));
    const bool found = it != h->plans.end();
    *plan_out = to_public(found ? it->second : R4Plan());
    if (pinned_out) *pinned_out = found ? 1 : 0;
    return KLINEAGE_OK;
}

klineage_status_t klineage_gemm_autotune(klineage_gemm_t h, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                         const void* B, int64_t ldb, void* C, int64_t ldc, int iters, void* stream,
                                         klineage_gemm_plan_t* best_out, float* best_us_out, float* heuristic_us_out)
{
    if (!h) return KLINEAGE_ERR_INVALID_ARG;
    const klineage_status_t chk =
        klineage_gemm_check_args(h->b_layout, h->c_dtype, M, N, K, A, lda, B, ldb, C, ldc, KLINEAGE_TCGEN05);
    if (chk != KLINEAGE_OK) return chk;
    if (M == 0 || N == 0 || K == 0) {
        if (best_out) *best_out = to_public(R4Plan());
        if (best_us_out) *best_us_out = 0.f;
        if (heuristic_us_out) *heuristic_us_out = 0.f;
        return KLINEAGE_OK;
    }
    if (iters <= 0) iters = 10;
    DeviceGuard guard(h->ctx.device);
    if (!guard.ok) return KLINEAGE_ERR_LAUNCH;
    const GemmArgs g = make_args(h, M, N, K, A, lda, B, ldb, nullptr, C, ldc);
    R4Plan cand[KLINEAGE_MAX_PLANS];
    const int n = r4_enumerate_plans(g, h->ctx, cand, KLINEAGE_MAX_PLANS);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
        cudaGetLastError();
        if (e0) cudaEventDestroy(e0);
        return KLINEAGE_ERR_INTERNAL;
    }
    float best = -1.f, heur = -1.f;
    int best_i = -1;
    klineage_status_t fatal = KLINEAGE_OK;
    // Two passes over the candidates, the minimum of each candidate's two averages: a pass
    // sees every candidate under similar clocks, the minimum discards a disturbed one.
    float t_min[KLINEAGE_MAX_PLANS];
    for (int i = 0; i < n; ++i) t_min[i] = -1.f;
    h->forcing = true;
    for (int pass = 0; pass < 2 && fatal == KLINEAGE_OK; ++pass) {
        for (int i = 0; i < n; ++i) {
            if (pass == 1 && t_min[i] < 0.f) continue;   // failed in the first pass
            h->forced = cand[i];
            // one untimed launch (instruction cache, tensor maps), then the timed ones
            klineage_status_t st = klineage_gemm_run(h, M, N, K, A, lda, B, ldb, C, ldc, KLINEAGE_TCGEN05, stream);
            if (st == KLINEAGE_OK) {
                cudaEventRecord(e0, s);
                for (int r = 0; r < iters && st == KLINEAGE_OK; ++r)
                    st = klineage_gemm_run(h, M, N, K, A, lda, B, ldb, C, ldc, KLINEAGE_TCGEN05, stream);
                cudaEventRecord(e1, s);
            }
            if (cudaStreamSynchronize(s) != cudaSuccess) {
                cudaGetLastError();
                fatal = KLINEAGE_ERR_LAUNCH;
                break;
            }
            int code = 0;
            if (klineage_gemm_get_device_status(h, &code, nullptr) != KLINEAGE_OK) {
                fatal = KLINEAGE_ERR_INTERNAL;
                break;
            }
            if (st != KLINEAGE_OK || code != KLINEAGE_OK) {
                t_min[i] = -1.f;
                continue;
            }
            float ms = 0.f;
            cudaEventElapsedTime(&ms, e0, e1);
            const float us = ms * 1e3f / static_cast<float>(iters);
            if (pass == 0 || us < t_min[i]) t_min[i] = us;
        }
    }
    h->forcing = false;
    h->forced = R4Plan();
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (fatal != KLINEAGE_OK) return fatal;
    for (int i = 0; i < n; ++i) {
        if (t_min[i] < 0.f) continue;
        if (i == 0) heur = t_min[i];
        if (best_i < 0 || t_min[i] < best) {
            best = t_min[i];
            best_i = i;
        }
    }
    if (best_i < 0) return KLINEAGE_ERR_LAUNCH;
    // keep the heuristic plan unless a candidate beats it by more than the timing noise (1 %)
    if (heur > 0.f && best > 0.99f * heur) {
        best_i = 0;
        best = heur;
    }
    // leave C holding the product computed by the chosen plan
    h->plans[plan_key(h, M, N, K, A, lda, B, ldb, C, ldc)] = cand[best_i];
    const klineage_status_t st = klineage_gemm_run(h, M, N, K, A, lda, B, ldb, C, ldc, KLINEAGE_TCGEN05, stream);
    if (best_out) *best_out = to_public(cand[best_i]);
    if (best_us_out) *best_us_out = best;
    if (heuristic_us_out) *heuristic_us_out = heur;
    return st;
}

klineage_status_t klineage_gemm_get_device_status(klineage_gemm_t h, int* code_out, int* kernel_id_out)
{
    if (!h || !code_out) return KLINEAGE_ERR_INVALID_ARG;
    DeviceGuard guard(h->ctx.device);
    unsigned w[4] = {0, 0, 0, 0};
    if (cudaMemcpy(w, h->status, sizeof w, cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        return KLINEAGE_ERR_INTERNAL;
    }
    *code_out = (w[0] == kDevOk) ? KLINEAGE_OK : KLINEAGE_ERR_TIMEOUT;
    if (kernel_id_out) *kernel_id_out = static_cast<int>(w[1]);
    if (w[0] != kDevOk) {
        fprintf(stderr, "klineage_gemm: device-side give-up code=%u block=%u where=0x%x\n", w[0], w[2], w[3]);
        h->give_up_block = w[2];
        h->give_up_where = w[3];
        if (cudaMemset(h->status, 0, sizeof(unsigned)) != cudaSuccess) cudaGetLastError();
        // A CTA that gave up may have left split-K arrival counters short of their self-reset; a later split
        // launch would then see a wrong last arriver.  The stream is idle by contract: start them from zero.
        if (cudaMemset(h->ctx.tile_counters, 0, sizeof(unsigned) * h->ctx.n_tile_counters) != cudaSuccess) cudaGetLastError();
    }
    return KLINEAGE_OK;
}

int klineage_gemm_last_kernel_id(klineage_gemm_t h) { return h ? h->last_kernel_id : -1; }

klineage_status_t klineage_gemm_last_give_up(klineage_gemm_t h, unsigned* block_out, unsigned* where_out)
{
    if (!h) return KLINEAGE_ERR_INVALID_ARG;
    if (block_out) *block_out = h->give_up_block;
    if (where_out) *where_out = h->give_up_where;
    return KLINEAGE_OK;
}

const char* klineage_status_string(int status)
{
    switch (status) {
        case KLINEAGE_OK: return "ok";
        case KLINEAGE_ERR_INVALID_ARG: return "invalid argument";
        case KLINEAGE_ERR_BAD_VARIANT: return "bad variant";
        case KLINEAGE_ERR_UNSUPPORTED_DEVICE: return "unsupported device";
        case KLINEAGE_ERR_ALLOC: return "allocation failed";
        case KLINEAGE_ERR_LAUNCH: return "launch failed";
        case KLINEAGE_ERR_TIMEOUT: return "device-side wait timed out";
        case KLINEAGE_ERR_INTERNAL: return "internal error";
        case KLINEAGE_ERR_SCRATCH_LIMIT: return "shape exceeds the fixed scratch of the allocation-free call";
        default: return "unknown status";
    }
}

const char* klineage_variant_name(int variant)
{
    switch (variant) {
        case KLINEAGE_NAIVE: return "naive";
        case KLINEAGE_TILED: return "tiled";
        case KLINEAGE_VECTORIZED: return "vectorized";
        case KLINEAGE_PIPELINED: return "pipelined";
        case KLINEAGE_TCGEN05: return "tcgen05";
        case KLINEAGE_MMA_SYNC: return "mma_sync";
        default: return "unknown";
    }
}

}  // extern "C"
