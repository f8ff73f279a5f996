/*
 * klineage_gemm.h - C ABI of the B200 (sm_100a) bf16 GEMM lineage.
 *
 * The library computes  C <- A . B  for bf16 A and B with fp32 accumulation and
 * an fp32 or bf16 C, for arbitrary (unaligned) M, N, K and leading dimensions.
 * It offers the same product through five separately selectable kernels that
 * form a forward lineage in the sense of the paper's Method section (a lineage
 * L = (K_0, tau_1, ..., K_n) from a naive kernel K_0 to an expert kernel K_n):
 * each rung adds one of the optimization intents the paper's Introduction and
 * Table 1 name, together with the precondition that makes it valid.
 *
 * C99, no C++ types, no exceptions cross this boundary.  All pointers named
 * "device" are device pointers on the handle's GPU; everything else is host
 * memory.  There is no CPU fallback and no cross-rung fallback: a variant
 * either runs its own kernel or the call returns an error (the paper's
 * harness notes, Appendix B, describe how wrappers that silently fall back to
 * a reference fake correctness).
 */
#ifndef KLINEAGE_GEMM_H
#define KLINEAGE_GEMM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Opaque handle, owned by the library, released by klineage_gemm_destroy. */
typedef struct klineage_gemm_s* klineage_gemm_t;

typedef enum {
    KLINEAGE_OK = 0,
    KLINEAGE_ERR_INVALID_ARG = 1,        /* null pointer, negative size, ld too small, aliasing ... */
    KLINEAGE_ERR_BAD_VARIANT = 2,        /* variant outside 0..5                                      */
    KLINEAGE_ERR_UNSUPPORTED_DEVICE = 3, /* the rung needs sm_100 hardware the device lacks          */
    KLINEAGE_ERR_ALLOC = 4,              /* device or host allocation failed in create                */
    KLINEAGE_ERR_LAUNCH = 5,             /* the CUDA runtime rejected a launch or a tensor map        */
    KLINEAGE_ERR_TIMEOUT = 6,            /* a bounded device-side wait gave up (see get_device_status) */
    KLINEAGE_ERR_INTERNAL = 7,
    KLINEAGE_ERR_SCRATCH_LIMIT = 8       /* klineage_gemm_run_noalloc: the shape needs more fixed scratch than exists */
} klineage_status_t;

/* Storage of B (K x N).  A is always row-major M x K, C always row-major M x N. */
typedef enum {
    KLINEAGE_B_ROW_MAJOR = 0, /* element (k, j) at B[k * ldb + j]  (N contiguous) */
    KLINEAGE_B_COL_MAJOR = 1  /* element (k, j) at B[j * ldb + k]  (K contiguous) */
} klineage_layout_t;

typedef enum {
    KLINEAGE_C_F32 = 0, /* C holds the fp32 accumulator                                  */
    KLINEAGE_C_BF16 = 1, /* C holds the accumulator rounded to bf16, round-to-nearest-even */
    KLINEAGE_C_F16 = 2   /* klineage_conv2d_run only: y holds the accumulator rounded to fp16 (RNE); the
                            GEMM calls refuse a handle of this dtype with KLINEAGE_ERR_INVALID_ARG       */
} klineage_ctype_t;

/*
 * The lineage rungs (paper: the Introduction's list of optimization intents -
 * tiles, staging through shared memory, wide loads, a software pipeline, matrix
 * instructions - and the transition vocabulary of Table 1).
 */
typedef enum {
    KLINEAGE_NAIVE = 0,      /* K_0: one thread per C element, K-loop over global memory                     */
    KLINEAGE_TILED = 1,      /* Table 1 "tile / sm_stage": block tile staged in shared memory, register tile */
    KLINEAGE_VECTORIZED = 2, /* Table 1 "vectorize_global": 128-bit accesses when aligned, masked tail,
                                scalar fallback when base or leading dimension is not 16-byte aligned        */
    KLINEAGE_PIPELINED = 3,  /* Table 1 "cp.async + pipeline" / "tma_load": multi-stage ring fed by TMA with
                                full/empty mbarriers; producer threads when TMA's alignment rules fail       */
    KLINEAGE_TCGEN05 = 4,    /* Table 1 "warp_specialize" + matrix intrinsics: tcgen05.mma into TMEM (the
                                sm_100 successor of the table's wgmma), producer / MMA / epilogue warps,
                                persistent tile scheduler, swizzled shared-memory epilogue, split-K          */
    KLINEAGE_MMA_SYNC = 5    /* "rung 3.5", outside the five-step ladder: Table 1 "ldmatrix.swizzle" + "mma
                                (m16n8k16)", the legacy warp-level tensor-core path on rung 3's TMA ring; it
                                sits between rungs 3 and 4 in speed and completes the table's vocabulary       */
} klineage_variant_t;

/*
 * KLINEAGE_FLAG_STATIC_B - a promise about the caller's B operands ("the weights are static"): no GPU work
 * that is still in flight when a klineage_gemm_run* call is enqueued writes B.  The tcgen05 rung then
 * starts streaming B for a short (single-wave) launch before it waits for the previous kernel in the
 * stream - launches go out with programmatic stream serialization, so the kernel may start while its
 * predecessor drains - and waits only before it reads A and before it writes C.  For back-to-back
 * weight-streaming calls (the decode shape) this hides the kernel boundary.  Without the flag every
 * global access waits for the previous kernel.  The paper has no counterpart; results are identical.
 */
#define KLINEAGE_FLAG_STATIC_B 1u

/*
 * KLINEAGE_FLAG_TEST_GIVE_UP - a test hook for the boundary's error path (KLINEAGE_ERR_TIMEOUT,
 * klineage_gemm_get_device_status).  The FIRST klineage_gemm_run(..., KLINEAGE_TCGEN05, ...) call on the
 * handle that takes the single-CTA, non-cluster, TMA-fed kernel with more than two k-blocks per tile makes
 * that launch give up in the permitted way: its TMA producer stops after two k-blocks and the MMA issuer's
 * bounded wait for the third runs out after about a millisecond, whereupon every CTA records the error,
 * raises its abort flag, lets its other roles leave their loops, frees its tensor memory and RETURNS
 * NORMALLY - no trap, no fault, nothing unbounded; C is not written.  Every later call on the handle runs
 * normally.  The paper's gate (Method: a candidate must compile, be correct and be profiled) needs failures
 * to surface as statuses, which is what this flag lets a test observe.
 */
#define KLINEAGE_FLAG_TEST_GIVE_UP 2u

/* Create-time configuration (host memory, read during create only). */
typedef struct {
    int device;             /* CUDA device ordinal the handle is bound to                              */
    int b_layout;           /* klineage_layout_t                                                       */
    int c_dtype;            /* klineage_ctype_t                                                        */
    size_t workspace_bytes; /* device scratch of rung 4: split-K partial sums, aligned copies of unaligned
                               operands, the tables of grouped / multi-destination launches; 0 selects
                               the default (64 MiB).  Calls on one handle share it: one stream at a time */
    unsigned flags;         /* 0, or an OR of KLINEAGE_FLAG_STATIC_B, KLINEAGE_FLAG_TEST_GIVE_UP              */
} klineage_gemm_config_t;

/*
 * Creates a handle bound to cfg->device with the given B layout and C dtype
 * (the paper's GEMM workload, Evaluation Table 2, fixes neither; they are
 * properties of the handle so that klineage_gemm_run keeps the BLAS-like
 * argument list).  Allocates the device workspace and status block (this is the
 * only allocating call besides destroy).  out and cfg are host pointers.
 * Errors: INVALID_ARG (null, bad enum, unknown flag bits, no such device), ALLOC.
 */
klineage_status_t klineage_gemm_create(klineage_gemm_t* out, const klineage_gemm_config_t* cfg);

/*
 * Enqueues C <- A . B on `stream` (a cudaStream_t, may be NULL for the default
 * stream) using exactly the rung `variant` (0..5); returns after the enqueue, performs
 * no device synchronisation and no allocation.
 *
 *   M, N, K   sizes, 0 <= value < 2^31.  M*N == 0: nothing is launched, OK.
 *             K == 0: C is set to zero.
 *   A         device, bf16 bits, row-major M x K, lda >= K  (elements)
 *   B         device, bf16 bits, K x N in the handle's layout,
 *             ldb >= N (row-major) or ldb >= K (column-major)
 *   C         device, fp32 or bf16 per the handle, row-major, ldc >= N; write-only
 *             (previous contents, NaN included, are ignored); padding between N and
 *             ldc is never written.  A and B must not overlap C.
 *   Pointers need only element alignment (2 bytes bf16, 4 bytes fp32); wider
 *   alignment is detected per call and selects the vector / TMA sub-paths
 *   (paper, Introduction: a wide load is valid only on aligned addresses and
 *   with its tail handled).  Buffers stay owned by the caller.
 *
 * Errors: INVALID_ARG, BAD_VARIANT, UNSUPPORTED_DEVICE (variant 3, 4 or 5 on a
 * device without sm_100 TMA/tcgen05), LAUNCH.  Device-side give-ups (a bounded
 * barrier wait that expired) are reported by klineage_gemm_get_device_status.
 * One handle must not be used from two host threads at once.
 */
klineage_status_t klineage_gemm_run(klineage_gemm_t h, int64_t M, int64_t N, int64_t K,
                                    const void* A, int64_t lda, const void* B, int64_t ldb,
                                    void* C, int64_t ldc, int variant, void* stream);

/*
 * AddMM:  C <- A . B + bias,  bias a vector of N bf16 values (device, 2-byte aligned,
 * not overlapping C) added to every row - the bias-epilogue fusion of the paper's
 * held-out plain-GEMM family (Appendix D, "Additional Held-out Verification": AddMM at
 * 4096^3).  The bias is added to the fp32 accumulator before the rounding to bf16 (bf16 C);
 * with a K split it is added once, by the final reduction.  K == 0 gives C[i][j] = bias[j].
 * Every other argument, rule and error is that of klineage_gemm_run; bias == NULL with
 * M*N > 0 is INVALID_ARG.
 */
klineage_status_t klineage_gemm_run_addmm(klineage_gemm_t h, int64_t M, int64_t N, int64_t K,
                                          const void* A, int64_t lda, const void* B, int64_t ldb,
                                          const void* bias, void* C, int64_t ldc, int variant, void* stream);

/*
 * The host-side argument checks of klineage_gemm_run, callable without a handle
 * or a device (pointers are only compared, never dereferenced).  Returns what
 * run would return for these arguments before touching the GPU: OK,
 * INVALID_ARG or BAD_VARIANT.  The paper states the principle (Introduction):
 * an optimization applied outside its precondition yields a wrong or failing
 * kernel, so preconditions are checked, not assumed.
 */
klineage_status_t klineage_gemm_check_args(int b_layout, int c_dtype, int64_t M, int64_t N, int64_t K,
                                           const void* A, int64_t lda, const void* B, int64_t ldb,
                                           const void* C, int64_t ldc, int variant);

/* Releases the handle, its workspace and status block.  NULL is accepted. */
klineage_status_t klineage_gemm_destroy(klineage_gemm_t h);

/*
 * Reads the device status block (synchronous copy; call after synchronising
 * the stream).  *code_out receives KLINEAGE_OK or KLINEAGE_ERR_TIMEOUT;
 * *kernel_id_out (may be NULL) receives the id the last finished kernel wrote
 * on the device, which identifies rung and sub-path (see
 * klineage_gemm_last_kernel_id).  The error code is cleared by the read; after a
 * give-up the handle's split-K arrival counters are reset as well, so that the
 * next call starts clean.
 * The paper's gate (Method: compile, correctness, profile) is what this serves.
 */
klineage_status_t klineage_gemm_get_device_status(klineage_gemm_t h, int* code_out, int* kernel_id_out);

/*
 * Where the last device-side give-up reported by klineage_gemm_get_device_status on this
 * handle happened: *block_out the CTA, *where_out the role and barrier -
 *   0x400|s producer / "stage s free",  0x410|b MMA issuer / "accumulator b drained",
 *   0x420|s MMA issuer / "operand stage s landed",  0x430|b epilogue / "accumulator b complete",
 *   0x440..0x470|s gathering producers and the Conv2d producers,  0x500.. the CTA-pair kernel's roles.
 * Both are 0 when no give-up has been read.  Either pointer may be NULL.
 */
klineage_status_t klineage_gemm_last_give_up(klineage_gemm_t h, unsigned* block_out, unsigned* where_out);

/*
 * Host-side record of the kernel the last successful run enqueued:
 *   0 naive | 100 tiled | 200 + 1*(A vector) + 2*(B vector) + 4*(C vector)
 *   300 TMA pipeline, 301 producer-thread pipeline
 *   400 + 1*(generic-proxy producer) + 2*(direct epilogue) + 4*(split-K) + 8*(skinny mode)
 *       + 16*(cluster reduce) + 32*(CTA-pair MMA) + 64*(unaligned operands repacked into the workspace)
 *       + 128*(last wave of CTA-pair tiles streamed along K)
 *       + 256*(CTA-pair MMA on 256-row tiles, two k-blocks per stage)
 *   500 mma.sync rung on the TMA ring, 501 on producer threads
 *   900 zero fill (K == 0); -1 before the first run or after a no-op.
 */
int klineage_gemm_last_kernel_id(klineage_gemm_t h);

/*
 * The tcgen05 rung (variant 4) for callers that must not allocate device memory.
 * (The paper has no counterpart to this call; it exists for integration.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a plug-in or
 * operator called by a host framework that owns the whole memory budget and
 * forbids outside allocations, a latency-critical serving loop (cudaMalloc can
 * synchronise the device and may fail late, under memory pressure), or a process
 * whose remaining device memory is already spoken for.  klineage_gemm_create
 * allocates a workspace, so such callers cannot even obtain a handle.
 *
 * This call takes no handle and calls no allocator: not cudaMalloc/cudaFree, not
 * an allocating library routine.  Its scratch memory (split-K partial sums,
 * arrival counters, status words) is a fixed array inside the library image:
 * 8 MiB of partial sums + 16 KiB of counters.  Every GPU that loads the library
 * holds those bytes until the process exits, whether or not this call is used.
 *
 *   b_layout, c_dtype   as in klineage_gemm_config_t
 *   M, N, K, A, lda, B, ldb, C, ldc, stream   exactly as for klineage_gemm_run;
 *                       the caller still owns and passes inputs and output
 *   The GEMM runs on the calling thread's current CUDA device; the pointers must
 *   belong to that device.
 *
 * Limits and rules:
 *   - A shape whose K split would need more than the 8 MiB of partial sums
 *     (splits * M * round_up(N,4) * 4 bytes; only shapes with few output tiles
 *     are split) is refused with KLINEAGE_ERR_SCRATCH_LIMIT and a message on
 *     stderr; nothing is launched.  Use a handle for such shapes.
 *   - The first call on each device looks up the array's device address (with
 *     that device current).  Make that first call outside any stream capture.
 *   - All calls share the one array, which keeps the previous call's contents;
 *     each call re-zeroes the counters and status words on `stream` before its
 *     kernel.  Two calls that overlap on the GPU (different streams, or several
 *     host threads) race on the array: keep calls to one stream at a time.
 *   - Device-side give-ups (bounded waits) cannot be read back through this call.
 * Results: for operands that satisfy TMA's alignment rules (16-byte aligned base
 * and pitch of A and B) the call runs the same kernels with the same schedule as
 * klineage_gemm_run(..., KLINEAGE_TCGEN05, ...) on a default handle and gives the
 * same bits.  Unaligned operands take another sub-path here (the handle copies
 * them into its workspace first, this call gathers them tile by tile, and the two
 * may split K differently): the result then carries the library's usual
 * guarantee - bit-exact where fp32 sums are exact, else within
 * K * 2^-23 * (|A| . |B|)_ij of the exact product - not bit equality with the
 * handle path.
 * Errors: as klineage_gemm_run, plus KLINEAGE_ERR_SCRATCH_LIMIT.
 */
klineage_status_t klineage_gemm_run_noalloc(int b_layout, int c_dtype, int64_t M, int64_t N, int64_t K,
                                            const void* A, int64_t lda, const void* B, int64_t ldb,
                                            void* C, int64_t ldc, void* stream);

/* ---------------------------------------------------------------------------
 * Batched and grouped GEMM (paper, Appendix D: BMM at batch 16 x 2048^3 and
 * batch 32 x 1024^3, GroupedGEMM at G = 4 and 8 are held-out members of the GEMM
 * family; the paper prints no interface for them, this one follows the
 * strided-batch and pointer-array conventions of BLAS libraries).
 *
 * klineage_gemm_run_batched: C_b <- A_b . B_b for b in [0, batch), every problem
 * of the shape and layout of klineage_gemm_run; operand b starts stride_a /
 * stride_b / stride_c ELEMENTS after operand b-1 (device memory).  stride_a or
 * stride_b may be 0 (one matrix shared by all batches); the C matrices must not
 * overlap (stride_c >= (M-1)*ldc + N when batch > 1) nor overlap A or B.
 * batch <= 65535; batch == 0 is a no-op.
 *
 * klineage_gemm_run_grouped: C_i <- A_i . B_i for i in [0, groups), each group
 * with its own M[i], N[i], K[i], pointers and pitches; all groups share the
 * handle's B layout and C dtype.  The ten arrays are HOST arrays of `groups`
 * entries, read before the call returns; the pointers in A, B, C are device
 * pointers.  Groups with M*N == 0 are skipped, K == 0 zero-fills that C.  No C
 * may overlap another group's C or any A or B.
 *
 * Execution: with variant KLINEAGE_TCGEN05 and TMA-loadable operands (16-byte
 * aligned bases, pitches and batch strides), ONE launch walks the tiles of all
 * problems (batched: the batch is the third dimension of the tensor maps;
 * grouped: a table of per-group tensor maps and sizes, built in the handle's
 * workspace and copied on `stream` ahead of the kernel; at most 256 groups per
 * launch) when they fill at least half of the SMs: on the CTA-pair kernel
 * (512 x 256 tiles, or 256 x 256 tiles when twice the tiles take fewer than
 * twice the rounds over the CTA pairs - see `stages` of the launch plan) or on
 * the single-CTA kernel (128 x 256 tiles, whose double-buffered accumulator
 * hides the epilogue), whichever schedule the rung's cycle estimate makes the
 * shorter over all problems of the call; grouped calls take the pair kernel
 * only when every problem has more than 256 rows or rounding every group's
 * rows up to a multiple of 256 adds at most a quarter (with 512-row tiles, a
 * tile with at most 256 live rows does half the work and such last tile rows
 * of the groups are scheduled last).  A plan pinned for the shape of the (first) problem
 * may name the kernel.  Every other case - lower
 * rungs, unaligned operands, a K == 0 group, too few tiles - runs the rung's
 * ordinary path once per problem, in order, on `stream`.
 * Results equal those of `batch` / `groups` separate klineage_gemm_run calls
 * with the same variant, bit for bit unless such a call would split K.
 * Errors: as klineage_gemm_run; everything is validated before the first launch.
 */
klineage_status_t klineage_gemm_run_batched(klineage_gemm_t h, int64_t batch, int64_t M, int64_t N, int64_t K,
                                            const void* A, int64_t lda, int64_t stride_a,
                                            const void* B, int64_t ldb, int64_t stride_b,
                                            void* C, int64_t ldc, int64_t stride_c,
                                            int variant, void* stream);

klineage_status_t klineage_gemm_run_grouped(klineage_gemm_t h, int groups,
                                            const int64_t* M, const int64_t* N, const int64_t* K,
                                            const void* const* A, const int64_t* lda,
                                            const void* const* B, const int64_t* ldb,
                                            void* const* C, const int64_t* ldc,
                                            int variant, void* stream);

/* ---------------------------------------------------------------------------
 * Conv2d as an implicit GEMM on the tcgen05 rung (paper, Evaluation, Table 2: Conv2d,
 * N=8, C=64, 56x56, F=128, 3x3, FP16; the paper fixes neither layout, padding nor
 * stride - channels-last and "same" padding are this library's reading for that
 * shape, the call takes any padding and stride).
 *
 *   y[n][p][q][f] = sum_{r,s,c} x[n][p*stride_h + r - pad_h][q*stride_w + s - pad_w][c] * w[f][r][s][c]
 *
 * (cross-correlation, zero outside the image), P = (H + 2 pad_h - R)/stride_h + 1,
 * Q likewise.  x: device, fp16 bits, (N, H, W, C) contiguous; w: device, fp16 bits,
 * (F, R, S, C) contiguous; y: device, (N, P, Q, F) contiguous, fp32 or fp16 per the
 * handle's c_dtype (KLINEAGE_C_F32 or KLINEAGE_C_F16; the handle's B layout is not
 * used); fp32 accumulation.  Pointers need element alignment only; 16-byte aligned x
 * with C % 8 == 0 selects 16-byte patch loads.  variant: KLINEAGE_NAIVE (direct
 * convolution, one thread per output) or KLINEAGE_TCGEN05 (rows = output pixels,
 * columns = filters, k = (r, s, c); the patches reach the swizzled shared-memory operand
 * layout as 4-D TMA boxes whose out-of-image part is zero-filled (C % 64 == 0, unit
 * stride) or are gathered by producer warps - no im2col buffer exists - and
 * tcgen05.mma.kind::f16 multiplies fp16 operands into TMEM).  No output pixel
 * (N*P*Q == 0) or F == 0: nothing is launched; C == 0: y is zero-filled.
 * Errors: INVALID_ARG (sizes, R or S outside 1..64, padding or stride outside
 * 0..64 / 1..64, a filter larger than the padded image, null or overlapping
 * buffers, a handle of dtype BF16), BAD_VARIANT, UNSUPPORTED_DEVICE, LAUNCH.
 */
klineage_status_t klineage_conv2d_check_args(int y_dtype, int64_t N, int64_t H, int64_t W, int64_t C,
                                             int64_t F, int64_t R, int64_t S, int64_t pad_h, int64_t pad_w,
                                             int64_t stride_h, int64_t stride_w,
                                             const void* x, const void* w, const void* y, int variant);
klineage_status_t klineage_conv2d_run(klineage_gemm_t h, int64_t N, int64_t H, int64_t W, int64_t C,
                                      int64_t F, int64_t R, int64_t S, int64_t pad_h, int64_t pad_w,
                                      int64_t stride_h, int64_t stride_w,
                                      const void* x, const void* w, void* y, int variant, void* stream);

/*
 * One product, several destinations:  C_d <- A . B  for d in [0, n_dst), n_dst <= 16.
 * C and ldc are HOST arrays of n_dst device pointers / pitches (read before the call
 * returns); every destination is an M x N matrix of the handle's C dtype and may
 * live on another GPU that this device can address (peer access enabled by the
 * caller).  This is the fused all-gather of a GEMM partitioned by columns over
 * several GPUs: rank r multiplies A by its column slice of B and passes, as
 * destinations, the address of that slice inside every rank's full-width C - no
 * operand is ever loaded from a peer, results leave through plain or TMA stores
 * (the paper has no multi-GPU design; its hardware section is single-GPU).
 * With variant KLINEAGE_TCGEN05, TMA-loadable A and B and a shape that needs neither
 * a K split nor the skinny orientation, one launch writes every output block to all
 * destinations from its epilogue; every other case computes into C_0 through the
 * rung's ordinary path and copies that matrix to the other destinations on `stream`.
 * Destinations must not overlap one another, A or B.  Errors: as klineage_gemm_run.
 */
klineage_status_t klineage_gemm_run_multi_dst(klineage_gemm_t h, int64_t M, int64_t N, int64_t K,
                                              const void* A, int64_t lda, const void* B, int64_t ldb,
                                              int n_dst, void* const* C, const int64_t* ldc,
                                              int variant, void* stream);

/* Number of GEMM kernels the last klineage_gemm_run / _run_addmm / _run_batched /
 * _run_grouped call on this handle enqueued (1 when a batched or grouped call took
 * its one-launch path; zero-fill launches count, repack pre-passes do not). */
int klineage_gemm_last_launch_count(klineage_gemm_t h);

/* ---------------------------------------------------------------------------
 * The product with HOST operands: copies and kernels overlapped by the library.
 *
 * The paper times kernels with their operands already on the device
 * (Evaluation, Setup); a caller whose matrices live in host memory pays the
 * transfers as well, and a GEMM splits by rows of A and C so that they overlap
 * the arithmetic.  klineage_gemm_run_host computes the same C = A . B as
 * klineage_gemm_run, through the same rung kernels, with A, B and C in HOST memory:
 *
 *   copy stream   B (whole), then A row slab by row slab        (host -> device)
 *   `stream`      slab i of C = slab i of A . B, on `variant`   (after its A slab landed)
 *   store stream  slab i of C                                   (device -> host, after its kernel)
 *
 * so that, after B, the link carries A while earlier slabs are multiplied and
 * their results travel back in the other direction.  Slabs are whole multiples
 * of 128 rows, at most 16 per call.
 *
 *   A, B, C    HOST pointers; same shapes, pitches (elements, any value >= the
 *              row length) and element types as in klineage_gemm_run.  Page-locked
 *              memory makes the copies asynchronous and lets them overlap; pageable
 *              memory is accepted and gives the same result without the overlap.
 *              Only the M x N (M x K, ...) elements are read or written, padding
 *              up to the pitch is not touched.  The buffers must stay valid, and A
 *              and B unmodified, until work enqueued on `stream` after this call
 *              has been reached (for instance until the stream is synchronised).
 *   scratch    DEVICE memory on the handle's GPU, owned by the caller, at least
 *              klineage_gemm_host_scratch_bytes(...) bytes, 256-byte aligned.  It
 *              holds the device copies of A, B and C (pitches rounded up to 16
 *              bytes, so the TMA sub-paths always apply) and may be reused by the
 *              caller once `stream` has passed this call.
 *   stream     work enqueued on it before the call precedes every copy, work
 *              enqueued after the call follows the last copy back to the host.
 *
 * The first call on a handle creates the two internal streams and their events
 * (no device memory); destroy releases them.  M == 0 or N == 0: OK, nothing is
 * done.  K == 0: C_host <- 0.  Errors: as klineage_gemm_run, plus INVALID_ARG for a
 * missing, misaligned or too small scratch and for host ranges of A or B that
 * overlap C; LAUNCH when a copy cannot be enqueued.
 * klineage_gemm_last_launch_count then reports the slab kernels of the call.
 */
size_t klineage_gemm_host_scratch_bytes(int b_layout, int c_dtype, int64_t M, int64_t N, int64_t K);

klineage_status_t klineage_gemm_run_host(klineage_gemm_t h, int64_t M, int64_t N, int64_t K,
                                         const void* A_host, int64_t lda, const void* B_host, int64_t ldb,
                                         void* C_host, int64_t ldc,
                                         void* scratch_device, size_t scratch_bytes,
                                         int variant, void* stream);

/* ---------------------------------------------------------------------------
 * Launch plans and the autotuner of the tcgen05 rung.
 *
 * Paper, Table 1 (transition vocabulary: `templatize`, `autotune`) and Appendix D
 * (the recipe parameters a skill carries - block size, stages, split - steered
 * by a short sweep on top of a fixed kernel structure).  The tcgen05 rung leaves
 * a few choices of its schedule open; each is a field of the plan below, 0 =
 * "let the rung's heuristic decide":
 *   kernel     1 single-CTA kernel (128 x 256 tiles), 2 CTA-pair kernel (512 x 256 tiles)
 *   splits     number of K splits (1 = none)
 *   split_via  with splits > 1: 1 partial sums through the global workspace,
 *              2 through a thread-block cluster (splits 2 / 4 / 8; M <= 32 or M > 64);
 *              with kernel 2 and splits 1: 3 streams the under-filled last wave of pair tiles along K (the
 *              k-blocks of its tiles are dealt out evenly over all CTA pairs; pieces that do not hold a tile's
 *              first k-block pass their fp32 partial tile through the workspace, the piece that does adds them
 *              in k order - a fixed order, so results repeat bit for bit), 1 never does
 *   group_m    tile-rows per raster group (L2 reuse pattern)
 *   half_tail  1 cut the last wave into 128-column half tiles, 2 never
 *   tile_n     columns per output tile (needs `kernel`): single-CTA kernel 256, 128 or 64; CTA-pair kernel a
 *              multiple of 64 up to 256
 *   tail_n     CTA-pair kernel only: tile_n = every tile of that width; a smaller multiple of 64 = tile rows
 *              start with tile_n-wide tiles and end with tiles of this width, dealt to the CTA pairs back and
 *              forth so that wide and narrow turns balance a last, under-filled wave
 *   stages     single-CTA kernel: depth of the operand ring in 64-deep k-blocks - 4; 6 with 128- or 64-column
 *              tiles; 8 with 64-column tiles.  Without a K split, 6 stages of 128-column tiles and 8 stages of
 *              64-column tiles are filled and freed two k-blocks at a time (3 / 4 stages of 128 k).
 *              CTA-pair kernel: 3 = tiles of 256 x 256 instead of 512 x 256, three stages of two k-blocks each,
 *              the two TMEM accumulators holding consecutive tiles of a pair (one fills while the other drains);
 *              256-column tiles only, no narrow tail, no streamed wave.  The heuristic takes it when such
 *              tiles make one round over more than half of the CTA pairs (K >= 3072, or K >= 1280 where the
 *              single-CTA kernel's wave would be less than 85 % full) or several rounds that its cycle estimate
 *              puts ahead of the 512-row tiles' rounds
 * Every plan computes the same C up to fp32 summation order (plans that differ
 * only in kernel / group_m / half_tail / tile shape / stages are bit-identical; K
 * splits change the order of the partial sums and stay within the parity bound).
 *   split_via  2 also covers 128-row tiles (M > 64): the K splits of a tile then run as one cluster whose
 *              CTAs exchange their partial tiles through the idle operand rings (one wave of clusters at most)
 *
 * A plan is pinned per handle for one (M, N, K) and alignment class of the
 * operands (16-byte alignment of base and pitch of A, B, C; the pointers are
 * used for nothing else and no memory is touched).  Later klineage_gemm_run /
 * klineage_gemm_run_addmm calls with variant KLINEAGE_TCGEN05 on that shape use
 * it.  All host-side; not thread-safe per handle.
 */
typedef struct {
    int kernel;
    int splits;
    int split_via;
    int group_m;
    int half_tail;
    int tile_n;
    int tail_n;
    int stages;
} klineage_gemm_plan_t;

#define KLINEAGE_MAX_PLANS 48

/* Writes the candidate plans of a problem to out[0 .. min(cap, *count)) and their
 * number to *count (at most KLINEAGE_MAX_PLANS); out[0] is the all-zero
 * heuristic plan.  Host only.  Errors: as klineage_gemm_check_args. */
klineage_status_t klineage_gemm_plan_candidates(klineage_gemm_t h, int64_t M, int64_t N, int64_t K,
                                                const void* A, int64_t lda, const void* B, int64_t ldb,
                                                const void* C, int64_t ldc,
                                                klineage_gemm_plan_t* out, int cap, int* count);

/* Pins `plan` for the shape (plan == NULL removes the pin).  A plan that cannot
 * run the shape (e.g. the pair kernel with unaligned operands, more splits than
 * k-blocks or than the workspace holds) is refused with KLINEAGE_ERR_INVALID_ARG
 * and nothing changes. */
klineage_status_t klineage_gemm_set_plan(klineage_gemm_t h, int64_t M, int64_t N, int64_t K,
                                         const void* A, int64_t lda, const void* B, int64_t ldb,
                                         const void* C, int64_t ldc, const klineage_gemm_plan_t* plan);

/* Reads the pinned plan (*pinned_out = 1) or the all-zero plan (*pinned_out = 0). */
klineage_status_t klineage_gemm_get_plan(klineage_gemm_t h, int64_t M, int64_t N, int64_t K,
                                         const void* A, int64_t lda, const void* B, int64_t ldb,
                                         const void* C, int64_t ldc,
                                         klineage_gemm_plan_t* plan_out, int* pinned_out);

/* Times every candidate plan on the caller's operands (device pointers, as for
 * klineage_gemm_run; `iters` launches per measurement, <= 0 means 10, CUDA events
 * on `stream`, two passes, minimum), pins the fastest - the heuristic plan unless
 * another beats it by more than 1 % - and leaves C = A.B computed by it.
 * Blocks the host until done (this call synchronises `stream`).  Candidates whose
 * launch fails or that report a device-side give-up are skipped.
 * best_out / best_us_out / heuristic_us_out (each optional): the pinned plan,
 * its time per launch and the heuristic plan's, in microseconds.
 * Errors: as klineage_gemm_run; KLINEAGE_ERR_LAUNCH when no candidate ran. */
klineage_status_t klineage_gemm_autotune(klineage_gemm_t h, int64_t M, int64_t N, int64_t K,
                                         const void* A, int64_t lda, const void* B, int64_t ldb,
                                         void* C, int64_t ldc, int iters, void* stream,
                                         klineage_gemm_plan_t* best_out, float* best_us_out,
                                         float* heuristic_us_out);

const char* klineage_status_string(int status);
const char* klineage_variant_name(int variant);

#ifdef __cplusplus
}
#endif
#endif /* KLINEAGE_GEMM_H */
