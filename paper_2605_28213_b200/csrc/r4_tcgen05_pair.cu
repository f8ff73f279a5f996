// Rung 4, CTA-pair form: tcgen05.mma.cta_group::2.
//
// Two CTAs on neighbouring SMs (a cluster of 2) share one 512 x 256 output
// tile, computed as two 256-row MMA blocks.  Each CTA holds its own 2 x 128 rows
// of A and ONE HALF (128 columns) of the B block in shared memory; the MMAs,
// issued by one thread of the pair's even CTA, feed both SMs' tensor cores,
// which fetch the other half of B from the peer's shared memory.  Per k-block a
// CTA loads 48 KiB for 256 x 256 x 64 multiply-adds (half the bytes per flop of
// the single-CTA 128 x 256 tile).  The two row blocks have separate fp32
// accumulators in TMEM (2 x 256 columns) and their MMAs ALTERNATE (row block 0,
// row block 1, next k-step); eight full-width MMAs per k-block need 1024 clocks
// of the tensor pipe, and the issuing thread keeps up with that (1033-1040 measured).
//
//   warp 0      TMA producer (each CTA loads its own A box and its half of B;
//               every byte is fetched by exactly one CTA, into its own memory).  Both
//               CTAs' loads complete on the EVEN CTA's "full" barrier
//               (cp.async.bulk.tensor ... .cta_group::2 lets the barrier live in
//               the partner), which expects the bytes of both
//   warp 1      even CTA: MMA issuer; idle in the odd CTA
//   warps 2..3  idle: they complete the first warp group, which as a whole hands most of its
//               registers to the epilogue groups (setmaxnreg)
//   warps 4..11 epilogue: four warps per row block drain its accumulator.  A full-width bf16
//               tile reads three of its four 64-column units raw into registers, rounds one to
//               make room for the fourth, releases the accumulator and only then rounds the
//               rest, stages and stores (TMA store or masked stores); other tiles go unit by
//               unit, software-pipelined, and release after the last load
// "Stage free" and "accumulator ready" reach both CTAs through two plain
// tcgen05.commit instructions (own barrier, peer's barrier), never the
// cluster-wide broadcast form.  All waits are bounded; both CTAs pass a cluster barrier
// before exit so that no remote arrive can hit shared memory of a finished CTA.
//
// Preconditions (paper, Introduction: a matrix instruction is valid only for
// tile shapes, layouts and hardware that fit it): A, B TMA-loadable (16-byte aligned
// base and pitch), no K split, not the skinny orientation.  Everything else
// runs on the single-CTA kernel of r4_tcgen05.cu.
#include "common.cuh"
#include "ptx.cuh"
#include <algorithm>
#include <cstring>
#include <new>

#ifdef KLIN_TRACE
static __device__ unsigned long long klin_trace_pair[klin::kTraceSlots * klin::kTraceCtas];
#define KLIN_TRACE_BUF klin_trace_pair
extern "C" int klin_trace_dump_pair(unsigned long long* host)
{
    cudaDeviceSynchronize();
    const cudaError_t e = cudaMemcpyFromSymbol(host, klin_trace_pair, sizeof klin_trace_pair);
    void* dev = nullptr;
    if (cudaGetSymbolAddress(&dev, klin_trace_pair) == cudaSuccess) cudaMemset(dev, 0, sizeof klin_trace_pair);
    return static_cast<int>(e);
}
#endif

namespace klin {
namespace {

constexpr int PM = 128;            // rows per CTA and MMA block; a pair tile has 2 blocks x 2 CTAs x 128 = 512 rows
constexpr int TILE_M = 4 * PM;
constexpr int PN = 256;            // columns of C per pair
constexpr int BK = 64;
constexpr int STAGES = 4;
constexpr int kABlockBytes = PM * BK * 2;      // 16 KiB per row block
constexpr int kABytes = 2 * kABlockBytes;      // 32 KiB
constexpr int kBHalfBytes = (PN / 2) * BK * 2; // 16 KiB
constexpr int kStageBytes = kABytes + kBHalfBytes;
constexpr int kEpiBufBytes = 32 * 128;
constexpr int kEpiBytes = 8 * kEpiBufBytes;       // one staging block per epilogue warp
constexpr int kBarBytes = 1536;                 // barriers, TMEM slot, abort flag, grouped schedule (<= 257 ints)
constexpr int kSmemBytes = 1024 + STAGES * kStageBytes + kEpiBytes + kBarBytes;
constexpr int kTmemCols = 512;
constexpr int kThreads = 12 * 32;                // warp group 0: producer, MMA issuer, two idle warps; groups 1, 2: 2 x 4 epilogue warps
constexpr int kEpiWarp0 = 4;                     // first epilogue warp
// Registers: the kernel is compiled for 168 per thread (three warps share a 16 K-register scheduler
// partition); the first warp group gives its surplus back (setmaxnreg.dec) and the epilogue groups
// take it (setmaxnreg.inc), so that three fp32 units of the accumulator fit in registers at once
// (the compiler allocates each region against its own limit: at 40 / 232 the epilogue spilled).
// The two amounts must balance (the pool the increase draws from holds only what was released:
// with 48 instead of 40 the increase never completed and the launch hung).
constexpr int kRegsLean = 24, kRegsEpilogue = 240;   // balanced: 128 x (168 - 24) released = 256 x (240 - 168) taken

struct PairParams {
    int tiles_m2, tiles_n;      // 512-row x 256-column tiles
    int nkb;
    int epi_tma;
    int kid;
    int group_m;
    int64_t total_tiles;
    // Column tiling of a single problem (MODE 0 / 3): per tile row, n_wide tiles of tile_n columns followed by
    // n_narrow tiles of tile_n2 columns (the last one clipped by N).  Wide tiles come first in the schedule and
    // the pairs walk it back and forth, so that a pair's turns add up to about the same work (see
    // plan_columns): the narrow tiles fill what would otherwise be an under-filled last wave.
    int tile_n, n_wide, tile_n2, n_narrow;
    int64_t wide_tiles;         // tiles_m2 * n_wide
    int snake;                  // 1: odd rounds of the schedule run over the pairs in reverse order
    int one_round;              // 1 (one problem): uniform tiles, at most one per pair - tile t is (t / n_wide, t % n_wide)
    uint32_t stage_tx;          // bytes the loads of both CTAs deliver per stage
    int b_boxes;                // row-major B: 64-column boxes per CTA and stage (1 or 2)
    // Streamed last wave (MODE 0, uniform 256-column tiles).  Tiles [0, sk_first) run whole, sk_rounds of them per
    // pair; the k-blocks of the remaining tiles - one under-filled wave - are laid end to end (sk_work of them) and
    // pair q takes the contiguous range [q * sk_work / pairs, (q + 1) * sk_work / pairs).  A range that starts
    // inside a tile begins with a piece that does not hold the tile's first k-block: the pair computes it FIRST,
    // writes the fp32 partial tile to its slot of the workspace and raises the slot's flags; the piece that holds
    // a tile's first k-block comes after it in its pair's order, reads the partials of the pairs after it (whose
    // first pieces are shorter than this pair's two) in k order, adds them and stores the tile; the whole tiles
    // come last.  No pair ever waits for work that has not been started, sums are added in a fixed order,
    // nothing is atomic.
    int sk;                     // 1: the schedule above
    int sk_rounds;
    int64_t sk_first;
    int64_t sk_work;
    float* sk_slots;            // [pair][128 blocks of 32 rows x 32 columns] fp32, a block laid out [column / 4][row][column % 4]
    unsigned* sk_flags;         // [pair][CTA of the pair][epilogue warp]: the launch's epoch once the warp's rows are written
    unsigned sk_epoch;
    uint32_t idesc;
    uint32_t b_desc_hi, b_desc_lbo, b_kstep;
    // batched launches (MODE 1): the schedule runs over batch x tiles_per_batch
    int tiles_per_batch;
    int64_t stride_c_bytes;
    // grouped launches (MODE 2): table in device memory, one entry per group
    const GroupEntry* groups;
    int n_groups;
    // multi-destination launches (MODE 3): every output block goes to each entry of the table
    const DstEntry* dsts;
    int n_dst;
};

// What a role needs to know about one tile of the schedule.
struct TileInfo {
    int m0, n0;                 // first row of this CTA's first row block / first column of the pair tile
    int width;                  // columns of the tile (the MMA's N): a multiple of 64, at most 256
    int M, N, nkb;              // extent of the problem the tile belongs to
    int z;                      // batch index (third tensor-map coordinate), 0 otherwise
    int epi_tma;
    const CUtensorMap *ma, *mb, *mc;
    uint8_t* C;                 // base of that problem's C
    int64_t ldc;
};

__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_dst, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(ptx::smem_u32(smem_dst)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_f16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                              uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Plain commit of the pair's MMAs onto a barrier given by its shared::cluster
// address (own CTA or the peer).
__device__ __forceinline__ void umma_commit_pair(uint32_t cluster_bar_addr)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(cluster_bar_addr)
                 : "memory");
}
// 2-D tiled load whose completion is counted on a barrier that may live in the
// partner CTA (shared::cluster address); the data lands in this CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t smem_dst, const void* tmap, int x, int y, uint32_t cluster_bar_addr)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.cta_group::2 [%0], [%1, {%2, "
        "%3}], [%4];"
        ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(cluster_bar_addr)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t smem_dst, const void* tmap, int x, int y, int z,
                                                 uint32_t cluster_bar_addr)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.cta_group::2 [%0], [%1, {%2, "
        "%3, %4}], [%5];"
        ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(z),
        "r"(cluster_bar_addr)
        : "memory");
}
template <int N>
__device__ __forceinline__ void setmaxnreg_dec()
{
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N>
__device__ __forceinline__ void setmaxnreg_inc()
{
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar_addr)
{
    // (The arrive only says "my TMEM reads have completed" - tcgen05.wait::ld has made sure of that before - and
    // publishes no memory.  With .release.cluster it took 1.3 k clocks per tile, on the path that keeps the next
    // tile's MMAs waiting; the default form - release at CTA scope - is what this needs.)
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar_addr) : "memory");
}

__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr, uint32_t lbo_field, uint32_t hi)
{
    const uint32_t lo = ((smem_addr >> 4) & 0x3FFFu) | (lbo_field << 16);
    return (static_cast<uint64_t>(hi) << 32) | lo;
}

// MODE 0: one problem (tensor maps 2-D).  MODE 1: batched (3-D tensor maps, z = batch).
// MODE 2: grouped (per-group tensor maps and sizes from a table in device memory).
// MODE 3: one problem whose C goes to several destinations (table of C maps / pointers).
// MODE 6, 7, 8: MODE 0, 1, 2 on 256-row tiles with two k-blocks per stage (see the ring geometry in the kernel).
// MODE 5: MODE 0 with its last wave streamed along K (a separate instantiation, so that the plain kernel does not carry
// the work-list arithmetic in its 24-register producer and MMA threads).
template <bool BCOL, int MODE_>
__global__ void __launch_bounds__(kThreads, 1)
r4_pair_kernel(GemmArgs g, const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_c, PairParams p)
{
    constexpr bool SK = MODE_ == 5;
    constexpr bool KP = MODE_ >= 6;              // 6, 7, 8: modes 0, 1, 2 on k-paired 256-row tiles
    constexpr int MODE = SK ? 0 : KP ? MODE_ - 6 : MODE_;
    // Ring and tile geometry.  The plain forms: 512-row tiles, four stages of one k-block (two row blocks of A and half
    // of B).  KP: 256-row tiles, three stages of TWO k-blocks (A and half of B of either), eight MMAs per stage into
    // ONE accumulator; the two accumulators belong to consecutive tiles of the pair, each drained by its own four
    // epilogue warps while the other fills.
    constexpr int NS = KP ? 3 : STAGES;
    constexpr int SB = KP ? 4 * kABlockBytes : kStageBytes;
    constexpr int TM = KP ? 2 * PM : TILE_M;
    constexpr int KSTAGE = KP ? 2 * BK : BK;     // k per stage
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* epi_smem = smem + STAGES * kStageBytes;     // (= 3 x 64 KiB: the k-paired ring ends at the same place)
    uint64_t* full = reinterpret_cast<uint64_t*>(epi_smem + kEpiBytes);   // even CTA: both CTAs' loads landed
    uint64_t* empty = full + STAGES;                                      // the pair's MMAs are done with the stage
    uint64_t* acc_full = empty + STAGES;                                  // [0]: the tile's accumulators are complete
    uint64_t* acc_empty = acc_full + 2;                                   // [0]: even CTA, both epilogues drained
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    int* gstart = reinterpret_cast<int*>(const_cast<uint32_t*>(abort_flag) + 2);   // MODE 2: first tile of every group
    // streamed schedule: six barriers per epilogue warp for the partial sums it streams through the idle ring (the
    // group table's space is free there)
    uint64_t* fix_bar = reinterpret_cast<uint64_t*>((reinterpret_cast<uintptr_t>(gstart) + 7) & ~uintptr_t(7));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();          // 0 = even CTA (issues the MMAs), 1 = odd CTA
    const int64_t pair_id = blockIdx.x >> 1;
    const int64_t n_pairs = gridDim.x >> 1;

    if (warp == 0 && lane == 0) {
        KLIN_T(0);
#ifdef KLIN_TRACE
        {
            unsigned long long ns;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));
            if (blockIdx.x < kTraceCtas) KLIN_TRACE_BUF[blockIdx.x * kTraceSlots + 5] = ns;
        }
#endif
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(&full[s], 1);
            ptx::mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(&acc_full[b], 1);
            ptx::mbar_init(&acc_empty[b], KP ? 8 : 16);    // the epilogue warps of both CTAs that drain it
        }
        abort_flag[0] = 0;
        abort_flag[1] = 0;
        if (SK)
            for (int i = 0; i < 8 * 6; ++i) ptx::mbar_init(&fix_bar[i], 1);
        ptx::fence_barrier_init();
        KLIN_T(24);
        if (MODE != 2) {
            ptx::prefetch_tensormap(&map_a);
            ptx::prefetch_tensormap(&map_b);
            if (p.epi_tma && MODE != 3) ptx::prefetch_tensormap(&map_c);
        }
        if (blockIdx.x == 0) g.status[1] = p.kid;
    }
    if (MODE == 2 && warp >= kEpiWarp0) {
        for (int i = threadIdx.x - kEpiWarp0 * 32; i <= p.n_groups; i += kThreads - kEpiWarp0 * 32)
            gstart[i] = (i < p.n_groups) ? p.groups[i].tile_start : static_cast<int>(p.total_tiles);
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, kTmemCols);
        tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    if (threadIdx.x == 32) KLIN_T(25);      // TMEM allocated
    __syncthreads();
    if (threadIdx.x == 0) KLIN_T(26);
    // Both CTAs' barriers exist before anyone signals across the pair (their initialisation was published by the
    // mbarrier-init fence above; the arrive itself publishes nothing and need not be a release).
    ptx::cluster_arrive_relaxed();
    ptx::cluster_wait_acquire();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    if (threadIdx.x == 0) KLIN_T(1);

    int group_hint = 0;     // MODE 2: a thread's tiles come in increasing order, so its search resumes here
    auto tile_info = [&](int64_t t) {
        TileInfo x;
        int tm, tn;
        if (MODE == 2) {
            const int ti = static_cast<int>(t);
            int gi = group_hint;
            while (gstart[gi + 1] <= ti) ++gi;              // gstart[n_groups] = total tiles > ti
            group_hint = gi;
            const GroupEntry* e = p.groups + gi;
            x.M = e->M;
            x.N = e->N;
            x.nkb = e->nkb;
            x.z = 0;
            x.epi_tma = e->epi_tma;
            x.ma = &e->map_a;
            x.mb = &e->map_b;
            x.mc = &e->map_c;
            x.C = static_cast<uint8_t*>(e->C);
            x.ldc = e->ldc;
            raster_tile(ti - gstart[gi], e->tiles_m, e->tiles_n, tm, tn, p.group_m);
            x.n0 = tn * PN;
            x.width = PN;
        } else {
            x.M = g.M;
            x.N = g.N;
            x.nkb = p.nkb;
            x.epi_tma = p.epi_tma;
            x.ma = &map_a;
            x.mb = &map_b;
            x.mc = &map_c;
            x.ldc = g.ldc;
            if (MODE == 1) {
                const uint32_t t32 = static_cast<uint32_t>(t), tpb = static_cast<uint32_t>(p.tiles_per_batch);
                const uint32_t b = t32 / tpb;
                x.z = static_cast<int>(b);
                x.C = static_cast<uint8_t*>(g.C) + static_cast<int64_t>(b) * p.stride_c_bytes;
                raster_tile(t32 - b * tpb, p.tiles_m2, p.tiles_n, tm, tn, p.group_m);
                x.n0 = tn * PN;
                x.width = PN;
            } else {
                x.z = 0;
                x.C = static_cast<uint8_t*>(g.C);
                if (p.one_round) {
                    // one round of uniform tiles, at most one per pair: their order does not matter, and the first
                    // decode is on the critical path of a short launch - one 32-bit division, row-major
                    const uint32_t t32 = static_cast<uint32_t>(t), per_row = static_cast<uint32_t>(p.n_wide);
                    tm = static_cast<int>(t32 / per_row);
                    tn = static_cast<int>(t32 - static_cast<uint32_t>(tm) * per_row);
                    x.n0 = tn * p.tile_n;
                    x.width = p.tile_n;
                } else if (t < p.wide_tiles) {
                    raster_tile(t, p.tiles_m2, p.n_wide, tm, tn, p.group_m);
                    x.n0 = tn * p.tile_n;
                    x.width = p.tile_n;
                } else {
                    raster_tile(t - p.wide_tiles, p.tiles_m2, p.n_narrow, tm, tn, p.group_m);
                    x.n0 = p.n_wide * p.tile_n + tn * p.tile_n2;
                    x.width = p.tile_n2;
                }
                // a tile clipped by the matrix edge runs a narrower MMA
                x.width = min(x.width, (g.N - x.n0 + 63) & ~63);
            }
        }
        x.m0 = tm * TM + static_cast<int>(rank) * PM;   // this CTA's rows: m0 + [0,128) and (512-row tiles) m0 + 256 + [0,128)
        return x;
    };
    // The r-th tile of this pair (-1: the schedule has ended).  Odd rounds run over the pairs in reverse
    // when the schedule mixes tile widths: a pair that took an early (wide) tile takes a late (narrow) one next.
    auto tile_at = [&](uint32_t r) -> int64_t {
        const int64_t idx = static_cast<int64_t>(r) * n_pairs + ((p.snake && (r & 1u)) ? n_pairs - 1 - pair_id : pair_id);
        return idx < p.total_tiles ? idx : -1;
    };
    // One item of this pair's work list: a tile and the k-blocks [kb0, kb1) of it.  kind 0: the whole tile;
    // 1: a piece without the tile's first k-block - its partial sums go to this pair's workspace slot;
    // 2: a piece with the first but not the last k-block - it adds the partial sums of the pairs after it.
    struct Work {
        int64_t tile;
        int kb0, kb1, kind;
    };
    struct WorkState {
        uint32_t i;             // whole-tile rounds handed out so far
        int64_t pos, end;       // streamed range still to hand out (k-blocks of the streamed region)
        bool first_done;
    };
    auto work_init = [&]() {
        WorkState st = {0u, 0, 0, false};
        if (SK) {
            st.pos = pair_id * p.sk_work / n_pairs;
            st.end = (pair_id + 1) * p.sk_work / n_pairs;
        }
        return st;
    };
    auto next_work = [&](WorkState& st, Work& w) -> bool {
        if (!SK) {
            const int64_t t = tile_at(st.i++);
            if (t < 0) return false;
            w.tile = t;
            w.kb0 = 0;
            w.kb1 = -1;         // the tile's own k-block count
            w.kind = 0;
            return true;
        }
        const int nkb = p.nkb;
        if (!st.first_done) {   // first: the piece that starts inside a tile
            st.first_done = true;
            const int off = static_cast<int>(st.pos % nkb);
            if (off != 0 && st.pos < st.end) {
                w.tile = p.sk_first + st.pos / nkb;
                w.kb0 = off;
                w.kb1 = static_cast<int>(min(static_cast<int64_t>(nkb), off + (st.end - st.pos)));
                w.kind = 1;
                st.pos += w.kb1 - w.kb0;
                return true;
            }
        }
        if (st.pos < st.end) {  // then the rest of the range, tile by tile (it starts at a tile's first k-block)
            w.tile = p.sk_first + st.pos / nkb;
            w.kb0 = 0;
            w.kb1 = static_cast<int>(min(static_cast<int64_t>(nkb), st.end - st.pos));
            w.kind = w.kb1 == nkb ? 0 : 2;
            st.pos += w.kb1;
            return true;
        }
        if (st.i < static_cast<uint32_t>(p.sk_rounds)) {       // last the whole tiles of the full rounds: the adding of
            w.tile = static_cast<int64_t>(st.i++) * n_pairs + pair_id;   // partial sums above hides behind their MMAs
            w.kb0 = 0;
            w.kb1 = nkb;
            w.kind = 0;
            return true;
        }
        return false;
    };
    // One operand box of a stage; completion is counted on the even CTA's barrier.
    auto load_box = [&](uint32_t dst, const CUtensorMap* map, int c0, int c1, int z, uint32_t bar) {
        if (MODE == 1)
            tma_load_3d_pair(dst, map, c0, c1, z, bar);
        else
            tma_load_2d_pair(dst, map, c0, c1, bar);
    };

    if (warp < kEpiWarp0) {
    // One instruction for the whole first warp group (the register release is warp-group wide), ahead of
    // the producer and MMA code, which run within the reduced budget.
    setmaxnreg_dec<kRegsLean>();
    if (threadIdx.x == 0) KLIN_T(27);
    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        // (One thread issues all of a stage's loads.  Measured: three threads - one per operand block, each
        // waiting for "stage free" on its own - made the main loop 4 % SLOWER, 1120 against 1077 clocks per
        // k-block: the loop is not waiting for the producer.  A k-block moves 48 KiB into shared memory and its
        // eight MMAs read 64 KiB from it, 112 of the 128 bytes per clock a CTA's shared memory delivers.)
        if (lane == 0) {
            // The ring position (stage s, parity ph of its "empty" barrier) is carried, barriers and stages are
            // addressed by their shared-window addresses, and everything a stage's loads need is in registers
            // before the wait: what follows the wait is the expect-tx arrive and the loads themselves.  (The time
            // from "stage free" to "loads issued" is part of every stage's round trip: four stages of 1024 MMA
            // clocks hide about 4 k clocks of it, and a load takes about 3 k to land.)
            uint32_t it = 0, s = 0, ph = 1;
            bool ok = true;
            const uint32_t smem0 = ptx::smem_u32(smem), empty0 = ptx::smem_u32(empty), full0 = ptx::smem_u32(full);
            const uint32_t full_even0 = ptx::map_to_cta(full0, 0);   // the even CTA's barriers (consecutive words)
            const uint32_t stage_tx = p.stage_tx;
            const bool two_boxes = !BCOL && p.b_boxes > 1;
            WorkState ws = work_init();
            Work wk;
            while (ok && next_work(ws, wk)) {
                const TileInfo x = tile_info(wk.tile);
                const int m0 = x.m0, z = x.z;
                const CUtensorMap *ma = x.ma, *mb = x.mb;
                const int nb = x.n0 + static_cast<int>(rank) * (x.width >> 1);    // this CTA's half of B
                const int kb_end = wk.kb1 < 0 ? x.nkb : wk.kb1;
                if (it == 0) KLIN_T(28);
                for (int kb = wk.kb0; kb < kb_end; ++kb, ++it) {
                    const uint32_t sa = smem0 + s * SB, sb = sa + kABytes;
                    const uint32_t bar = full_even0 + 8 * s;
                    const int kx = kb * KSTAGE;
                    if (!ptx::mbar_wait_addr(empty0 + 8 * s, ph, abort_flag)) {
                        report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x500u | s);
                        abort_flag[0] = 1;
                        ok = false;
                        break;
                    }
                    // The even CTA's barrier counts the bytes of both CTAs' loads of this stage.
                    if (rank == 0) ptx::mbar_arrive_expect_tx_addr(full0 + 8 * s, stage_tx);
                    load_box(sa, ma, kx, m0, z, bar);
                    if (KP) {
                        // the stage's second k-block (past the end of K the boxes read zeros and its MMAs add nothing)
                        load_box(sa + kABlockBytes, ma, kx + BK, m0, z, bar);
                        if (BCOL) {
                            load_box(sb, mb, kx, nb, z, bar);
                            load_box(sb + kBHalfBytes, mb, kx + BK, nb, z, bar);
                        } else {
                            load_box(sb, mb, nb, kx, z, bar);
                            if (two_boxes) load_box(sb + 64 * BK * 2, mb, nb + 64, kx, z, bar);
                            load_box(sb + kBHalfBytes, mb, nb, kx + BK, z, bar);
                            if (two_boxes) load_box(sb + kBHalfBytes + 64 * BK * 2, mb, nb + 64, kx + BK, z, bar);
                        }
                    } else {
                    load_box(sa + kABlockBytes, ma, kx, m0 + 2 * PM, z, bar);
                    if (BCOL) {
                        load_box(sb, mb, kx, nb, z, bar);
                    } else {
                        load_box(sb, mb, nb, kx, z, bar);
                        if (two_boxes) load_box(sb + 64 * BK * 2, mb, nb + 64, kx, z, bar);
                    }
                    }
                    if (it == 0) KLIN_T(2);
                    if (it == NS - 1) KLIN_T(3);
                    if (++s == NS) {
                        s = 0;
                        ph ^= 1u;
                    }
                }
            }
            // Drain: in the even CTA wait for the last fills; the odd CTA's loads are covered by
            // the same barriers (the MMAs that consumed them have completed before the epilogue ends).
            if (rank == 0) {
                const uint32_t first = it > NS ? it - NS : 0;
                for (uint32_t j = first; j < it; ++j)
                    ptx::mbar_wait(&full[j % NS], (j / NS) & 1, abort_flag + 1);
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // -------------------------------------------------------- MMA issuer (even CTA)
            // Ring position carried, barriers by shared-window address, a stage's descriptors = the first stage's
            // plus s * (stage bytes >> 4) in the 14-bit start-address field (the ring ends below 256 KiB).  The next
            // tile's coordinates are worked out BEFORE the wait for the drained accumulators, not after it.
            uint32_t tcount = 0, s = 0, ph = 0;
            bool ok = true;
            const uint32_t full0 = ptx::smem_u32(full), empty0 = ptx::smem_u32(empty);
            const uint32_t empty_odd0 = ptx::map_to_cta(empty0, 1);
            const uint32_t accf = ptx::smem_u32(&acc_full[0]), accf_odd = ptx::map_to_cta(accf, 1);
            // descriptors: the high words never change, the low words step by 16-byte units (no carry out of the
            // 14-bit address field inside the ring)
            const uint64_t a_desc0 = make_desc(ptx::smem_u32(smem), 1, (1024u >> 4) | (1u << 14) | (2u << 29));
            const uint64_t b_desc0 = make_desc(ptx::smem_u32(smem) + kABytes, p.b_desc_lbo, p.b_desc_hi);
            const uint32_t a_lo0 = static_cast<uint32_t>(a_desc0), a_hi = static_cast<uint32_t>(a_desc0 >> 32);
            const uint32_t b_lo0 = static_cast<uint32_t>(b_desc0), b_hi = static_cast<uint32_t>(b_desc0 >> 32);
            const uint32_t kstep = p.b_kstep;
            auto desc = [](uint32_t hi, uint32_t lo) { return (static_cast<uint64_t>(hi) << 32) | lo; };
            WorkState ws = work_init();
            Work wk;
            for (; ok && next_work(ws, wk); ++tcount) {
                const TileInfo x = tile_info(wk.tile);
                const int kb_first = wk.kb0, kb_end = wk.kb1 < 0 ? x.nkb : wk.kb1;
                // the MMA's N is the tile's width
                const uint32_t idesc = (p.idesc & ~(0x3Fu << 17)) | (static_cast<uint32_t>(x.width >> 3) << 17);
                // A tile whose second row block lies wholly past the matrix (at most 256 live rows) issues the first
                // block's MMAs only: this thread's instruction stream bounds the loop, so such a tile takes about
                // half the time (its second accumulator is never read: the epilogue warps of that block have no rows).
                const bool two_blocks = x.M - x.m0 > 2 * PM;
                // Both accumulators are rewritten: wait until both CTAs' epilogues drained the last tile.  (KP: the
                // accumulator of this tile's parity, drained of the tile before the last.)
                const uint32_t buf = KP ? (tcount & 1u) : 0u;
                if (!ptx::mbar_wait(&acc_empty[buf], ((KP ? tcount >> 1 : tcount) & 1) ^ 1, abort_flag)) {
                    report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x520u);
                    abort_flag[0] = 1;
                    break;
                }
                ptx::tc_fence_after_sync();
                KLIN_T(tcount < 4 ? 8 + 4 * static_cast<int>(tcount) : -1);
                for (int kb = kb_first; kb < kb_end; ++kb) {
                    if (!ptx::mbar_wait_addr(full0 + 8 * s, ph, abort_flag)) {
                        report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x530u | s);
                        abort_flag[0] = 1;
                        ok = false;
                        break;
                    }
                    // (no tcgen05 fence: the operands came through the async proxy, which is how the MMA reads them.)
                    // This thread's instruction stream bounds the main loop - eight MMAs at ~85 clocks of issue each
                    // plus what surrounds them, against the 1024 clocks the tensor pipe needs - so nothing is derived
                    // here that can be carried.  (A look-ahead probe of the next stage's barrier changed nothing.)
                    const uint32_t s_next = (s + 1 == NS) ? 0u : s + 1, ph_next = (s + 1 == NS) ? ph ^ 1u : ph;
                    if (kb == kb_first) KLIN_T(tcount < 4 ? 9 + 4 * static_cast<int>(tcount) : -1);
                    if (kb == kb_end - 1) KLIN_T(tcount < 4 ? 10 + 4 * static_cast<int>(tcount) : -1);
                    const uint32_t a_lo = a_lo0 + s * static_cast<uint32_t>(SB >> 4);
                    const uint32_t b_lo = b_lo0 + s * static_cast<uint32_t>(SB >> 4);
                    if (KP) {
                        const uint32_t d = tmem_base + buf * PN;
#pragma unroll
                        for (int k8 = 0; k8 < 2 * (BK / 16); ++k8) {
                            const uint32_t sub = static_cast<uint32_t>(k8 >> 2), k4 = static_cast<uint32_t>(k8 & 3);
                            umma_f16_pair(d, desc(a_hi, a_lo + sub * (kABlockBytes >> 4) + k4 * 2u),
                                          desc(b_hi, b_lo + sub * (kBHalfBytes >> 4) + k4 * kstep), idesc,
                                          (kb > kb_first || k8 > 0) ? 1u : 0u);
                        }
                    } else {
#pragma unroll
                        for (int k4 = 0; k4 < BK / 16; ++k4) {
                            const uint32_t acc = (kb > kb_first || k4 > 0) ? 1u : 0u;
                            // alternate the two row blocks: consecutive MMAs never share an accumulator
                            const uint64_t bd = desc(b_hi, b_lo + static_cast<uint32_t>(k4) * kstep);
                            umma_f16_pair(tmem_base, desc(a_hi, a_lo + static_cast<uint32_t>(k4 * 2)), bd, idesc, acc);
                            if (two_blocks)
                                umma_f16_pair(tmem_base + PN,
                                              desc(a_hi, a_lo + static_cast<uint32_t>((kABlockBytes >> 4) + k4 * 2)), bd, idesc, acc);
                        }
                    }
                    umma_commit_pair(empty0 + 8 * s);
                    umma_commit_pair(empty_odd0 + 8 * s);
                    s = s_next;
                    ph = ph_next;
                }
                if (ok) {
                    umma_commit_pair(accf + 8 * buf);
                    umma_commit_pair(accf_odd + 8 * buf);
                    KLIN_T(tcount < 4 ? 11 + 4 * static_cast<int>(tcount) : -1);
                }
            }
        }
    }
    } else {
        // ------------------------------------------------------------ epilogue
        setmaxnreg_inc<kRegsEpilogue>();
        // Warps 4..7 drain the first row block's accumulator, warps 8..11 the second; a warp
        // reads the TMEM lane quarter (warp & 3).  TMEM loads of the next 128-byte unit are in
        // flight while the current one is converted, staged and stored, and the accumulator is
        // handed back as soon as its last load has landed.
        const int q = warp & 3;
        const int mb = (warp - kEpiWarp0) >> 2;
        uint8_t* b = epi_smem + (warp - kEpiWarp0) * kEpiBufBytes;
        const bool out_bf16 = g.c_bf16 != 0;
        const int cpc = out_bf16 ? 64 : 32;                   // columns per 128-byte staging row
        uint32_t tcount = 0;
        bool ok = true;
        WorkState ws = work_init();
        Work wk;
        for (; ok && next_work(ws, wk); ++tcount) {
            // KP: a tile belongs to the warp group of its parity - except the pair's LAST tile, which both groups drain,
            // the owner the first half of its 128-byte units and the other group (idle by then) the second half.
            const int ab = KP ? static_cast<int>(tcount & 1u) : mb;           // the accumulator (KP) / row block read here
            const bool helper = KP && ab != mb;
            if (helper && tile_at(ws.i) >= 0) continue;
            const TileInfo x = tile_info(wk.tile);
            const int m0 = x.m0, n0 = x.n0;
            float* dst_f = reinterpret_cast<float*>(x.C);
            uint16_t* dst_h = reinterpret_cast<uint16_t*>(x.C);
            const int row0 = m0 + (KP ? 0 : mb * 2 * PM) + q * 32;
            const int rows = min(32, x.M - row0);
            const int nunits = (row0 < x.M) ? (min(x.width, x.N - n0) + cpc - 1) / cpc : 0;
            const uint32_t tbase = tmem_base + ab * PN + (static_cast<uint32_t>(q * 32) << 16);
            const bool shared = KP && nunits >= 2 && tile_at(ws.i) < 0;       // both warp groups drain this tile
            if (helper && !shared) continue;
            const int u_lo = (shared && helper) ? nunits / 2 : 0, u_hi = (shared && !helper) ? nunits / 2 : nunits;
            // first 4 KiB block of this warp's rows inside a partial-tile slot: (CTA, row block, lane quarter) x 8 column blocks
            const int64_t sk_block = ((static_cast<int64_t>(rank) * 2 + mb) * 4 + q) * (PN / 32);

            // A piece with the tile's first but not its last k-block: the pairs after this one hold the rest of the
            // tile's K range, each as one partial tile in its slot, in k order.  They computed those pieces first of
            // all, so the flags are up long before this piece's own MMAs end: the (bounded) wait for them happens
            // here, ahead of the wait for the accumulator.
            int n_part = 0;
            if (SK && wk.kind == 2) {
                const int64_t rel = wk.tile - p.sk_first;
                for (int64_t j = pair_id + 1; j < n_pairs; ++j) {
                    const int64_t sj = j * p.sk_work / n_pairs;
                    if (sj % p.nkb == 0 || sj / p.nkb != rel) break;
                    ++n_part;
                }
                bool seen = true;
                if (lane == 0) {
                    for (int j = 1; j <= n_part && seen; ++j) {
                        const volatile unsigned* f = p.sk_flags + ((pair_id + j) * 2 + rank) * 8 + (warp - kEpiWarp0);
                        seen = false;
                        for (uint32_t i = 0; i < ptx::kMbarPollLimit; ++i) {
                            if (*f == p.sk_epoch) {
                                seen = true;
                                break;
                            }
                            if ((i & 1023u) == 1023u && abort_flag[0]) break;
                        }
                    }
                    if (!seen) {
                        report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x560u);
                        abort_flag[0] = 1;
                    }
                }
                seen = __shfl_sync(0xFFFFFFFFu, seen ? 1 : 0, 0) != 0;
                __threadfence();
                if (!seen) {       // give up: nothing is stored; the raised flag ends the other roles' waits
                    ok = false;
                    break;
                }
            }
            // AddMM: this lane's bias values of the tile's eight 32-column blocks, fetched while the MMAs still run (inside
            // the drain their ~600-clock loads stood in the way of every unit: 4096^3 with bias 97.2 us against 95.0 without)
            float pb[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) pb[k] = (g.bias && n0 + 32 * k + lane < x.N) ? bias_at(g, n0 + 32 * k + lane) : 0.f;
            if (!ptx::mbar_wait(&acc_full[KP ? ab : 0], (KP ? tcount >> 1 : tcount) & 1, abort_flag)) {
                if (lane == 0) report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x540u);
                abort_flag[0] = 1;
                ok = false;
                break;
            }
            ptx::tc_fence_after_sync();
            if (warp == kEpiWarp0 && lane == 0) KLIN_T(tcount < 8 ? 40 + 3 * static_cast<int>(tcount) : -1);

            auto release = [&]() {
                ptx::tc_fence_before_sync();
                if (tcount == 0 && warp == kEpiWarp0 && lane == 0) KLIN_T(60);
                __syncwarp();
                if (tcount == 0 && warp == kEpiWarp0 && lane == 0) KLIN_T(61);
                // (a shared tile is the pair's last: nobody waits for its accumulator)
                if (lane == 0 && !shared) mbar_arrive_cluster(ptx::map_to_cta(ptx::smem_u32(&acc_empty[KP ? ab : 0]), 0));
            };
            auto issue = [&](int u, uint32_t (&r0)[32], uint32_t (&r1)[32]) {
                ptx::tmem_ld_32x32b_x32(tbase + u * cpc, r0);
                if (out_bf16) ptx::tmem_ld_32x32b_x32(tbase + u * cpc + 32, r1);
            };
            // pack: bias and rounding of one unit (r0, r1 -> 32 words of output); stage_store: the words
            // go through the warp's staging block to global memory
            // (`pre`: u is a literal at the call site - the prefetched values are picked at compile time; the general
            // loops, whose u is a variable, fetch the unit's bias here)
            auto pack = [&](int u, uint32_t (&r0)[32], uint32_t (&r1)[32], uint32_t (&w)[32], bool pre = false) {
                const int col0 = n0 + u * cpc;
                if (g.bias) {   // AddMM: this unit's columns get their bias in fp32, before any rounding
                    // lane l holds the bias of columns col0 + l and col0 + 32 + l; a shuffle hands column i's
                    // value to every lane (every lane holds a different row of the same columns)
                    float b0, b1;
                    if (pre) {
                        b0 = out_bf16 ? pb[(2 * u) & 7] : pb[u & 7];
                        b1 = out_bf16 ? pb[(2 * u + 1) & 7] : 0.f;
                    } else {
                        b0 = (col0 + lane < x.N) ? bias_at(g, col0 + lane) : 0.f;
                        b1 = (out_bf16 && col0 + 32 + lane < x.N) ? bias_at(g, col0 + 32 + lane) : 0.f;
                    }
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        r0[i] = __float_as_uint(__uint_as_float(r0[i]) + __shfl_sync(0xFFFFFFFFu, b0, i));
                        if (out_bf16) r1[i] = __float_as_uint(__uint_as_float(r1[i]) + __shfl_sync(0xFFFFFFFFu, b1, i));
                    }
                }
                if (out_bf16) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        w[i] = pack_bf16x2(__uint_as_float(r0[2 * i]), __uint_as_float(r0[2 * i + 1]));
                        w[16 + i] = pack_bf16x2(__uint_as_float(r1[2 * i]), __uint_as_float(r1[2 * i + 1]));
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) w[i] = r0[i];
                }
            };
            auto stage_store = [&](int u, const uint32_t (&w)[32]) {
                const int col0 = n0 + u * cpc;
                // (a warp's staging buffer may still be read by its previous TMA store, possibly of
                // another group's tile: wait whenever any tile of the launch can take that path)
                if (p.epi_tma) {
                    if (lane == 0) ptx::tma_store_wait_read<0>();   // the previous store has read the buffer
                    __syncwarp();
                }
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    *reinterpret_cast<uint4*>(b + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                        make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
                if (x.epi_tma) {
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        if (MODE == 1) {
                            ptx::tma_store_3d(x.mc, col0, row0, x.z, b);
                        } else if (MODE == 3) {
                            for (int d = 0; d < p.n_dst; ++d) ptx::tma_store_2d(&p.dsts[d].map_c, col0, row0, b);
                        } else {
                            ptx::tma_store_2d(x.mc, col0, row0, b);
                        }
                        ptx::tma_store_commit();
                    }
                } else {
                    __syncwarp();
                    for (int d = 0; d < (MODE == 3 ? p.n_dst : 1); ++d) {
                    if (MODE == 3) {
                        dst_f = static_cast<float*>(p.dsts[d].C);
                        dst_h = static_cast<uint16_t*>(p.dsts[d].C);
                    }
                    const int64_t ldd = (MODE == 3) ? p.dsts[d].ldc : x.ldc;
                    for (int rr = 0; rr < rows; ++rr) {
                        const uint32_t word = *reinterpret_cast<const uint32_t*>(
                            b + rr * 128 + (((lane >> 2) ^ (rr & 7)) << 4) + (lane & 3) * 4);
                        const int64_t row = row0 + rr;
                        if (out_bf16) {
                            const int col = col0 + 2 * lane;
                            uint16_t* o = dst_h + row * ldd + col;
                            if (col + 1 < x.N && (reinterpret_cast<uintptr_t>(o) & 3) == 0) {
                                *reinterpret_cast<uint32_t*>(o) = word;
                            } else {
                                if (col < x.N) o[0] = static_cast<uint16_t>(word & 0xFFFFu);
                                if (col + 1 < x.N) o[1] = static_cast<uint16_t>(word >> 16);
                            }
                        } else {
                            const int col = col0 + lane;
                            if (col < x.N) dst_f[row * ldd + col] = __uint_as_float(word);
                        }
                    }
                    }
                    __syncwarp();
                }
            };
            if (SK && wk.kind == 1) {
                // A piece without the tile's first k-block: this warp's 32 rows of the raw fp32 partial tile go to the
                // pair's workspace slot, as 4 KiB blocks of 32 rows x 32 columns laid out [column / 4][row][column % 4]
                // (a warp's store instruction writes 512 contiguous bytes); then the accumulator is handed back and
                // the warp's flag tells the owner its rows are there.
                uint4* dst = reinterpret_cast<uint4*>(p.sk_slots + pair_id * (TILE_M * PN) + sk_block * 1024) + lane;
                uint32_t v0[32], v1[32];
#pragma unroll 1
                for (int c = 0; c < PN / 32; c += 2) {
                    ptx::tmem_ld_32x32b_x32(tbase + c * 32, v0);
                    ptx::tmem_ld_32x32b_x32(tbase + c * 32 + 32, v1);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        __stcg(dst + c * 256 + j * 32, make_uint4(v0[4 * j], v0[4 * j + 1], v0[4 * j + 2], v0[4 * j + 3]));
                        __stcg(dst + (c + 1) * 256 + j * 32, make_uint4(v1[4 * j], v1[4 * j + 1], v1[4 * j + 2], v1[4 * j + 3]));
                    }
                }
                release();
                __threadfence();
                __syncwarp();
                if (lane == 0)
                    *reinterpret_cast<volatile unsigned*>(p.sk_flags + (pair_id * 2 + rank) * 8 + (warp - kEpiWarp0)) = p.sk_epoch;
                continue;
            }
            if (nunits == 0) {
                release();
                continue;
            }
            uint32_t a0[32], a1[32], c0[32], c1[32];
            // adds the partial sums of unit u (this lane's row, the unit's columns) to r0 / r1, slot by slot = in k order;
            // all of a slot's loads for the unit (eight, or sixteen for a 2-byte C) are in flight together
            auto add_partials = [&](int u, uint32_t (&r0)[32], uint32_t (&r1)[32]) {
#pragma unroll 1
                for (int j = 1; j <= n_part; ++j) {
                    // unit u = 32-column blocks u * (cpc / 32) and, for a 2-byte C, the next one
                    const float4* src = reinterpret_cast<const float4*>(p.sk_slots + (pair_id + j) * (TILE_M * PN) + sk_block * 1024) +
                                        u * (cpc / 32) * 256 + lane;
                    float4 t[8], t2[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) t[i] = __ldcg(src + i * 32);
                    // (unconditional: values defined on one side of a branch only cost the register allocator
                    // dearly here - 1.4 KB of spills; a 4-byte C re-reads its block and ignores the copy)
#pragma unroll
                    for (int i = 0; i < 8; ++i) t2[i] = __ldcg(src + (out_bf16 ? 256 : 0) + i * 32);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        r0[4 * i] = __float_as_uint(__uint_as_float(r0[4 * i]) + t[i].x);
                        r0[4 * i + 1] = __float_as_uint(__uint_as_float(r0[4 * i + 1]) + t[i].y);
                        r0[4 * i + 2] = __float_as_uint(__uint_as_float(r0[4 * i + 2]) + t[i].z);
                        r0[4 * i + 3] = __float_as_uint(__uint_as_float(r0[4 * i + 3]) + t[i].w);
                    }
                    if (out_bf16) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            r1[4 * i] = __float_as_uint(__uint_as_float(r1[4 * i]) + t2[i].x);
                            r1[4 * i + 1] = __float_as_uint(__uint_as_float(r1[4 * i + 1]) + t2[i].y);
                            r1[4 * i + 2] = __float_as_uint(__uint_as_float(r1[4 * i + 2]) + t2[i].z);
                            r1[4 * i + 3] = __float_as_uint(__uint_as_float(r1[4 * i + 3]) + t2[i].w);
                        }
                    }
                }
            };
            if (SK && n_part > 0 && p.sk_rounds == 0) {
                // The owner's piece is the pair's LAST work here (no whole tiles follow), its MMAs have completed and
                // no load is in flight or to come: the operand ring is idle.  The partial sums stream through it -
                // 4 KiB blocks by bulk copies, six in flight per warp on barriers of their own, in the order they are
                // added (unit, half, slot) - instead of through registers, where one slot's sixteen loads per lane at
                // a time left this epilogue, which nothing hides, at 25-28 k clocks.
                const int wi = warp - kEpiWarp0;
                const uint32_t buf0 = ptx::smem_u32(smem) + static_cast<uint32_t>(wi) * (6u * 4096u);
                const uint32_t bar0 = ptx::smem_u32(fix_bar + wi * 6);
                const int per_unit = (cpc / 32) * n_part;          // items of a unit: (half, slot), slots in k order
                const int total = nunits * per_unit;
                auto issue_item = [&](int i) {
                    if (lane == 0) {
                        const int blk = i / n_part, j = 1 + i % n_part;
                        const float* src = p.sk_slots + (pair_id + j) * (TILE_M * PN) + (sk_block + blk) * 1024;
                        const uint32_t slot = static_cast<uint32_t>(i % 6);
                        ptx::fence_proxy_async_smem();             // the buffer's last readers were generic loads
                        ptx::mbar_arrive_expect_tx_addr(bar0 + 8 * slot, 4096u);
                        ptx::bulk_load_1d(buf0 + slot * 4096u, src, 4096u, bar0 + 8 * slot);
                    }
                };
                for (int i = 0; i < total && i < 6; ++i) issue_item(i);
                bool fine = true;
#pragma unroll 1
                for (int u = 0; u < nunits && fine; ++u) {
                    issue(u, a0, a1);
                    ptx::tmem_ld_wait();
                    if (u == nunits - 1) release();
#pragma unroll 1
                    for (int k = 0; k < per_unit; ++k) {
                        const int i = u * per_unit + k;
                        const uint32_t slot = static_cast<uint32_t>(i % 6);
                        if (!ptx::mbar_wait_addr(bar0 + 8 * slot, static_cast<uint32_t>(i / 6) & 1u, abort_flag)) {
                            if (lane == 0) report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x570u | slot);
                            abort_flag[0] = 1;
                            fine = false;
                            break;
                        }
                        const float4* sp = reinterpret_cast<const float4*>(smem + wi * (6 * 4096) + slot * 4096) + lane;
                        float4 t[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) t[e] = sp[e * 32];
                        if (k >= n_part) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                a1[4 * e] = __float_as_uint(__uint_as_float(a1[4 * e]) + t[e].x);
                                a1[4 * e + 1] = __float_as_uint(__uint_as_float(a1[4 * e + 1]) + t[e].y);
                                a1[4 * e + 2] = __float_as_uint(__uint_as_float(a1[4 * e + 2]) + t[e].z);
                                a1[4 * e + 3] = __float_as_uint(__uint_as_float(a1[4 * e + 3]) + t[e].w);
                            }
                        } else {
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                a0[4 * e] = __float_as_uint(__uint_as_float(a0[4 * e]) + t[e].x);
                                a0[4 * e + 1] = __float_as_uint(__uint_as_float(a0[4 * e + 1]) + t[e].y);
                                a0[4 * e + 2] = __float_as_uint(__uint_as_float(a0[4 * e + 2]) + t[e].z);
                                a0[4 * e + 3] = __float_as_uint(__uint_as_float(a0[4 * e + 3]) + t[e].w);
                            }
                        }
                        __syncwarp();
                        if (i + 6 < total) issue_item(i + 6);
                    }
                    if (!fine) {
                        if (u != nunits - 1) release();
                        break;
                    }
                    pack(u, a0, a1, c0);
                    stage_store(u, c0);
                }
                if (!fine) {
                    ok = false;
                    break;
                }
                continue;
            }
            if (SK && n_part > 0) {
                // The owner of a streamed tile when whole tiles follow (its epilogue then hides behind their MMAs, and
                // the ring is theirs), unit by unit: the accumulator's values plus the partial sums of the
                // later k ranges.  (One unit of the accumulator in registers at a time: the registers go to the
                // sixteen loads per lane that are in flight for every slot.)
#pragma unroll 1
                for (int u = 0; u < nunits; ++u) {
                    issue(u, a0, a1);
                    ptx::tmem_ld_wait();
                    if (u == nunits - 1) release();
                    if (warp == kEpiWarp0 && lane == 0) KLIN_T(48 + 3 * u);
                    add_partials(u, a0, a1);
                    if (warp == kEpiWarp0 && lane == 0) KLIN_T(49 + 3 * u);
                    pack(u, a0, a1, c0);
                    stage_store(u, c0);
                    if (warp == kEpiWarp0 && lane == 0) KLIN_T(50 + 3 * u);
                }
                continue;
            }
            if (out_bf16 && nunits == 4 && n_part == 0 && !shared) {
                // Full-width bf16 tile: the accumulator is handed back before anything is staged or stored.
                // Rounding (F2F, 16 results per clock and SM) is what the drain costs: three units are read
                // raw (192 registers), one is rounded to make room for the fourth, the accumulator is
                // released, and the other roundings, staging and the TMA stores run while the next tile's
                // MMAs already fill it again.
                uint32_t d0[32], d1[32], w0[32];
                issue(0, a0, a1);
                ptx::tmem_ld_wait();
                if (tcount == 0 && warp == kEpiWarp0 && lane == 0) KLIN_T(56);
                issue(1, c0, c1);
                issue(2, d0, d1);
                if (tcount == 0 && warp == kEpiWarp0 && lane == 0) KLIN_T(57);
                pack(0, a0, a1, w0, true);     // (while units 1 and 2 are on their way) frees a0, a1 for the fourth unit
                if (tcount == 0 && warp == kEpiWarp0 && lane == 0) KLIN_T(58);
                issue(3, a0, a1);
                ptx::tmem_ld_wait();
                if (tcount == 0 && warp == kEpiWarp0 && lane == 0) KLIN_T(59);
                release();
                if (warp == kEpiWarp0 && lane == 0) KLIN_T(tcount < 8 ? 41 + 3 * static_cast<int>(tcount) : -1);
                stage_store(0, w0);
                pack(1, c0, c1, w0, true);
                stage_store(1, w0);
                pack(2, d0, d1, w0, true);
                stage_store(2, w0);
                pack(3, a0, a1, w0, true);
                stage_store(3, w0);
                if (warp == kEpiWarp0 && lane == 0) KLIN_T(tcount < 8 ? 42 + 3 * static_cast<int>(tcount) : -1);
                continue;
            }
            if (!out_bf16 && nunits == 8 && n_part == 0 && !shared) {
                // Full-width fp32 tile (eight 32-column units, nothing to round): six units are read raw, two
                // are staged and stored to make room for the last two, then the accumulator is released.
                uint32_t d0[32], d1[32];
                issue(0, a0, a1);
                issue(1, a1, a0);          // (a unit is one 32-column load here: the second array is unused)
                issue(2, c0, c1);
                issue(3, c1, c0);
                issue(4, d0, d1);
                issue(5, d1, d0);
                ptx::tmem_ld_wait();
                if (g.bias) pack(0, a0, a0, a0, true);
                stage_store(0, a0);
                issue(6, a0, a0);
                if (g.bias) pack(1, a1, a1, a1, true);
                stage_store(1, a1);
                issue(7, a1, a1);
                ptx::tmem_ld_wait();
                release();
                if (g.bias) pack(2, c0, c0, c0, true);
                stage_store(2, c0);
                if (g.bias) pack(3, c1, c1, c1, true);
                stage_store(3, c1);
                if (g.bias) pack(4, d0, d0, d0, true);
                stage_store(4, d0);
                if (g.bias) pack(5, d1, d1, d1, true);
                stage_store(5, d1);
                if (g.bias) pack(6, a0, a0, a0, true);
                stage_store(6, a0);
                if (g.bias) pack(7, a1, a1, a1, true);
                stage_store(7, a1);
                continue;
            }
            if (u_lo < u_hi) issue(u_lo, a0, a1);
            for (int u = u_lo; u < u_hi; u += 2) {
                ptx::tmem_ld_wait();
                if (u + 1 < u_hi) issue(u + 1, c0, c1); else release();
                {
                    uint32_t w[32];
                    pack(u, a0, a1, w);
                    stage_store(u, w);
                }
                if (u + 1 < u_hi) {
                    ptx::tmem_ld_wait();
                    if (u + 2 < u_hi) issue(u + 2, a0, a1); else release();
                    uint32_t w[32];
                    pack(u + 1, c0, c1, w);
                    stage_store(u + 1, w);
                }
            }
        }
        // shared memory may go once the stores have read it; their writes complete with the grid
        if (p.epi_tma && lane == 0) ptx::tma_store_wait_read<0>();
    }

    // No CTA leaves while its partner may still signal into its shared memory.
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_arrive_relaxed();      // (an execution barrier only: no memory is handed over here)
    ptx::cluster_wait_acquire();
    if (threadIdx.x == 0) KLIN_T(4);
#ifdef KLIN_TRACE
    if (threadIdx.x == 0) {
        unsigned long long ns;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));
        if (blockIdx.x < kTraceCtas) KLIN_TRACE_BUF[blockIdx.x * kTraceSlots + 6] = ns;
    }
#endif
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

template <bool BCOL, int MODE>
cudaError_t launch(const GemmArgs& g, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc,
                   const PairParams& p, unsigned grid, int device, cudaStream_t stream)
{
    auto kern = r4_pair_kernel<BCOL, MODE>;
    static bool attr_set[64] = {};
    if (device < 0 || device >= 64 || !attr_set[device]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        if (device >= 0 && device < 64) attr_set[device] = true;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, g, ma, mb, mc, p);
}

}  // namespace

bool r4_pair_possible(const GemmArgs& g, const RunContext& ctx)
{
    auto ok2 = [](const void* base, int64_t ld) {
        return reinterpret_cast<uintptr_t>(base) % 16 == 0 && (ld * 2) % 16 == 0 && ld * 2 < (int64_t(1) << 40);
    };
    if (!ctx.encode_tiled || ctx.max_smem_optin < kSmemBytes) return false;
    return ok2(g.A, g.lda) && ok2(g.B, g.ldb);
}

// Estimated cycles of the single-CTA kernel's schedule: per wave of 128 x 256 tiles 580 per k-block (the issuing
// thread and the shared-memory port; the epilogue hides behind the next tile) plus ~4 k that no main loop hides; a
// launch that is one under-filled wave cut into half tiles counts 0.8.  Fitted to graph replays (operands in the L2)
// of 1536^3 ... 2560^3, 4096 x 4096 x {256, 512, 1024}, 8192 x 8192 x {128, 512}.
static double single_schedule_cycles(int64_t tiles1, int64_t nkb, bool halves, const RunContext& ctx)
{
    const int64_t full = tiles1 / ctx.sm_count, tail = tiles1 % ctx.sm_count;
    const double waves = full + (tail == 0 ? 0.0 : (full == 0 && 2 * tail <= ctx.sm_count && halves ? 0.8 : 1.0));
    return waves * (4000.0 + 580.0 * static_cast<double>(nkb));
}
static double single_schedule_cycles(const GemmArgs& g, const RunContext& ctx)
{
    return single_schedule_cycles(static_cast<int64_t>((g.M + PM - 1) / PM) * ((g.N + PN - 1) / PN), (g.K + BK - 1) / BK,
                                  g.N > PN / 2, ctx);
}

// Batched and grouped launches: the same comparison on the launch's tile counts (128 x 256 and 512 x 256 tiles over all
// problems, the longest K).  Measured cold / warm in us, single-CTA against pair: BMM 32 x 1024 x 1024 x 512 41.8 / 37.6
// against 41.7 / 36.8, 16 x 2048 x 2048 x 512 69.7 / 69.3 against 62.4 / 62.8, 32 x 1024 x 1024 x 256 31.7 / 27.0 against
// 28.7 / 24.2, 24 x 768 x 3072 x 768 85.0 / 83.9 against 82.9 / 84.5 (73.8 / 77.6 on 256-row tiles).
bool r4_pair_faster_multi(int64_t tiles128, int64_t tiles256, int64_t tiles512, int64_t nkb, const RunContext& ctx)
{
    const int64_t pairs = ctx.sm_count / 2;
    if (pairs <= 0) return false;
    // the pair kernel's better form: 512-row tiles, or 256-row tiles at 1170 per stage of two k-blocks + 1.2 k per tile
    const double t512 = static_cast<double>((tiles512 + pairs - 1) / pairs) * (nkb * 1035.0 + 3600.0);
    const double t256 = static_cast<double>((tiles256 + pairs - 1) / pairs) * (((nkb + 1) / 2) * 1170.0 + 1200.0);
    return (t512 < t256 ? t512 : t256) < single_schedule_cycles(tiles128, nkb, false, ctx);
}

bool r4_pair_applicable(const GemmArgs& g, const RunContext& ctx)
{
    if (!r4_pair_possible(g, ctx) || g.M <= 2 * PM) return false;
    // Which kernel finishes first?  Estimated cycles of either schedule, from measured rates: a 512 x 256 pair tile
    // takes ~1035 cycles per k-block (two accumulators alternate: full rate) plus ~3.6 k cycles per tile that the main
    // loop does not hide (accumulator drain, barrier round trips); the single-CTA kernel as estimated above.  Timed
    // with operands in the L2 (graph replay) and after an L2 flush; the rule follows the former where they disagree
    // (2304^3: 26.3 against 31.2 us warm, 31.6 / 36.9 cold; 4096 x 4096 x 1024 28.1 / 31.2 and 33.7 / 37.9; 8192 x 8192
    // x 128 29.7 / 40.5 and 33.6 / 45.1; 2048^3 23.8 / 16.7 and 29.7 / 23.0 - the single-CTA kernel's).
    const int64_t nkb = (g.K + BK - 1) / BK;
    const int64_t pairs = ctx.sm_count / 2;
    const int64_t tiles2 = static_cast<int64_t>((g.M + TILE_M - 1) / TILE_M) * ((g.N + PN - 1) / PN);
    const double t_pair = static_cast<double>((tiles2 + pairs - 1) / pairs) * (nkb * 1035.0 + 3600.0);
    return t_pair < single_schedule_cycles(g, ctx);
}

namespace {

bool tma2(const void* base, int64_t ld_elems, int elt)
{
    return reinterpret_cast<uintptr_t>(base) % 16 == 0 && (ld_elems * elt) % 16 == 0 &&
           ld_elems * elt < (int64_t(1) << 40);
}

// The fields of PairParams that depend only on the operand layout.
void fill_layout(PairParams& p, const GemmArgs& g, const RunContext& ctx)
{
    p.group_m = ctx.plan.group_m > 0 ? ctx.plan.group_m : 4;
    const uint32_t w_major = g.b_col ? 0u : 1u;
    p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | (w_major << 16) | (static_cast<uint32_t>(PN >> 3) << 17) |
              (static_cast<uint32_t>((2 * PM) >> 4) << 24);
    p.b_desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    p.b_desc_lbo = g.b_col ? 1u : ((64u * BK * 2u) >> 4);
    p.b_kstep = g.b_col ? 2u : (2048u >> 4);
}

// Rounds of 256-row tiles against rounds of 512-row tiles, for launches of several rounds.  Per tile, fitted to graph
// replays of batched and single launches (K = 128 ... 4096): 2.4 k + 1350 per stage of two k-blocks for a 256 x 256 tile
// (its drain overlaps the next tile's MMAs; a third more L2 traffic per flop than the 512-row tile), 3.9 k + 1257 per
// k-block for a 512 x 256 tile.  Twice the tiles in fewer than twice the rounds is what pays: 3584^3 70.7 us against
// 77.3 (three rounds against two), 2560 x 4096 x 4096 76.8 / 84.5, BMM 32 x 1024^3 60.4 / 62.4 (seven against four),
// 24 x 768 x 3072 x 768 73.8 / 82.9, ragged groups 201 / 219; with both counts a whole number of rounds (4096^3: four
// against two) 100 against 94, 8192 x 8192 x 128 32.8 against 29.7.
bool pair_k_paired_faster(int64_t tiles256, int64_t tiles512, int64_t nkb, int64_t pairs)
{
    if (pairs <= 0 || nkb < 1) return false;
    const int64_t r256 = (tiles256 + pairs - 1) / pairs, r512 = (tiles512 + pairs - 1) / pairs;
    const double t256 = static_cast<double>(r256) * (static_cast<double>((nkb + 1) / 2) * 1350.0 + 2400.0);
    const double t512 = static_cast<double>(r512) * (static_cast<double>(nkb) * 1257.0 + 3900.0);
    return t256 < 0.97 * t512;
}

// Batched and grouped launches: k-paired 256-row tiles when the plan that names the pair kernel asks for them
// (stages 3), and by the estimate above when no plan names a kernel.
bool pair_k_paired_multi(const RunContext& ctx, int64_t tiles256, int64_t tiles512, int64_t nkb)
{
    if (ctx.plan.kernel == 2) return ctx.plan.stages == 3;
    return ctx.plan.kernel == 0 && pair_k_paired_faster(tiles256, tiles512, nkb, ctx.sm_count / 2);
}

bool c_takes_tma_store(const GemmArgs& g)
{
    const int celt = g.c_bf16 ? 2 : 4;
    return tma2(g.C, g.ldc, celt) && (static_cast<int64_t>(g.N) * celt) % 16 == 0;
}

}  // namespace

bool r4_pair_batched_possible(const GemmArgs& g, const BatchArgs& b, const RunContext& ctx)
{
    if (!r4_pair_possible(g, ctx) || b.batch < 1 || b.batch > 65535) return false;
    // batch strides become tensor-map strides: multiples of 16 bytes, below 2^40
    auto ok = [](int64_t stride_elems) {
        return stride_elems > 0 && (stride_elems * 2) % 16 == 0 && stride_elems * 2 < (int64_t(1) << 40);
    };
    if (!ok(b.stride_a) || !ok(b.stride_b)) return false;
    const int64_t tiles = static_cast<int64_t>((g.M + TILE_M - 1) / TILE_M) * ((g.N + PN - 1) / PN);
    return tiles * b.batch < 0x7FFFFFFFll;
}

cudaError_t launch_r4_pair_batched(const GemmArgs& g, const BatchArgs& b, RunContext& ctx, cudaStream_t stream,
                                   int* kernel_id)
{
    if (!r4_pair_batched_possible(g, b, ctx)) return cudaErrorInvalidValue;
    PairParams p;
    memset(&p, 0, sizeof p);
    fill_layout(p, g, ctx);
    const int64_t tn = (g.N + PN - 1) / PN;
    const bool kp = pair_k_paired_multi(ctx, (g.M + 2 * PM - 1) / (2 * PM) * tn * b.batch, (g.M + TILE_M - 1) / TILE_M * tn * b.batch,
                                        (g.K + BK - 1) / BK);
    p.tiles_m2 = kp ? (g.M + 2 * PM - 1) / (2 * PM) : (g.M + TILE_M - 1) / TILE_M;
    p.tiles_n = (g.N + PN - 1) / PN;
    p.tiles_per_batch = p.tiles_m2 * p.tiles_n;
    p.total_tiles = static_cast<int64_t>(p.tiles_per_batch) * b.batch;
    p.stage_tx = kp ? 2 * 4 * kABlockBytes : 2 * kStageBytes;
    p.b_boxes = 2;
    p.nkb = (g.K + BK - 1) / BK;
    if (kp) p.nkb = (p.nkb + 1) / 2;        // stages of two k-blocks
    const int celt = g.c_bf16 ? 2 : 4;
    p.stride_c_bytes = b.stride_c * celt;
    p.epi_tma = (c_takes_tma_store(g) && p.stride_c_bytes % 16 == 0 && p.stride_c_bytes > 0 &&
                 p.stride_c_bytes < (int64_t(1) << 40))
                    ? 1
                    : 0;
    CUtensorMap ma, mb, mc;
    memset(&ma, 0, sizeof ma);
    memset(&mb, 0, sizeof mb);
    memset(&mc, 0, sizeof mc);
    const uint64_t nb = static_cast<uint64_t>(b.batch);
    bool ok = encode_map_3d(ctx, &ma, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.A, g.K, g.M, nb, g.lda * 2, b.stride_a * 2, BK,
                            PM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (g.b_col)
        ok = ok && encode_map_3d(ctx, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B, g.K, g.N, nb, g.ldb * 2, b.stride_b * 2,
                                 BK, PN / 2, CU_TENSOR_MAP_SWIZZLE_128B);
    else
        ok = ok && encode_map_3d(ctx, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B, g.N, g.K, nb, g.ldb * 2, b.stride_b * 2,
                                 64, BK, CU_TENSOR_MAP_SWIZZLE_128B);
    if (p.epi_tma)
        ok = ok && encode_map_3d(ctx, &mc, g.c_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                                 g.C, g.N, g.M, nb, g.ldc * celt, static_cast<uint64_t>(p.stride_c_bytes),
                                 g.c_bf16 ? 64 : 32, 32, CU_TENSOR_MAP_SWIZZLE_128B);
    if (!ok) return cudaErrorInvalidValue;
    p.kid = kIdTcgen05 + (p.epi_tma ? 0 : 2) + 32 + (kp ? 256 : 0) + ctx.kid_flags;
    *kernel_id = p.kid;
    const int64_t max_pairs = ctx.sm_count / 2;
    const unsigned grid = 2u * static_cast<unsigned>(p.total_tiles < max_pairs ? p.total_tiles : max_pairs);
    if (kp)
        return g.b_col ? launch<true, 7>(g, ma, mb, mc, p, grid, ctx.device, stream)
                       : launch<false, 7>(g, ma, mb, mc, p, grid, ctx.device, stream);
    return g.b_col ? launch<true, 1>(g, ma, mb, mc, p, grid, ctx.device, stream)
                   : launch<false, 1>(g, ma, mb, mc, p, grid, ctx.device, stream);
}

bool r4_pair_grouped_possible(const GemmArgs* groups, int n, const RunContext& ctx)
{
    if (n < 1 || n > kMaxGroups || ctx.workspace_bytes < static_cast<size_t>(n) * sizeof(GroupEntry)) return false;
    int64_t tiles = 0;
    for (int i = 0; i < n; ++i) {
        const GemmArgs& g = groups[i];
        if (g.M <= 0 || g.N <= 0 || g.K <= 0) return false;          // the caller drops empty groups
        if (!r4_pair_possible(g, ctx)) return false;
        tiles += static_cast<int64_t>((g.M + TILE_M - 1) / TILE_M) * ((g.N + PN - 1) / PN);
    }
    return tiles < 0x7FFFFFFFll;
}

cudaError_t launch_r4_pair_grouped(const GemmArgs* groups, int n, RunContext& ctx, cudaStream_t stream, int* kernel_id)
{
    if (!r4_pair_grouped_possible(groups, n, ctx)) return cudaErrorInvalidValue;
    static_assert(sizeof(GroupEntry) % 128 == 0, "table entries keep their tensor maps 128-byte aligned");
    // Ragged groups: a tile row with at most 256 live rows costs about half a tile (its second row block issues no
    // MMAs).  Such a last tile row becomes a table entry of its own (the group's A and C from that row on), all of
    // them go to the END of the schedule, and odd rounds run over the pairs in reverse: the pairs that got a full
    // tile in the last full round get the half tiles last.  (Dealt round-robin in group order, a G = 8 launch of
    // 320 tiles kept some pairs busy for 5 tiles' time where 4 suffice.)
    int64_t t256 = 0, t512 = 0, nkb_max = 0;
    for (int i = 0; i < n; ++i) {
        const int64_t tn = (groups[i].N + PN - 1) / PN;
        t256 += (groups[i].M + 2 * PM - 1) / (2 * PM) * tn;
        t512 += (groups[i].M + TILE_M - 1) / TILE_M * tn;
        nkb_max = std::max<int64_t>(nkb_max, (groups[i].K + BK - 1) / BK);
    }
    const bool kp = pair_k_paired_multi(ctx, t256, t512, nkb_max);        // 256-row tiles: no tile row is worth splitting off
    GemmArgs* ents = new (std::nothrow) GemmArgs[2 * n];
    if (!ents) return cudaErrorMemoryAllocation;
    int n_full = 0, n_half = 0;
    GemmArgs* halves = ents + n;
    for (int i = 0; i < n && !kp; ++i) {
        const GemmArgs& g = groups[i];
        const int rem = g.M % TILE_M;
        if (rem == 0 || rem > 2 * PM) {
            ents[n_full++] = g;
            continue;
        }
        GemmArgs h = g;                       // the last (or only) tile row
        const int64_t off = g.M - rem;
        h.A = g.A + off * g.lda;
        h.C = static_cast<uint8_t*>(g.C) + off * g.ldc * (g.c_bf16 ? 2 : 4);
        h.M = rem;
        halves[n_half++] = h;
        if (off > 0) {
            GemmArgs f = g;
            f.M = static_cast<int>(off);
            ents[n_full++] = f;
        }
    }
    const bool reorder = n_half > 0 && n_full > 0 && n_full + n_half <= kMaxGroups &&
                         ctx.workspace_bytes >= static_cast<size_t>(n_full + n_half) * sizeof(GroupEntry);
    if (reorder) {
        for (int i = 0; i < n_half; ++i) ents[n_full + i] = halves[i];
        n = n_full + n_half;
        groups = ents;
    }
    GroupEntry* table = new (std::nothrow) GroupEntry[n];
    if (!table) {
        delete[] ents;
        return cudaErrorMemoryAllocation;
    }
    memset(table, 0, sizeof(GroupEntry) * n);
    PairParams p;
    memset(&p, 0, sizeof p);
    fill_layout(p, groups[0], ctx);
    int tile_start = 0;
    bool ok = true, any_tma = false;
    for (int i = 0; i < n && ok; ++i) {
        const GemmArgs& g = groups[i];
        GroupEntry& e = table[i];
        const int celt = g.c_bf16 ? 2 : 4;
        e.C = g.C;
        e.ldc = g.ldc;
        e.M = g.M;
        e.N = g.N;
        e.K = g.K;
        e.nkb = (g.K + BK - 1) / BK;
        e.tiles_m = (g.M + TILE_M - 1) / TILE_M;
        if (kp) {
            e.nkb = (e.nkb + 1) / 2;        // stages of two k-blocks
            e.tiles_m = (g.M + 2 * PM - 1) / (2 * PM);
        }
        e.tiles_n = (g.N + PN - 1) / PN;
        e.tile_start = tile_start;
        tile_start += e.tiles_m * e.tiles_n;
        e.epi_tma = c_takes_tma_store(g) ? 1 : 0;
        any_tma = any_tma || e.epi_tma;
        ok = encode_map_2d(ctx, &e.map_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.A, g.K, g.M, g.lda * 2, BK, PM,
                           CU_TENSOR_MAP_SWIZZLE_128B);
        if (g.b_col)
            ok = ok && encode_map_2d(ctx, &e.map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B, g.K, g.N, g.ldb * 2, BK, PN / 2,
                                     CU_TENSOR_MAP_SWIZZLE_128B);
        else
            ok = ok && encode_map_2d(ctx, &e.map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B, g.N, g.K, g.ldb * 2, 64, BK,
                                     CU_TENSOR_MAP_SWIZZLE_128B);
        if (e.epi_tma)
            ok = ok && encode_map_2d(ctx, &e.map_c,
                                     g.c_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, g.C, g.N,
                                     g.M, g.ldc * celt, g.c_bf16 ? 64 : 32, 32, CU_TENSOR_MAP_SWIZZLE_128B);
    }
    cudaError_t err = ok ? cudaSuccess : cudaErrorInvalidValue;
    // The table travels on the launch's stream, ahead of the kernel that reads it (from pageable
    // memory the copy is staged before the call returns, so the host array can go).
    if (err == cudaSuccess)
        err = cudaMemcpyAsync(ctx.workspace, table, sizeof(GroupEntry) * n, cudaMemcpyHostToDevice, stream);
    delete[] table;
    const GemmArgs g0 = groups[0];
    delete[] ents;
    if (err != cudaSuccess) return err;
    p.groups = static_cast<const GroupEntry*>(ctx.workspace);
    p.n_groups = n;
    p.total_tiles = tile_start;
    p.snake = reorder ? 1 : 0;
    p.stage_tx = kp ? 2 * 4 * kABlockBytes : 2 * kStageBytes;
    p.b_boxes = 2;
    p.epi_tma = any_tma ? 1 : 0;
    p.kid = kIdTcgen05 + (any_tma ? 0 : 2) + 32 + (kp ? 256 : 0) + ctx.kid_flags;
    *kernel_id = p.kid;
    const int64_t max_pairs = ctx.sm_count / 2;
    const unsigned grid = 2u * static_cast<unsigned>(p.total_tiles < max_pairs ? p.total_tiles : max_pairs);
    CUtensorMap none;
    memset(&none, 0, sizeof none);
    if (kp)
        return g0.b_col ? launch<true, 8>(g0, none, none, none, p, grid, ctx.device, stream)
                        : launch<false, 8>(g0, none, none, none, p, grid, ctx.device, stream);
    return g0.b_col ? launch<true, 2>(g0, none, none, none, p, grid, ctx.device, stream)
                    : launch<false, 2>(g0, none, none, none, p, grid, ctx.device, stream);
}

namespace {
cudaError_t launch_pair_one_problem(const GemmArgs& g, void* const* dst_c, const int64_t* dst_ldc, int n_dst,
                                    RunContext& ctx, cudaStream_t stream, int* kernel_id);

// Column tiling of one problem on the pair kernel (paper, Table 1 `templatize` / `autotune`: the tile shape is a
// recipe parameter).  tile_n == 0: the pinned widths cannot run.
struct PairColumns {
    int tile_n, n_wide, tile_n2, n_narrow;
    double cycles;      // estimated tensor-pipe cycles of the launch
};

// Tensor-pipe cycles of one k-block of a 512-row pair tile `w` columns wide (eight MMAs, two accumulators
// alternating), measured with uniform-width launches.
double pair_kblock_cycles(int w)
{
    // (single under-filled waves at K = 8192: 256 / 192 / 128 columns 90.1 / 84.0 / 81 us per tile - the issuing thread
    // and the A operand's bytes do not shrink with the width)
    return w >= 256 ? 1035.0 : w >= 192 ? 960.0 : w >= 128 ? 930.0 : 900.0;
}

// Makespan (cycles) of the static schedule: tiles in schedule order (all wide ones, then the narrow ones),
// dealt to `pairs` CTA pairs round by round, odd rounds in reverse order when widths are mixed.
double pair_makespan(int64_t n_wide_tiles, int64_t n_narrow_tiles, double c_wide, double c_narrow, int64_t pairs)
{
    const int64_t total = n_wide_tiles + n_narrow_tiles;
    const bool snake = n_wide_tiles > 0 && n_narrow_tiles > 0;
    double worst = 0.0;
    // a pair's load depends only on its position; positions 0, pairs-1 and those next to the wide / narrow
    // boundary of each round bound the maximum, but the count is small: evaluate every pair
    for (int64_t q = 0; q < pairs; ++q) {
        double t = 0.0;
        for (int64_t r = 0; r * pairs < total; ++r) {
            const int64_t idx = r * pairs + ((snake && (r & 1)) ? pairs - 1 - q : q);
            if (idx >= total) break;
            t += idx < n_wide_tiles ? c_wide : c_narrow;
        }
        if (t > worst) worst = t;
    }
    return worst;
}

// Whether and how the last, under-filled wave of pair tiles is streamed along K (see PairParams).
struct StreamK {
    bool on;
    int rounds;
    int64_t first, work;
};
// CTA pairs of this kernel that the device holds at once (asked of the runtime once per device): a streamed wave
// has pairs waiting on one another's partial tiles, so every pair of the grid must be resident.
int resident_pairs(const RunContext& ctx)
{
    static int cache[64] = {};
    const bool cacheable = ctx.device >= 0 && ctx.device < 64;
    if (cacheable && cache[ctx.device] != 0) return cache[ctx.device];
    auto kern = r4_pair_kernel<false, 0>;
    int n = 0;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>(ctx.sm_count / 2 * 2));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess ||
        cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n < 0) {
        cudaGetLastError();
        n = 0;
    }
    if (cacheable) cache[ctx.device] = n > 0 ? n : -1;
    return n > 0 ? n : -1;
}

StreamK plan_stream_k(int64_t tiles, int nkb, int64_t pairs, const RunContext& ctx, bool forced)
{
    StreamK sk = {false, 0, 0, 0};
    if (!ctx.sk_flags || pairs < 2 || tiles <= 0) return sk;
    if (resident_pairs(ctx) < pairs) return sk;
    const int64_t rounds = tiles / pairs, rem = tiles % pairs;
    if (rem == 0) return sk;
    const int64_t work = rem * nkb;
    const int64_t share = (work + pairs - 1) / pairs;             // k-blocks of the streamed wave per pair
    // every piece at least 8 k-blocks deep on average, and no tile cut into more than 6 pieces
    if (share < 8 || share * 6 < nkb || work / pairs < 1) return sk;
    if (static_cast<size_t>(pairs) * TILE_M * PN * sizeof(float) > ctx.workspace_bytes) return sk;
    if (rounds > 0x7FFFFFFF) return sk;
    // Not chosen unless a plan asks for it.  Measured on B200 (single launches after an L2 flush): 4096^3 107 us
    // streamed against 92 us in whole tiles, 3072 x 2048 x 8192 91 against 87, 2048 x 4096 x 4096 71 against 52 -
    // although the schedule alone (partial tiles neither written nor read) would take 89 / 75 / 54 us.  The pair
    // kernel's main loop already draws about 9 TB/s from the L2; the partial tiles' trip through it (1 MiB per
    // pair) comes on top, and a power-capped part clocks lower with every SM busy.  The autotuner times the
    // candidate and may pin it where it wins.
    if (!forced) return sk;
    sk.on = true;
    sk.rounds = static_cast<int>(rounds);
    sk.first = rounds * pairs;
    sk.work = work;
    return sk;
}

PairColumns plan_columns_uncached(const GemmArgs& g, const RunContext& ctx);

// The search below evaluates up to fifty schedules of seventy-four pairs each: 8-20 us of host time, which a launch of a
// dozen microseconds enqueued in a loop cannot hide (4096 x 4096 x 256: 21.5 us per call against 13.4 for the single-CTA
// kernel's launch).  Its result depends on the sizes and the plan only: the last few are remembered per thread.
PairColumns plan_columns(const GemmArgs& g, const RunContext& ctx)
{
    struct Entry {
        int64_t M, N, K;
        int sm, tile_n, tail_n, split_via;
        bool used;
        PairColumns cols;
    };
    static thread_local Entry memo[8] = {};
    static thread_local unsigned next = 0;
    for (const Entry& e : memo)
        if (e.used && e.M == g.M && e.N == g.N && e.K == g.K && e.sm == ctx.sm_count && e.tile_n == ctx.plan.tile_n &&
            e.tail_n == ctx.plan.tail_n && e.split_via == ctx.plan.split_via)
            return e.cols;
    Entry& e = memo[next++ % 8];
    e = Entry{g.M, g.N, g.K, ctx.sm_count, ctx.plan.tile_n, ctx.plan.tail_n, ctx.plan.split_via, true,
              plan_columns_uncached(g, ctx)};
    return e.cols;
}

PairColumns plan_columns_uncached(const GemmArgs& g, const RunContext& ctx)
{
    const int64_t tiles_m2 = (g.M + TILE_M - 1) / TILE_M;
    const int64_t nkb = (g.K + BK - 1) / BK;
    const int64_t pairs = ctx.sm_count / 2 > 0 ? ctx.sm_count / 2 : 1;
    const double per_tile = 5000.0;        // cycles per tile that the main loop does not hide
    auto valid_w = [](int w) { return w >= 64 && w <= PN && w % 64 == 0; };   // whole 128-byte store units in either C type
    const int wide = ctx.plan.tile_n > 0 ? ctx.plan.tile_n : PN;
    PairColumns best = {0, 0, 0, 0, 0.0};
    if (!valid_w(wide)) return best;
    auto consider = [&](int n_wide, int w2) {
        const int64_t rest = static_cast<int64_t>(g.N) - static_cast<int64_t>(n_wide) * wide;
        const int n_narrow = rest > 0 ? static_cast<int>((rest + w2 - 1) / w2) : 0;
        if (n_wide + n_narrow > 0x3FFFFF) return;
        const double cw = nkb * pair_kblock_cycles(wide) + per_tile, cn = nkb * pair_kblock_cycles(w2) + per_tile;
        const double t = pair_makespan(tiles_m2 * n_wide, tiles_m2 * n_narrow, cw, cn, pairs);
        // (a mixed schedule has to win by 2 %: its narrow MMAs run below the full rate and it re-reads more of B)
        const double score = (n_narrow > 0 && n_wide > 0) ? t * 1.02 : t;
        if (best.tile_n == 0 || score < best.cycles) best = {wide, n_wide, n_narrow > 0 ? w2 : 0, n_narrow, score};
    };
    const int all_wide = static_cast<int>((static_cast<int64_t>(g.N) + wide - 1) / wide);
    consider(all_wide, wide);              // uniform tiles
    if (ctx.plan.tile_n == 0 && ctx.plan.tail_n == 0 && ctx.plan.split_via != 3 && tiles_m2 * all_wide <= pairs) {
        // One under-filled round: narrower uniform tiles that still fit one round finish sooner (a tile's time falls by
        // 7-10 %, nothing else changes): 3072 x 2048 x 8192 90.1 -> 84.0 us with 192 columns.
        for (int w : {192, 128}) {
            const int64_t cols = (static_cast<int64_t>(g.N) + w - 1) / w;
            if (tiles_m2 * cols > pairs) continue;
            const double t = nkb * pair_kblock_cycles(w) + per_tile;
            if (t < best.cycles * 0.97) best = {w, static_cast<int>(cols), 0, 0, t};
        }
        return best;
    }
    if (ctx.plan.tail_n == wide) return best;
    if (ctx.plan.tail_n > 0 && !valid_w(ctx.plan.tail_n)) return PairColumns{0, 0, 0, 0, 0.0};
    if (ctx.plan.tail_n > 0) best.tile_n = 0;        // a pinned narrow width must be used
    for (int w2 = 128; w2 < wide; w2 += 64) {
        if (ctx.plan.tail_n > 0 && w2 != ctx.plan.tail_n) continue;
        if (tiles_m2 * all_wide <= pairs && ctx.plan.tail_n == 0) break;      // one round: nothing to balance
        const int lo = all_wide > 24 ? all_wide - 24 : 0;
        for (int n_wide = all_wide - 1; n_wide >= lo; --n_wide) consider(n_wide, w2);
    }
    if (ctx.plan.tail_n > 0 && ctx.plan.tail_n < 128 && best.tile_n == 0) {
        for (int n_wide = all_wide - 1; n_wide >= 0 && n_wide >= all_wide - 24; --n_wide) consider(n_wide, ctx.plan.tail_n);
    }
    return best;
}

// Whether a single problem runs as k-paired 256-row tiles: when a plan asks for it (stages = 3), else - with nothing
// pinned - by the rule of r4_pair_k_paired_auto.  Never with a tile width other than 256, a narrow tail or a streamed
// last wave.
bool pair_k_paired(const GemmArgs& g, const RunContext& ctx)
{
    const R4Plan& pl = ctx.plan;
    if (pl.stages != 0 && pl.stages != 3) return false;
    if ((pl.tile_n != 0 && pl.tile_n != PN) || pl.tail_n != 0 || pl.split_via == 3) return false;
    if (pl.stages == 3) return true;
    return pl.kernel == 0 && pl.split_via == 0 && pl.tile_n == 0 && r4_pair_k_paired_auto(g, ctx);
}
}

// One problem, nothing pinned.  One round of 256 x 256 tiles that fills more than half of the CTA pairs, K >= 3072: at
// 2048^3 the form is level with the single-CTA kernel in graph replay (15.9 against 16.1 us) but its cluster launch
// costs the host more, and launches enqueued one by one fall behind (18.5 against 16.9 us per launch) - measured (single launches after an L2 flush, against the single-CTA kernel's one
// wave of 128 x 256 tiles): 2048 x 2048 x 8192 56.2 against 61.4 us, 512 x 8192 x 8192 61.5 / 65.5, 1536 x 2048 x 4096
// 32.8 / 34.8, 2304 x 2048 x 6144 45.6 / 49.1, 2048 x 2048 x 3072 28.2 / 28.8; with 32 tiles (1024 x 2048 x 8192) 54
// against 42 for the single-CTA kernel's cluster split.  Several rounds: when they beat the 512-row tiles' rounds
// (pair_k_paired_faster) and the single-CTA kernel's estimate
// (3072 x 4096 x 2048: 46.1 against 50.2 and 52.2 us).
bool r4_pair_k_paired_auto(const GemmArgs& g, const RunContext& ctx)
{
    if (!r4_pair_possible(g, ctx) || g.M <= 2 * PM) return false;
    const int64_t tn = (g.N + PN - 1) / PN;
    const int64_t tiles = static_cast<int64_t>((g.M + 2 * PM - 1) / (2 * PM)) * tn;
    const int64_t pairs = ctx.sm_count / 2;
    if (tiles <= pairs) {
        // (not where one wave of the single-CTA kernel's 128-column tiles fills the matrix's columns much better: at
        // 1912 x 1064 x 3544 - the fifth 256-column tile holds 40 columns - they take 25.7 us against 29.2, at 3104 x
        // 528 x 4784 24.0 against 28.8)
        // K: from 3072 on; from 1280 on where the single-CTA kernel's wave of 128 x 256 tiles would be less than 85 % full
        // (launches enqueued one by one, us: 1328 x 1944 x 2128 18.6 against 22.9, 544 x 5896 x 1776 18.0 / 20.2, 1472 x 2040 x
        // 1496 18.4 / 19.7; at 2048^3 - 128 tiles on 148 SMs - 18.5 against 16.9)
        const int64_t tiles1 = static_cast<int64_t>((g.M + PM - 1) / PM) * tn;
        const bool k_ok = g.K >= 3072 || (g.K >= 1280 && tiles1 * 100 < static_cast<int64_t>(ctx.sm_count) * 85);
        return 2 * tiles > pairs && k_ok && !r4_narrow_tiles_fill_better(g.M, g.N, ctx.sm_count);
    }
    const int64_t nkb = (g.K + BK - 1) / BK;
    if (!pair_k_paired_faster(tiles, static_cast<int64_t>((g.M + TILE_M - 1) / TILE_M) * tn, nkb, pairs)) return false;
    const int64_t r256 = (tiles + pairs - 1) / pairs;
    const double t256 = static_cast<double>(r256) * (static_cast<double>((nkb + 1) / 2) * 1170.0 + 1200.0);
    return t256 < single_schedule_cycles(g, ctx);
}

bool r4_pair_stream_k_possible(const GemmArgs& g, const RunContext& ctx)
{
    if (!r4_pair_possible(g, ctx) || g.M <= 0 || g.N <= 0 || g.K <= 0) return false;
    const int64_t tiles = static_cast<int64_t>((g.M + TILE_M - 1) / TILE_M) * ((g.N + PN - 1) / PN);
    return plan_stream_k(tiles, (g.K + BK - 1) / BK, ctx.sm_count / 2, ctx, true).on;
}

cudaError_t launch_r4_tcgen05_pair(const GemmArgs& g, RunContext& ctx, cudaStream_t stream, int* kernel_id)
{
    return launch_pair_one_problem(g, nullptr, nullptr, 0, ctx, stream, kernel_id);
}

cudaError_t launch_r4_pair_multi_dst(const GemmArgs& g, void* const* C, const int64_t* ldc, int n_dst, RunContext& ctx,
                                     cudaStream_t stream, int* kernel_id)
{
    if (n_dst < 1 || n_dst > kMaxDst || !C || !ldc) return cudaErrorInvalidValue;
    return launch_pair_one_problem(g, C, ldc, n_dst, ctx, stream, kernel_id);
}

namespace {

// n_dst == 0: the plain launch (C and its pitch from g).  n_dst >= 1: the multi-destination launch;
// g.C / g.ldc are ignored, the destination table is built in the workspace on `stream`.
cudaError_t launch_pair_one_problem(const GemmArgs& g, void* const* dst_c, const int64_t* dst_ldc, int n_dst,
                                    RunContext& ctx, cudaStream_t stream, int* kernel_id)
{
    PairParams p;
    memset(&p, 0, sizeof p);
    // k-paired 256-row tiles (see the kernel): one problem, one destination, uniform 256-column tiles, whole tiles
    const bool kp = n_dst == 0 && pair_k_paired(g, ctx);
    if (ctx.plan.stages == 3 && !kp) return cudaErrorInvalidValue;
    p.tiles_m2 = kp ? (g.M + 2 * PM - 1) / (2 * PM) : (g.M + TILE_M - 1) / TILE_M;
    p.nkb = (g.K + BK - 1) / BK;
    if (kp) p.nkb = (p.nkb + 1) / 2;        // the kernel's k-loop counts stages of two k-blocks
    PairColumns cols = plan_columns(g, ctx);
    if (kp) {
        const int n_tiles = (g.N + PN - 1) / PN;
        cols = PairColumns{PN, n_tiles, 0, 0, 0.0};
    }
    if (cols.tile_n == 0) return cudaErrorInvalidValue;
    p.tile_n = cols.tile_n;
    p.n_wide = cols.n_wide;
    p.tile_n2 = cols.tile_n2;
    p.n_narrow = cols.n_narrow;
    p.tiles_n = cols.n_wide + cols.n_narrow;
    p.wide_tiles = static_cast<int64_t>(p.tiles_m2) * p.n_wide;
    p.total_tiles = static_cast<int64_t>(p.tiles_m2) * p.tiles_n;
    p.snake = cols.n_narrow > 0 && cols.n_wide > 0 ? 1 : 0;
    // every tile loads a B box as wide as the widest tile's half (a narrower tile ignores the rest)
    const int widest = cols.n_wide > 0 ? cols.tile_n : cols.tile_n2;
    const uint32_t b_box_rows = static_cast<uint32_t>(widest / 2);
    p.b_boxes = (widest / 2 + 63) / 64;
    p.stage_tx = 2u * (kABytes + (g.b_col ? b_box_rows * 128u : static_cast<uint32_t>(p.b_boxes) * 8192u));
    if (kp) p.stage_tx = 2u * (kABytes + 2u * (g.b_col ? b_box_rows * 128u : static_cast<uint32_t>(p.b_boxes) * 8192u));
    // default raster group: 4 x 512 rows; 8 when the problem has at least 16 tile rows (measured at 8192^3 in rested
    // 10-launch bursts: 672-674 us against 676-678 us for 4 and 684-686 us for 1, 2, 3 or 16)
    p.group_m = ctx.plan.group_m > 0 ? ctx.plan.group_m : (p.tiles_m2 >= 16 ? 8 : 4);
    const int celt = g.c_bf16 ? 2 : 4;
    // (row length a multiple of 16 bytes too: a store box ending inside a 16-byte unit at the tensor's
    // right edge writes the whole unit)
    p.epi_tma = (reinterpret_cast<uintptr_t>(g.C) % 16 == 0 && (g.ldc * celt) % 16 == 0 &&
                 (static_cast<int64_t>(g.N) * celt) % 16 == 0 && g.ldc * celt < (int64_t(1) << 40))
                    ? 1
                    : 0;
    DstEntry table[kMaxDst];
    if (n_dst > 0) {
        // TMA stores only when every destination qualifies (one epilogue form per launch)
        if (ctx.workspace_bytes < sizeof(DstEntry) * n_dst) return cudaErrorInvalidValue;
        memset(table, 0, sizeof(DstEntry) * n_dst);
        p.epi_tma = 1;
        for (int d = 0; d < n_dst; ++d) {
            GemmArgs gd = g;
            gd.C = dst_c[d];
            gd.ldc = dst_ldc[d];
            if (!c_takes_tma_store(gd)) p.epi_tma = 0;
            table[d].C = dst_c[d];
            table[d].ldc = dst_ldc[d];
        }
    }
    // Instruction descriptor: fp32 accumulator, bf16 A/B, A K-major, B K-major (column-major B) or
    // MN-major (row-major B), N = 256, M = 256 (128 rows in each CTA of the pair).
    const uint32_t w_major = g.b_col ? 0u : 1u;
    p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | (w_major << 16) | (static_cast<uint32_t>(PN >> 3) << 17) |
              (static_cast<uint32_t>((2 * PM) >> 4) << 24);
    // B half in shared memory: 128 columns.  K-major: 128 rows of 128 bytes; MN-major: two
    // 64-column blocks 8192 bytes apart, 8-k groups 1024 bytes apart.
    p.b_desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    p.b_desc_lbo = g.b_col ? 1u : ((64u * BK * 2u) >> 4);
    p.b_kstep = g.b_col ? 2u : (2048u >> 4);

    CUtensorMap ma, mb, mc;
    memset(&ma, 0, sizeof ma);
    memset(&mb, 0, sizeof mb);
    memset(&mc, 0, sizeof mc);
    bool ok = encode_map_2d(ctx, &ma, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.A, g.K, g.M, g.lda * 2, BK, PM,
                            CU_TENSOR_MAP_SWIZZLE_128B);
    if (g.b_col)
        ok = ok && encode_map_2d(ctx, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B, g.K, g.N, g.ldb * 2, BK, b_box_rows,
                                 CU_TENSOR_MAP_SWIZZLE_128B);
    else
        ok = ok && encode_map_2d(ctx, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B, g.N, g.K, g.ldb * 2, 64, BK,
                                 CU_TENSOR_MAP_SWIZZLE_128B);
    if (p.epi_tma && n_dst == 0)
        ok = ok && encode_map_2d(ctx, &mc, g.c_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                                 g.C, g.N, g.M, g.ldc * celt, g.c_bf16 ? 64 : 32, 32, CU_TENSOR_MAP_SWIZZLE_128B);
    for (int d = 0; d < n_dst && p.epi_tma && ok; ++d)
        ok = encode_map_2d(ctx, &table[d].map_c,
                           g.c_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, table[d].C, g.N, g.M,
                           table[d].ldc * celt, g.c_bf16 ? 64 : 32, 32, CU_TENSOR_MAP_SWIZZLE_128B);
    if (!ok) return cudaErrorInvalidValue;

    const int64_t max_pairs = ctx.sm_count / 2;
    unsigned grid = 2u * static_cast<unsigned>(p.total_tiles < max_pairs ? p.total_tiles : max_pairs);
    // Stream the under-filled last wave along K?  (one problem, one destination, uniform 256-column tiles)
    if (n_dst == 0 && !kp && cols.n_narrow == 0 && cols.tile_n == PN && ctx.plan.split_via != 1) {
        const StreamK sk = plan_stream_k(p.total_tiles, p.nkb, max_pairs, ctx, ctx.plan.split_via == 3);
        if (sk.on) {
            p.sk = 1;
            p.sk_rounds = sk.rounds;
            p.sk_first = sk.first;
            p.sk_work = sk.work;
            p.sk_slots = static_cast<float*>(ctx.workspace);
            p.sk_flags = ctx.sk_flags;
            p.sk_epoch = ++ctx.sk_epoch;
            grid = 2u * static_cast<unsigned>(max_pairs);
        } else if (ctx.plan.split_via == 3) {
            return cudaErrorInvalidValue;
        }
    } else if (ctx.plan.split_via == 3) {
        return cudaErrorInvalidValue;
    }
    p.one_round = (!p.sk && cols.n_narrow == 0 && p.total_tiles <= max_pairs && p.tiles_m2 > 1) ? 1 : 0;
    p.kid = kIdTcgen05 + (p.epi_tma ? 0 : 2) + 32 + (p.sk ? 128 : 0) + (kp ? 256 : 0) + ctx.kid_flags;
    *kernel_id = p.kid;
    if (n_dst > 0) {
        // the table travels on the launch's stream, ahead of the kernel (staged before the call returns)
        const cudaError_t e = cudaMemcpyAsync(ctx.workspace, table, sizeof(DstEntry) * n_dst, cudaMemcpyHostToDevice, stream);
        if (e != cudaSuccess) return e;
        p.dsts = static_cast<const DstEntry*>(ctx.workspace);
        p.n_dst = n_dst;
        return g.b_col ? launch<true, 3>(g, ma, mb, mc, p, grid, ctx.device, stream)
                       : launch<false, 3>(g, ma, mb, mc, p, grid, ctx.device, stream);
    }
    if (p.sk)
        return g.b_col ? launch<true, 5>(g, ma, mb, mc, p, grid, ctx.device, stream)
                       : launch<false, 5>(g, ma, mb, mc, p, grid, ctx.device, stream);
    if (kp)
        return g.b_col ? launch<true, 6>(g, ma, mb, mc, p, grid, ctx.device, stream)
                       : launch<false, 6>(g, ma, mb, mc, p, grid, ctx.device, stream);
    return g.b_col ? launch<true, 0>(g, ma, mb, mc, p, grid, ctx.device, stream)
                   : launch<false, 0>(g, ma, mb, mc, p, grid, ctx.device, stream);
}

}  // namespace

}  // namespace klin
