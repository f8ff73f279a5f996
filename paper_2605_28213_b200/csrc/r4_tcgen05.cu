// Rung 4 - the expert kernel K_n of the lineage: "warp_specialize" plus matrix
// intrinsics (paper, Table 1; Introduction: a matrix instruction is valid only
// for tile shapes, layouts and hardware that fit it).  On sm_100a the
// intrinsic is tcgen05.mma with the accumulator in tensor memory (TMEM); the
// table's wgmma does not exist on this architecture.
//
// One persistent CTA per SM walks a static schedule of work units
// (128 x 256 output tile, optional K split).  Warp roles:
//   warp 0      TMA producer: per k-block (64 deep) loads the A box and the B
//               box(es) into a 4-stage shared-memory ring, 128-byte swizzled
//   warp 1      MMA issuer: owns TMEM (512 columns = two 128x256 fp32
//               accumulators); one lane issues 4 tcgen05.mma (K = 16 each) per
//               k-block and commits to the stage's "empty" barrier; after the
//               last k-block commits to the accumulator's "full" barrier
//   warps 2..5  epilogue: tcgen05.ld the accumulator (each warp its 32 TMEM
//               lanes), round to bf16 if asked, stage 32-row x 128-byte blocks
//               in swizzled shared memory, then TMA-store them (aligned C) or
//               copy them out with coalesced masked stores (any C); the double
//               buffered accumulator lets this overlap the next tile's MMAs
//   warps 6..9  only when A or B breaks TMA's alignment rules: generic-proxy
//               producers that gather the operands with masked loads into the
//               same swizzled layout and fence them towards the async proxy
// Split-K (few tiles, long K): each unit writes an fp32 partial tile to the
// workspace; the last unit to arrive per block of the tile adds the partials in
// split order (deterministic) and writes C.
// Skinny mode (M <= 64, the decode-like weight-streaming shape): the operands
// swap roles - the 256 weight columns of the tile become the 2 x 128 MMA rows
// (TMEM lanes) and the few activation rows become the MMA's N (16..64).  All
// four epilogue warps then hold useful lanes, a lane's registers run over m,
// and stores are coalesced along n straight from registers.  With M <= 32 the
// K splits of a tile form a thread-block cluster and reduce through distributed
// shared memory instead of the global workspace: every CTA sends each 32-column
// block of its partial tile to the block's owner CTA (plain st.shared::cluster),
// one cluster barrier, and each owner adds the partials in rank order and stores
// its columns of C.  No atomics, no round trip through L2.
//
// Every barrier wait is bounded; on expiry the CTA records an error, stops
// issuing work, lets its copies drain, frees TMEM and returns.
#include "../../include/klineage_gemm.h"
#include "common.cuh"
#include "ptx.cuh"
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#ifdef KLIN_TRACE
static __device__ unsigned long long klin_trace_single[klin::kTraceSlots * klin::kTraceCtas];
#define KLIN_TRACE_BUF klin_trace_single
extern "C" int klin_trace_dump_single(unsigned long long* host)
{
    cudaDeviceSynchronize();
    const cudaError_t e = cudaMemcpyFromSymbol(host, klin_trace_single, sizeof klin_trace_single);
    void* dev = nullptr;
    if (cudaGetSymbolAddress(&dev, klin_trace_single) == cudaSuccess) cudaMemset(dev, 0, sizeof klin_trace_single);
    return static_cast<int>(e);
}
static __device__ int klin_trace_knob;      // experiments: MMAs issued per k-block (0 = all four)
extern "C" int klin_trace_set_knob(int v)
{
    return static_cast<int>(cudaMemcpyToSymbol(klin_trace_knob, &v, sizeof v));
}
#define KLIN_TNS(slot)                                                                             \
    do {                                                                                           \
        unsigned long long ns_;                                                                    \
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns_));                                    \
        if (blockIdx.x < klin::kTraceCtas) KLIN_TRACE_BUF[blockIdx.x * klin::kTraceSlots + (slot)] = ns_; \
    } while (0)
#else
#define KLIN_TNS(slot) ((void)0)
#endif

namespace klin {
namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4;
constexpr int kABytes = BM * BK * 2;              // 16 KiB
constexpr int kBBytes = BN * BK * 2;              // 32 KiB
constexpr int kStageBytes = kABytes + kBBytes;    // 48 KiB
// Conv2d by TMA with at most 128 filters: a stage is a 16 KiB patch box plus a 16 KiB filter block, so the ring
// area holds six stages instead of four (their barriers live in the grouped schedule's space, unused in that mode).
constexpr int kConvFilterBytes = (BN / 2) * BK * 2;                                  // 16 KiB
constexpr int kConvStageBytes = kABytes + kConvFilterBytes;                          // 32 KiB
constexpr int kConvStages = 6;
constexpr int kMaxStages = 8;                     // deepest ring (24 KiB stages of 64-column tiles; 6 x 32 KiB with 128 columns)
static_assert(kConvStages * kConvStageBytes <= STAGES * kStageBytes, "conv ring exceeds the ring area");
constexpr int kEpiBufBytes = 32 * 128;            // one 32-row x 128-byte staging block
constexpr int kEpiBytes = 4 * 2 * kEpiBufBytes;   // 4 warps x 2 buffers
constexpr int kBarBytes = 1536;                   // barriers, TMEM slot, abort flag, grouped schedule (<= 257 ints)
constexpr int kSmemBytes = 1024 + STAGES * kStageBytes + kEpiBytes + kBarBytes;
constexpr int kTmemCols = 512;
constexpr int kThreadsTma = 6 * 32, kThreadsGeneric = 10 * 32;
constexpr int kProducerThreads = 128;

struct R4Params {
    int tiles_m, tiles_n;
    int splits, kb_per_split, nkb;
    int epi_tma;            // 1: TMA-store epilogue, 0: coalesced masked stores
    int kid;
    float* ws;              // split-K partials [split][M][ldw]
    int64_t ldw;
    unsigned* counters;     // [tile * 4 + row block], zero between launches
    uint32_t idesc;
    uint32_t b_desc_hi, b_desc_lbo, b_kstep;   // B operand descriptor pieces (depend on the layout of B)
    int n_mma;              // skinny mode: M rounded up to 16 = the MMA's N
    uint32_t stage_tx;      // bytes one stage's TMA loads deliver (A box + B boxes)
    int cluster;            // 1: the splits of a tile are one cluster and reduce through DSMEM
    int splits_log2;        // cluster mode: splits is 2, 4 or 8
    int b_box3d;            // row-major B whose four 64-column blocks of a stage arrive as ONE 3-D box
    int static_b;           // the caller promised static B: the first ring fill's B boxes go out before the dependency wait
    int group_m;            // tile raster: tile-rows per group
    int64_t full_units;     // units [0, full_units) are whole tiles; later ones are 128-column half tiles
    int64_t total_units;
    uint32_t idesc_half;    // instruction descriptor for a half tile (N = 128)
    // several problems in one launch (MODE 1: batched over 3-D tensor maps; MODE 2: grouped, a
    // table of per-group tensor maps and sizes in device memory); never combined with a K split
    int tiles_per_batch;
    int64_t stride_c_bytes;
    const GroupEntry* groups;
    int n_groups;
    // MODE 3: one problem, every output block stored to each entry of a destination table
    const DstEntry* dsts;
    int n_dst;
    // MODE 4: Conv2d as an implicit GEMM (the A producers gather input patches)
    ConvGeom conv;
    int conv_fast;          // 1: C % 8 == 0 and x 16-byte aligned - an 8-k chunk is one 16-byte load
    int half_only;          // every unit is the first 128-column half of its tile (problems with N <= 128)
    int one_wave;           // whole unsplit tiles, at most one per CTA: unit u is tile (u / tiles_n, u % tiles_n)
    int conv_ring6;         // Conv2d by TMA, F <= 128: six 32 KiB stages with their own barriers and a lean producer loop
    int conv_t;             // Conv2d by TMA, F <= 128, transposed: filters are the 128-row MMA operand, a unit is TWO patch
                            // tiles (256 pixels as the N operand: full-width MMAs), the epilogue stores y transposed
    int conv_nimg;          // images (conv_t: a unit's second patch tile may lie past the last image)
    int conv_b_tma;         // MODE 4: the weights come by TMA (warp 0), only the patches are gathered
    int conv_b_rows;        // rows of the weight box (128 with half_only, else 256)
    int conv_patch;         // patches by TMA: row tile t = 8 x 16 output patch (t % tq, (t / tq) % tp) of image t / (tq tp)
    int conv_tq, conv_tp;
    // Give-up test hook (KLINEAGE_FLAG_TEST_GIVE_UP, one launch): the TMA producer stops after this many k-blocks
    // and the MMA issuer's wait for the next operand stage runs out after test_poll_limit polls, so that the
    // kernel's give-up path - error word, abort flag, every role leaving its loop, TMEM freed - really runs.
    int test_stop_after;
    uint32_t test_poll_limit;
    // Tile width and ring depth (MODE 0, TMA-fed, regular orientation; every other form runs 256 columns and 4
    // stages): 256 columns with four 48 KiB stages, or 128 / 64 columns with four or six 32 / 24 KiB stages.
    int tile_n;
    int kpair;              // 1: a stage holds TWO 64-deep k-blocks (one barrier round trip per eight MMAs); nkb counts such pairs
    int n_stages;
    uint32_t stage_bytes;
};

// One entry of the static schedule.
struct Unit {
    int64_t tile;
    int m0, n0;             // first row / column of C it computes
    int ncols;              // 256, or 128 for the half tiles that fill the last wave
    int split, kb0, kb1;    // K split index and k-block range
    // the problem the unit belongs to (MODE 1 / 2 only)
    int M, N, z, epi_tma;
    const CUtensorMap *ma, *mb, *mc;
    uint8_t* C;
    int64_t ldc;
};
// MODE 1 / 2: a launch-wide tile index -> its problem and its (tile_m, tile_n) there.
template <int MODE>
__device__ __forceinline__ void decode_multi(Unit& x, const GemmArgs& g, const R4Params& p, const int* gstart, int& hint)
{
    int tm, tn;
    if (MODE == 2) {
        const int ti = static_cast<int>(x.tile);
        int gi = hint;
        while (gstart[gi + 1] <= ti) ++gi;                  // gstart[n_groups] = number of tiles > ti
        hint = gi;
        const GroupEntry* e = p.groups + gi;
        x.M = e->M;
        x.N = e->N;
        x.z = 0;
        x.epi_tma = e->epi_tma;
        x.ma = &e->map_a;
        x.mb = &e->map_b;
        x.mc = &e->map_c;
        x.C = static_cast<uint8_t*>(e->C);
        x.ldc = e->ldc;
        x.kb0 = 0;
        x.kb1 = e->nkb;
        raster_tile(ti - gstart[gi], e->tiles_m, e->tiles_n, tm, tn, p.group_m);
    } else {
        const uint32_t t32 = static_cast<uint32_t>(x.tile), tpb = static_cast<uint32_t>(p.tiles_per_batch);
        const uint32_t b = t32 / tpb;
        x.M = g.M;
        x.N = g.N;
        x.z = static_cast<int>(b);
        x.epi_tma = p.epi_tma;
        x.C = static_cast<uint8_t*>(g.C) + static_cast<int64_t>(b) * p.stride_c_bytes;
        x.ldc = g.ldc;
        x.kb0 = 0;
        x.kb1 = p.nkb;
        raster_tile(t32 - b * tpb, p.tiles_m, p.tiles_n, tm, tn, p.group_m);
    }
    x.m0 = tm * BM;
    x.n0 = tn * BN;
}
__device__ __forceinline__ Unit decode_unit(int64_t u, const R4Params& p)
{
    Unit x;
    int half = 0;
    const int tile_n = p.tile_n;
    x.ncols = tile_n;
    if (p.one_wave) {
        // One wave of whole tiles: the order they are dealt in does not matter, so the unit decodes with one 32-bit
        // division (this arithmetic is the first thing every role runs: cold code on the critical path of short kernels).
        const uint32_t u32 = static_cast<uint32_t>(u), tn_count = static_cast<uint32_t>(p.tiles_n);
        const uint32_t tm = u32 / tn_count, tn = u32 - tm * tn_count;
        x.tile = u;
        x.split = 0;
        x.m0 = static_cast<int>(tm) * BM;
        x.n0 = static_cast<int>(tn) * tile_n;
        x.kb0 = 0;
        x.kb1 = p.nkb;
        return x;
    }
    if (p.cluster) {              // splits is a power of two: no division on the critical path of short kernels
        x.tile = u >> p.splits_log2;
        x.split = static_cast<int>(u & (p.splits - 1));
    } else if (p.splits > 1) {
        if (u < 0x7FFFFFFFll) {   // 32-bit division: this sits on the critical path of short kernels
            const uint32_t u32 = static_cast<uint32_t>(u), sp = static_cast<uint32_t>(p.splits);
            x.tile = u32 / sp;
            x.split = static_cast<int>(u32 - static_cast<uint32_t>(x.tile) * sp);
        } else {
            x.tile = u / p.splits;
            x.split = static_cast<int>(u % p.splits);
        }
    } else {
        x.split = 0;
        if (p.half_only) {
            x.tile = u;
            x.ncols = tile_n / 2;
        } else if (u < p.full_units) {
            x.tile = u;
        } else {
            const int64_t v = u - p.full_units;
            x.tile = p.full_units + (v >> 1);
            half = static_cast<int>(v & 1);
            x.ncols = tile_n / 2;
        }
    }
    int tm, tn;
    raster_tile(x.tile, p.tiles_m, p.tiles_n, tm, tn, p.group_m);
    x.m0 = tm * BM;
    x.n0 = tn * tile_n + half * (tile_n / 2);
    x.kb0 = x.split * p.kb_per_split;
    x.kb1 = min(p.nkb, x.kb0 + p.kb_per_split);
    return x;
}

// 64-bit shared-memory matrix descriptor: start address, leading / stride byte
// offsets (all >> 4), descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    const uint32_t lo = ((smem_addr >> 4) & 0x3FFFu) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
    const uint32_t hi = ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
    return (static_cast<uint64_t>(hi) << 32) | lo;
}

// 8 consecutive bf16 starting at p, `valid` of them in range, as one 16-byte chunk.
__device__ __forceinline__ uint4 gather8(const uint16_t* p, int valid)
{
    if (valid >= 8 && (reinterpret_cast<uintptr_t>(p) & 15) == 0) return __ldg(reinterpret_cast<const uint4*>(p));
    uint16_t v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = (e < valid) ? __ldg(p + e) : uint16_t(0);
    uint4 r;
    r.x = v[0] | (uint32_t(v[1]) << 16);
    r.y = v[2] | (uint32_t(v[3]) << 16);
    r.z = v[4] | (uint32_t(v[5]) << 16);
    r.w = v[6] | (uint32_t(v[7]) << 16);
    return r;
}

template <bool BCOL, bool GENERIC, bool SWAP, int MODE>
__global__ void __launch_bounds__(GENERIC ? kThreadsGeneric : kThreadsTma, 1)
r4_tcgen05_kernel(GemmArgs g, const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const __grid_constant__ CUtensorMap map_c, R4Params p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* epi_smem = smem + STAGES * kStageBytes;
    uint64_t* full = reinterpret_cast<uint64_t*>(epi_smem + kEpiBytes);
    uint64_t* empty = full + kMaxStages;
    uint64_t* acc_full = empty + kMaxStages;
    uint64_t* acc_empty = acc_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
    volatile uint32_t* abort_flag = tmem_slot + 1;   // [0] raised on give-up, [1] stays 0
    int* gstart = reinterpret_cast<int*>(const_cast<uint32_t*>(abort_flag) + 2);   // MODE 2: first tile of every group
    // MODE 4 with the six-stage ring: its full / empty barriers (the group table's space is free there)
    uint64_t* cfull = reinterpret_cast<uint64_t*>((reinterpret_cast<uintptr_t>(gstart) + 7) & ~uintptr_t(7));
    uint64_t* cempty = cfull + kConvStages;
    const bool ring6 = MODE == 4 && !GENERIC && p.conv_ring6;
    // Ring geometry: a parameter of the plain TMA-fed GEMM only, the constants everywhere else
    constexpr bool kTunable = MODE == 0 && !GENERIC && !SWAP;
    const uint32_t NS = kTunable ? static_cast<uint32_t>(p.n_stages) : static_cast<uint32_t>(STAGES);
    const uint32_t SB = kTunable ? p.stage_bytes : static_cast<uint32_t>(kStageBytes);
    const int TN = kTunable ? p.tile_n : BN;
    // Narrow tiles may pair their k-blocks: a stage is two sub-stages of the usual layout, 64 k each, filled and freed
    // together.  The issuing thread spends ~350 clocks per barrier round trip (probe, commit, descriptor step) on top
    // of ~85 per MMA; with eight MMAs per round trip instead of four a k-block of 64 costs ~515 clocks instead of ~690.
    const int NSUB = (kTunable && p.kpair) ? 2 : 1;
    const uint32_t SUB = SB / static_cast<uint32_t>(NSUB);          // bytes of a sub-stage
    // (Measured: a tcgen05.mma of this kernel issues every ~159 clocks whatever its N - 64, 128 or 256 - and
    // whether or not consecutive ones share an accumulator: letting a narrow tile's k-steps alternate between
    // two or four accumulators, summed by the epilogue, left the main loop at 636 clocks per k-block and only made
    // the epilogue longer.  What a narrow tile buys is a shorter epilogue and more CTAs, not cheaper MMAs.)
    int group_hint = 0;     // MODE 2: a thread's units come in increasing order; its group search resumes here
    // One unit of the schedule for this thread's role.
    auto unit_of = [&](int64_t u) {
        Unit x = decode_unit(u, p);
        if (MODE == 1 || MODE == 2) {
            const int half_cols = x.n0 % BN;                // 0, or 128 for the second half tile
            decode_multi<MODE>(x, g, p, gstart, group_hint);
            x.n0 += half_cols;
        } else {
            x.M = g.M;
            x.N = g.N;
            x.z = 0;
            x.epi_tma = p.epi_tma;
            x.ma = &map_a;
            x.mb = &map_b;
            x.mc = &map_c;
            x.C = static_cast<uint8_t*>(g.C);
            x.ldc = g.ldc;
        }
        if (MODE == 1) {
            x.ma = &map_a;
            x.mb = &map_b;
            x.mc = &map_c;
        }
        return x;
    };

    // (the warp index by a broadcast: the compiler then knows it, and every role branch, to be uniform across the warp)
    const int warp = __shfl_sync(0xFFFFFFFFu, static_cast<int>(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    // Cluster mode: no CTA may touch a peer's shared memory before that peer runs and has initialised the barrier
    // its incoming partial sums are counted on (warp 0 arrives after it has done that, below).
    if (SWAP && p.cluster && warp != 0) ptx::cluster_arrive_relaxed();
    uint64_t* xchg_bar = cfull;      // skinny cluster mode only (the six-stage ring's barriers are another mode's)
    const int64_t total_units = p.total_units;

    // TMA producer state (used by warp 0, lane 0 only): position in the static schedule.
    struct {
        int64_t u;
        int kb, kb1, m0, n0, z;
        const CUtensorMap *ma, *mb;
        uint32_t it;
        bool live;
        int cw, ch, cn;                 // MODE 4 on TMA: input origin (w, h) and image of the tile's 8 x 16 pixel patch
        uint32_t st, ph;                // ring stage of load `it` and the parity its "empty" barrier is waited with
    } prod = {static_cast<int64_t>(blockIdx.x), 0, 0, 0, 0, 0, &map_a, &map_b, 0u, false, 0, 0, 0, 0u, 1u};
    auto prod_enter_unit = [&]() {
        prod.live = prod.u < total_units;
        if (!prod.live) return;
        const Unit x = unit_of(prod.u);
        prod.kb = x.kb0;
        prod.kb1 = x.kb1;
        prod.m0 = x.m0;
        prod.n0 = x.n0;     // a half tile still loads 256 columns from n0; its MMA reads the first 128
        if (MODE == 1 || MODE == 2) {
            prod.z = x.z;
            prod.ma = x.ma;
            prod.mb = x.mb;
        }
        if (MODE == 4 && !GENERIC) {
            // patch tiling: row tile t of the launch is the 8 x 16 output patch (pt, qt) of image n
            const int t = x.m0 / BM;
            const int qt = t % p.conv_tq, u2 = t / p.conv_tq;
            prod.cw = qt * 16 - p.conv.pad_w;
            prod.ch = (u2 % p.conv_tp) * 8 - p.conv.pad_h;
            prod.cn = u2 / p.conv_tp;
        }
    };
    auto load_box = [&](void* dst, const CUtensorMap* map, int c0, int c1, uint64_t* bar) {
        if (MODE == 1)
            ptx::tma_load_3d(dst, map, c0, c1, prod.z, bar);
        else
            ptx::tma_load_2d(dst, map, c0, c1, bar);
    };
    // The expect-tx arrive and the loads of one stage: k-block kb of the tile at (m0, n0) of the producer's unit.
    auto stage_loads = [&](uint32_t s, int kb_stage, int m0, int n0) {
        ptx::mbar_arrive_expect_tx(&full[s], p.stage_tx);
        const CUtensorMap* pa = (MODE == 2) ? prod.ma : &map_a;
        const CUtensorMap* pb = (MODE == 2) ? prod.mb : &map_b;
        // the loads of one 64-deep (sub-)stage: k-block kb into the sub-stage at sa
        auto sub_loads = [&](int kb, uint8_t* sa) {
            uint8_t* sb = sa + kABytes;
            if (MODE == 4) {
                // Conv2d: k-block = (filter tap, 64-channel group); the A stage is ONE box of 64 channels
                // x 16 x 8 pixels (the tile's output patch shifted by the tap) - where it leaves the
                // image the TMA unit fills zeros, which is the padding.  GEMM row = 16 * patch row + column.
                const int cpb = p.conv.C >> 6;
                const int tap = kb / cpb, cg = kb - tap * cpb;
                const int fr = tap / p.conv.S, fs = tap - fr * p.conv.S;
                ptx::tma_load_4d(sa, &map_a, cg * 64, prod.cw + fs, prod.ch + fr, prod.cn, &full[s]);
            } else
                load_box(sa, pa, kb * BK, m0, &full[s]);
            if (BCOL) {
                load_box(sb, pb, kb * BK, n0, &full[s]);
            } else if (MODE == 1 && p.b_box3d) {
                ptx::tma_load_4d(sb, pb, 0, kb * BK, n0 >> 6, prod.z, &full[s]);   // the same box, batch as 4th coordinate
            } else if ((MODE == 0 || MODE == 3) && p.b_box3d) {
                // B viewed as (64 columns, K rows, N / 64 column blocks): one box of 64 x 64 x 4 lands as the
                // four consecutive 8 KiB blocks the MN-major descriptor expects - one TMA instruction, not four
                // (a producer thread issues a TMA instruction every ~110 cycles)
                ptx::tma_load_3d(sb, pb, 0, kb * BK, n0 >> 6, &full[s]);
            } else {
#pragma unroll
                for (int cb = 0; cb < BN / 64; ++cb)
                    if (cb * 64 < TN) load_box(sb + cb * (64 * BK * 2), pb, n0 + cb * 64, kb * BK, &full[s]);
            }
        };
        if (kTunable && NSUB == 2) {
            // (a sub-stage past the end of K reads zeros: out-of-range boxes are filled, and its MMAs add nothing)
            sub_loads(2 * kb_stage, smem + s * SB);
            sub_loads(2 * kb_stage + 1, smem + s * SB + SUB);
        } else {
            sub_loads(kb_stage, smem + s * SB);
        }
    };
    // Issues loads until `limit` k-blocks have been issued in total or the schedule ends.
    auto produce = [&](uint32_t limit) {
        while (prod.live && prod.it < limit) {
            const uint32_t it = prod.it;
            if (p.test_stop_after > 0 && it == static_cast<uint32_t>(p.test_stop_after)) {   // test hook: a stage never arrives
                prod.live = false;
                break;
            }
            const uint32_t s = prod.st;
            if (!ptx::mbar_wait(&empty[s], prod.ph, abort_flag)) {
                report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x400u | s);
                abort_flag[0] = 1;
                prod.live = false;
                break;
            }
            stage_loads(s, prod.kb, prod.m0, prod.n0);
            ++prod.it;
            if (++prod.st == NS) {
                prod.st = 0;
                prod.ph ^= 1u;
            }
            if (++prod.kb == prod.kb1) {
                prod.u += gridDim.x;
                prod_enter_unit();
            }
        }
    };

    // The rest of the schedule after the first ring fill, for the TMA-fed GEMM forms: the ring position is carried in
    // registers and a unit's k-blocks run in a loop of their own - wait, expect-tx arrive, loads, nothing else.  (Short
    // k-blocks are bound by the round trip "stage freed -> loads issued -> data landed", about 2 k clocks of TMA
    // latency under load plus this thread's own instruction stream: the general loop above spent 500 clocks per
    // stage on itself.)
    auto produce_rest = [&]() {
        uint32_t st = prod.st, ph = prod.ph, it = prod.it;
        const uint32_t empty0 = ptx::smem_u32(empty);
        while (prod.live) {
            const int m0 = prod.m0, n0 = prod.n0, kb1 = prod.kb1;
            for (int kb = prod.kb; kb < kb1; ++kb, ++it) {
                if (it == 8) KLIN_T(20);
                if (it == 9) KLIN_T(23);
                if (!ptx::mbar_wait_addr(empty0 + 8 * st, ph, abort_flag)) {
                    report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x400u | st);
                    abort_flag[0] = 1;
                    prod.live = false;
                    break;
                }
                if (it == 8) KLIN_T(21);
                if (it == 9) KLIN_T(24);
                const uint32_t st_next = (st + 1 == NS) ? 0u : st + 1, ph_next = (st + 1 == NS) ? ph ^ 1u : ph;
                stage_loads(st, kb, m0, n0);
                if (it == 8) KLIN_T(22);
                if (it == 9) KLIN_T(25);
                st = st_next;
                ph = ph_next;
            }
            if (!prod.live) break;
            prod.u += gridDim.x;
            prod_enter_unit();
        }
        prod.it = it;
    };

    // Set-up.  In the TMA-fed GEMM forms warp 0 does not wait for the other warps: it initialises the barriers,
    // signals (a named barrier the others wait on) and goes straight on to the first ring fill, while warp 1
    // allocates TMEM and the MMA and epilogue threads work out their first unit.  (The fill used to come before a
    // CTA-wide barrier that every warp waited on: on 256^3 the first MMA was issued 4.9 k clocks after the CTA's
    // start, 2.2 k of them spent issuing four stages of loads one after the other.)
    constexpr bool kEarlyProducer = !GENERIC && (MODE == 0 || MODE == 1 || MODE == 3);
    // The first ring fill in one pass of the instruction stream: lane l issues stage l (plain GEMM forms).
    constexpr bool kLockstepFill = !GENERIC && (MODE == 0 || MODE == 3);
    if (warp == 0) {
        if (lane == 0) {
            KLIN_T(0);
            KLIN_TNS(6);
            for (uint32_t s = 0; s < NS; ++s) {
                ptx::mbar_init(&full[s], GENERIC ? kProducerThreads + ((MODE == 4 && p.conv_b_tma) ? 1 : 0) : 1);
                ptx::mbar_init(&empty[s], 1);
            }
            for (int b = 0; b < 2; ++b) {
                ptx::mbar_init(&acc_full[b], 1);
                ptx::mbar_init(&acc_empty[b], 4);
            }
            if (ring6)
                for (int i = 0; i < 2 * kConvStages; ++i) ptx::mbar_init(&cfull[i], 1);
            abort_flag[0] = 0;
            abort_flag[1] = 0;
            if (SWAP && p.cluster) ptx::mbar_init(xchg_bar, 1);
            ptx::fence_barrier_init();
            if (!GENERIC && MODE != 2) {
                ptx::prefetch_tensormap(&map_a);
                ptx::prefetch_tensormap(&map_b);
            }
            if (p.epi_tma && MODE != 2 && MODE != 3) ptx::prefetch_tensormap(&map_c);
            KLIN_T(1);
        }
        if (SWAP && p.cluster) {
            __syncwarp();
            ptx::cluster_arrive_relaxed();
        }
        if (kEarlyProducer) {
            __syncwarp();
            ptx::named_barrier_arrive(1, blockDim.x);
        }
        // The launch is a programmatic dependent one: everything above (and the TMEM
        // allocation in warp 1) may overlap the tail of the previous kernel in the stream;
        // nothing below the wait touches global memory before that kernel has completed.
        if (lane == 0 && !GENERIC && MODE != 2) prod_enter_unit();           // schedule arithmetic only
        if (lane == 0) KLIN_T(2);
        const bool lockstep = kLockstepFill && !ring6 && !p.static_b && p.test_stop_after == 0;
        if (lockstep) {
            const int kb = __shfl_sync(0xFFFFFFFFu, prod.kb, 0), kb1 = __shfl_sync(0xFFFFFFFFu, prod.kb1, 0);
            const int m0 = __shfl_sync(0xFFFFFFFFu, prod.m0, 0), n0 = __shfl_sync(0xFFFFFFFFu, prod.n0, 0);
            const int live = __shfl_sync(0xFFFFFFFFu, prod.live ? 1 : 0, 0);
            const int nfill = live ? min(static_cast<int>(NS), kb1 - kb) : 0;
            ptx::grid_dependency_wait();
            if (lane == 0) KLIN_T(3);
            // (the "empty" barriers are fresh: the first NS loads wait for nothing)
            if (lane < nfill) stage_loads(static_cast<uint32_t>(lane), kb + lane, m0, n0);
            __syncwarp();
            if (lane == 0 && nfill > 0) {
                prod.it = static_cast<uint32_t>(nfill);
                if (static_cast<uint32_t>(nfill) == NS) {
                    prod.st = 0;
                    prod.ph ^= 1u;
                } else {
                    prod.st = static_cast<uint32_t>(nfill);
                }
                prod.kb += nfill;
                if (prod.kb == prod.kb1) {
                    prod.u += gridDim.x;
                    prod_enter_unit();
                }
            }
            if (lane == 0) KLIN_T(4);
        } else if (lane == 0) {
        if (!GENERIC && MODE == 0 && p.static_b && prod.live && prod.kb1 - prod.kb >= STAGES) {
            // Static B: the B boxes of the first ring fill do not depend on the previous kernel in
            // the stream and go out at once; only A waits (C is written much later, after the wait
            // that every thread passes below).  The fresh "empty" barriers need no wait.
            for (int s = 0; s < STAGES; ++s) {
                uint8_t* sb = smem + s * kStageBytes + kABytes;
                const int kb = prod.kb + s;
                ptx::mbar_arrive_expect_tx(&full[s], p.stage_tx);
                if (BCOL) {
                    ptx::tma_load_2d(sb, &map_b, kb * BK, prod.n0, &full[s]);
                } else {
#pragma unroll
                    for (int cb = 0; cb < BN / 64; ++cb)
                        ptx::tma_load_2d(sb + cb * (64 * BK * 2), &map_b, prod.n0 + cb * 64, kb * BK, &full[s]);
                }
            }
            ptx::grid_dependency_wait();
            for (int s = 0; s < STAGES; ++s)
                ptx::tma_load_2d(smem + s * kStageBytes, &map_a, (prod.kb + s) * BK, prod.m0, &full[s]);
            prod.it = STAGES;          // (the host grants this path to the 4-stage, 256-column form only)
            prod.st = 0;
            prod.ph ^= 1u;
            prod.kb += STAGES;
            if (prod.kb == prod.kb1) {
                prod.u += gridDim.x;
                prod_enter_unit();
            }
        } else {
            ptx::grid_dependency_wait();
            KLIN_T(3);
            if (!GENERIC && MODE != 2) {
                // The first ring fill needs nothing from the other warps: start it before the
                // set-up barrier so that TMEM allocation hides behind the first loads' latency.
                if (!ring6 && !(MODE == 4 && p.conv_t)) produce(NS);
            }
            KLIN_T(4);
        }
        }
        if (lane == 0 && blockIdx.x == 0) g.status[1] = p.kid;
    }
    if (MODE == 2 && warp >= 2) {
        // the grouped schedule's prefix sums (written on the stream before this launch)
        ptx::grid_dependency_wait();
        for (int i = static_cast<int>(threadIdx.x) - 64; i <= p.n_groups; i += blockDim.x - 64)
            gstart[i] = (i < p.n_groups) ? p.groups[i].tile_start : static_cast<int>(p.full_units + (p.total_units - p.full_units) / 2);
    }
    if (warp == 1) {
        ptx::tmem_alloc(tmem_slot, kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    if (threadIdx.x == 32) KLIN_T(16);
    if (kEarlyProducer) {
        if (warp != 0) ptx::named_barrier_sync(1, blockDim.x);
    } else {
        __syncthreads();
    }
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    if (threadIdx.x == 0) KLIN_T(5);
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();
    if (SWAP && p.cluster) ptx::cluster_wait_acquire();
    // Cluster mode: what the final reduce needs, computed now, off the kernel's tail.
    const int fin_rank = (SWAP && p.cluster) ? static_cast<int>(blockIdx.x & static_cast<unsigned>(p.splits - 1)) : 0;
    const int fin_n0 = (SWAP && p.cluster) ? static_cast<int>(blockIdx.x >> p.splits_log2) * BN : 0;
    const float* fin_slots = reinterpret_cast<const float*>(epi_smem) + lane * 4;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (MODE == 4 && !GENERIC && p.conv_t && lane == 0) {
            // Conv2d, transposed orientation: per k-block the filter block goes to the 16 KiB slot of the 128-row
            // operand and the patch boxes of the unit's two patch tiles to the two halves of the 256-row slot
            // (a tile past the last image reads zeros: out-of-range coordinates).  Lean loop as below.
            const uint32_t ring0 = ptx::smem_u32(smem), full0 = ptx::smem_u32(full), empty0 = ptx::smem_u32(empty);
            const int cpb = p.conv.C >> 6, fS = p.conv.S, nkb = p.nkb, tq = p.conv_tq, tp = p.conv_tp;
            uint32_t st = 0, ph = 1;
            while (prod.live) {
                int cw[2], ch[2], cn[2];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int t = 2 * (prod.m0 / BM) + h;
                    const int qt = t % tq, u2 = t / tq;
                    cw[h] = qt * 16 - p.conv.pad_w;
                    ch[h] = (u2 % tp) * 8 - p.conv.pad_h;
                    cn[h] = u2 / tp;
                }
                int cg = 0, fs = 0, fr = 0;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!ptx::mbar_wait_addr(empty0 + 8 * st, ph, abort_flag)) {
                        report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x470u | st);
                        abort_flag[0] = 1;
                        prod.live = false;
                        break;
                    }
                    const uint32_t dst = ring0 + st * kStageBytes, bar = full0 + 8 * st;
                    ptx::mbar_arrive_expect_tx_addr(bar, static_cast<uint32_t>(kStageBytes));
                    ptx::tma_load_2d_addr(dst, &map_b, kb * BK, 0, bar);
                    ptx::tma_load_4d_addr(dst + kABytes, &map_a, cg * 64, cw[0] + fs, ch[0] + fr, cn[0], bar);
                    ptx::tma_load_4d_addr(dst + kABytes + kABytes, &map_a, cg * 64, cw[1] + fs, ch[1] + fr, cn[1], bar);
                    if (++cg == cpb) {
                        cg = 0;
                        if (++fs == fS) {
                            fs = 0;
                            ++fr;
                        }
                    }
                    if (++st == STAGES) {
                        st = 0;
                        ph ^= 1u;
                    }
                    ++prod.it;
                }
                if (!prod.live) break;
                prod.u += gridDim.x;
                prod_enter_unit();
            }
            const uint32_t it = prod.it;
            const uint32_t first = it > STAGES ? it - STAGES : 0;
            for (uint32_t j = first; j < it; ++j) ptx::mbar_wait(&full[j % STAGES], (j / STAGES) & 1, abort_flag + 1);
        } else if (ring6 && lane == 0) {
            // Conv2d, six-stage ring.  With k-blocks this short (four N = 128 MMAs) the producer's own instruction
            // stream bounds the kernel, so this loop carries everything it needs instead of deriving it: stage
            // addresses and parity, the tap (fr, fs) and channel group of the k-block, all by increments.
            const uint32_t ring0 = ptx::smem_u32(smem), cfull0 = ptx::smem_u32(cfull), cempty0 = ptx::smem_u32(cempty);
            const int cpb = p.conv.C >> 6, fS = p.conv.S, nkb = p.nkb;
            uint32_t st = 0, ph = 1;                  // stage and the parity its "empty" barrier is waited with
            while (prod.live) {
                const int cw = prod.cw, ch = prod.ch, cn = prod.cn, n0 = prod.n0;
                int cg = 0, fs = 0, fr = 0;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!ptx::mbar_wait_addr(cempty0 + 8 * st, ph, abort_flag)) {
                        report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x460u | st);
                        abort_flag[0] = 1;
                        prod.live = false;
                        break;
                    }
                    const uint32_t dst = ring0 + st * kConvStageBytes, bar = cfull0 + 8 * st;
                    ptx::mbar_arrive_expect_tx_addr(bar, static_cast<uint32_t>(kConvStageBytes));
                    ptx::tma_load_4d_addr(dst, &map_a, cg * 64, cw + fs, ch + fr, cn, bar);
                    ptx::tma_load_2d_addr(dst + kABytes, &map_b, kb * BK, n0, bar);
                    if (++cg == cpb) {
                        cg = 0;
                        if (++fs == fS) {
                            fs = 0;
                            ++fr;
                        }
                    }
                    if (++st == kConvStages) {
                        st = 0;
                        ph ^= 1u;
                    }
                    ++prod.it;
                }
                if (!prod.live) break;
                prod.u += gridDim.x;
                prod_enter_unit();
            }
            // Drain: every load issued must have landed before shared memory is released.
            const uint32_t it = prod.it;
            const uint32_t first = it > kConvStages ? it - kConvStages : 0;
            for (uint32_t j = first; j < it; ++j)
                ptx::mbar_wait(&cfull[j % kConvStages], (j / kConvStages) & 1, abort_flag + 1);
        } else if (!GENERIC && lane == 0) {
            if (MODE == 2) prod_enter_unit();      // (its group search reads the table the other warps just staged)
            if (MODE == 4 || p.test_stop_after > 0)
                produce(0xFFFFFFFFu);
            else
                produce_rest();
            // Drain: every load issued must have landed before shared memory is released.
            const uint32_t it = prod.it;
            const uint32_t first = it > NS ? it - NS : 0;
            for (uint32_t j = first; j < it; ++j) ptx::mbar_wait(&full[j % NS], (j / NS) & 1, abort_flag + 1);
        }
        if (GENERIC && MODE == 4 && lane == 0 && p.conv_b_tma) {
            // Conv2d: the filter block of every k-block by TMA (the patches come from warps 6..9)
            uint32_t it = 0;
            bool ok = true;
            for (int64_t u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
                const Unit x = decode_unit(u, p);
                for (int kb = x.kb0; kb < x.kb1; ++kb, ++it) {
                    const int s = it % STAGES;
                    if (!ptx::mbar_wait(&empty[s], ((it / STAGES) & 1) ^ 1, abort_flag)) {
                        report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x450u | s);
                        abort_flag[0] = 1;
                        ok = false;
                        break;
                    }
                    ptx::mbar_arrive_expect_tx(&full[s], static_cast<uint32_t>(p.conv_b_rows) * 128u);
                    ptx::tma_load_2d(smem + s * kStageBytes + kABytes, &map_b, kb * BK, x.n0, &full[s]);
                }
            }
            const uint32_t first = it > STAGES ? it - STAGES : 0;
            for (uint32_t j = first; j < it; ++j) ptx::mbar_wait(&full[j % STAGES], (j / STAGES) & 1, abort_flag + 1);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        // The whole warp walks the schedule and waits on the barriers; lane 0 alone issues the MMAs and commits.  (With
        // the loop inside a one-lane branch every descriptor is a per-thread value that has to be moved into the uniform
        // registers the MMA instruction reads, instruction by instruction; in converged code the compiler keeps ring
        // position and descriptors there from the start.)
        {
            const bool issuer = lane == 0;
            uint32_t t = 0;
            bool ok = true;
            // The ring position (stage s, phase ph) is carried instead of derived, barriers are addressed by their
            // shared-window address, and a stage's descriptors are the first stage's plus s * (stage bytes >> 4)
            // in the 14-bit start-address field (the ring ends below 256 KiB: no carry out of the field).
            // (Measured: the length of this instruction stream does not bound the kernel - trimming it changed no
            // timing, and releasing stages in pairs to halve the commits was slower, because the ring got shallower.)
            uint32_t s = 0, ph = 0;
#ifdef KLIN_TRACE
            const int trace_knob = klin_trace_knob > 0 ? klin_trace_knob : 4;
#endif
            const uint32_t full0 = ptx::smem_u32(ring6 ? cfull : full), empty0 = ptx::smem_u32(ring6 ? cempty : empty);
            const uint32_t n_stages = ring6 ? kConvStages : NS;
            const uint32_t stage_step = (ring6 ? static_cast<uint32_t>(kConvStageBytes) : SB) >> 4;
            const uint64_t a_desc0 = make_desc(ptx::smem_u32(smem), 16, 1024);
            const uint32_t a_lo0 = static_cast<uint32_t>(a_desc0), a_hi = static_cast<uint32_t>(a_desc0 >> 32);
            const uint32_t b_lo0 = (((ptx::smem_u32(smem) + kABytes) >> 4) & 0x3FFFu) | (p.b_desc_lbo << 16);
            const uint32_t b_hi = p.b_desc_hi, kstep = p.b_kstep;
            const uint32_t full_limit = p.test_poll_limit ? p.test_poll_limit : ptx::kMbarPollLimit;
            for (int64_t u = blockIdx.x; u < total_units && ok; u += gridDim.x, ++t) {
                const Unit x = unit_of(u);
                const int kb0 = x.kb0, kb1 = x.kb1;
                const uint32_t idesc = (x.ncols == TN) ? p.idesc : p.idesc_half;
                const uint32_t buf = t & 1;
                if (!ptx::mbar_wait(&acc_empty[buf], ((t >> 1) & 1) ^ 1, abort_flag)) {
                    if (issuer) {
                        report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x410u | buf);
                        abort_flag[0] = 1;
                    }
                    break;
                }
                ptx::tc_fence_after_sync();
                if (issuer && t == 0) KLIN_T(8);
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (issuer && t == 0 && kb == kb0 + 8) KLIN_T(26);
                    if (issuer && t == 0 && kb == kb0 + 9) KLIN_T(29);
                    if (!ptx::mbar_wait_addr(full0 + 8 * s, ph, abort_flag, full_limit)) {
                        if (issuer) {
                            report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x420u | s);
                            abort_flag[0] = 1;
                        }
                        ok = false;
                        break;
                    }
                    // (TMA-fed operands need no tcgen05 fence here: they were written through the async proxy, which
                    // is also how the MMA reads them.)
                    if (GENERIC) ptx::tc_fence_after_sync();
                    // (A look-ahead probe of the next stage's barrier cost this kernel's long-K launches 6 %, 63.5 -> 67.6 us
                    // at 2048 x 2048 x 8192, ahead of the MMAs and 3 % behind them: not used.)
                    const uint32_t s_next = (s + 1 == n_stages) ? 0u : s + 1, ph_next = (s + 1 == n_stages) ? ph ^ 1u : ph;
                    if (issuer && t == 0 && kb == kb0) KLIN_T(9);
                    if (issuer && t == 0 && kb == kb1 - 1) KLIN_T(10);
                    if (issuer && t == 0 && kb == kb0 + 8) KLIN_T(27);
                    if (issuer && t == 0 && kb == kb0 + 9) KLIN_T(30);
                    // the MMAs of one 64-deep (sub-)stage; `later`: not the unit's first sub-stage
                    auto issue_sub = [&](uint32_t a_lo, uint32_t b_lo, bool later) {
#pragma unroll
                        for (int k4 = 0; k4 < BK / 16; ++k4) {
#ifdef KLIN_TRACE
                            if (k4 >= trace_knob) continue;
#endif
                            // K-major operand: +32 bytes per 16 k inside the 128-byte swizzle row.
                            const uint32_t acc = (later || k4 > 0) ? 1u : 0u;
                            const uint64_t a_desc = (static_cast<uint64_t>(a_hi) << 32) | (a_lo + 2u * k4);
                            if (SWAP) {
                                // weights are the 128-row operand (two halves of the tile's 256 columns,
                                // 16 KiB apart in the stage), activations the N operand
#pragma unroll
                                for (int hh = 0; hh < 2; ++hh)
                                    ptx::umma_f16(d_tmem + hh * 128,
                                                  (static_cast<uint64_t>(b_hi) << 32) | (b_lo + hh * (16384u >> 4) + k4 * kstep),
                                                  a_desc, idesc, acc);
                            } else {
                                ptx::umma_f16(d_tmem, a_desc, (static_cast<uint64_t>(b_hi) << 32) | (b_lo + k4 * kstep), idesc,
                                              acc);
                            }
                        }
                    };
                    const uint32_t a_lo = a_lo0 + s * stage_step, b_lo = b_lo0 + s * stage_step;
                    if (issuer) {
                        issue_sub(a_lo, b_lo, kb > kb0);
                        // (the paired form is a branch of its own so that the one-k-block form keeps its straight-line
                        // code: as a loop over the sub-stages it cost the 256-column tiles 6 % - 2048^3 16.2 -> 17.2 us)
                        if (kTunable && NSUB == 2) issue_sub(a_lo + (SUB >> 4), b_lo + (SUB >> 4), true);
                        ptx::umma_commit_addr(empty0 + 8 * s);
                    }
                    if (issuer && t == 0 && kb == kb0 + 8) KLIN_T(28);
                    if (issuer && t == 0 && kb == kb0 + 9) KLIN_T(31);
                    s = s_next;
                    ph = ph_next;
                }
                if (ok && issuer) ptx::umma_commit(&acc_full[buf]);
                if (issuer && t == 0) KLIN_T(11);
            }
        }
    } else if (warp < 6) {
        // ------------------------------------------------------------ epilogue
        if (SWAP && p.cluster && warp == 2 && lane == 0) {
            // what this CTA will receive: every source's partial of each block it owns that lies inside the matrix
            const int nblk = 8 >> p.splits_log2;
            uint32_t blocks = 0;
            for (int bl = 0; bl < nblk; ++bl) {
                const int bi = (bl << p.splits_log2) + fin_rank;
                if (fin_n0 + (bi >> 2) * 128 + (bi & 3) * 32 < g.N) ++blocks;
            }
            ptx::mbar_arrive_expect_tx(xchg_bar, blocks * static_cast<uint32_t>(p.splits) * static_cast<uint32_t>(p.n_mma) * 128u);
        }
        const int q = warp & 3;                              // TMEM lane quarter this warp may read
        uint8_t* stg = epi_smem + (warp - 2) * 2 * kEpiBufBytes;
        uint32_t t = 0;
        uint32_t nstaged = 0;                                // staging blocks written so far (buffer = parity)
        bool ok = true;
        for (int64_t u = blockIdx.x; u < total_units && ok; u += gridDim.x, ++t) {
            const Unit x = unit_of(u);
            const int64_t tile = x.tile;
            const int split = x.split;
            const int m0 = x.m0, n0 = x.n0;
            const uint32_t buf = t & 1;
            if (!ptx::mbar_wait(&acc_full[buf], (t >> 1) & 1, abort_flag)) {
                if (lane == 0) report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x430u | buf);
                abort_flag[0] = 1;
                ok = false;
                break;
            }
            ptx::tc_fence_after_sync();
            if (t == 0 && warp == 2 && lane == 0) KLIN_T(12);
            if (SWAP) {
                // lane = weight column n, registers = activation rows m
                const bool partial = p.splits > 1 && !p.cluster;
                float* dst_f = partial ? p.ws + static_cast<int64_t>(split) * g.M * p.ldw : static_cast<float*>(g.C);
                const int64_t ld = partial ? p.ldw : g.ldc;
                const bool out_bf16 = g.c_bf16 && !partial;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int nbase = n0 + h * 128 + q * 32;
                    if (nbase >= g.N) continue;
                    const int n = nbase + lane;
                    for (int mc = 0; mc < p.n_mma; mc += 16) {
                        uint32_t v[16];
                        ptx::tmem_ld_32x32b_x16(tmem_base + buf * BN + h * 128 + mc + (static_cast<uint32_t>(q * 32) << 16), v);
                        uint32_t remote = 0, remote_bar = 0;
                        if (p.cluster) {
                            // block (h, q) of the tile belongs to CTA (block % splits); this CTA's
                            // partial goes to slot [split][block / splits] of the owner, laid out
                            // [m / 4][lane][m % 4] so that four rows travel as one 16-byte store
                            // (address arithmetic while the TMEM load is in flight)
                            const int bi = h * 4 + q;
                            const uint32_t owner = static_cast<uint32_t>(bi & (p.splits - 1));
                            const int nblk = 8 >> p.splits_log2;
                            float* slot = reinterpret_cast<float*>(epi_smem) +
                                          ((split * nblk + (bi >> p.splits_log2)) * p.n_mma + mc) * 32 + lane * 4;
                            remote = ptx::map_to_cta(ptx::smem_u32(slot), owner);
                            remote_bar = ptx::map_to_cta(ptx::smem_u32(xchg_bar), owner);
                        }
                        ptx::tmem_ld_wait();
                        if (p.cluster) {
                            // asynchronous stores counted on the owner's barrier: the owner waits for its bytes, no
                            // cluster-wide barrier stands between the last MMA and the reduce
#pragma unroll
                            for (int j = 0; j < 16; j += 4)
                                ptx::st_async_v4_f32(remote + j * 128, __uint_as_float(v[j]), __uint_as_float(v[j + 1]),
                                                     __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]), remote_bar);
                        } else if (n < g.N) {
                            const float bn = partial ? 0.f : bias_at(g, n);
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                v[j] = __float_as_uint(__uint_as_float(v[j]) + bn);
                                const int m = mc + j;
                                if (m < g.M) {
                                    if (out_bf16)
                                        static_cast<uint16_t*>(g.C)[m * ld + n] = float_to_bf16_bits(__uint_as_float(v[j]));
                                    else
                                        dst_f[m * ld + n] = __uint_as_float(v[j]);
                                }
                            }
                        }
                    }
                }
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&acc_empty[buf]);

                if (partial) {
                    // One arrival counter per (tile, lane quarter); the last arriver sums its 2 x 32
                    // columns over all rows, partials in split order, loads batched to hide latency.
                    const int64_t plane = static_cast<int64_t>(g.M) * p.ldw;
                    if (n0 + q * 32 < g.N) {
                        __syncwarp();
                        unsigned old = 0;
                        unsigned* cnt = p.counters + tile * 4 + q;
                        if (lane == 0) {
                            __threadfence();
                            old = atomicAdd(cnt, 1u);
                            __threadfence();
                        }
                        old = __shfl_sync(0xFFFFFFFFu, old, 0);
                        if (old == static_cast<unsigned>(p.splits - 1)) {
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                const int n = n0 + h * 128 + q * 32 + lane;
                                if (n >= g.N) continue;
                                for (int mb = 0; mb < g.M; mb += 16) {
                                    float acc[16];
#pragma unroll
                                    for (int j = 0; j < 16; ++j) acc[j] = 0.f;
                                    for (int sp = 0; sp < p.splits; sp += 4) {
                                        float x[4][16];
#pragma unroll
                                        for (int s4 = 0; s4 < 4; ++s4)
#pragma unroll
                                            for (int j = 0; j < 16; ++j)
                                                x[s4][j] = (sp + s4 < p.splits && mb + j < g.M)
                                                               ? __ldcg(p.ws + (sp + s4) * plane + (mb + j) * p.ldw + n)
                                                               : 0.f;
#pragma unroll
                                        for (int s4 = 0; s4 < 4; ++s4)
#pragma unroll
                                            for (int j = 0; j < 16; ++j) acc[j] += x[s4][j];
                                    }
#pragma unroll
                                    for (int j = 0; j < 16; ++j)
                                        if (mb + j < g.M) store_c(g.C, g.c_bf16, (mb + j) * g.ldc + n, acc[j] + bias_at(g, n));
                                }
                            }
                            __syncwarp();
                            if (lane == 0) *cnt = 0;   // ready for the next launch
                        }
                    }
                }
                continue;
            }
            if (MODE == 4 && !GENERIC && p.conv_t) {
                // Transposed Conv2d tile: TMEM lane = filter, column = pixel (128 per patch tile, 16 per patch row).
                // A warp owns 32 filters: per step it stages 64 pixels x 32 filters (64-byte rows, its private 4 KiB
                // block) and stores them as ONE 4-D box of y (32 filters x 16 x 4 pixels, clipped at the image).
                const bool f_live = q * 32 < g.N;                    // (warp-uniform) filters of this warp exist
#pragma unroll 1
                for (int hc = 0; hc < 4; ++hc) {                     // (patch tile h, 4-row half c)
                    const int h = hc >> 1, c = hc & 1;
                    const int tt = 2 * (m0 / BM) + h;
                    const int qt = tt % p.conv_tq, u2 = tt / p.conv_tq;
                    const int cq0 = qt * 16, cp0 = (u2 % p.conv_tp) * 8 + c * 4, cimg = u2 / p.conv_tp;
                    if (!f_live || cimg >= p.conv_nimg || cp0 >= p.conv.P) continue;
                    uint32_t v[32], v2[32];
                    const uint32_t taddr = tmem_base + buf * BN + h * 128 + c * 64 + (static_cast<uint32_t>(q * 32) << 16);
                    ptx::tmem_ld_32x32b_x32(taddr, v);
                    ptx::tmem_ld_32x32b_x32(taddr + 32, v2);
                    uint8_t* b = stg + (nstaged++ & 1) * kEpiBufBytes;
                    if (lane == 0) ptx::tma_store_wait_read<1>();    // the store that last read this block
                    __syncwarp();
                    ptx::tmem_ld_wait();
                    uint16_t* row = reinterpret_cast<uint16_t*>(b) + lane;     // [pixel][32 filters]
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        const uint32_t w0 = pack_out2(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), g.f16);
                        const uint32_t w1 = pack_out2(__uint_as_float(v2[j]), __uint_as_float(v2[j + 1]), g.f16);
                        row[j * 32] = static_cast<uint16_t>(w0 & 0xFFFFu);
                        row[(j + 1) * 32] = static_cast<uint16_t>(w0 >> 16);
                        row[(j + 32) * 32] = static_cast<uint16_t>(w1 & 0xFFFFu);
                        row[(j + 33) * 32] = static_cast<uint16_t>(w1 >> 16);
                    }
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        ptx::tma_store_4d(&map_c, q * 32, cq0, cp0, cimg, b);
                        ptx::tma_store_commit();
                    }
                }
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&acc_empty[buf]);
                continue;
            }
            if (MODE == 0 && p.cluster) continue;     // drained after the cluster-wide barrier below
            const int row0 = m0 + q * 32;
            if (row0 < x.M) {
                const bool partial = p.splits > 1;
                const bool out_bf16 = g.c_bf16 && !partial;
                const bool use_tma = x.epi_tma && !partial;
                const int cpc = out_bf16 ? 64 : 32;           // columns per 128-byte staging row
                float* dst_f = partial ? p.ws + static_cast<int64_t>(split) * g.M * p.ldw : reinterpret_cast<float*>(x.C);
                uint16_t* dst_h = reinterpret_cast<uint16_t*>(x.C);
                const int64_t ld = partial ? p.ldw : x.ldc;
                const int rows = min(32, x.M - row0);
                // Conv2d with patch tiling: this warp's 32 rows are patch rows 2q, 2q+1 (16 pixels each) of
                // the 8 x 16 output patch (pt, qt) of image cn
                int cq0 = 0, cp0 = 0, cimg = 0;
                bool below = false;
                if (MODE == 4 && !GENERIC) {
                    const int t = m0 / BM;
                    const int qt = t % p.conv_tq, u2 = t / p.conv_tq;
                    cq0 = qt * 16;
                    cp0 = (u2 % p.conv_tp) * 8 + 2 * q;
                    cimg = u2 / p.conv_tp;
                    below = cp0 >= p.conv.P;                      // the patch rows of this warp lie below the image
                }
                for (int c = 0; c * cpc < x.ncols && !below; ++c) {
                    const int col0 = n0 + c * cpc;
                    if (col0 >= x.N) break;
                    uint32_t v[32], w[32];
                    const uint32_t taddr = tmem_base + buf * BN + c * cpc + (static_cast<uint32_t>(q * 32) << 16);
                    ptx::tmem_ld_32x32b_x32(taddr, v);
                    if (out_bf16) {
                        uint32_t v2[32];
                        ptx::tmem_ld_32x32b_x32(taddr + 32, v2);
                        ptx::tmem_ld_wait();
                        if (g.bias) {   // lane l fetches two columns' bias, shuffles hand them round
                            const float b0 = (col0 + lane < x.N) ? bias_at(g, col0 + lane) : 0.f;
                            const float b1 = (col0 + 32 + lane < x.N) ? bias_at(g, col0 + 32 + lane) : 0.f;
#pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                v[i] = __float_as_uint(__uint_as_float(v[i]) + __shfl_sync(0xFFFFFFFFu, b0, i));
                                v2[i] = __float_as_uint(__uint_as_float(v2[i]) + __shfl_sync(0xFFFFFFFFu, b1, i));
                            }
                        }
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            w[i] = pack_out2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]), g.f16);
                            w[16 + i] = pack_out2(__uint_as_float(v2[2 * i]), __uint_as_float(v2[2 * i + 1]), g.f16);
                        }
                    } else {
                        ptx::tmem_ld_wait();
                        if (g.bias && !partial) {
                            const float b0 = (col0 + lane < x.N) ? bias_at(g, col0 + lane) : 0.f;
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                v[i] = __float_as_uint(__uint_as_float(v[i]) + __shfl_sync(0xFFFFFFFFu, b0, i));
                        }
#pragma unroll
                        for (int i = 0; i < 32; ++i) w[i] = v[i];
                    }
                    if (partial) {
                        // K-split partial sums to the workspace straight from registers: a lane holds 32 consecutive
                        // fp32 columns of its row (128 bytes, 16-byte aligned) - eight 16-byte stores, no staging
                        if (lane < rows) {
                            float* prow = dst_f + (row0 + lane) * ld + col0;
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                if (col0 + 4 * j < x.N)
                                    *reinterpret_cast<uint4*>(prow + 4 * j) = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
                        }
                        continue;
                    }
                    uint8_t* b = stg + (nstaged++ & 1) * kEpiBufBytes;   // (bias was added above)
                    if (MODE == 2 ? p.epi_tma != 0 : use_tma) {   // (grouped: an earlier group's store may be in flight)
                        if (lane == 0) ptx::tma_store_wait_read<1>();   // the store that last read this buffer
                        __syncwarp();
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<uint4*>(b + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                            make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
                    if (use_tma) {
                        ptx::fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) {
                            if (MODE == 1) {
                                ptx::tma_store_3d(x.mc, col0, row0, x.z, b);
                            } else if (MODE == 4 && !GENERIC) {
                                ptx::tma_store_4d(x.mc, col0, cq0, cp0, cimg, b);   // box: columns x 16 x 2 pixels, clipped at the image
                            } else if (MODE == 3) {
                                for (int d = 0; d < p.n_dst; ++d) ptx::tma_store_2d(&p.dsts[d].map_c, col0, row0, b);
                            } else {
                                ptx::tma_store_2d(x.mc, col0, row0, b);
                            }
                            ptx::tma_store_commit();
                        }
                    } else {
                        __syncwarp();
                        // lane l owns 32-bit word l of every staged row: coalesced 128-byte rows.
                        for (int dd = 0; dd < (MODE == 3 ? p.n_dst : 1); ++dd) {
                        if (MODE == 3) {
                            dst_f = static_cast<float*>(p.dsts[dd].C);
                            dst_h = static_cast<uint16_t*>(p.dsts[dd].C);
                        }
                        const int64_t ldd = (MODE == 3) ? p.dsts[dd].ldc : ld;
                        for (int rr = 0; rr < rows; ++rr) {
                            const uint32_t word =
                                *reinterpret_cast<const uint32_t*>(b + rr * 128 + (((lane >> 2) ^ (rr & 7)) << 4) +
                                                                   (lane & 3) * 4);
                            int64_t row = row0 + rr;
                            if (MODE == 4 && !GENERIC) {     // staged row rr = pixel (cp0 + rr / 16, cq0 + rr % 16)
                                const int pp = cp0 + (rr >> 4), qq = cq0 + (rr & 15);
                                if (pp >= p.conv.P || qq >= p.conv.Q) continue;
                                row = (static_cast<int64_t>(cimg) * p.conv.P + pp) * p.conv.Q + qq;
                            }
                            if (out_bf16) {
                                const int col = col0 + 2 * lane;
                                uint16_t* d = dst_h + row * ldd + col;
                                if (col + 1 < x.N && (reinterpret_cast<uintptr_t>(d) & 3) == 0) {
                                    *reinterpret_cast<uint32_t*>(d) = word;
                                } else {
                                    if (col < x.N) d[0] = static_cast<uint16_t>(word & 0xFFFFu);
                                    if (col + 1 < x.N) d[1] = static_cast<uint16_t>(word >> 16);
                                }
                            } else {
                                const int col = col0 + lane;
                                if (col < x.N) dst_f[row * ldd + col] = __uint_as_float(word);
                            }
                        }
                        }
                        __syncwarp();
                    }
                }
            }
            // TMEM reads of this tile are done: hand the accumulator back.
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&acc_empty[buf]);
            if (t == 0 && warp == 2 && lane == 0) KLIN_T(13);

            if (p.splits > 1 && row0 < g.M) {
                // Arrival per (tile, 32-row block); the last arriver adds the partials in split order.
                __threadfence();
                __syncwarp();
                unsigned old = 0;
                unsigned* cnt = p.counters + tile * 4 + q;
                if (lane == 0) old = atomicAdd(cnt, 1u);
                old = __shfl_sync(0xFFFFFFFFu, old, 0);
                if (old == static_cast<unsigned>(p.splits - 1)) {
                    __threadfence();
                    const int rows = min(32, g.M - row0);
                    const int64_t plane = static_cast<int64_t>(g.M) * p.ldw;
                    // Four rows x both 128-column passes x two splits per step: sixteen independent 16-byte loads
                    // per lane are in flight before the first add (one load at a time made this reduce cost as
                    // much as a hundred k-blocks).  Every element still adds its partials in split order.
                    const int celt_out = g.c_bf16 ? 2 : 4;
                    const bool fast = n0 + BN <= g.N && (reinterpret_cast<uintptr_t>(g.C) % (4 * celt_out)) == 0 &&
                                      (g.ldc * celt_out) % (4 * celt_out) == 0;
                    float4 bias4[2] = {make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f)};
                    if (fast && g.bias) {
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            const int col = n0 + lane * 4 + c * 128;
                            bias4[c] = make_float4(bias_at(g, col), bias_at(g, col + 1), bias_at(g, col + 2), bias_at(g, col + 3));
                        }
                    }
                    for (int r4 = 0; r4 < rows; r4 += 4) {
                        float4 acc[4][2];
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int c = 0; c < 2; ++c) acc[i][c] = make_float4(0.f, 0.f, 0.f, 0.f);
                        // (rows and columns past the matrix are clamped to valid addresses and never stored, the
                        // odd last split is read twice and added once: the loads stay unconditional, so that all
                        // sixteen are issued before the first use)
                        const float* base[4][2];
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int c = 0; c < 2; ++c) {
                                const int col = min(n0 + lane * 4 + c * 128, static_cast<int>(p.ldw) - 4);
                                base[i][c] = p.ws + (row0 + min(r4 + i, rows - 1)) * p.ldw + col;
                            }
                        for (int sp = 0; sp < p.splits; sp += 2) {
                            float4 x[2][4][2];
                            const int64_t off1 = (sp + 1 < p.splits ? sp + 1 : sp) * plane;
#pragma unroll
                            for (int i = 0; i < 4; ++i)
#pragma unroll
                                for (int c = 0; c < 2; ++c) {
                                    x[0][i][c] = __ldcg(reinterpret_cast<const float4*>(base[i][c] + sp * plane));
                                    x[1][i][c] = __ldcg(reinterpret_cast<const float4*>(base[i][c] + off1));
                                }
                            if (sp + 1 >= p.splits) {
#pragma unroll
                                for (int i = 0; i < 4; ++i)
#pragma unroll
                                    for (int c = 0; c < 2; ++c) x[1][i][c] = make_float4(0.f, 0.f, 0.f, 0.f);
                            }
#pragma unroll
                            for (int s2 = 0; s2 < 2; ++s2)
#pragma unroll
                                for (int i = 0; i < 4; ++i)
#pragma unroll
                                    for (int c = 0; c < 2; ++c) {
                                        acc[i][c].x += x[s2][i][c].x;
                                        acc[i][c].y += x[s2][i][c].y;
                                        acc[i][c].z += x[s2][i][c].z;
                                        acc[i][c].w += x[s2][i][c].w;
                                    }
                        }
                        if (fast && r4 + 3 < rows) {
                            // whole rows of a tile inside the matrix, C aligned for vector stores: no per-element
                            // tests (this tail runs on one warp: its instruction count is its time)
                            const int64_t idx0 = (row0 + r4) * g.ldc + n0 + lane * 4;
#pragma unroll
                            for (int i = 0; i < 4; ++i)
#pragma unroll
                                for (int c = 0; c < 2; ++c) {
                                    const int64_t idx = idx0 + i * g.ldc + c * 128;
                                    const float4 o = make_float4(acc[i][c].x + bias4[c].x, acc[i][c].y + bias4[c].y,
                                                                 acc[i][c].z + bias4[c].z, acc[i][c].w + bias4[c].w);
                                    if (g.c_bf16)
                                        *reinterpret_cast<uint2*>(static_cast<uint16_t*>(g.C) + idx) =
                                            make_uint2(pack_bf16x2(o.x, o.y), pack_bf16x2(o.z, o.w));
                                    else
                                        *reinterpret_cast<float4*>(static_cast<float*>(g.C) + idx) = o;
                                }
                            continue;
                        }
#pragma unroll
                        for (int i = 0; i < 4; ++i)
#pragma unroll
                            for (int c = 0; c < 2; ++c) {
                                const int col = n0 + lane * 4 + c * 128;
                                const int64_t row = row0 + r4 + i;
                                if (r4 + i >= rows) continue;
                                if (col >= g.N) continue;
                                float o[4] = {acc[i][c].x, acc[i][c].y, acc[i][c].z, acc[i][c].w};
#pragma unroll
                                for (int e = 0; e < 4; ++e)
                                    if (col + e < g.N) o[e] += bias_at(g, col + e);
                                const int64_t idx = row * g.ldc + col;
                                if (col + 3 < g.N && g.c_bf16 && (reinterpret_cast<uintptr_t>(static_cast<uint16_t*>(g.C) + idx) & 7) == 0) {
                                    *reinterpret_cast<uint2*>(static_cast<uint16_t*>(g.C) + idx) =
                                        make_uint2(pack_bf16x2(o[0], o[1]), pack_bf16x2(o[2], o[3]));
                                } else if (col + 3 < g.N && !g.c_bf16 &&
                                           (reinterpret_cast<uintptr_t>(static_cast<float*>(g.C) + idx) & 15) == 0) {
                                    *reinterpret_cast<float4*>(static_cast<float*>(g.C) + idx) = make_float4(o[0], o[1], o[2], o[3]);
                                } else {
#pragma unroll
                                    for (int e = 0; e < 4; ++e)
                                        if (col + e < g.N) store_c(g.C, g.c_bf16, idx + e, o[e]);
                                }
                            }
                    }
                    __syncwarp();
                    if (lane == 0) *cnt = 0;   // ready for the next launch
                }
            }
                }
        // shared memory may go once the stores have read it; their writes complete with the grid
        if (p.epi_tma && lane == 0) ptx::tma_store_wait_read<0>();
    } else if (GENERIC) {
        // ------------------------------------------------------------ generic-proxy producers
        const int pt = threadIdx.x - 6 * 32;                 // 0..127
        uint32_t it = 0;
        bool ok = true;
        if (MODE == 4 && p.conv_fast) {
            // Conv2d, 16-byte chunks (C % 8 == 0, aligned x).  Row m of the implicit GEMM is the output
            // pixel (n, p, q), k the filter tap and channel (r, s, c); the element is
            // x[n][p*stride_h + r - pad_h][q*stride_w + s - pad_w][c], zero outside the image.  A thread
            // owns chunk kc of rows (pt >> 3) + 16 j: its chunk's tap is the same for all eight rows,
            // whose pixel origins are decoded once per tile.  The eight loads of the NEXT k-block are
            // issued before this k-block is stored, so a load's latency hides behind the ring.
            const ConvGeom& cv = p.conv;
            const int kc = pt & 7;
            for (int64_t u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
                const Unit x = decode_unit(u, p);
                int h0[8], w0[8], nn[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int gm = x.m0 + (pt >> 3) + 16 * j;
                    const int q = gm % cv.Q, t = gm / cv.Q;
                    nn[j] = gm < g.M ? t / cv.P : -1;
                    h0[j] = (t % cv.P) * cv.stride_h - cv.pad_h;
                    w0[j] = q * cv.stride_w - cv.pad_w;
                }
                auto fetch = [&](int kb, uint4 (&v)[8]) {
                    const int gk = kb * BK + kc * 8;
                    const int tap = gk / cv.C, ch = gk - tap * cv.C;
                    const int fr = tap / cv.S, fs = tap - fr * cv.S;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int h = h0[j] + fr, w = w0[j] + fs;
                        v[j] = make_uint4(0u, 0u, 0u, 0u);
                        if (nn[j] >= 0 && gk < g.K && h >= 0 && h < cv.H && w >= 0 && w < cv.W)
                            v[j] = __ldg(reinterpret_cast<const uint4*>(
                                g.A + ((static_cast<int64_t>(nn[j]) * cv.H + h) * cv.W + w) * cv.C + ch));
                    }
                };
                auto commit = [&](int kb, const uint4 (&v)[8]) -> bool {
                    const int s = it % STAGES;
                    if (!ptx::mbar_wait(&empty[s], ((it / STAGES) & 1) ^ 1, abort_flag)) {
                        if (pt == 0) report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x460u | s);
                        abort_flag[0] = 1;
                        return false;
                    }
                    uint8_t* sa = smem + s * kStageBytes;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int r = (pt >> 3) + 16 * j;
                        *reinterpret_cast<uint4*>(sa + r * 128 + ((kc ^ (r & 7)) << 4)) = v[j];
                    }
                    if (!p.conv_b_tma) {
                        // filters [F][K], K contiguous: 8-k chunks of rows n0 .. n0 + ncols
                        uint8_t* sb = sa + kABytes;
#pragma unroll 4
                        for (int c = pt; c < x.ncols * 8; c += kProducerThreads) {
                            const int n = c >> 3, kc2 = c & 7;
                            const int64_t gn = x.n0 + n;
                            const int gk = kb * BK + kc2 * 8;
                            const int valid = (gn < g.N) ? min(8, max(0, g.K - gk)) : 0;
                            *reinterpret_cast<uint4*>(sb + n * 128 + ((kc2 ^ (n & 7)) << 4)) =
                                gather8(g.B + gn * g.ldb + gk, valid);
                        }
                    }
                    ptx::fence_proxy_async_smem();
                    ptx::mbar_arrive(&full[s]);
                    ++it;
                    return true;
                };
                uint4 va[8], vb[8];
                fetch(x.kb0, va);
                for (int kb = x.kb0; kb < x.kb1 && ok; kb += 2) {
                    if (kb + 1 < x.kb1) fetch(kb + 1, vb);
                    ok = commit(kb, va);
                    if (ok && kb + 1 < x.kb1) {
                        if (kb + 2 < x.kb1) fetch(kb + 2, va);
                        ok = commit(kb + 1, vb);
                    }
                }
            }
        } else
        for (int64_t u = blockIdx.x; u < total_units && ok; u += gridDim.x) {
            const Unit x = decode_unit(u, p);
            const int kb0 = x.kb0, kb1 = x.kb1;
            const int m0 = x.m0, n0 = x.n0;
            for (int kb = kb0; kb < kb1; ++kb, ++it) {
                const int s = it % STAGES;
                if (!ptx::mbar_wait(&empty[s], ((it / STAGES) & 1) ^ 1, abort_flag)) {
                    if (pt == 0) report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x440u | s);
                    abort_flag[0] = 1;
                    ok = false;
                    break;
                }
                uint8_t* sa = smem + s * kStageBytes;
                uint8_t* sb = sa + kABytes;
                const int k0 = kb * BK;
                // A: 128 rows x 8 chunks of 8 k (K-major, 128-byte swizzle)
                if (MODE == 4) {
                    // (the 16-byte-chunk form has a loop of its own above)
                    // channel counts that are not multiples of 8 (a chunk may straddle two taps) or an
                    // unaligned x: element by element
                    const ConvGeom& cv = p.conv;
                    for (int c = pt; c < BM * 8; c += kProducerThreads) {
                        const int r = c >> 3, kc = c & 7;
                        const int gm = m0 + r;
                        const int gk = k0 + kc * 8;
                        uint16_t e8[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) e8[e] = 0;
                        if (gm < g.M && gk < g.K) {
                            const int q = gm % cv.Q, t = gm / cv.Q;
                            const int pp = t % cv.P, n = t / cv.P;
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                const int k = gk + e;
                                if (k < g.K) {
                                    const int tap = k / cv.C, ch = k - tap * cv.C;
                                    const int fr = tap / cv.S, fs = tap - fr * cv.S;
                                    const int h = pp * cv.stride_h + fr - cv.pad_h, w = q * cv.stride_w + fs - cv.pad_w;
                                    if (h >= 0 && h < cv.H && w >= 0 && w < cv.W)
                                        e8[e] = __ldg(g.A + ((static_cast<int64_t>(n) * cv.H + h) * cv.W + w) * cv.C + ch);
                                }
                            }
                        }
                        uint4 v;
                        v.x = e8[0] | (uint32_t(e8[1]) << 16);
                        v.y = e8[2] | (uint32_t(e8[3]) << 16);
                        v.z = e8[4] | (uint32_t(e8[5]) << 16);
                        v.w = e8[6] | (uint32_t(e8[7]) << 16);
                        *reinterpret_cast<uint4*>(sa + r * 128 + ((kc ^ (r & 7)) << 4)) = v;
                    }
                } else {
#pragma unroll 4
                for (int c = pt; c < BM * 8; c += kProducerThreads) {
                    const int r = c >> 3, kc = c & 7;
                    const int64_t gm = m0 + r;
                    const int gk = k0 + kc * 8;
                    const int valid = (gm < g.M) ? min(8, max(0, g.K - gk)) : 0;
                    *reinterpret_cast<uint4*>(sa + r * 128 + ((kc ^ (r & 7)) << 4)) =
                        gather8(g.A + gm * g.lda + gk, valid);
                }
                }
                if (BCOL) {
                    // B column-major: 256 n-rows x 8 chunks of 8 k (K-major)
#pragma unroll 4
                    for (int c = pt; c < x.ncols * 8; c += kProducerThreads) {
                        const int n = c >> 3, kc = c & 7;
                        const int64_t gn = n0 + n;
                        const int gk = k0 + kc * 8;
                        const int valid = (gn < g.N) ? min(8, max(0, g.K - gk)) : 0;
                        *reinterpret_cast<uint4*>(sb + n * 128 + ((kc ^ (n & 7)) << 4)) =
                            gather8(g.B + gn * g.ldb + gk, valid);
                    }
                } else {
                    // B row-major: 64 k-rows x 32 chunks of 8 n (MN-major): 64-column blocks of
                    // 64 k-rows x 128 bytes, chunk index swizzled with the k-row.
#pragma unroll 4
                    for (int c = pt; c < BK * 32; c += kProducerThreads) {
                        const int k = c >> 5, nc = c & 31;
                        const int64_t gk = k0 + k;
                        const int gn = n0 + nc * 8;
                        const int valid = (gk < g.K) ? min(8, max(0, g.N - gn)) : 0;
                        *reinterpret_cast<uint4*>(sb + (nc >> 3) * (64 * BK * 2) + k * 128 + (((nc & 7) ^ (k & 7)) << 4)) =
                            gather8(g.B + gk * g.ldb + gn, valid);
                    }
                }
                ptx::fence_proxy_async_smem();
                ptx::mbar_arrive(&full[s]);
            }
        }
    }

    if (!SWAP && MODE == 0 && p.cluster) {
        // K split of a 128-row tile inside a thread-block cluster (2, 4 or 8 CTAs, one K range each).  The tile
        // is cut into (32-row lane quarter, store unit of 128 bytes per row) pairs: 16 for a 2-byte C, 32 for
        // fp32; CTA r owns pairs [r * per, (r + 1) * per).  After a first cluster barrier - every CTA's MMAs have
        // completed, so every operand ring is idle - each CTA sends the 32 x 32 blocks of its partial tile that
        // it does not own to their owners (plain st.shared::cluster into the owner's ring), laid out
        // [column / 4][row][column % 4] so that a lane's four columns travel as one conflict-free 16-byte
        // store.  After a second barrier the owner adds the partials in rank order (deterministic; its own
        // comes straight from TMEM), adds the bias once, rounds and stores its pairs.  No workspace, no
        // atomics, no trip through L2.
        const uint32_t rank = ptx::cluster_ctarank();
        if (warp == 2 && lane == 0) KLIN_T(32);
        ptx::cluster_arrive_relaxed();      // (an execution barrier: "my MMAs are done"; the data follows behind the second one)
        ptx::cluster_wait_acquire();
        if (warp == 2 && lane == 0) KLIN_T(33);
        const bool epi_warp = warp >= 2 && warp < 6;
        const bool out_bf16 = g.c_bf16 != 0;
        const int sub_log2 = out_bf16 ? 1 : 0;                          // 32-column blocks per store unit
        const int per_log2 = (out_bf16 ? 4 : 5) - (TN == BN ? 0 : TN == BN / 2 ? 1 : 2) - p.splits_log2;   // pairs per CTA
        const int q = warp & 3;                                         // TMEM lane quarter of this warp
        const uint32_t tlane = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
        float* recv = reinterpret_cast<float*>(smem);
        // slot of 32-column block c (of lane quarter qq) sent by CTA `src`, inside its owner's ring
        auto slot_of = [&](int src, int c, int qq) {
            const int idx = ((c >> sub_log2) << 2) + qq;
            const int lp = idx & ((1 << per_log2) - 1);
            return recv + ((((src << per_log2) + lp) << sub_log2) + (c & ((1 << sub_log2) - 1))) * 1024 + lane * 4;
        };
        if (epi_warp && !abort_flag[0]) {
            ptx::tc_fence_after_sync();
            // two blocks per step: both TMEM loads are in flight before the first remote store
#pragma unroll 1
            for (int c = 0; c < TN / 32; c += 2) {
                const uint32_t own0 = static_cast<uint32_t>((((c >> sub_log2) << 2) + q) >> per_log2);
                const uint32_t own1 = static_cast<uint32_t>(((((c + 1) >> sub_log2) << 2) + q) >> per_log2);
                if (own0 == rank && own1 == rank) continue;
                uint32_t v0[32], v1[32];
                ptx::tmem_ld_32x32b_x32(tlane + c * 32, v0);
                ptx::tmem_ld_32x32b_x32(tlane + c * 32 + 32, v1);
                const uint32_t r0 = ptx::map_to_cta(ptx::smem_u32(slot_of(static_cast<int>(rank), c, q)), own0);
                const uint32_t r1 = ptx::map_to_cta(ptx::smem_u32(slot_of(static_cast<int>(rank), c + 1, q)), own1);
                ptx::tmem_ld_wait();
                if (own0 != rank) {
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        ptx::st_cluster_v4_f32(r0 + j * 512, __uint_as_float(v0[4 * j]), __uint_as_float(v0[4 * j + 1]),
                                               __uint_as_float(v0[4 * j + 2]), __uint_as_float(v0[4 * j + 3]));
                }
                if (own1 != rank) {
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        ptx::st_cluster_v4_f32(r1 + j * 512, __uint_as_float(v1[4 * j]), __uint_as_float(v1[4 * j + 1]),
                                               __uint_as_float(v1[4 * j + 2]), __uint_as_float(v1[4 * j + 3]));
                }
            }
        }
        if (warp == 2 && lane == 0) KLIN_T(34);
        ptx::cluster_arrive_release();
        ptx::cluster_wait_acquire();
        if (warp == 2 && lane == 0) KLIN_T(35);
        if (epi_warp && !abort_flag[0]) {
            const Unit x = decode_unit(static_cast<int64_t>(blockIdx.x), p);
            uint8_t* stg = epi_smem + (warp - 2) * 2 * kEpiBufBytes;
            const int cpc = out_bf16 ? 64 : 32;
            uint32_t nstaged = 0;
            // a warp takes the pairs of its own TMEM lane quarter (this CTA's partial is read from TMEM)
#pragma unroll 1
            for (int lp = 0; lp < (1 << per_log2); ++lp) {
                const int idx = (static_cast<int>(rank) << per_log2) + lp;
                if ((idx & 3) != q) continue;
                const int u = idx >> 2;
                const int row0 = x.m0 + q * 32, col0 = x.n0 + u * cpc;
                if (row0 >= g.M || col0 >= g.N) continue;
                const int rows = min(32, g.M - row0);
                uint32_t own[2][32];
                ptx::tmem_ld_32x32b_x32(tlane + (u << sub_log2) * 32, own[0]);
                if (out_bf16) ptx::tmem_ld_32x32b_x32(tlane + (u << sub_log2) * 32 + 32, own[1]);
                float acc[2][32];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) acc[h][i] = 0.f;
                }
                bool own_added = false;
                for (int src = 0; src < p.splits; ++src) {
                    if (src == static_cast<int>(rank)) {
                        ptx::tmem_ld_wait();
                        own_added = true;
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            if (h > sub_log2) continue;
#pragma unroll
                            for (int i = 0; i < 32; ++i) acc[h][i] += __uint_as_float(own[h][i]);
                        }
                        continue;
                    }
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (h > sub_log2) continue;
                        const float4* sl = reinterpret_cast<const float4*>(slot_of(src, (u << sub_log2) + h, q));
                        float4 t[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) t[j] = sl[j * 32];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            acc[h][4 * j] += t[j].x;
                            acc[h][4 * j + 1] += t[j].y;
                            acc[h][4 * j + 2] += t[j].z;
                            acc[h][4 * j + 3] += t[j].w;
                        }
                    }
                }
                if (!own_added) ptx::tmem_ld_wait();
                if (g.bias) {   // lane l fetches the bias of columns col0 + l (and + 32), shuffles hand them round
                    const float b0 = (col0 + lane < g.N) ? bias_at(g, col0 + lane) : 0.f;
                    const float b1 = (out_bf16 && col0 + 32 + lane < g.N) ? bias_at(g, col0 + 32 + lane) : 0.f;
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        acc[0][i] += __shfl_sync(0xFFFFFFFFu, b0, i);
                        acc[1][i] += __shfl_sync(0xFFFFFFFFu, b1, i);
                    }
                }
                uint32_t w[32];
                if (out_bf16) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        w[i] = pack_bf16x2(acc[0][2 * i], acc[0][2 * i + 1]);
                        w[16 + i] = pack_bf16x2(acc[1][2 * i], acc[1][2 * i + 1]);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) w[i] = __float_as_uint(acc[0][i]);
                }
                uint8_t* b = stg + (nstaged++ & 1) * kEpiBufBytes;
                if (p.epi_tma) {
                    if (lane == 0) ptx::tma_store_wait_read<1>();   // the store that last read this buffer
                    __syncwarp();
                }
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    *reinterpret_cast<uint4*>(b + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                        make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
                if (p.epi_tma) {
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        ptx::tma_store_2d(&map_c, col0, row0, b);
                        ptx::tma_store_commit();
                    }
                } else {
                    __syncwarp();
                    // lane l owns 32-bit word l of every staged row: coalesced 128-byte rows
                    for (int rr = 0; rr < rows; ++rr) {
                        const uint32_t word = *reinterpret_cast<const uint32_t*>(
                            b + rr * 128 + (((lane >> 2) ^ (rr & 7)) << 4) + (lane & 3) * 4);
                        const int64_t row = row0 + rr;
                        if (out_bf16) {
                            const int col = col0 + 2 * lane;
                            uint16_t* d = static_cast<uint16_t*>(g.C) + row * g.ldc + col;
                            if (col + 1 < g.N && (reinterpret_cast<uintptr_t>(d) & 3) == 0) {
                                *reinterpret_cast<uint32_t*>(d) = word;
                            } else {
                                if (col < g.N) d[0] = static_cast<uint16_t>(word & 0xFFFFu);
                                if (col + 1 < g.N) d[1] = static_cast<uint16_t>(word >> 16);
                            }
                        } else {
                            const int col = col0 + lane;
                            if (col < g.N) static_cast<float*>(g.C)[row * g.ldc + col] = __uint_as_float(word);
                        }
                    }
                    __syncwarp();
                }
            }
            // shared memory may go once the stores have read it; their writes complete with the grid
            if (p.epi_tma && lane == 0) ptx::tma_store_wait_read<0>();
        }
    }

    if (SWAP && p.cluster) {
        // The owner waits until every byte sent to it has landed: (splits) sources x its blocks inside the matrix
        // x n_mma rows x 128 bytes, announced on its barrier by one thread at the start of the epilogue role.
        bool got = true;
        if (warp >= 2 && warp < 6) {
            got = ptx::mbar_wait(xchg_bar, 0, abort_flag);
            if (!got) {
                if (lane == 0) report_error(g.status, kDevBarrierTimeout, blockIdx.x, 0x480u);
                abort_flag[0] = 1;
            }
        }
        if (warp >= 2 && warp < 6 && got && !abort_flag[0]) {
            // This CTA owns blocks bi = bl * splits + rank of the tile; slot (src * nblk + bl) holds
            // CTA src's partial of local block bl as [m / 4][lane][m % 4].  A warp takes four
            // consecutive rows (one 16-byte load per source); all of a block's loads are issued
            // before the adds (in rank order: deterministic), lanes run along n.
            const int nblk = 8 >> p.splits_log2;
            for (int m4 = (warp - 2) * 4; m4 < g.M; m4 += 16) {
                for (int bl = 0; bl < nblk; ++bl) {
                    const int bi = (bl << p.splits_log2) + fin_rank;
                    const int n = fin_n0 + (bi >> 2) * 128 + (bi & 3) * 32 + lane;
                    if (n >= g.N) continue;
                    const float4* sl = reinterpret_cast<const float4*>(fin_slots + (bl * p.n_mma + m4) * 32);
                    const int src_stride = nblk * p.n_mma * 8;      // in float4
                    float4 v[8];
#pragma unroll
                    for (int src = 0; src < 8; ++src)
                        v[src] = (src < p.splits) ? sl[src * src_stride] : make_float4(0.f, 0.f, 0.f, 0.f);
                    const float bn = bias_at(g, n);
                    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int src = 0; src < 8; ++src)
                        if (src < p.splits) {
                            acc[0] += v[src].x;
                            acc[1] += v[src].y;
                            acc[2] += v[src].z;
                            acc[3] += v[src].w;
                        }
#pragma unroll
                    for (int r = 0; r < 4; ++r)
                        if (m4 + r < g.M) store_c(g.C, g.c_bf16, static_cast<int64_t>(m4 + r) * g.ldc + n, acc[r] + bn);
                }
            }
        }
        // No CTA leaves while a peer could still send into its shared memory (on the ordinary path every byte has
        // been counted by now; a peer that gave up sends nothing more after it arrives here).  Execution only.
        ptx::cluster_arrive_relaxed();
        ptx::cluster_wait_acquire();
    }

    if (warp == 2 && lane == 0) KLIN_T(14);
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0) {
        KLIN_T(15);
        KLIN_TNS(7);
    }
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

// Row-major B (K x N, N a multiple of 64) as a 3-D tensor: 64 columns innermost, the K rows, then the
// N / 64 column blocks (128 bytes apart); the box takes `blocks` column blocks of 64 x BK.
bool encode_b_blocks_3d(const RunContext& ctx, CUtensorMap* map, const GemmArgs& g, uint32_t blocks)
{
    if (!ctx.encode_tiled) return false;
    const cuuint64_t dims[3] = {64, static_cast<cuuint64_t>(g.K), static_cast<cuuint64_t>(g.N / 64)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(g.ldb) * 2, 128};
    const cuuint32_t box[3] = {64, BK, blocks};
    const cuuint32_t estr[3] = {1, 1, 1};
    return ctx.encode_tiled(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<uint16_t*>(g.B), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool tma_ok(const void* base, int64_t ld_elems, int elt)
{
    return reinterpret_cast<uintptr_t>(base) % 16 == 0 && (ld_elems * elt) % 16 == 0 &&
           ld_elems * elt < (int64_t(1) << 40);
}

// Chooses the number of K splits: minimise waves x (k-blocks per unit + fixed
// per-unit cost), within the workspace and counter budgets.
// `fixed` is the per-unit cost of splitting in k-block times, `per_split` what every further split adds to it:
// small for the skinny orientation (coalesced partial stores, batched reduce), large for 128-row tiles, whose
// partial tile goes through the workspace and whose last arriver reads it back for every split (measured at
// 256 x 256 x 8192 in 2 .. 16 splits: overhead = 10 us + 2.2 us per split, a k-block being 0.34 us - i.e.
// splitting only pays for long K).
int choose_splits(int64_t tiles, int nkb, int sm, int64_t M, int64_t ldw, const RunContext& ctx, int fixed,
                  int per_split)
{
    if (tiles * 2 > sm || nkb < 8 || tiles * 4 > ctx.n_tile_counters) return 1;
    const int kFixed = fixed;
    int best = 1;
    int64_t best_cost = ((tiles + sm - 1) / sm) * static_cast<int64_t>(nkb);
    for (int s = 2; s <= 32 && s * 4 <= nkb; ++s) {
        const int per = (nkb + s - 1) / s;
        const int eff = (nkb + per - 1) / per;        // splits that actually get work
        if (eff != s) continue;
        if (static_cast<size_t>(s) * M * ldw * sizeof(float) > ctx.workspace_bytes) break;
        const int64_t cost = ((tiles * s + sm - 1) / sm) * (per + kFixed + per_split * s);
        if (cost < best_cost) {
            best_cost = cost;
            best = s;
        }
    }
    return best;
}

// Skinny shapes with M <= 32: the K splits of a tile run as one thread-block cluster
// (2, 4 or 8 CTAs) and need no workspace.  Returns 1 when splitting does not pay.
int choose_cluster_splits(int64_t tiles, int nkb, int sm)
{
    if (tiles * 2 > sm || nkb < 8) return 1;
    const int kFixed = 3;
    int best = 1;
    int64_t best_cost = ((tiles + sm - 1) / sm) * (nkb + kFixed);
    for (int s = 2; s <= 8 && s * 4 <= nkb; s *= 2) {
        const int per = (nkb + s - 1) / s;
        if ((nkb + per - 1) / per != s) continue;
        const int64_t cost = ((tiles * s + sm - 1) / sm) * (per + kFixed);
        if (cost < best_cost) {
            best_cost = cost;
            best = s;
        }
    }
    return best;
}

// 128-row tiles split inside a cluster: what the two cluster barriers, the exchange of the partial tile through
// the operand rings and the owner's reduce cost, in k-block times (0.31 us), measured in CUDA-graph replay on
// products of 1 .. 64 tiles: 4.0 / 5.0 / 6.6 us for 2 / 4 / 8 CTAs, about 4 us more when the launch fills
// most of the GPU (768 x 768 x 3072: 72 CTAs in pairs 12.3 us, 144 CTAs in fours 14.4 us).  A launch never exceeds one wave of clusters: a CTA runs exactly one unit, and a second
// wave would pay the kernel's set-up again (measured: 2048^3 in 4 splits 54 us against 17 us unsplit).
int cluster_fixed_cost(int s, int64_t ctas, int sm, int tile_n)
{
    // (128-column tiles exchange half as much: 1.7 / 2.0 / 2.5 us less)
    const int base = tile_n == BN ? (s == 2 ? 13 : s == 4 ? 16 : 22) : (s == 2 ? 8 : s == 4 ? 10 : 14);
    // (a launch of fours or eights over most of the GPU: 35 k-block times measured at 768 x 768 x 3072 and at 1024 x 1024 x
    // 4096 - 16.3 us in fours against 14.4 in pairs - where 16 + 12 said 28)
    // 256-column tiles pay it from a third of the GPU on: 1024 x 1024 x 4096 in pairs of 256-column tiles (64 CTAs) 17.9 us
    // = 26 k-block times over its 32 k-blocks, in pairs of 128-column tiles (128 CTAs) 14.4 us.
    const bool crowded = tile_n == BN ? ctas * 3 > static_cast<int64_t>(sm) : ctas * 3 > static_cast<int64_t>(sm) * 2;
    return base + (crowded ? (s >= 4 && ctas * 3 > static_cast<int64_t>(sm) * 2 ? 19 : 12) : 0);
}
// Clusters of `s` CTAs of this kernel that the device can hold at once (GPC boundaries make this less than
// SMs / s for large clusters); asked of the runtime once per size and device.
int max_resident_clusters(int s, const RunContext& ctx);

// K splits of the cluster route for a regular-orientation problem and their estimated cost (k-block times);
// 1 when no split fits or pays.
// A k-block of an UNSPLIT launch in fifths of a wide tile's k-block time: 128-column tiles take 4 (paired k-blocks) while
// the launch is small and 5 once a third of the SMs or more are at work (1208 x 992 x 4936, 80 such tiles: 0.32 us per
// k-block, 28.9 us against 24.6 in pairs; 592 x 1688 x 2744, 70 tiles: 18.4 against 15.2).  The splits themselves keep 4:
// 160 x 4016 x 4000 in pairs of 128-column tiles runs 0.27 us per k-block on 128 CTAs.
int64_t unsplit_kb_cost(int tile_n, int64_t tiles, int sm)
{
    return (tile_n == BN || tiles * 3 > sm) ? 5 : 4;
}

int choose_regular_cluster_splits(int64_t tiles, int nkb, const RunContext& ctx, int tile_n, int64_t* cost_out)
{
    int best = 1;
    // costs in fifths of a k-block time; a k-block of a narrow tile (paired k-blocks) takes about 0.8 of a wide one's
    const int64_t kb_cost = tile_n == BN ? 5 : 4;
    int64_t best_cost = ((tiles + ctx.sm_count - 1) / ctx.sm_count) * static_cast<int64_t>(nkb) * unsplit_kb_cost(tile_n, tiles, ctx.sm_count);
    for (int s = 2; s <= 8 && s * 2 <= nkb; s *= 2) {
        const int per = (nkb + s - 1) / s;
        if ((nkb + per - 1) / per != s) continue;
        if (tiles > max_resident_clusters(s, ctx)) continue;
        const int64_t cost = per * kb_cost + 5 * cluster_fixed_cost(s, tiles * s, ctx.sm_count, tile_n);
        if (cost < best_cost) {
            best_cost = cost;
            best = s;
        }
    }
    *cost_out = best_cost;
    return best;
}

// How a shape is split along K: not at all, through the global workspace, or
// through a cluster.  One function so that every caller plans the same way.
struct SplitPlan {
    int splits;
    bool cluster;
    bool swap;
    int64_t cost;       // the heuristic's estimate for its own choice, in k-block times (0 when not computed)
};

SplitPlan plan_split(int M, int64_t tiles, int nkb, int64_t ldw, const RunContext& ctx, int tile_n = BN)
{
    SplitPlan sp;
    sp.swap = M <= 64;
    sp.cluster = false;
    sp.cost = 0;
    if (sp.swap && M <= 32) {
        const int s = choose_cluster_splits(tiles, nkb, ctx.sm_count);
        if (s > 1) {
            sp.splits = s;
            sp.cluster = true;
            return sp;
        }
    }
    // (the workspace reduce of 128-row tiles is written for 256-column tiles)
    sp.splits = (sp.swap || tile_n == BN) ? choose_splits(tiles, nkb, ctx.sm_count, M, ldw, ctx, sp.swap ? 6 : 30, sp.swap ? 0 : 6) : 1;
    if (!sp.swap) {
        // 128-row tiles: the cluster route against the workspace route chosen above and against no split
        const int sm = ctx.sm_count;
        const int per_w = (nkb + sp.splits - 1) / sp.splits;
        // (in fifths of a k-block time, like the cluster route's estimate)
        sp.cost = sp.splits > 1 ? ((tiles * sp.splits + sm - 1) / sm) * static_cast<int64_t>(per_w + 30 + 6 * sp.splits) * 5
                                : ((tiles + sm - 1) / sm) * static_cast<int64_t>(nkb) * unsplit_kb_cost(tile_n, tiles, sm);
        int64_t cost_c = 0;
        const int sc = choose_regular_cluster_splits(tiles, nkb, ctx, tile_n, &cost_c);
        if (sc > 1 && cost_c <= sp.cost) {
            sp.splits = sc;
            sp.cluster = true;
            sp.cost = cost_c;
        }
    }
    return sp;
}

// Whether `splits` K splits can run: every split gets k-blocks, and the partial sums fit
// the cluster (skinny orientation, M <= 32, 2 / 4 / 8 CTAs) or the workspace and counters.
bool split_feasible(int M, int64_t tiles, int nkb, int64_t ldw, const RunContext& ctx, int splits, bool cluster)
{
    if (splits == 1) return !cluster;
    if (splits < 1 || splits > 64 || splits > nkb) return false;
    const int per = (nkb + splits - 1) / splits;
    if ((nkb + per - 1) / per != splits) return false;
    if (cluster) {
        if (splits != 2 && splits != 4 && splits != 8) return false;
        return M <= 32 || (M > 64 && tiles <= max_resident_clusters(splits, ctx));   // 128-row tiles: one wave of clusters
    }
    if (tiles * 4 > ctx.n_tile_counters) return false;
    return static_cast<size_t>(splits) * M * ldw * sizeof(float) <= ctx.workspace_bytes;
}

// The heuristic plan with the pinned fields of `pl` applied; false when they cannot run.
bool resolve_split(int M, int64_t tiles, int nkb, int64_t ldw, const RunContext& ctx, const R4Plan& pl, SplitPlan* out,
                   int tile_n = BN)
{
    SplitPlan sp = plan_split(M, tiles, nkb, ldw, ctx, tile_n);
    if (pl.splits > 0) {
        sp.cost = 0;
        sp.splits = pl.splits;
        if (pl.splits == 1)
            sp.cluster = false;
        else if (pl.split_via == 2)
            sp.cluster = true;
        else if (pl.split_via == 1)
            sp.cluster = false;
        else
            sp.cluster = (M <= 32 || !sp.swap) && (pl.splits == 2 || pl.splits == 4 || pl.splits == 8);
        if (!split_feasible(M, tiles, nkb, ldw, ctx, sp.splits, sp.cluster)) return false;
    }
    *out = sp;
    return true;
}

template <bool BCOL, bool GENERIC, bool SWAP, int MODE = 0>
cudaError_t launch(const GemmArgs& g, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc,
                   const R4Params& p, unsigned grid, int device, cudaStream_t stream)
{
    auto kern = r4_tcgen05_kernel<BCOL, GENERIC, SWAP, MODE>;
    static bool attr_set[64] = {};
    if (device < 0 || device >= 64 || !attr_set[device]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        if (device >= 0 && device < 64) attr_set[device] = true;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(GENERIC ? kThreadsGeneric : kThreadsTma);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attrs[2];
    unsigned na = 0;
    // Programmatic dependent launch for single-wave launches (short kernels, where the gap
    // between back-to-back launches is a visible share of the time): the kernel's set-up may
    // overlap the previous kernel's tail; the kernel itself waits (griddepcontrol.wait) before
    // it touches global memory.  Multi-wave launches measured slower with it and do without.
    if (p.total_units <= static_cast<int64_t>(grid)) {
        attrs[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attrs[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    if (p.cluster) {
        attrs[na].id = cudaLaunchAttributeClusterDimension;
        attrs[na].val.clusterDim.x = static_cast<unsigned>(p.splits);
        attrs[na].val.clusterDim.y = 1;
        attrs[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.attrs = attrs;
    cfg.numAttrs = na;
    return cudaLaunchKernelEx(&cfg, kern, g, ma, mb, mc, p);
}

int max_resident_clusters(int s, const RunContext& ctx)
{
    static int cache[64][4] = {};      // [device][log2 s], 0 = not asked yet
    const int l2 = s == 2 ? 1 : s == 4 ? 2 : 3;
    const bool cacheable = ctx.device >= 0 && ctx.device < 64;
    if (cacheable && cache[ctx.device][l2] != 0) return cache[ctx.device][l2];
    auto kern = r4_tcgen05_kernel<false, false, false, 0>;
    int n = 0;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(static_cast<unsigned>(ctx.sm_count / s * s));
    cfg.blockDim = dim3(kThreadsTma);
    cfg.dynamicSmemBytes = kSmemBytes;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = static_cast<unsigned>(s);
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess ||
        cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        n = ctx.sm_count / (2 * s);    // the runtime would not say: assume half
        if (n < 1) n = 1;
    }
    if (cacheable) cache[ctx.device][l2] = n;
    return n;
}

}  // namespace

namespace {

// Copies a rows x cols bf16 matrix with an arbitrary (element-aligned) base and pitch into a
// buffer whose pitch is a multiple of 8 elements, zero-filling the pitch padding: the
// precondition repair that lets an unaligned operand use the TMA / tcgen05 path.  One
// 16-byte store per thread; consecutive threads take consecutive 8-element groups.
// Both operands of a call go through ONE launch: blocks [0, blocks_first) copy the first matrix, the rest
// the second (a matrix with rows == 0 has no blocks).
struct RepackJob {
    const uint16_t* src;
    int64_t ld_src;
    uint16_t* dst;
    int64_t ld_dst, rows;
    int cols;
};
__global__ void __launch_bounds__(256) repack_rows_kernel(RepackJob first, RepackJob second, unsigned blocks_first)
{
    const bool is_first = blockIdx.x < blocks_first;
    const RepackJob& j = is_first ? first : second;
    const unsigned block = is_first ? blockIdx.x : blockIdx.x - blocks_first;
    const unsigned nblocks = is_first ? blocks_first : gridDim.x - blocks_first;
    const uint16_t* __restrict__ src = j.src;
    uint16_t* __restrict__ dst = j.dst;
    const int64_t ld_src = j.ld_src, ld_dst = j.ld_dst;
    const int cols = j.cols;
    const int64_t groups_per_row = ld_dst >> 3;
    const int64_t total = j.rows * groups_per_row;
    for (int64_t i = block * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(nblocks) * blockDim.x) {
        const int64_t r = i / groups_per_row;
        const int c0 = static_cast<int>(i - r * groups_per_row) * 8;
        const uint16_t* s = src + r * ld_src + c0;
        uint16_t v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = (c0 + e < cols) ? __ldg(s + e) : uint16_t(0);
        uint4 o;
        o.x = v[0] | (uint32_t(v[1]) << 16);
        o.y = v[2] | (uint32_t(v[3]) << 16);
        o.z = v[4] | (uint32_t(v[5]) << 16);
        o.w = v[6] | (uint32_t(v[7]) << 16);
        *reinterpret_cast<uint4*>(dst + r * ld_dst + c0) = o;
    }
}

bool c_store_by_tma(const GemmArgs& g);
// Tile width, ring depth and K split of a single-CTA launch (paper, Table 1 `templatize` / `autotune`; Appendix D:
// block size, stages and split are recipe parameters swept on a fixed kernel structure).  One function, so
// that the launcher, the plan checks and the allocation-free entry point all plan the same way.
struct LaunchPlan {
    int tile_n, stages;
    SplitPlan split;
};
bool plan_launch(const GemmArgs& g, const RunContext& ctx, bool generic, bool multi_dst, LaunchPlan* out)
{
    const R4Plan& pl = ctx.plan;
    const int nkb = (g.K + BK - 1) / BK;
    const int64_t ldw = (static_cast<int64_t>(g.N) + 3) & ~int64_t(3);
    const int64_t tiles_m = (g.M + BM - 1) / BM;
    // 128-column tiles and deeper rings: the plain TMA-fed GEMM in the regular orientation only
    const bool tunable = !generic && !multi_dst && g.M > 64 && ctx.encode_tiled != nullptr;
    auto try_shape = [&](int tn, int st, LaunchPlan* lp) {
        lp->tile_n = tn;
        lp->stages = st;
        const int64_t tiles = tiles_m * ((g.N + tn - 1) / tn);
        if (tiles > 0x3FFFFFFFll) return false;
        if (!resolve_split(g.M, tiles, nkb, ldw, ctx, pl, &lp->split, tn)) return false;
        return tn == BN || lp->split.splits == 1 || lp->split.cluster;
    };
    if (pl.kernel != 2 && (pl.tile_n != 0 || pl.stages != 0)) {        // pinned (the pair kernel reads the fields its own way)
        const int tn = pl.tile_n != 0 ? pl.tile_n : BN;
        const int st = pl.stages != 0 ? pl.stages : STAGES;
        const bool ok = (tn == BN && st == STAGES) ||
                        (tunable && ((tn == BN / 2 && (st == 4 || st == 6)) || (tn == BN / 4 && (st == 4 || st == 6 || st == 8))));
        return ok && try_shape(tn, st, out);
    }
    LaunchPlan wide;
    const bool wide_ok = try_shape(BN, STAGES, &wide);
    if (!tunable || g.N <= BN / 2 || pl.half_tail != 0 || pl.kernel == 2) {
        *out = wide;
        return wide_ok;
    }
    LaunchPlan narrow;
    const int64_t tiles256 = tiles_m * ((g.N + BN - 1) / BN);
    if (!try_shape(BN / 2, STAGES, &narrow)) {
        *out = wide;
        return wide_ok;
    }
    if (!wide_ok) {
        *out = narrow;
        return true;
    }
    // Measured (CUDA-graph replay): a cluster split with 128-column tiles exchanges half as much and wins at equal
    // splits; unsplit, 128-column tiles match the half-tile tail when one under-filled wave is all there is (they load
    // only the columns they use) and lose once the tiles no longer fit one wave.
    bool take_narrow;
    // Columns that 256-wide tiles fill badly (N just above a multiple of 256) while one wave of 128-wide tiles fills
    // them well: measured unsplit, 128 against 256 columns, 1912 x 1064 x 3544 25.6 against 37.1 us, 3104 x 528 x 4784
    // 24.1 / 34.1, 3632 x 616 x 816 9.2 / 12.0, 4848 x 304 x 1144 10.4 / 13.4, 1808 x 1112 x 320 6.3 / 7.7.
    const bool fuller = pl.splits == 0 && pl.split_via == 0 && wide.split.splits == 1 && narrow.split.splits == 1 &&
                        r4_narrow_tiles_fill_better(g.M, g.N, ctx.sm_count);
    if (fuller)
        take_narrow = true;
    else if (pl.splits > 0)
        take_narrow = narrow.split.cluster || (narrow.split.splits == 1 && tiles256 * 2 <= ctx.sm_count);
    else if (narrow.split.cost != wide.split.cost)
        take_narrow = narrow.split.cost < wide.split.cost;
    else
        take_narrow = narrow.split.splits > 1 || tiles256 * 2 <= ctx.sm_count;
    // the deepest ring: six real stages for a cluster split; unsplit, three stages of two k-blocks each (one barrier round
    // trip per eight MMAs: 1024^3 9.1 -> 8.4 us, 1536^3 13.2 -> 11.5 in graph replay)
    if (take_narrow && (narrow.split.cluster || narrow.split.splits == 1)) narrow.stages = 6;
    if (fuller && nkb < 16) narrow.stages = 4;      // (short K: the plain four-stage ring was the faster one in those runs)
    if (take_narrow && narrow.split.splits == 1 && g.N > BN / 4) {
        // still at most half a wave of 128-column tiles: 64 columns (measured 0.4 - 0.5 us off a 5 - 7 us launch at
        // 256^3, 512^3 and 300 x 520 x 200: an MMA takes as long whatever its width, the epilogue of a tile shrinks)
        const int64_t tiles128 = tiles_m * ((g.N + BN / 2 - 1) / (BN / 2));
        LaunchPlan tiny;
        if (tiles128 * 2 <= ctx.sm_count && try_shape(BN / 4, 8, &tiny) && tiny.split.splits == 1) narrow = tiny;
    }
    *out = take_narrow ? narrow : wide;
    return true;
}
struct MultiDst {
    void* const* C;
    const int64_t* ldc;
    int n;
};
cudaError_t launch_r4_planned(const GemmArgs& g, RunContext& ctx, cudaStream_t stream, int* kernel_id,
                              const MultiDst* md = nullptr);

}  // namespace

// Entry of rung 4.  Operands that break TMA's alignment rules (base not 16-byte aligned or
// pitch not a multiple of 16 bytes) are first copied into the handle's workspace with an
// aligned pitch when they fit there - one streaming pass over the operand, after which the
// aligned kernels apply; otherwise the generic-proxy producers gather them tile by tile.
cudaError_t launch_r4_tcgen05(const GemmArgs& g, RunContext& ctx, cudaStream_t stream, int* kernel_id)
{
    const bool bad_a = !tma_ok(g.A, g.lda, 2), bad_b = !tma_ok(g.B, g.ldb, 2);
    if (!(bad_a || bad_b) || !ctx.allow_repack || !ctx.encode_tiled) return launch_r4_planned(g, ctx, stream, kernel_id);
    const int64_t b_rows = g.b_col ? g.N : g.K, b_cols = g.b_col ? g.K : g.N;
    const int64_t lda2 = (static_cast<int64_t>(g.K) + 7) & ~int64_t(7), ldb2 = (b_cols + 7) & ~int64_t(7);
    const size_t bytes_a = bad_a ? static_cast<size_t>(g.M) * lda2 * 2 : 0;
    const size_t bytes_b = bad_b ? static_cast<size_t>(b_rows) * ldb2 * 2 : 0;
    const size_t used = ((bytes_a + 255) & ~size_t(255)) + ((bytes_b + 255) & ~size_t(255));
    // keep at least a quarter of the workspace for split-K partial sums (the split heuristic sees what is left)
    if (used > ctx.workspace_bytes / 4 * 3) return launch_r4_planned(g, ctx, stream, kernel_id);

    GemmArgs g2 = g;
    uint8_t* ws = static_cast<uint8_t*>(ctx.workspace);
    RepackJob ja = {nullptr, 0, nullptr, 8, 0, 0}, jb = ja;
    auto blocks_of = [](const RepackJob& j) {
        const int64_t blocks = (j.rows * (j.ld_dst >> 3) + 255) / 256;
        return static_cast<unsigned>(blocks < 8 * 148 ? blocks : 8 * 148);
    };
    if (bad_a) {
        ja = {g.A, g.lda, reinterpret_cast<uint16_t*>(ws), lda2, g.M, g.K};
        g2.A = reinterpret_cast<const uint16_t*>(ws);
        g2.lda = lda2;
    }
    if (bad_b) {
        uint16_t* dst = reinterpret_cast<uint16_t*>(ws + ((bytes_a + 255) & ~size_t(255)));
        jb = {g.B, g.ldb, dst, ldb2, b_rows, static_cast<int>(b_cols)};
        g2.B = dst;
        g2.ldb = ldb2;
    }
    {
        const unsigned na = blocks_of(ja), nb = blocks_of(jb);
        repack_rows_kernel<<<na + nb, 256, 0, stream>>>(ja, jb, na);
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    RunContext c2 = ctx;
    c2.workspace = ws + used;
    c2.workspace_bytes = ctx.workspace_bytes - used;
    c2.kid_flags = 64;
    // The promise "no in-flight work writes B" is about the caller's B; the copy just enqueued IS in-flight
    // work that writes the B this launch reads, so its loads must wait for it like every other access.
    if (bad_b) c2.flags &= ~1u;
    const cudaError_t e = launch_r4_planned(g2, c2, stream, kernel_id);
    ctx.sk_epoch = c2.sk_epoch;          // (state the launch advanced lives in the caller's context)
    ctx.flags &= c2.flags | 1u;          // a one-shot test hook that fired stays fired
    return e;
}

namespace {

cudaError_t launch_r4_planned(const GemmArgs& g, RunContext& ctx, cudaStream_t stream, int* kernel_id, const MultiDst* md)
{
    if (ctx.max_smem_optin < kSmemBytes) return cudaErrorInvalidConfiguration;
    const R4Plan& pinned = ctx.plan;
    const bool generic = !(ctx.encode_tiled && tma_ok(g.A, g.lda, 2) && tma_ok(g.B, g.ldb, 2));
    // Tile width and ring depth of the single-CTA kernel (plain TMA-fed GEMM in the regular orientation only).
    LaunchPlan shape;
    if (!plan_launch(g, ctx, generic, md != nullptr, &shape)) return cudaErrorInvalidValue;
    const int64_t tiles_m = (g.M + BM - 1) / BM, tiles_n = (g.N + shape.tile_n - 1) / shape.tile_n;
    const int64_t tiles = tiles_m * tiles_n;
    if (tiles > 0x3FFFFFFFll) return cudaErrorInvalidConfiguration;

    R4Params p;
    memset(&p, 0, sizeof p);
    p.tile_n = shape.tile_n;
    p.n_stages = shape.stages;
    p.stage_bytes = static_cast<uint32_t>(kABytes + shape.tile_n * BK * 2);
    // Unsplit narrow tiles on their deepest ring pair their k-blocks: 8 x 24 KiB -> 4 stages of two, 6 x 32 KiB -> 3
    // (with a cluster split only if every split still gets work when K is counted in pairs of k-blocks)
    const int nkb_pairs = (g.K + 2 * BK - 1) / (2 * BK);
    const int per_pairs = (nkb_pairs + shape.split.splits - 1) / shape.split.splits;
    const bool pairs_split_evenly = shape.split.splits == 1 || (shape.split.cluster && (nkb_pairs + per_pairs - 1) / per_pairs == shape.split.splits);
    const bool kpair = !generic && md == nullptr && !shape.split.swap && pairs_split_evenly &&
                       ((shape.tile_n == BN / 4 && shape.stages == 8) || (shape.tile_n == BN / 2 && shape.stages == 6));
    if (kpair) {
        p.kpair = 1;
        p.n_stages = shape.stages / 2;
        p.stage_bytes *= 2;
    }
    p.tiles_m = static_cast<int>(tiles_m);
    p.tiles_n = static_cast<int>(tiles_n);
    p.nkb = kpair ? (g.K + 2 * BK - 1) / (2 * BK) : (g.K + BK - 1) / BK;
    p.ldw = (static_cast<int64_t>(g.N) + 3) & ~int64_t(3);
    const SplitPlan plan = shape.split;
    p.splits = plan.splits;
    p.cluster = plan.cluster ? 1 : 0;
    p.static_b = ((ctx.flags & 1u) && shape.tile_n == BN && shape.stages == STAGES) ? 1 : 0;
    p.splits_log2 = plan.splits >= 8 ? 3 : plan.splits >= 4 ? 2 : plan.splits >= 2 ? 1 : 0;
    p.kb_per_split = (p.nkb + p.splits - 1) / p.splits;
    p.ws = static_cast<float*>(ctx.workspace);
    p.counters = ctx.tile_counters;

    // Large aligned problems run on the CTA-pair kernel (tcgen05.mma.cta_group::2).
    if (pinned.kernel == 2 && (plan.swap || plan.splits != 1 || !r4_pair_possible(g, ctx))) return cudaErrorInvalidValue;
    const bool use_pair = pinned.kernel == 2 || (pinned.kernel == 0 && (r4_pair_applicable(g, ctx) || (!md && plan.splits == 1 && !plan.swap && r4_pair_k_paired_auto(g, ctx))));
    if (md && (plan.swap || plan.splits != 1)) return cudaErrorNotSupported;
    if (!plan.swap && plan.splits == 1 && use_pair)
        return md ? launch_r4_pair_multi_dst(g, md->C, md->ldc, md->n, ctx, stream, kernel_id)
                  : launch_r4_tcgen05_pair(g, ctx, stream, kernel_id);

    if (md && generic) return cudaErrorNotSupported;
    const int celt = g.c_bf16 ? 2 : 4;
    // Skinny mode: few activation rows -> they become the MMA's N, the weights its 128 rows.
    const bool swap = plan.swap;
    p.n_mma = (g.M + 15) & ~15;
    // TMA store needs C 16-byte aligned with a 16-byte-multiple pitch, and a row length that is a
    // multiple of 16 bytes: measured on B200, a store box that ends inside a 16-byte unit at the
    // right edge of the tensor writes that whole unit, i.e. up to 12 bytes of row padding.
    p.epi_tma = (!swap && (p.splits == 1 || p.cluster) && ctx.encode_tiled && tma_ok(g.C, g.ldc, celt) &&
                 (static_cast<int64_t>(g.N) * celt) % 16 == 0)
                    ? 1
                    : 0;

    // Instruction descriptor: fp32 accumulator (bits 4-5), bf16 A and B (bits 7-9, 10-12),
    // operand majors (bit 15 A, bit 16 B; 0 = K-major, 1 = MN-major), N >> 3 (bits 17-22),
    // M >> 4 (bits 24-28).  Row-major B is MN-major, column-major B is K-major.
    const uint32_t w_major = g.b_col ? 0u : 1u;
    if (swap)
        p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | (w_major << 15) | (static_cast<uint32_t>(p.n_mma >> 3) << 17) |
                  (static_cast<uint32_t>(128 >> 4) << 24);
    else
        p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | (w_major << 16) | (static_cast<uint32_t>(shape.tile_n >> 3) << 17) |
                  (static_cast<uint32_t>(BM >> 4) << 24);
    // Shared-memory descriptor of B (version 1, 128-byte swizzle):
    //   K-major : 8-row groups 1024 bytes apart; +32 bytes per 16 k
    //   MN-major: 64-column blocks 8192 bytes apart (leading offset), 8-k groups 1024 bytes
    //             apart (stride offset); +2048 bytes per 16 k
    p.b_desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    p.b_desc_lbo = g.b_col ? 1u : ((64u * BK * 2u) >> 4);
    p.b_kstep = g.b_col ? 2u : (2048u >> 4);

    CUtensorMap ma, mb, mc;
    memset(&ma, 0, sizeof ma);
    memset(&mb, 0, sizeof mb);
    memset(&mc, 0, sizeof mc);
    bool ok = true;
    DstEntry table[kMaxDst];
    if (md) {
        // TMA stores only when every destination qualifies (one epilogue form per launch)
        if (md->n < 1 || md->n > kMaxDst || ctx.workspace_bytes < sizeof(DstEntry) * md->n) return cudaErrorInvalidValue;
        memset(table, 0, sizeof(DstEntry) * md->n);
        p.epi_tma = ctx.encode_tiled ? 1 : 0;
        for (int d = 0; d < md->n; ++d) {
            GemmArgs gd = g;
            gd.C = md->C[d];
            gd.ldc = md->ldc[d];
            if (!c_store_by_tma(gd)) p.epi_tma = 0;
            table[d].C = md->C[d];
            table[d].ldc = md->ldc[d];
        }
        for (int d = 0; d < md->n && p.epi_tma && ok; ++d)
            ok = encode_map_2d(ctx, &table[d].map_c,
                               g.c_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, table[d].C, g.N,
                               g.M, table[d].ldc * celt, g.c_bf16 ? 64 : 32, 32, CU_TENSOR_MAP_SWIZZLE_128B);
    }
    // Skinny mode fetches only the activation rows the MMA reads (n_mma of them).
    const uint32_t a_box_rows = swap ? static_cast<uint32_t>(p.n_mma) : BM;
    p.stage_tx = (a_box_rows * BK * 2 + static_cast<uint32_t>(shape.tile_n) * BK * 2) * (p.kpair ? 2u : 1u);
    if (!generic) {
        ok = encode_map_2d(ctx, &ma, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.A, g.K, g.M, g.lda * 2, BK, a_box_rows,
                           CU_TENSOR_MAP_SWIZZLE_128B);
        if (g.b_col)
            ok = ok && encode_map_2d(ctx, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B, g.K, g.N, g.ldb * 2, BK,
                                     static_cast<uint32_t>(shape.tile_n), CU_TENSOR_MAP_SWIZZLE_128B);
        else if (g.N % 64 == 0 && !p.static_b && encode_b_blocks_3d(ctx, &mb, g, static_cast<uint32_t>(shape.tile_n / 64)))
            p.b_box3d = 1;
        else
            ok = ok && encode_map_2d(ctx, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B, g.N, g.K, g.ldb * 2, 64, BK,
                                     CU_TENSOR_MAP_SWIZZLE_128B);
    }
    if (p.epi_tma && !md)
        ok = ok && encode_map_2d(ctx, &mc, g.c_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                                 g.C, g.N, g.M, g.ldc * celt, g.c_bf16 ? 64 : 32, 32, CU_TENSOR_MAP_SWIZZLE_128B);
    if (!ok) return cudaErrorInvalidValue;

    p.kid = kIdTcgen05 + (generic ? 1 : 0) + (p.epi_tma ? 0 : 2) + (p.splits > 1 ? 4 : 0) + (swap ? 8 : 0) +
            (p.cluster ? 16 : 0) + ctx.kid_flags;
    *kernel_id = p.kid;
    // Static schedule.  Without a K split, a last wave that would leave at least half of the
    // SMs idle is cut into 128-column half tiles (twice as many units, half as long).
    p.group_m = pinned.group_m > 0 ? pinned.group_m : 16;   // measured: 16 tile-rows per group re-read least from HBM at 8192^3
    p.full_units = tiles;
    if (p.splits == 1 && !swap && pinned.half_tail != 2 && shape.tile_n == BN) {
        const int64_t tail = tiles % ctx.sm_count;
        const bool pays = 2 * tail <= ctx.sm_count;
        if (tail != 0 && (pays || pinned.half_tail == 1) && g.N > BN / 2) p.full_units = tiles - tail;
    }
    p.total_units = p.splits > 1 ? tiles * p.splits : p.full_units + 2 * (tiles - p.full_units);
    p.idesc_half = (p.idesc & ~(0x3Fu << 17)) | (static_cast<uint32_t>((shape.tile_n / 2) >> 3) << 17);
    const int64_t units = p.total_units;
    p.one_wave = (p.splits == 1 && !p.cluster && p.full_units == tiles && units <= ctx.sm_count && tiles_m > 1) ? 1 : 0;
    // A cluster handles exactly one tile, so the cluster path launches every unit as a CTA.
    const unsigned grid = static_cast<unsigned>((p.cluster || units < ctx.sm_count) ? units : ctx.sm_count);
    if (md) {
        // the table travels on the launch's stream, ahead of the kernel (staged before the call returns)
        const cudaError_t e = cudaMemcpyAsync(ctx.workspace, table, sizeof(DstEntry) * md->n, cudaMemcpyHostToDevice, stream);
        if (e != cudaSuccess) return e;
        p.dsts = static_cast<const DstEntry*>(ctx.workspace);
        p.n_dst = md->n;
        return g.b_col ? launch<true, false, false, 3>(g, ma, mb, mc, p, grid, ctx.device, stream)
                       : launch<false, false, false, 3>(g, ma, mb, mc, p, grid, ctx.device, stream);
    }
    if ((ctx.flags & 2u) && !generic && !p.cluster && !swap && p.kb_per_split > 2) {
        // give-up test hook, this one launch only (never on a cluster or CTA-pair launch: there a CTA that gives
        // up leaves its peers waiting for their own limits)
        p.test_stop_after = 2;
        p.test_poll_limit = 1u << 14;
        ctx.flags &= ~2u;
    }
#define KLIN_R4_LAUNCH(BC, GE, SW) launch<BC, GE, SW>(g, ma, mb, mc, p, grid, ctx.device, stream)
    if (swap) {
        if (g.b_col) return generic ? KLIN_R4_LAUNCH(true, true, true) : KLIN_R4_LAUNCH(true, false, true);
        return generic ? KLIN_R4_LAUNCH(false, true, true) : KLIN_R4_LAUNCH(false, false, true);
    }
    if (g.b_col) return generic ? KLIN_R4_LAUNCH(true, true, false) : KLIN_R4_LAUNCH(true, false, false);
    return generic ? KLIN_R4_LAUNCH(false, true, false) : KLIN_R4_LAUNCH(false, false, false);
#undef KLIN_R4_LAUNCH
}

}  // namespace

namespace {

// The parts of R4Params that depend only on the operand layout (128 x 256 tiles, no K split,
// operands on TMA): shared by the batched and grouped launchers.
void fill_multi_params(R4Params& p, const GemmArgs& g, const RunContext& ctx)
{
    memset(&p, 0, sizeof p);
    p.splits = 1;
    const uint32_t w_major = g.b_col ? 0u : 1u;
    p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | (w_major << 16) | (static_cast<uint32_t>(BN >> 3) << 17) |
              (static_cast<uint32_t>(BM >> 4) << 24);
    p.idesc_half = (p.idesc & ~(0x3Fu << 17)) | (static_cast<uint32_t>((BN / 2) >> 3) << 17);
    p.b_desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    p.b_desc_lbo = g.b_col ? 1u : ((64u * BK * 2u) >> 4);
    p.b_kstep = g.b_col ? 2u : (2048u >> 4);
    p.n_mma = 16;
    p.stage_tx = kABytes + kBBytes;
    p.group_m = ctx.plan.group_m > 0 ? ctx.plan.group_m : 16;
    p.tile_n = BN;
    p.n_stages = STAGES;
    p.stage_bytes = kStageBytes;
}

// Static schedule over `tiles` whole tiles: a last wave that would leave at least half of the
// SMs idle is cut into 128-column half tiles (when every problem is wider than 128 columns).
unsigned finish_multi_schedule(R4Params& p, int64_t tiles, bool halves_ok, const RunContext& ctx)
{
    p.full_units = tiles;
    const int64_t tail = tiles % ctx.sm_count;
    if (halves_ok && tail != 0 && 2 * tail <= ctx.sm_count) p.full_units = tiles - tail;
    p.total_units = p.full_units + 2 * (tiles - p.full_units);
    return static_cast<unsigned>(p.total_units < ctx.sm_count ? p.total_units : ctx.sm_count);
}

bool c_store_by_tma(const GemmArgs& g)
{
    const int celt = g.c_bf16 ? 2 : 4;
    return tma_ok(g.C, g.ldc, celt) && (static_cast<int64_t>(g.N) * celt) % 16 == 0;
}

}  // namespace

bool r4_single_batched_possible(const GemmArgs& g, const BatchArgs& b, const RunContext& ctx)
{
    if (!ctx.encode_tiled || ctx.max_smem_optin < kSmemBytes || b.batch < 1 || b.batch > 65535) return false;
    if (!tma_ok(g.A, g.lda, 2) || !tma_ok(g.B, g.ldb, 2)) return false;
    auto ok = [](int64_t stride_elems) {
        return stride_elems > 0 && (stride_elems * 2) % 16 == 0 && stride_elems * 2 < (int64_t(1) << 40);
    };
    if (!ok(b.stride_a) || !ok(b.stride_b)) return false;
    const int64_t tiles = static_cast<int64_t>((g.M + BM - 1) / BM) * ((g.N + BN - 1) / BN);
    return tiles * b.batch < 0x3FFFFFFFll;
}

cudaError_t launch_r4_single_batched(const GemmArgs& g, const BatchArgs& b, RunContext& ctx, cudaStream_t stream,
                                     int* kernel_id)
{
    if (!r4_single_batched_possible(g, b, ctx)) return cudaErrorInvalidValue;
    R4Params p;
    fill_multi_params(p, g, ctx);
    p.tiles_m = (g.M + BM - 1) / BM;
    p.tiles_n = (g.N + BN - 1) / BN;
    p.tiles_per_batch = p.tiles_m * p.tiles_n;
    p.nkb = (g.K + BK - 1) / BK;
    p.kb_per_split = p.nkb;
    const int celt = g.c_bf16 ? 2 : 4;
    p.stride_c_bytes = b.stride_c * celt;
    p.epi_tma = (c_store_by_tma(g) && p.stride_c_bytes % 16 == 0 && p.stride_c_bytes > 0 &&
                 p.stride_c_bytes < (int64_t(1) << 40))
                    ? 1
                    : 0;
    CUtensorMap ma, mb, mc;
    memset(&ma, 0, sizeof ma);
    memset(&mb, 0, sizeof mb);
    memset(&mc, 0, sizeof mc);
    const uint64_t nb = static_cast<uint64_t>(b.batch);
    bool ok = encode_map_3d(ctx, &ma, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.A, g.K, g.M, nb, g.lda * 2, b.stride_a * 2, BK,
                            BM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (g.b_col)
        ok = ok && encode_map_3d(ctx, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B, g.K, g.N, nb, g.ldb * 2, b.stride_b * 2,
                                 BK, BN, CU_TENSOR_MAP_SWIZZLE_128B);
    else if (g.N % 64 == 0 && ctx.encode_tiled) {
        // the four 64-column blocks of a stage as one box: B as (64 columns, K rows, N / 64 blocks, batch)
        const cuuint64_t dims[4] = {64, static_cast<cuuint64_t>(g.K), static_cast<cuuint64_t>(g.N / 64), nb};
        const cuuint64_t strides[3] = {static_cast<cuuint64_t>(g.ldb) * 2, 128, static_cast<cuuint64_t>(b.stride_b) * 2};
        const cuuint32_t box[4] = {64, BK, BN / 64, 1};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        ok = ok && ctx.encode_tiled(&mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<uint16_t*>(g.B), dims, strides, box,
                                    estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
        p.b_box3d = 1;
    } else
        ok = ok && encode_map_3d(ctx, &mb, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B, g.N, g.K, nb, g.ldb * 2, b.stride_b * 2,
                                 64, BK, CU_TENSOR_MAP_SWIZZLE_128B);
    if (p.epi_tma)
        ok = ok && encode_map_3d(ctx, &mc, g.c_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                                 g.C, g.N, g.M, nb, g.ldc * celt, static_cast<uint64_t>(p.stride_c_bytes),
                                 g.c_bf16 ? 64 : 32, 32, CU_TENSOR_MAP_SWIZZLE_128B);
    if (!ok) return cudaErrorInvalidValue;
    p.kid = kIdTcgen05 + (p.epi_tma ? 0 : 2) + ctx.kid_flags;
    *kernel_id = p.kid;
    const unsigned grid = finish_multi_schedule(p, static_cast<int64_t>(p.tiles_per_batch) * b.batch, g.N > BN / 2, ctx);
    return g.b_col ? launch<true, false, false, 1>(g, ma, mb, mc, p, grid, ctx.device, stream)
                   : launch<false, false, false, 1>(g, ma, mb, mc, p, grid, ctx.device, stream);
}

bool r4_single_grouped_possible(const GemmArgs* groups, int n, const RunContext& ctx)
{
    if (!ctx.encode_tiled || ctx.max_smem_optin < kSmemBytes) return false;
    if (n < 1 || n > kMaxGroups || ctx.workspace_bytes < static_cast<size_t>(n) * sizeof(GroupEntry)) return false;
    int64_t tiles = 0;
    for (int i = 0; i < n; ++i) {
        const GemmArgs& g = groups[i];
        if (g.M <= 0 || g.N <= 0 || g.K <= 0) return false;          // the caller drops empty groups
        if (!tma_ok(g.A, g.lda, 2) || !tma_ok(g.B, g.ldb, 2)) return false;
        tiles += static_cast<int64_t>((g.M + BM - 1) / BM) * ((g.N + BN - 1) / BN);
    }
    return tiles < 0x3FFFFFFFll;
}

cudaError_t launch_r4_single_grouped(const GemmArgs* groups, int n, RunContext& ctx, cudaStream_t stream,
                                     int* kernel_id)
{
    if (!r4_single_grouped_possible(groups, n, ctx)) return cudaErrorInvalidValue;
    GroupEntry* table = new (std::nothrow) GroupEntry[n];
    if (!table) return cudaErrorMemoryAllocation;
    memset(table, 0, sizeof(GroupEntry) * n);
    R4Params p;
    fill_multi_params(p, groups[0], ctx);
    p.tiles_m = p.tiles_n = 1;      // unused by the grouped schedule; kept non-zero
    int tile_start = 0;
    bool ok = true, any_tma = false, halves_ok = true;
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
        e.tiles_m = (g.M + BM - 1) / BM;
        e.tiles_n = (g.N + BN - 1) / BN;
        e.tile_start = tile_start;
        tile_start += e.tiles_m * e.tiles_n;
        e.epi_tma = c_store_by_tma(g) ? 1 : 0;
        any_tma = any_tma || e.epi_tma;
        halves_ok = halves_ok && g.N > BN / 2;
        ok = encode_map_2d(ctx, &e.map_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.A, g.K, g.M, g.lda * 2, BK, BM,
                           CU_TENSOR_MAP_SWIZZLE_128B);
        if (g.b_col)
            ok = ok && encode_map_2d(ctx, &e.map_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B, g.K, g.N, g.ldb * 2, BK, BN,
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
    // The table travels on the launch's stream, ahead of the kernel that reads it (the copy from
    // pageable memory is staged before the call returns, so the host array can go).
    if (err == cudaSuccess)
        err = cudaMemcpyAsync(ctx.workspace, table, sizeof(GroupEntry) * n, cudaMemcpyHostToDevice, stream);
    delete[] table;
    if (err != cudaSuccess) return err;
    p.groups = static_cast<const GroupEntry*>(ctx.workspace);
    p.n_groups = n;
    p.epi_tma = any_tma ? 1 : 0;
    p.kid = kIdTcgen05 + (any_tma ? 0 : 2) + ctx.kid_flags;
    *kernel_id = p.kid;
    const unsigned grid = finish_multi_schedule(p, tile_start, halves_ok, ctx);
    CUtensorMap none;
    memset(&none, 0, sizeof none);
    const GemmArgs& g0 = groups[0];
    return g0.b_col ? launch<true, false, false, 2>(g0, none, none, none, p, grid, ctx.device, stream)
                    : launch<false, false, false, 2>(g0, none, none, none, p, grid, ctx.device, stream);
}

cudaError_t launch_r4_conv2d(const GemmArgs& g, const ConvGeom& geom, RunContext& ctx, cudaStream_t stream,
                             int* kernel_id)
{
    if (ctx.max_smem_optin < kSmemBytes || !g.b_col || g.M <= 0 || g.N <= 0 || g.K <= 0) return cudaErrorInvalidValue;
    R4Params p;
    fill_multi_params(p, g, ctx);
    if (g.f16) {   // operand format fields of the instruction descriptor: 0 = fp16, 1 = bf16
        p.idesc &= ~((1u << 7) | (1u << 10));
        p.idesc_half &= ~((1u << 7) | (1u << 10));
    }
    p.tiles_m = (g.M + BM - 1) / BM;
    p.tiles_n = (g.N + BN - 1) / BN;
    p.nkb = (g.K + BK - 1) / BK;
    p.kb_per_split = p.nkb;
    p.conv = geom;
    p.conv_fast = (geom.C % 8 == 0 && reinterpret_cast<uintptr_t>(g.A) % 16 == 0) ? 1 : 0;
    p.half_only = g.N <= BN / 2 ? 1 : 0;
    p.conv_b_rows = p.half_only ? BN / 2 : BN;
    CUtensorMap mb;
    memset(&mb, 0, sizeof mb);
    p.conv_b_tma = (p.conv_fast && ctx.encode_tiled && tma_ok(g.B, g.ldb, 2) &&
                    encode_map_2d(ctx, &mb, g.f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, g.B,
                                  g.K, g.N, g.ldb * 2, BK, static_cast<uint32_t>(p.conv_b_rows), CU_TENSOR_MAP_SWIZZLE_128B))
                       ? 1
                       : 0;
    const int celt = g.c_bf16 ? 2 : 4;
    p.epi_tma = (ctx.encode_tiled && c_store_by_tma(g)) ? 1 : 0;
    CUtensorMap none, mc;          // (every tensor map is encoded only on the path that uses it: an encode costs ~1 us of host time)
    memset(&none, 0, sizeof none);
    memset(&mc, 0, sizeof mc);
    const int64_t tiles = static_cast<int64_t>(p.tiles_m) * p.tiles_n;
    if (tiles > 0x3FFFFFFFll) return cudaErrorInvalidValue;
    unsigned grid;
    if (p.half_only) {      // one 128-column half tile per row block: the MMA runs at N = 128
        p.full_units = 0;
        p.total_units = tiles;
        grid = static_cast<unsigned>(tiles < ctx.sm_count ? tiles : ctx.sm_count);
    } else {
        grid = finish_multi_schedule(p, tiles, true, ctx);
    }
    // Patches by TMA: 64-channel groups (a k-block is one tap of one group) and unit stride.  The rows are
    // then tiled as 8 x 16 pixel patches of the output (one 16 KiB TMA box per k-block, clipped stores at the
    // image edges) instead of 128 consecutive pixels.
    CUtensorMap mx;
    memset(&mx, 0, sizeof mx);
    const int64_t n_img = g.M / (static_cast<int64_t>(geom.P) * geom.Q);
    const int tq = (geom.Q + 15) / 16, tp = (geom.P + 7) / 8;
    const int64_t patch_tiles = n_img * tp * tq * p.tiles_n;
    bool patch_tma = p.conv_b_tma && geom.C % 64 == 0 && geom.stride_h == 1 && geom.stride_w == 1 &&
                     patch_tiles < 0x3FFFFFFFll / BM &&
                     encode_map_nhwc(ctx, &mx, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, g.A, geom.C, geom.W, geom.H,
                                     static_cast<uint64_t>(n_img), 64, 16, 8, 2, CU_TENSOR_MAP_SWIZZLE_128B);
    CUtensorMap my;
    memset(&my, 0, sizeof my);
    const bool transposed = patch_tma && p.half_only && patch_tiles >= 2 && g.c_bf16 && p.epi_tma &&
                            encode_map_nhwc(ctx, &my, g.f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                                            g.C, g.N, geom.Q, geom.P, static_cast<uint64_t>(n_img), 32, 16, 4, 2,
                                            CU_TENSOR_MAP_SWIZZLE_NONE);
    if (patch_tma && p.epi_tma && !transposed)   // y as a 4-D tensor (F, Q, P, N): a warp stores 2 patch rows x 16 pixels per box
        patch_tma = encode_map_nhwc(ctx, &mc, g.c_bf16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                                    g.C, g.N, geom.Q, geom.P, static_cast<uint64_t>(n_img), g.c_bf16 ? 64 : 32, 16, 2, celt,
                                    CU_TENSOR_MAP_SWIZZLE_128B);
    if (!patch_tma && p.epi_tma &&
        !encode_map_2d(ctx, &mc, g.c_bf16 ? (g.f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16)
                                          : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                       g.C, g.N, g.M, g.ldc * celt, g.c_bf16 ? 64 : 32, 32, CU_TENSOR_MAP_SWIZZLE_128B))
        return cudaErrorInvalidValue;
    p.kid = kIdConvTcgen05 + (patch_tma ? 0 : 4) + (p.epi_tma ? 0 : 2) + (p.conv_fast ? 0 : 1);
    *kernel_id = p.kid;
    if (patch_tma) {
        // the schedule runs over patch tiles: a virtual row count of 128 per patch (clipping happens in the stores)
        GemmArgs gp = g;
        gp.M = static_cast<int>(n_img * tp * tq * BM);
        p.conv_patch = 1;
        p.conv_tq = tq;
        p.conv_tp = tp;
        p.tiles_m = static_cast<int>(n_img * tp * tq);
        p.stage_tx = kABytes + static_cast<uint32_t>(p.conv_b_rows) * 128u;
        p.conv_ring6 = p.half_only;         // 16 KiB filter blocks: six stages fit where four full ones do
        if (transposed) {
            // At most 128 filters: run the product transposed (filters = the 128-row operand, two patch tiles =
            // 256 pixels as the N operand), so that every MMA is full width; the epilogue stores y transposed.
            const int64_t units = (patch_tiles + 1) / 2;
            p.conv_t = 1;
            p.conv_ring6 = 0;
            p.conv_nimg = static_cast<int>(n_img);
            p.half_only = 0;
            p.epi_tma = 1;                 // (the kernel end waits for its stores; the map is this mode's own)
            p.tiles_m = static_cast<int>(units);
            p.tiles_n = 1;
            p.full_units = p.total_units = units;
            p.stage_tx = kStageBytes;
            gp.M = static_cast<int>(units * BM);
            p.kid = kIdConvTcgen05 + 8;
            *kernel_id = p.kid;
            const unsigned tgrid = static_cast<unsigned>(units < ctx.sm_count ? units : ctx.sm_count);
            return launch<true, false, false, 4>(gp, mx, mb, my, p, tgrid, ctx.device, stream);
        }
        unsigned pgrid;
        if (p.half_only) {
            p.full_units = 0;
            p.total_units = patch_tiles;
            pgrid = static_cast<unsigned>(patch_tiles < ctx.sm_count ? patch_tiles : ctx.sm_count);
        } else {
            pgrid = finish_multi_schedule(p, patch_tiles, true, ctx);
        }
        return launch<true, false, false, 4>(gp, mx, mb, mc, p, pgrid, ctx.device, stream);
    }
    return launch<true, true, false, 4>(g, none, mb, mc, p, grid, ctx.device, stream);
}

bool r4_multi_dst_possible(const GemmArgs& g, const RunContext& ctx)
{
    if (!ctx.encode_tiled || ctx.max_smem_optin < kSmemBytes || g.M <= 0 || g.N <= 0 || g.K <= 0) return false;
    if (!tma_ok(g.A, g.lda, 2) || !tma_ok(g.B, g.ldb, 2)) return false;
    LaunchPlan lp;
    if (!plan_launch(g, ctx, false, true, &lp)) return false;
    return !lp.split.swap && lp.split.splits == 1;
}

cudaError_t launch_r4_multi_dst(const GemmArgs& g, void* const* C, const int64_t* ldc, int n_dst, RunContext& ctx,
                                cudaStream_t stream, int* kernel_id)
{
    if (!C || !ldc || n_dst < 1 || n_dst > kMaxDst) return cudaErrorInvalidValue;
    const MultiDst md = {C, ldc, n_dst};
    return launch_r4_planned(g, ctx, stream, kernel_id, &md);
}

bool r4_narrow_tiles_fill_better(int64_t M, int64_t N, int sm_count)
{
    if (M <= 0 || N <= 0) return false;
    const int64_t tm = (M + BM - 1) / BM, wide = (N + BN - 1) / BN, narrow = (N + BN / 2 - 1) / (BN / 2);
    if (tm * narrow > sm_count) return false;
    const double fill_wide = static_cast<double>(N) / static_cast<double>(wide * BN);
    const double fill_narrow = static_cast<double>(N) / static_cast<double>(narrow * (BN / 2));
    return fill_narrow >= fill_wide + 0.08;
}

bool r4_plan_valid(const GemmArgs& g, const RunContext& ctx, const R4Plan& pl)
{
    if (pl.kernel < 0 || pl.kernel > 2 || pl.splits < 0 || pl.split_via < 0 || pl.split_via > 3 || pl.group_m < 0 ||
        pl.group_m > 1024 || pl.half_tail < 0 || pl.half_tail > 2 || pl.tile_n < 0 || pl.tail_n < 0 || pl.stages < 0)
        return false;
    // tile widths: the pair kernel takes multiples of 64 columns (and a second, narrower width for the tiles
    // that balance its last wave)
    if (pl.tile_n != 0 && (pl.tile_n < 64 || pl.tile_n > 256 || pl.tile_n % 64 != 0)) return false;
    if (pl.tail_n != 0 && (pl.tail_n < 64 || pl.tail_n > 256 || pl.tail_n % 64 != 0 || pl.tail_n > (pl.tile_n ? pl.tile_n : 256)))
        return false;
    if (pl.tail_n != 0 && pl.kernel != 2) return false;
    if (pl.split_via == 3 && (pl.kernel != 2 || pl.splits > 1)) return false;     // streaming the last wave is the pair kernel's
    // CTA-pair kernel: stages = 3 asks for k-paired 256-row tiles (three stages of two k-blocks), 256 columns wide
    if (pl.kernel == 2 && pl.stages != 0 &&
        !(pl.stages == 3 && (pl.tile_n == 0 || pl.tile_n == BN) && pl.tail_n == 0 && pl.split_via != 3))
        return false;
    if (pl.kernel != 2 && (pl.tile_n != 0 || pl.stages != 0)) {
        // single-CTA kernel: 256 columns x 4 stages, 128 columns x 4 or 6, 64 columns x 4, 6 or 8 (plain TMA-fed GEMM, M > 64)
        if (pl.tile_n != 0 && pl.tile_n != BN && pl.tile_n != BN / 2 && pl.tile_n != BN / 4) return false;
        if (pl.stages != 0 && pl.stages != 4 && pl.stages != 6 && !(pl.stages == 8 && pl.tile_n == BN / 4)) return false;
    }
    // a tile shape is a property of one of the two kernels: name the kernel with it
    if ((pl.tile_n != 0 || pl.tail_n != 0 || pl.stages != 0) && pl.kernel == 0) return false;
    if (g.M <= 0 || g.N <= 0 || g.K <= 0) return true;   // nothing to launch; any plan is moot
    RunContext c2 = ctx;
    c2.plan = pl;
    // (unaligned operands that the launch repacks into the workspace run the TMA-fed kernel)
    const bool aligned = ctx.encode_tiled && tma_ok(g.A, g.lda, 2) && tma_ok(g.B, g.ldb, 2);
    LaunchPlan lp;
    if (!plan_launch(g, c2, !aligned && !ctx.allow_repack, false, &lp)) return false;
    const SplitPlan& sp = lp.split;
    if (pl.kernel == 2 && (sp.swap || sp.splits != 1 || !r4_pair_possible(g, ctx))) return false;
    if (pl.split_via == 3 && (pl.tile_n % 256 != 0 || (pl.tail_n != 0 && pl.tail_n != 256) || !r4_pair_stream_k_possible(g, ctx)))
        return false;
    return true;
}

// Candidates: both kernels where the pair kernel can run, a few raster groups, the half-tile
// tail on and off, and K splits around the heuristic's choice.  Unaligned operands are tuned
// as they run (after the repack, aligned): the caller passes the problem it will run.
int r4_enumerate_plans(const GemmArgs& g, const RunContext& ctx, R4Plan* out, int cap)
{
    int n = 0;
    auto push = [&](const R4Plan& pl) {
        if (n >= cap || !r4_plan_valid(g, ctx, pl)) return;
        for (int i = 0; i < n; ++i)
            if (out[i].kernel == pl.kernel && out[i].splits == pl.splits && out[i].split_via == pl.split_via &&
                out[i].group_m == pl.group_m && out[i].half_tail == pl.half_tail && out[i].tile_n == pl.tile_n &&
                out[i].tail_n == pl.tail_n && out[i].stages == pl.stages)
                return;
        out[n++] = pl;
    };
    push(R4Plan());
    if (g.M <= 0 || g.N <= 0 || g.K <= 0) return n;
    const int64_t tiles_m = (g.M + BM - 1) / BM, tiles_n = (g.N + BN - 1) / BN;
    const int64_t tiles = tiles_m * tiles_n;
    const int nkb = (g.K + BK - 1) / BK;
    const bool swap = g.M <= 64;
    if (!swap) {
        if (r4_pair_possible(g, ctx) && g.M > BM)
            for (int gm : {2, 4, 8, 16}) {
                if (gm > 2 && gm / 2 >= (g.M + 511) / 512) continue;   // more rows per group than there are
                R4Plan pl;
                pl.kernel = 2;
                pl.splits = 1;
                pl.group_m = gm;
                push(pl);
            }
        if (r4_pair_possible(g, ctx) && g.M > BM) {
            // tile widths of the pair kernel: uniform 192 / 128 columns, and 256 with a narrow tail
            for (int w : {192, 128}) {
                R4Plan pl;
                pl.kernel = 2;
                pl.splits = 1;
                pl.tile_n = w;
                pl.tail_n = w;
                push(pl);
            }
            R4Plan pl;
            pl.kernel = 2;
            pl.splits = 1;
            pl.tile_n = 256;
            pl.tail_n = 192;
            push(pl);
            // 256-row tiles, two k-blocks per stage
            if (g.M > 2 * BM) {
                R4Plan pk;
                pk.kernel = 2;
                pk.splits = 1;
                pk.stages = 3;
                push(pk);
            }
            // last wave streamed along K, and never streamed
            for (int via : {3, 1}) {
                R4Plan ps;
                ps.kernel = 2;
                ps.splits = 1;
                ps.split_via = via;
                push(ps);
            }
        }
        // tile shapes of the single-CTA kernel: 128 columns on a 4- or 6-stage ring
        for (int st : {4, 6}) {
            R4Plan pl;
            pl.kernel = 1;
            pl.splits = 1;
            pl.tile_n = BN / 2;
            pl.stages = st;
            push(pl);
        }
        if (tiles * 2 <= ctx.sm_count) {     // few tiles: 64 columns
            for (int st : {4, 8}) {
                R4Plan pl;
                pl.kernel = 1;
                pl.splits = 1;
                pl.tile_n = BN / 4;
                pl.stages = st;
                push(pl);
            }
        }
        for (int gm : {4, 8, 16, 32}) {
            if (gm > 4 && gm / 2 >= tiles_m) continue;
            for (int ht : {1, 2}) {
                if (ht == 1 && tiles % ctx.sm_count == 0) continue;
                R4Plan pl;
                pl.kernel = 1;
                pl.splits = 1;
                pl.group_m = gm;
                pl.half_tail = ht;
                push(pl);
            }
        }
    }
    // K splits: when the unsplit tiles leave SMs idle
    if (tiles < ctx.sm_count) {
        const int64_t want = ctx.sm_count / tiles;   // splits that fill one wave
        for (int s : {2, 3, 4, 6, 8, 12, 16, 24, 32}) {
            if (s > 2 * want + 1) continue;
            R4Plan pl;
            pl.kernel = 1;
            pl.splits = s;
            pl.split_via = 1;
            push(pl);
            if ((!swap || g.M <= 32) && (s == 2 || s == 4 || s == 8)) {
                pl.split_via = 2;
                push(pl);
                if (!swap) {
                    pl.tile_n = BN / 2;
                    pl.stages = 6;
                    push(pl);
                }
            }
        }
        R4Plan pl;
        pl.kernel = 1;
        pl.splits = 1;
        push(pl);
    }
    (void)nkb;
    return n;
}

}  // namespace klin

// ---------------------------------------------------------------------------
// Allocation-free entry point.
//
// klineage_gemm_run_noalloc runs the tcgen05 rung without a handle and without
// ever asking the CUDA allocator for memory.  Everything the kernel needs beyond
// the caller's A, B and C - the split-K partial sums, the per-row-block arrival
// counters and the four status words - lives in the fixed array below, which is
// part of the library image: each GPU that loads the library reserves these
// bytes until the process exits.
namespace klin {
namespace {

constexpr size_t kNoAllocPartialBytes = size_t(8) << 20;   // split-K partial sums (fp32)
constexpr int kNoAllocCounters = 4096;                     // arrival counters (one per tile and 32-row block)
constexpr size_t kNoAllocScratchBytes = kNoAllocPartialBytes + kNoAllocCounters * sizeof(unsigned) + 256;

}  // namespace
}  // namespace klin

static __device__ __align__(256) unsigned char g_noalloc_scratch[klin::kNoAllocScratchBytes];

namespace klin {
namespace {

// Per-device state of the entry point.  In host code the name g_noalloc_scratch
// is only a stand-in for the device array, so the real device address is looked
// up once per device (with that device current) and kept here.
struct NoAllocDevice {
    bool ready = false;
    unsigned char* scratch = nullptr;
    unsigned* status = nullptr;
    RunContext ctx;
};
NoAllocDevice g_noalloc_devices[64];
std::mutex g_noalloc_mutex;

klineage_status_t noalloc_setup(int device, NoAllocDevice** out)
{
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    NoAllocDevice& d = g_noalloc_devices[device];
    if (!d.ready) {
        unsigned char* ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_scratch);
        if (e != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            fprintf(stderr, "klineage_gemm_run_noalloc: cudaGetSymbolAddress failed: %s\n", cudaGetErrorString(e));
            return KLINEAGE_ERR_INTERNAL;
        }
        RunContext& c = d.ctx;
        c.device = device;
        cudaDeviceGetAttribute(&c.sm_count, cudaDevAttrMultiProcessorCount, device);
        cudaDeviceGetAttribute(&c.cc_major, cudaDevAttrComputeCapabilityMajor, device);
        cudaDeviceGetAttribute(&c.cc_minor, cudaDevAttrComputeCapabilityMinor, device);
        cudaDeviceGetAttribute(&c.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            c.encode_tiled = reinterpret_cast<TensorMapEncodeTiledFn>(fn);
        else
            cudaGetLastError();
        d.scratch = ptr;
        c.workspace = ptr;
        c.workspace_bytes = kNoAllocPartialBytes;
        c.tile_counters = reinterpret_cast<unsigned*>(ptr + kNoAllocPartialBytes);
        c.n_tile_counters = kNoAllocCounters;
        d.status = c.tile_counters + kNoAllocCounters;
        c.allow_repack = false;   // its fixed scratch is reserved for split-K partial sums
        d.ready = true;
    }
    *out = &d;
    return KLINEAGE_OK;
}

}  // namespace
}  // namespace klin

extern "C" klineage_status_t klineage_gemm_run_noalloc(int b_layout, int c_dtype, int64_t M, int64_t N, int64_t K,
                                                       const void* A, int64_t lda, const void* B, int64_t ldb,
                                                       void* C, int64_t ldc, void* stream)
{
    using namespace klin;
    const klineage_status_t chk =
        klineage_gemm_check_args(b_layout, c_dtype, M, N, K, A, lda, B, ldb, C, ldc, KLINEAGE_TCGEN05);
    if (chk != KLINEAGE_OK) return chk;
    if (M == 0 || N == 0) return KLINEAGE_OK;

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) {
        cudaGetLastError();
        return KLINEAGE_ERR_INVALID_ARG;
    }
    // (before the symbol lookup: the library image holds sm_100a code only, so on any other device the
    // lookup itself fails and would hide the real reason)
    int cc_major = 0;
    if (cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) {
        cudaGetLastError();
        return KLINEAGE_ERR_INTERNAL;
    }
    if (cc_major != 10) return KLINEAGE_ERR_UNSUPPORTED_DEVICE;
    NoAllocDevice* d = nullptr;
    const klineage_status_t st = noalloc_setup(device, &d);
    if (st != KLINEAGE_OK) return st;

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
    g.b_col = b_layout == KLINEAGE_B_COL_MAJOR ? 1 : 0;
    g.c_bf16 = c_dtype == KLINEAGE_C_BF16 ? 1 : 0;
    g.status = d->status;
    g.bias = nullptr;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int kid = -1;
    if (K == 0) return launch_zero_fill(g, s, &kid) == cudaSuccess ? KLINEAGE_OK : KLINEAGE_ERR_LAUNCH;

    // Refuse, rather than quietly change the schedule, when the K split this
    // shape would get needs more partial-sum space than the fixed array holds.
    const int64_t ldw = (N + 3) & ~int64_t(3);
    RunContext unlimited = d->ctx;
    unlimited.workspace_bytes = ~size_t(0);
    unlimited.plan = R4Plan();
    SplitPlan plan;
    plan.splits = 1;
    plan.cluster = false;
    {
        const bool generic = !(unlimited.encode_tiled && tma_ok(g.A, g.lda, 2) && tma_ok(g.B, g.ldb, 2));
        LaunchPlan lp;
        if (plan_launch(g, unlimited, generic, false, &lp)) plan = lp.split;
    }
    const size_t need =
        (plan.splits > 1 && !plan.cluster) ? static_cast<size_t>(plan.splits) * M * ldw * sizeof(float) : 0;
    if (need > kNoAllocPartialBytes) {
        fprintf(stderr,
                "klineage_gemm_run_noalloc: M=%lld N=%lld K=%lld needs %zu bytes of split-K scratch, the fixed "
                "array holds %zu; use klineage_gemm_run with a handle for this shape\n",
                static_cast<long long>(M), static_cast<long long>(N), static_cast<long long>(K), need,
                kNoAllocPartialBytes);
        return KLINEAGE_ERR_SCRATCH_LIMIT;
    }

    // The array keeps whatever the previous call left: counters and status must start at zero.
    if (cudaMemsetAsync(d->ctx.tile_counters, 0, (kNoAllocCounters + 4) * sizeof(unsigned), s) != cudaSuccess) {
        cudaGetLastError();
        return KLINEAGE_ERR_LAUNCH;
    }
    if (launch_r4_tcgen05(g, d->ctx, s, &kid) != cudaSuccess) {
        cudaGetLastError();
        return KLINEAGE_ERR_LAUNCH;
    }
    return KLINEAGE_OK;
}
