// Shared pieces of the pvf_score projection kernels: tile constants, pipeline control block, PTX wrappers
// (mbarrier, TMA, tcgen05), the vocabulary work split and the running softmax state of one row.
// (A part of pvf_score.cu's translation unit; see that file for the overview.)
#pragma once
#include <math.h>

#include "pvf_internal.h"


namespace {


// Tile shapes and the row windows of the four kernels (settled by measurement).
constexpr int kGeneralTileN = 256;         // 128-row GEMM kernel: vocabulary entries per accumulator
constexpr int kGeneralPanels = 1;          //   64-element k-panels per pipeline stage
constexpr int kGeneralStages = 4;          //   pipeline stages
constexpr int kPairMinTiles = 2;           // 128-row tiles from which the paired (cta_group::2) kernel takes over
constexpr int kSwapSmallMaxRows = 64;      // 33 .. this many rows take the swapped paired kernel
constexpr int kSwapRaggedMaxRows = 192;    // and so do 129 .. this many rows (at most 256)
constexpr int kSwapWideWarps = 3;          // epilogue warps per lane quadrant of the swapped paired kernel above 256 rows
constexpr int kSwapWideMaxRows = 448;      // and 257 .. this many rows (at most 512), in two column groups

constexpr int kTileM = 128;                // rows per accumulator (tensor-memory lanes)
constexpr int kUnit = 16;                  // vocabulary granule
constexpr int kBlockK = 64;                // bf16 per k-panel = one 128-byte swizzle row
constexpr int kRowBytes = kBlockK * 2;     // 128
constexpr int kUnitBytes = kUnit * kRowBytes;          // 2 KiB
constexpr int kThreads = 192;
constexpr int kEpilogueThreads = 128;
constexpr int kMaxStages = 16;
constexpr int kStreamRows = 32;            // the streaming kernel handles at most this many rows
constexpr int kWBoxSizes = PVF_W_BOX_SIZES;             // W boxes of 16, 32, ..., 256 vocabulary entries
constexpr int kMaxConcurrentTiles = 64;    // cap on the wave's L2-resident H tiles
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

template <int TILE_N, int PANELS, int STAGES>
struct GemmCfg {
    static constexpr int kTileN = TILE_N;              // vocabulary entries per accumulator (columns)
    static constexpr int kPanels = PANELS;             // 64-element k-panels per stage
    static constexpr int kStages = STAGES;
    static constexpr int kAPanelBytes = kTileM * kRowBytes;
    static constexpr int kBPanelBytes = TILE_N * kRowBytes;
    static constexpr int kStageBytes = PANELS * (kAPanelBytes + kBPanelBytes);
    static constexpr int kUnitsPerTile = TILE_N / kUnit;
    static constexpr int kTmemCols = 2 * TILE_N;
    static constexpr int kControlBytes = 512;
    static constexpr int kSmemBytes = STAGES * kStageBytes + 1024 /*alignment slack*/ + kControlBytes;
    static_assert(TILE_N == 64 || TILE_N == 128 || TILE_N == 256, "accumulator width");
    static_assert(STAGES >= 2 && STAGES <= kMaxStages, "stages");
    static_assert(kSmemBytes <= 227 * 1024, "shared memory");
};

using GeneralCfg = GemmCfg<kGeneralTileN, kGeneralPanels, kGeneralStages>;

struct __align__(8) SharedControl {
    unsigned long long full[kMaxStages];   // TMA bytes landed
    unsigned long long empty[kMaxStages];  // MMAs that read the stage have completed
    unsigned long long acc_full[2];        // accumulator complete
    unsigned long long acc_empty[2];       // epilogue has drained the accumulator
    unsigned long long drain;              // abort path: all issued MMAs completed
    unsigned long long drain2;             // the same for the streaming kernel's second issuer
    uint32_t tmem_base;
    volatile int abort_flag;
};
static_assert(sizeof(SharedControl) <= 512, "control block");

// W as [V][D] seen through boxes of 16 * n rows x 64 columns, n = 1 .. 16: a vocabulary tile of any
// whole number of granules is one TMA instruction (the producer thread is bound by the instructions
// it issues, not by the bytes they move).
struct WMaps {
    CUtensorMap size[kWBoxSizes];
};

struct ScoreArgs {
    int M, V, D;
    int num_kb;          // ceil(D / 64)
    int units;           // ceil(V / 16)
    int m_tiles, mb, splits, waves;
    int mb_last, splits_last;   // paired kernel: geometry of a partial last wave (mb_last = 0: every wave is full)
    int a_rows;          // rows per H box
    int n_pad, stages;   // swapped paired kernel: rows per row tile (MMA N), pipeline stages
    int w_once;          // 1: the launch reads every W tile exactly once (its L2 lines are marked evict-first)
    int parts;           // partial states per row (row stride of `partials`)
    float4 *partials;    // [M][parts]
    int32_t *status;
    uint32_t *wave_sync; // paired kernel with several waves: {arrivals, done} counters of the wave boundaries, else nullptr
    unsigned long long *clock_acc;   // {ns, cycles, launches} sums of block 0's run (see LaunchClock), or nullptr
};

// ---------------------------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Block 0 measures its own run in wall time (%globaltimer) and in SM cycles (clock64) and adds both to the context's
// sums: cycles / time is the SM clock the launch really ran at (the power cap moves it from launch to launch), and the
// cycle count is what separates a kernel's efficiency from the clock it was given.
struct LaunchClock {
    unsigned long long t0, c0;
    __device__ __forceinline__ void begin()
    {
        if (blockIdx.x == 0 && threadIdx.x == 0) { t0 = global_timer_ns(); c0 = (unsigned long long)clock64(); }
    }
    __device__ __forceinline__ void end(unsigned long long *acc) const
    {
        if (blockIdx.x == 0 && threadIdx.x == 0 && acc) {
            atomicAdd(acc, global_timer_ns() - t0);
            atomicAdd(acc + 1, (unsigned long long)clock64() - c0);
            atomicAdd(acc + 2, 1ull);
        }
    }
};

// Bounded wait.  Returns false when the block is aborting (this wait ran out, or another did).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, SharedControl *ctl, int32_t *status,
                                            unsigned long long limit_ns = kWaitLimitNs)
{
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (ctl->abort_flag) return false;
        if (global_timer_ns() - t0 > limit_ns) {
            ctl->abort_flag = 1;
            atomicExch(status, (int32_t)PVF_ERR_TIMEOUT);
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, SharedControl *ctl, int32_t *status)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, ctl, status);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"((unsigned long long)map), "r"(bar), "r"(x), "r"(y) : "memory");
}

// L2 eviction priority for the W tiles.  Where a launch reads W exactly once (one wave, one row tile in flight) the
// tiles are marked evict-first: a gigabyte of weights then streams through L2 without pushing out what the small
// kernels behind the projection need (their instructions, the partial states, the hidden states).  Where blocks share
// W tiles through L2 (several row tiles in flight) the loads carry no hint at all: the hinted form of the instruction,
// even with the normal priority, cost 3 % (paired kernel) to 11 % (128-row kernel) at 32768 rows.
__device__ __forceinline__ uint64_t w_evict_first_policy()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"((unsigned long long)map), "r"(bar), "r"(x), "r"(y), "l"(policy) : "memory");
}

// Asks TMA to bring the box at (x, y) into L2 (no shared memory, no barrier: a hint).
__device__ __forceinline__ void tma_prefetch_l2_2d(const CUtensorMap *map, int x, int y, uint64_t policy)
{
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile.L2::cache_hint [%0, {%1, %2}], %3;"
                 ::"l"((unsigned long long)map), "r"(x), "r"(y), "l"(policy) : "memory");
}

__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]^T, one 128 x N x 16 bf16 MMA.
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16) with the
// 128-byte swizzle: 8-row groups are 1024 bytes apart (stride offset), the leading offset is unused.
__device__ __forceinline__ uint64_t smem_desc_k_major_sw128(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);         // start address, 16-byte units
    d |= (uint64_t)1 << 16;                          // leading byte offset (ignored for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset
    d |= (uint64_t)1 << 46;                          // descriptor version of sm_100
    d |= (uint64_t)2 << 61;                          // 128-byte swizzle
    return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t instr_desc_bf16(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
}

#define PVF_TMEM_LD_ARGS(v, o) \
    "=r"(v[o + 0]), "=r"(v[o + 1]), "=r"(v[o + 2]), "=r"(v[o + 3]), "=r"(v[o + 4]), "=r"(v[o + 5]), \
    "=r"(v[o + 6]), "=r"(v[o + 7]), "=r"(v[o + 8]), "=r"(v[o + 9]), "=r"(v[o + 10]), "=r"(v[o + 11]), \
    "=r"(v[o + 12]), "=r"(v[o + 13]), "=r"(v[o + 14]), "=r"(v[o + 15])

// 16 consecutive fp32 columns of this thread's lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : PVF_TMEM_LD_ARGS(v, 0) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float fast_exp2(float x) { return pvf_fast_exp2(x); }

// Bounded wait (no more than kWaitLimitNs) until the copies a producer thread armed on full[0 .. stages) have
// landed: the abort path's drain, so that no copy is in flight into shared memory that is about to be released.
// The producer keeps two bit sets (registers, no local memory): bit s of `armed` is set once full[s] has been armed,
// bit s of `parity` is the phase parity the barrier had when it was last armed.
struct ArmedStages {
    uint32_t armed = 0, parity = 0;
    __device__ __forceinline__ void note(int stage, uint32_t phase)
    {
        armed |= 1u << stage;
        parity = (parity & ~(1u << stage)) | (phase << stage);
    }
};
__device__ __forceinline__ void drain_armed_stages(SharedControl *ctl, const ArmedStages &a, int stages)
{
    for (int s = 0; s < stages; ++s)
        if ((a.armed >> s) & 1u) {
            const unsigned long long t0 = global_timer_ns();
            while (!mbar_try_wait(smem_u32(&ctl->full[s]), (a.parity >> s) & 1u) && global_timer_ns() - t0 < kWaitLimitNs) {}
        }
}

// Barrier set-up shared by the three projection kernels (one thread): `issuers` threads commit every stage and
// every accumulator, `drainers` epilogue threads release an accumulator.
__device__ __forceinline__ void init_pipeline_barriers(SharedControl *ctl, int stages, int issuers, int drainers)
{
    for (int s = 0; s < stages; ++s) {
        mbar_init(smem_u32(&ctl->full[s]), 1);
        mbar_init(smem_u32(&ctl->empty[s]), issuers);
    }
    for (int b = 0; b < 2; ++b) {
        mbar_init(smem_u32(&ctl->acc_full[b]), issuers);
        mbar_init(smem_u32(&ctl->acc_empty[b]), drainers);
    }
    mbar_init(smem_u32(&ctl->drain), 1);
    mbar_init(smem_u32(&ctl->drain2), 1);
    ctl->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---------------------------------------------------------------------------------- work split
// Vocabulary granules [u0, u1) of split q.
__device__ __forceinline__ void split_range(int units, int splits, int q, int *u0, int *u1)
{
    *u0 = (int)((long long)units * q / splits);
    *u1 = (int)((long long)units * (q + 1) / splits);
}

__device__ __forceinline__ int widest_range(int units, int splits) { return (units + splits - 1) / splits; }

// Vocabulary tiles of a range of `range` granules starting at u0.  A short range (up to
// kBalanceMaxTiles tiles) is cut into near-equal tiles: with full tiles plus a small ragged one, the
// ragged tile's pipeline stages would hold too few bytes to keep HBM busy, and in the weight-streaming
// regime that tile is a tenth of the block's work.  A long range keeps full tiles (one TMA box each).
// `widest` (streaming kernel; 0 elsewhere) = the granules of the launch's widest range, ceil(units / splits): every
// block then cuts its range into as many tiles as the widest one needs.  When HBM is saturated a block's share of it
// follows the bytes it has in flight, i.e. its stage size; with V = 152064 a block of 64 granules (4 tiles of 16)
// and its neighbour of 65 (5 tiles of 13) differ by a fifth in stage size, and the launch ended with the 65-granule
// blocks 12 % after the others (measured per block: 181 us per launch, 173 with the same tile count everywhere).
// The paired kernels lose more on the extra, narrower MMA tiles than they gain (measured), so they keep their own count.
constexpr int kBalanceMaxTiles = 16;
struct TileSplit {
    int u0, range, n_tiles, units_per_tile;
    bool balanced;
    __device__ __forceinline__ TileSplit(int u0_, int u1_, int units_per_tile_, int widest)
        : u0(u0_), range(u1_ - u0_), n_tiles((max(u1_ - u0_, widest) + units_per_tile_ - 1) / units_per_tile_),
          units_per_tile(units_per_tile_), balanced(n_tiles <= kBalanceMaxTiles)
    {
        if (!balanced) n_tiles = (range + units_per_tile - 1) / units_per_tile;
        else if (n_tiles > range) n_tiles = max(range, 1);         // never an empty tile
    }
    // first granule and number of granules of tile t
    __device__ __forceinline__ void tile(int t, int *tu0, int *tun) const
    {
        if (balanced) {
            const int a = range * t / n_tiles, b = range * (t + 1) / n_tiles;
            *tu0 = u0 + a;
            *tun = b - a;
        } else {
            *tu0 = u0 + t * units_per_tile;
            *tun = min(units_per_tile, u0 + range - *tu0);
        }
    }
};

// Running softmax state of one row over the columns seen so far.  The term of the maximum itself (e^0 = 1) is
// kept OUT of the sum: beside it, the other terms of a peaked row (e^-17 = 4e-8 each, a hundred thousand of them,
// half a per cent of the mass together) lie below the fp32 rounding unit of 1.0 and would be rounded away one by
// one.  The row's normaliser is 1 + s.  The state is empty while arg is kNoArg.
constexpr int kNoArg = kPvfNoArg;
struct RowState {
    float m;      // running max
    float s;      // sum of e^{x - m} over every column except the one that holds the max
    float t;      // sum (x - m) e^{x - m}
    int arg;      // lowest id attaining m
};

// Folds 16 logits (ids col0 .. col0+15; only the first n are real when !kFull) into the state.
template <bool kFull>
__device__ __forceinline__ void fold16(RowState &st, const uint32_t (&raw)[16], int col0, int n)
{
    constexpr float kLog2e = 1.4426950408889634f;
    float x[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) x[i] = (kFull || i < n) ? __uint_as_float(raw[i]) : -INFINITY;
    float cm = x[0];
#pragma unroll
    for (int i = 1; i < 16; ++i) cm = fmaxf(cm, x[i]);
    int skip = -1;                                     // the column that becomes the new max: not a term of s
    if (cm > st.m) {                                   // strict: an equal later logit keeps the lower id
        int idx = 15;
#pragma unroll
        for (int i = 14; i >= 0; --i) idx = (x[i] == cm) ? i : idx;
        if (st.arg != kNoArg) {                        // the old max turns into an ordinary term
            const float d = st.m - cm;
            const float c = fast_exp2(d * kLog2e);
            const float total = st.s + 1.f;
            st.t = (st.t + d * total) * c;
            st.s = total * c;
        }
        st.m = cm;
        st.arg = col0 + idx;
        skip = idx;
    }
    float group = 0.f;                                 // the group's small terms are added up among themselves first
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        if (kFull || i < n) {
            const float d = x[i] - st.m;
            const float e = fast_exp2(d * kLog2e);
            group += (i == skip) ? 0.f : e;
            st.t = fmaf(d, e, st.t);
        }
    }
    st.s += group;
}


// One W tile of `tun` granules starting at granule tu0, columns x .. x+63, into b_dst.
template <bool kReadOnce>
__device__ __forceinline__ void load_w_tile(uint32_t b_dst, const WMaps &maps, uint32_t full, int x, int tu0, int tun, uint64_t policy)
{
    if (kReadOnce) tma_load_2d_hint(b_dst, &maps.size[tun - 1], full, x, tu0 * kUnit, policy);
    else tma_load_2d(b_dst, &maps.size[tun - 1], full, x, tu0 * kUnit);
}

}  // namespace
