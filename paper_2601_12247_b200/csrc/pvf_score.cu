// pvf_score: LM-head projection fused with a streaming softmax (sm_100a).
//
//   logits[m][v] = sum_k H[m][k] * W[v][k]      bf16 operands, fp32 accumulation in tensor memory
//   per row m:     top-1 token, its probability, the entropy of softmax(logits[m][:])
//
// The logits never leave the SM.  Scored rows sit on the 128 lanes of a tcgen05 accumulator, the
// vocabulary on its columns, so one epilogue thread owns one row and keeps that row's running
// softmax state (max, argmax, sum e^{x-max}, sum (x-max) e^{x-max}) in registers while the thread
// block sweeps a contiguous vocabulary range.  Each (row, range) pair leaves one 16-byte partial
// state; a small second kernel merges the partials of a row.
//
// Thread block = 6 warps:  warp 0 issues TMA loads (W and H tiles, 128-byte swizzle, a ring of
// stages), warp 1 owns tensor memory and issues the MMAs, warps 2-5 are the softmax epilogue.  Two
// accumulators alternate, so the epilogue of one vocabulary tile overlaps the MMAs of the next.
//
// The GEMM kernel is a template over its tile shape (GemmCfg): vocabulary entries per accumulator,
// 64-element k-panels per pipeline stage, stages; it serves 33 .. 128 rows and more than 8192 rows.
// 129 .. 8192 rows take the paired kernel (pvf_score_gemm_pair_kernel: two blocks per 256-row tile,
// tcgen05 cta_group::2, each loading half of every W tile) where the cost model prefers it.  Calls
// with at most 32 rows take a kernel with the operands swapped
// (pvf_score_stream_kernel): vocabulary on the lanes, rows on the columns, so that no tensor work is
// spent on padding rows.  33 .. 64 and 129 .. 192 rows, where 128- and 256-row tiles would be mostly
// padding, take the paired kernel with swapped operands (pvf_score_swap_pair_kernel).
//
// Work split.  Rows form tiles of 128, the vocabulary granules of 16 entries.  `mb` row tiles are
// in flight at once, each swept by `splits` blocks over disjoint vocabulary ranges (mb * splits
// <= number of SMs); blocks that share a range stream the same W tiles at the same time, so W is
// read from HBM once per wave, and the wave's H tiles stay L2-resident.
//
// Every wait on an mbarrier is bounded: when one runs out the block records PVF_ERR_TIMEOUT in
// the status word, raises a block-wide abort flag, drains its outstanding copies and MMAs with
// bounded waits, frees its tensor memory and returns.
#include <math.h>

#include "pvf_internal.h"

// Tile shapes (overridable at build time for tuning sweeps).
#ifndef PVF_STREAM_STAGES
#define PVF_STREAM_STAGES 6
#endif
#ifndef PVF_GENERAL_TILE_N
#define PVF_GENERAL_TILE_N 256
#endif
#ifndef PVF_GENERAL_PANELS
#define PVF_GENERAL_PANELS 1
#endif
#ifndef PVF_GENERAL_STAGES
#define PVF_GENERAL_STAGES 4
#endif
#ifndef PVF_PAIR_MIN_TILES
#define PVF_PAIR_MIN_TILES 2     // 128-row tiles from which the paired (cta_group::2) kernel takes over
#endif
#ifndef PVF_PAIR_MAX_ROWS
#define PVF_PAIR_MAX_ROWS 8192   // rows up to which the paired kernel is considered
#endif
#ifndef PVF_SWAP_SMALL_MAX_ROWS
#define PVF_SWAP_SMALL_MAX_ROWS 64     // 33 .. this many rows take the swapped paired kernel
#endif
#ifndef PVF_SWAP_RAGGED_MAX_ROWS
#define PVF_SWAP_RAGGED_MAX_ROWS 192   // and so do 129 .. this many rows (at most 256)
#endif

namespace {

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

using GeneralCfg = GemmCfg<PVF_GENERAL_TILE_N, PVF_GENERAL_PANELS, PVF_GENERAL_STAGES>;

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
    int a_rows;          // rows per H box
    int n_pad, stages;   // swapped paired kernel: rows per row tile (MMA N), pipeline stages
    int parts;           // partial states per row (row stride of `partials`)
    float4 *partials;    // [M][parts]
    int32_t *status;
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

// Bounded wait.  Returns false when the block is aborting (this wait ran out, or another did).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, SharedControl *ctl, int32_t *status)
{
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (ctl->abort_flag) return false;
        if (global_timer_ns() - t0 > kWaitLimitNs) {
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

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
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

// Vocabulary tiles of a range of `range` granules starting at u0.  A short range (up to
// kBalanceMaxTiles tiles) is cut into near-equal tiles: with full tiles plus a small ragged one, the
// ragged tile's pipeline stages would hold too few bytes to keep HBM busy, and in the weight-streaming
// regime that tile is a tenth of the block's work.  A long range keeps full tiles (one TMA box each).
constexpr int kBalanceMaxTiles = 16;
struct TileSplit {
    int u0, range, n_tiles, units_per_tile;
    bool balanced;
    __device__ __forceinline__ TileSplit(int u0_, int u1_, int units_per_tile_)
        : u0(u0_), range(u1_ - u0_), n_tiles((u1_ - u0_ + units_per_tile_ - 1) / units_per_tile_),
          units_per_tile(units_per_tile_), balanced(n_tiles <= kBalanceMaxTiles) {}
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
constexpr int kNoArg = 0x7fffffff;
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
__device__ __forceinline__ void load_w_tile(uint32_t b_dst, const WMaps &maps, uint32_t full, int x, int tu0, int tun)
{
    tma_load_2d(b_dst, &maps.size[tun - 1], full, x, tu0 * kUnit);
}

// ---------------------------------------------------------------------------------- GEMM kernel
template <class Cfg>
__global__ void __launch_bounds__(kThreads, 1)
pvf_score_gemm_kernel(const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ WMaps tm_w, const ScoreArgs args)
{
    constexpr int kStages = Cfg::kStages;
    constexpr int kPanels = Cfg::kPanels;
    constexpr int kTileN = Cfg::kTileN;
    constexpr int kUnitsPerTile = Cfg::kUnitsPerTile;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t tiles_addr = (raw_addr + 1023u) & ~1023u;           // swizzled tiles need 1024-byte alignment
    uint8_t *tiles_ptr = smem_raw + (tiles_addr - raw_addr);
    SharedControl *ctl = reinterpret_cast<SharedControl *>(tiles_ptr + kStages * Cfg::kStageBytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int mt_local = blockIdx.x % args.mb;
    const int q = blockIdx.x / args.mb;
    int u0, u1;
    split_range(args.units, args.splits, q, &u0, &u1);
    const TileSplit split(u0, u1, kUnitsPerTile);
    const int n_tiles = split.n_tiles;                                   // vocabulary tiles per sweep
    const int k_steps = (args.num_kb + kPanels - 1) / kPanels;

    if (threadIdx.x == 0) init_pipeline_barriers(ctl, kStages, 1, kEpilogueThreads);
    if (warp == 0 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"((unsigned long long)&tm_h) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"((unsigned long long)&tm_w.size[kWBoxSizes - 1]) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&ctl->tmem_base)), "r"(Cfg::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = ctl->tmem_base;

    // Everything above touched no global memory: it may overlap the tail of the kernel before this
    // one in the stream.  From here on the hidden states are read and the partial states written.
    pvf_grid_dependency_wait();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int armed_parity[kStages];
#pragma unroll
            for (int s = 0; s < kStages; ++s) armed_parity[s] = -1;
            bool alive = true;
            for (int w = 0; w < args.waves && alive; ++w) {
                const int m_tile = w * args.mb + mt_local;
                if (m_tile >= args.m_tiles) continue;
                for (int tile = 0; tile < n_tiles && alive; ++tile) {
                    int tu0, tun;                                              // first granule, granules of this tile
                    split.tile(tile, &tu0, &tun);
                    const uint32_t panel_bytes = (uint32_t)args.a_rows * kRowBytes + (uint32_t)tun * kUnitBytes;
                    for (int step = 0; step < k_steps; ++step) {
                        const int kb0 = step * kPanels;
                        const int np = min(kPanels, args.num_kb - kb0);
                        if (!mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, args.status)) { alive = false; break; }
                        const uint32_t full = smem_u32(&ctl->full[stage]);
                        const uint32_t a_base = tiles_addr + stage * Cfg::kStageBytes;
                        const uint32_t b_base = a_base + kPanels * Cfg::kAPanelBytes;
                        mbar_arrive_expect_tx(full, panel_bytes * (uint32_t)np);
                        armed_parity[stage] = (int)phase;
                        for (int p = 0; p < np; ++p) {
                            const int x = (kb0 + p) * kBlockK;
                            tma_load_2d(a_base + p * Cfg::kAPanelBytes, &tm_h, full, x, m_tile * kTileM);
                            load_w_tile(b_base + p * Cfg::kBPanelBytes, tm_w, full, x, tu0, tun);
                        }
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                }
            }
            if (!alive) {
                // Abort: let every copy this thread started land before the block's memory is released.
                for (int s = 0; s < kStages; ++s)
                    if (armed_parity[s] >= 0) {
                        const unsigned long long t0 = global_timer_ns();
                        while (!mbar_try_wait(smem_u32(&ctl->full[s]), (uint32_t)armed_parity[s]) &&
                               global_timer_ns() - t0 < kWaitLimitNs) {}
                    }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            uint32_t tile_count = 0;
            bool alive = true;
            for (int w = 0; w < args.waves && alive; ++w) {
                const int m_tile = w * args.mb + mt_local;
                if (m_tile >= args.m_tiles) continue;
                for (int tile = 0; tile < n_tiles && alive; ++tile, ++tile_count) {
                    int tu0, tun;
                    split.tile(tile, &tu0, &tun);
                    const uint32_t idesc = instr_desc_bf16(tun * kUnit);
                    const uint32_t buf = tile_count & 1u;
                    const uint32_t acc_phase = (tile_count >> 1) & 1u;
                    if (!mbar_wait(smem_u32(&ctl->acc_empty[buf]), acc_phase ^ 1u, ctl, args.status)) { alive = false; break; }
                    tc_fence_after_sync();
                    const uint32_t tmem_d = tmem_base + buf * kTileN;
                    for (int step = 0; step < k_steps; ++step) {
                        const int kb0 = step * kPanels;
                        const int np = min(kPanels, args.num_kb - kb0);
                        if (!mbar_wait(smem_u32(&ctl->full[stage]), phase, ctl, args.status)) { alive = false; break; }
                        tc_fence_after_sync();
                        const uint32_t a_base = tiles_addr + stage * Cfg::kStageBytes;
                        const uint32_t b_base = a_base + kPanels * Cfg::kAPanelBytes;
                        for (int p = 0; p < np; ++p) {
                            const uint64_t a_desc = smem_desc_k_major_sw128(a_base + p * Cfg::kAPanelBytes);
                            const uint64_t b_desc = smem_desc_k_major_sw128(b_base + p * Cfg::kBPanelBytes);
#pragma unroll
                            for (int k = 0; k < kBlockK / 16; ++k)       // 16 bf16 = 32 bytes further along K
                                tc_mma_bf16(tmem_d, a_desc + (uint64_t)(k * 2), b_desc + (uint64_t)(k * 2), idesc,
                                            (step | p | k) != 0 ? 1u : 0u);
                        }
                        tc_commit(smem_u32(&ctl->empty[stage]));
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                    if (alive) tc_commit(smem_u32(&ctl->acc_full[buf]));
                }
            }
            if (!alive) {
                // Abort: wait (bounded) until every MMA issued so far has retired.
                tc_commit(smem_u32(&ctl->drain));
                const unsigned long long t0 = global_timer_ns();
                while (!mbar_try_wait(smem_u32(&ctl->drain), 0u) && global_timer_ns() - t0 < kWaitLimitNs) {}
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax epilogue
        const int quad = warp & 3;                               // tensor-memory lanes quad*32 .. quad*32+31
        const int row_in_tile = quad * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        uint32_t tile_count = 0;
        bool alive = true;
        for (int w = 0; w < args.waves && alive; ++w) {
            const int m_tile = w * args.mb + mt_local;
            if (m_tile >= args.m_tiles) continue;
            const int row = m_tile * kTileM + row_in_tile;
            const bool warp_has_rows = m_tile * kTileM + quad * 32 < args.M;
            RowState st;
            st.m = -INFINITY; st.s = 0.f; st.t = 0.f; st.arg = kNoArg;
            for (int tile = 0; tile < n_tiles && alive; ++tile, ++tile_count) {
                int tu0, tun;
                split.tile(tile, &tu0, &tun);
                const uint32_t buf = tile_count & 1u;
                const uint32_t acc_phase = (tile_count >> 1) & 1u;
                if (!mbar_wait(smem_u32(&ctl->acc_full[buf]), acc_phase, ctl, args.status)) { alive = false; break; }
                tc_fence_after_sync();
                if (warp_has_rows) {
                    const int v0 = tu0 * kUnit;
                    for (int u = 0; u < tun; ++u) {
                        uint32_t raw[16];
                        tmem_ld16(lane_addr + buf * kTileN + u * kUnit, raw);
                        tmem_ld_wait();
                        const int col0 = v0 + u * kUnit;
                        const int n = args.V - col0;
                        if (n >= kUnit) fold16<true>(st, raw, col0, kUnit);
                        else fold16<false>(st, raw, col0, n);
                    }
                }
                tc_fence_before_sync();
                mbar_arrive(smem_u32(&ctl->acc_empty[buf]));
            }
            if (alive && row < args.M)
                args.partials[(size_t)row * args.splits + q] = make_float4(st.m, st.s, st.t, __int_as_float(st.arg));
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    // Only now may the next kernel's blocks become resident: while they wait for this grid they would
    // share the SM with the MMA and epilogue warps.
    pvf_launch_dependents();
    if (warp == 1) {
        tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(Cfg::kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------------- paired GEMM kernel
// More than 128 rows: two thread blocks on neighbouring SMs (a cluster of 2) share one 256-row x N tile
// with tcgen05 cta_group::2.  Block r of the pair holds rows r*128 .. r*128+127 of the tile in its own
// tensor memory, loads its own 128-row H tile and only HALF of every W tile (N/2 vocabulary entries);
// the MMA, issued by one thread of the even block, reads both halves from both blocks' shared memory.
// Per MMA cycle each SM so pulls a third less through L2 than with two independent 128-row blocks, and a
// 32 KiB stage leaves room for 6 stages instead of 4: the single-block kernel's MMA thread waits a quarter
// of its time for operands.
//
// Protocol (bounded waits as everywhere):
//   full[s]      lives in the even block; it arms the barrier for the bytes of both blocks, and both blocks'
//                TMA loads complete their bytes on it
//   empty[s]     one in each block, released by the MMA thread's commit, multicast to both
//   acc_full[b]  one in each block, multicast commit;  acc_empty[b] in the even block, 2 x 128 arrivals
// Vocabulary granule here = 32 entries (each block loads 16 of them), tile = up to 8 granules.
constexpr int kPairStages = 6;
constexpr int kPairUnit = 32;
constexpr int kPairUnitsPerTile = 8;
constexpr int kPairTileN = 256;
constexpr int kPairABytes = kTileM * kRowBytes;                      // 16 KiB: this block's H tile
constexpr int kPairBBytes = (kPairTileN / 2) * kRowBytes;            // 16 KiB: this block's half of the W tile
constexpr int kPairStageBytes = kPairABytes + kPairBBytes;
constexpr int kPairTmemCols = 512;
constexpr int kPairSmemBytes = kPairStages * kPairStageBytes + 1024 + 512;
constexpr uint32_t kPeerBitMask = 0xFEFFFFFFu;                       // shared::cluster address of the even block of a pair
static_assert(kPairSmemBytes <= 227 * 1024, "paired ring");

__device__ __forceinline__ uint32_t cluster_cta_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA load of one block of a pair: data into this block's shared memory, bytes counted on the even block's barrier.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"((unsigned long long)map), "r"(bar & kPeerBitMask), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate)
{
    const uint32_t zero = 0;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(zero) : "memory");
}
// Arrives on the barrier at this shared-memory offset in both blocks of the pair once the MMAs issued so far retire.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar)
{
    const uint16_t both = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(both) : "memory");
}
// The same on this block's own barrier only.
__device__ __forceinline__ void tc_commit_pair_local(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_even_block(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar & kPeerBitMask) : "memory");
}
__device__ __forceinline__ uint32_t instr_desc_bf16_m256(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

__global__ void __launch_bounds__(kThreads, 1)
pvf_score_gemm_pair_kernel(const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ WMaps tm_w, const ScoreArgs args)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t tiles_addr = (raw_addr + 1023u) & ~1023u;
    uint8_t *tiles_ptr = smem_raw + (tiles_addr - raw_addr);
    SharedControl *ctl = reinterpret_cast<SharedControl *>(tiles_ptr + kPairStages * kPairStageBytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_cta_rank();                            // 0: even block (issues the MMAs), 1: its peer
    const int pair = blockIdx.x >> 1;
    const int st_local = pair % args.mb;                                 // 256-row tile of the wave
    const int q = pair / args.mb;                                        // vocabulary range
    int u0, u1;
    split_range(args.units, args.splits, q, &u0, &u1);                   // granules of 32 entries
    const TileSplit split(u0, u1, kPairUnitsPerTile);
    const int n_tiles = split.n_tiles;
    const int k_steps = args.num_kb;

    if (threadIdx.x == 0) init_pipeline_barriers(ctl, kPairStages, 1, 2 * kEpilogueThreads);
    if (warp == 0 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"((unsigned long long)&tm_h) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"((unsigned long long)&tm_w.size[kPairUnitsPerTile - 1]) : "memory");
    }
    if (warp == 1) {                                                     // the same warp in both blocks
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&ctl->tmem_base)), "r"(kPairTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                                                  // the peer's barriers exist before anything signals them
    tc_fence_after_sync();
    const uint32_t tmem_base = ctl->tmem_base;
    pvf_grid_dependency_wait();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (one per block)
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool alive = true;
            for (int w = 0; w < args.waves && alive; ++w) {
                const int s_tile = w * args.mb + st_local;
                if (s_tile >= args.m_tiles) continue;
                const int row0 = s_tile * 2 * kTileM + (int)rank * kTileM;          // this block's rows
                for (int tile = 0; tile < n_tiles && alive; ++tile) {
                    int tu0, tun;
                    split.tile(tile, &tu0, &tun);
                    const uint32_t bytes = 2u * ((uint32_t)kPairABytes + (uint32_t)tun * kUnitBytes);   // both blocks
                    const int w_row = tu0 * kPairUnit + (int)rank * tun * kUnit;                        // this block's half
                    for (int step = 0; step < k_steps; ++step) {
                        if (!mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, args.status)) { alive = false; break; }
                        const uint32_t full = smem_u32(&ctl->full[stage]);
                        const uint32_t a_dst = tiles_addr + stage * kPairStageBytes;
                        if (rank == 0) mbar_arrive_expect_tx(full, bytes);
                        tma_load_2d_pair(a_dst, &tm_h, full, step * kBlockK, row0);
                        tma_load_2d_pair(a_dst + kPairABytes, &tm_w.size[tun - 1], full, step * kBlockK, w_row);
                        if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
                    }
                }
            }
            if (!alive) {
                // Abort: give the copies in flight time to land before the pair leaves.
                const unsigned long long t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 200000ull) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (even block only)
        if (lane == 0 && rank == 0) {
            int stage = 0;
            uint32_t phase = 0;
            uint32_t tile_count = 0;
            bool alive = true;
            for (int w = 0; w < args.waves && alive; ++w) {
                const int s_tile = w * args.mb + st_local;
                if (s_tile >= args.m_tiles) continue;
                for (int tile = 0; tile < n_tiles && alive; ++tile, ++tile_count) {
                    int tu0, tun;
                    split.tile(tile, &tu0, &tun);
                    const uint32_t idesc = instr_desc_bf16_m256(tun * kPairUnit);
                    const uint32_t buf = tile_count & 1u;
                    const uint32_t acc_phase = (tile_count >> 1) & 1u;
                    if (!mbar_wait(smem_u32(&ctl->acc_empty[buf]), acc_phase ^ 1u, ctl, args.status)) { alive = false; break; }
                    tc_fence_after_sync();
                    const uint32_t tmem_d = tmem_base + buf * kPairTileN;
                    for (int step = 0; step < k_steps; ++step) {
                        if (!mbar_wait(smem_u32(&ctl->full[stage]), phase, ctl, args.status)) { alive = false; break; }
                        tc_fence_after_sync();
                        const uint32_t a_addr = tiles_addr + stage * kPairStageBytes;
                        const uint64_t a_desc = smem_desc_k_major_sw128(a_addr);
                        const uint64_t b_desc = smem_desc_k_major_sw128(a_addr + kPairABytes);
#pragma unroll
                        for (int k = 0; k < kBlockK / 16; ++k)
                            tc_mma_bf16_pair(tmem_d, a_desc + (uint64_t)(k * 2), b_desc + (uint64_t)(k * 2), idesc,
                                             (step | k) != 0 ? 1u : 0u);
                        tc_commit_pair(smem_u32(&ctl->empty[stage]));
                        if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
                    }
                    if (alive) tc_commit_pair(smem_u32(&ctl->acc_full[buf]));
                }
            }
            if (!alive) {
                tc_commit_pair_local(smem_u32(&ctl->drain));
                const unsigned long long t0 = global_timer_ns();
                while (!mbar_try_wait(smem_u32(&ctl->drain), 0u) && global_timer_ns() - t0 < kWaitLimitNs) {}
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax epilogue (both blocks)
        const int quad = warp & 3;
        const int row_in_tile = quad * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        uint32_t tile_count = 0;
        bool alive = true;
        for (int w = 0; w < args.waves && alive; ++w) {
            const int s_tile = w * args.mb + st_local;
            if (s_tile >= args.m_tiles) continue;
            const int row_base = s_tile * 2 * kTileM + (int)rank * kTileM;
            const int row = row_base + row_in_tile;
            const bool warp_has_rows = row_base + quad * 32 < args.M;
            RowState st;
            st.m = -INFINITY; st.s = 0.f; st.t = 0.f; st.arg = kNoArg;
            for (int tile = 0; tile < n_tiles && alive; ++tile, ++tile_count) {
                int tu0, tun;
                split.tile(tile, &tu0, &tun);
                const uint32_t buf = tile_count & 1u;
                const uint32_t acc_phase = (tile_count >> 1) & 1u;
                if (!mbar_wait(smem_u32(&ctl->acc_full[buf]), acc_phase, ctl, args.status)) { alive = false; break; }
                tc_fence_after_sync();
                if (warp_has_rows) {
                    const int v0 = tu0 * kPairUnit;
                    for (int u = 0; u < 2 * tun; ++u) {
                        uint32_t raw[16];
                        tmem_ld16(lane_addr + buf * kPairTileN + u * kUnit, raw);
                        tmem_ld_wait();
                        const int col0 = v0 + u * kUnit;
                        const int n = args.V - col0;
                        if (n >= kUnit) fold16<true>(st, raw, col0, kUnit);
                        else if (n > 0) fold16<false>(st, raw, col0, n);
                    }
                }
                tc_fence_before_sync();
                mbar_arrive_even_block(smem_u32(&ctl->acc_empty[buf]));
            }
            if (alive && row < args.M)
                args.partials[(size_t)row * args.splits + q] = make_float4(st.m, st.s, st.t, __int_as_float(st.arg));
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                                                  // neither block leaves while the other may still signal it
    pvf_launch_dependents();
    if (warp == 1) {
        tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kPairTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------------- streaming kernel
// At most 32 scored rows: the call is a pure stream of W through the SMs, and the only thing that
// matters is to keep HBM busy while spending as little power as possible on everything else (the
// SM clocks are power-capped in this regime).  Running 32 rows through 128-row MMAs wastes three
// quarters of the tensor work, so here the operands are swapped: a 128-entry slice of the vocabulary
// sits on the 128 lanes of the accumulator and the scored rows are its N = 16 or 32 columns,
//     D[v][m] = sum_k W[v][k] * H[m][k],
// one 128 x N x 16 MMA per 16 elements of k and vocabulary slice, nothing wasted.  An epilogue thread
// now owns a vocabulary lane: it keeps one running softmax state per scored row (for the vocabulary
// entries that passed through its lane) and the block folds the 128 lanes' states once, at the end,
// through shared memory.  The per-(row, range) partial state it leaves is the GEMM kernel's.
constexpr int kStreamStages = PVF_STREAM_STAGES;
constexpr int kStreamTileN = 256;                                   // vocabulary entries per W tile (two 128-lane slices)
constexpr int kStreamUnitsPerTile = kStreamTileN / kUnit;
constexpr int kStreamHBytes = kStreamRows * kRowBytes;              // 4 KiB
constexpr int kStreamWBytes = kStreamTileN * kRowBytes;             // 32 KiB
constexpr int kStreamStageBytes = kStreamHBytes + kStreamWBytes;
constexpr int kStreamTmemCols = 128;                                // 2 buffers x 2 slices x 32 columns
constexpr int kStreamControlBytes = 512;
constexpr int kStreamIssuers = 2;                                   // MMA-issuing threads (one per vocabulary slice)
constexpr int kStreamSecondIssuerWarp = 6;
constexpr int kStreamThreads = 224;                                 // producer, issuer, 4 epilogue warps, issuer
constexpr int kStreamSmemBytes = kStreamStages * kStreamStageBytes + 1024 + kStreamControlBytes;
static_assert(kStreamStages >= 2 && kStreamStages <= kMaxStages && kStreamSmemBytes <= 227 * 1024, "streaming ring");
static_assert(kStreamTileN == 2 * kTileM, "each of the two MMA slices reads kTileM W rows of the stage");
// the end-of-block fold reuses the tile ring: 128 lanes x 32 rows x 16 bytes
static_assert(kStreamStages * kStreamStageBytes >= kTileM * kStreamRows * 16, "fold scratch");

// State (m, s, t, arg) absorbs one more logit x of vocabulary id v (s leaves out the max's own term, see RowState).
__device__ __forceinline__ void state_push(float &m, float &s, float &t, int &arg, float x, int v)
{
    constexpr float kLog2e = 1.4426950408889634f;
    if (x > m) {                                        // strict: ids ascend, so the lowest id keeps a tie
        if (arg != kNoArg) {
            const float d = m - x;
            const float c = fast_exp2(d * kLog2e);
            const float total = s + 1.f;
            t = (t + d * total) * c;
            s = total * c;
        }
        m = x;
        arg = v;
    } else {
        const float d = x - m;
        const float e = fast_exp2(d * kLog2e);
        s += e;
        t = fmaf(d, e, t);
    }
}

// a <- a merged with b (two states over disjoint vocabulary sets).  The larger max stays outside the sum; the
// other state's max joins it as an ordinary term.
__device__ __forceinline__ void state_merge(float4 &a, const float4 b)
{
    constexpr float kLog2e = 1.4426950408889634f;
    const int ia = __float_as_int(a.w), ib = __float_as_int(b.w);
    if (ib == kNoArg) return;
    if (ia == kNoArg) { a = b; return; }
    if (a.x > b.x || (a.x == b.x && ia < ib)) {
        const float d = b.x - a.x;                      // <= 0
        const float c = fast_exp2(d * kLog2e);
        const float total = b.y + 1.f;
        a.y += total * c;
        a.z += (b.z + d * total) * c;
    } else {
        const float d = a.x - b.x;
        const float c = fast_exp2(d * kLog2e);
        const float total = a.y + 1.f;
        a.y = b.y + total * c;
        a.z = b.z + (a.z + d * total) * c;
        a.x = b.x;
        a.w = b.w;
    }
}

__global__ void __launch_bounds__(kStreamThreads, 1)
pvf_score_stream_kernel(const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ WMaps tm_w, const ScoreArgs args)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t tiles_addr = (raw_addr + 1023u) & ~1023u;
    uint8_t *tiles_ptr = smem_raw + (tiles_addr - raw_addr);
    SharedControl *ctl = reinterpret_cast<SharedControl *>(tiles_ptr + kStreamStages * kStreamStageBytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int q = blockIdx.x;                                            // one vocabulary range per block
    int u0, u1;
    split_range(args.units, args.splits, q, &u0, &u1);
    const TileSplit split(u0, u1, kStreamUnitsPerTile);
    const int n_tiles = split.n_tiles;
    const int n_cols = args.M <= 16 ? 16 : 32;                           // MMA N: scored rows, padded
    const int k_steps = args.num_kb;

    if (threadIdx.x == 0) init_pipeline_barriers(ctl, kStreamStages, kStreamIssuers, kEpilogueThreads);
    if (warp == 0 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"((unsigned long long)&tm_h) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"((unsigned long long)&tm_w.size[kWBoxSizes - 1]) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&ctl->tmem_base)), "r"(kStreamTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = ctl->tmem_base;
    pvf_grid_dependency_wait();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int armed_parity[kStreamStages];
#pragma unroll
            for (int s = 0; s < kStreamStages; ++s) armed_parity[s] = -1;
            bool alive = true;
            for (int tile = 0; tile < n_tiles && alive; ++tile) {
                int tu0, tun;
                split.tile(tile, &tu0, &tun);
                const uint32_t bytes = (uint32_t)args.a_rows * kRowBytes + (uint32_t)tun * kUnitBytes;
                for (int step = 0; step < k_steps; ++step) {
                    if (!mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, args.status)) { alive = false; break; }
                    const uint32_t full = smem_u32(&ctl->full[stage]);
                    const uint32_t h_dst = tiles_addr + stage * kStreamStageBytes;
                    mbar_arrive_expect_tx(full, bytes);
                    armed_parity[stage] = (int)phase;
                    tma_load_2d(h_dst, &tm_h, full, step * kBlockK, 0);
                    load_w_tile(h_dst + kStreamHBytes, tm_w, full, step * kBlockK, tu0, tun);
                    if (++stage == kStreamStages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!alive) {
                for (int s = 0; s < kStreamStages; ++s)
                    if (armed_parity[s] >= 0) {
                        const unsigned long long t0 = global_timer_ns();
                        while (!mbar_try_wait(smem_u32(&ctl->full[s]), (uint32_t)armed_parity[s]) &&
                               global_timer_ns() - t0 < kWaitLimitNs) {}
                    }
            }
        }
    } else if (warp == 1 || warp == kStreamSecondIssuerWarp) {
        // ------------------------------------------------------------------ MMA issuers
        // One thread per 128-entry vocabulary slice: a single thread cannot issue the eight small MMAs
        // of a stage as fast as the stage's bytes arrive.  Both commit every stage and every tile (a
        // commit with nothing outstanding arrives at once), so the barrier counts never depend on
        // how many slices a ragged tile has.
        if (lane == 0) {
            const int sl = warp == 1 ? 0 : 1;                            // this thread's slice
            int stage = 0;
            uint32_t phase = 0;
            bool alive = true;
            const uint32_t idesc = instr_desc_bf16(n_cols);
            for (int tile = 0; tile < n_tiles && alive; ++tile) {
                int tu0, tun;
                split.tile(tile, &tu0, &tun);
                const int n_slices = tun > kTileM / kUnit ? 2 : 1;       // 128-entry vocabulary slices of this tile
                const uint32_t buf = (uint32_t)tile & 1u;
                const uint32_t acc_phase = ((uint32_t)tile >> 1) & 1u;
                if (!mbar_wait(smem_u32(&ctl->acc_empty[buf]), acc_phase ^ 1u, ctl, args.status)) { alive = false; break; }
                tc_fence_after_sync();
                const uint32_t tmem_d = tmem_base + buf * (2 * kStreamRows);
                for (int step = 0; step < k_steps; ++step) {
                    if (!mbar_wait(smem_u32(&ctl->full[stage]), phase, ctl, args.status)) { alive = false; break; }
                    tc_fence_after_sync();
                    const uint32_t h_addr = tiles_addr + stage * kStreamStageBytes;
                    const uint64_t h_desc = smem_desc_k_major_sw128(h_addr);
                    if (sl < n_slices) {
                        // Slice sl = rows sl*128 .. sl*128+127 of the W tile.  A ragged tile's last slice reads
                        // rows past its end: stale bytes of the same stage, on lanes the epilogue skips.
                        const uint64_t w_desc = smem_desc_k_major_sw128(h_addr + kStreamHBytes + sl * (kTileM * kRowBytes));
#pragma unroll
                        for (int k = 0; k < kBlockK / 16; ++k)
                            tc_mma_bf16(tmem_d + sl * kStreamRows, w_desc + (uint64_t)(k * 2), h_desc + (uint64_t)(k * 2), idesc,
                                        (step | k) != 0 ? 1u : 0u);
                    }
                    tc_commit(smem_u32(&ctl->empty[stage]));
                    if (++stage == kStreamStages) { stage = 0; phase ^= 1u; }
                }
                if (alive) tc_commit(smem_u32(&ctl->acc_full[buf]));
            }
            if (!alive) {
                const uint32_t drain = smem_u32(sl == 0 ? &ctl->drain : &ctl->drain2);
                tc_commit(drain);
                const unsigned long long t0 = global_timer_ns();
                while (!mbar_try_wait(drain, 0u) && global_timer_ns() - t0 < kWaitLimitNs) {}
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax epilogue
        const int quad = warp & 3;
        const int acc_lane = quad * 32 + lane;                           // this thread's accumulator lane
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        float sm[kStreamRows], ss[kStreamRows], st[kStreamRows];
        int sa[kStreamRows];
#pragma unroll
        for (int i = 0; i < kStreamRows; ++i) { sm[i] = -INFINITY; ss[i] = 0.f; st[i] = 0.f; sa[i] = kNoArg; }
        bool alive = true;
        for (int tile = 0; tile < n_tiles && alive; ++tile) {
            int tu0, tun;
            split.tile(tile, &tu0, &tun);
            const int n_slices = tun > kTileM / kUnit ? 2 : 1;
            const uint32_t buf = (uint32_t)tile & 1u;
            const uint32_t acc_phase = ((uint32_t)tile >> 1) & 1u;
            if (!mbar_wait(smem_u32(&ctl->acc_full[buf]), acc_phase, ctl, args.status)) { alive = false; break; }
            tc_fence_after_sync();
            const int tile_end = min((tu0 + tun) * kUnit, args.V);
            for (int sl = 0; sl < n_slices; ++sl) {
                const int v = tu0 * kUnit + sl * kTileM + acc_lane;      // vocabulary id on this lane
                const bool real = v < tile_end;
#pragma unroll
                for (int half = 0; half < kStreamRows / 16; ++half) {
                    if (half * 16 < n_cols) {                            // block-uniform
                        uint32_t raw[16];
                        tmem_ld16(lane_addr + buf * (2 * kStreamRows) + sl * kStreamRows + half * 16, raw);
                        tmem_ld_wait();
                        if (real) {
#pragma unroll
                            for (int i = 0; i < 16; ++i)
                                state_push(sm[half * 16 + i], ss[half * 16 + i], st[half * 16 + i], sa[half * 16 + i],
                                           __uint_as_float(raw[i]), v);
                        }
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive(smem_u32(&ctl->acc_empty[buf]));
        }
        // Fold the 128 lanes.  The tile ring is idle now (every copy landed and every MMA that read it
        // retired before the last accumulator was published), so it serves as scratch [row][lane].
        if (alive) {
            float4 *scratch = reinterpret_cast<float4 *>(tiles_ptr);
#pragma unroll
            for (int i = 0; i < kStreamRows; ++i)
                scratch[i * kTileM + acc_lane] = make_float4(sm[i], ss[i], st[i], __int_as_float(sa[i]));
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kEpilogueThreads) : "memory");
        if (alive && !ctl->abort_flag) {
            // 4 threads per scored row, each folds 32 lanes in lane order, then the 4 fold together
            const float4 *scratch = reinterpret_cast<const float4 *>(tiles_ptr);
            const int e = threadIdx.x - 64;                              // 0..127
            const int row = e >> 2, part = e & 3;
            float4 acc = make_float4(-INFINITY, 0.f, 0.f, __int_as_float(kNoArg));
            for (int l = 0; l < 32; ++l) state_merge(acc, scratch[row * kTileM + part * 32 + l]);
            for (int o = 1; o < 4; o <<= 1) {
                float4 other;
                other.x = __shfl_xor_sync(0xffffffffu, acc.x, o);
                other.y = __shfl_xor_sync(0xffffffffu, acc.y, o);
                other.z = __shfl_xor_sync(0xffffffffu, acc.z, o);
                other.w = __shfl_xor_sync(0xffffffffu, acc.w, o);
                state_merge(acc, other);
            }
            if (part == 0 && row < args.M) args.partials[(size_t)row * args.splits + q] = acc;
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    pvf_launch_dependents();
    if (warp == 1) {
        tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kStreamTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------------- swapped paired kernel
// 33 .. 256 rows in one row tile: the launch sits at the ridge, where HBM, the tensor pipe and the power cap all
// matter, and 128- or 256-row MMAs over a ragged row count waste tensor work (and with it clock).  Here the
// operands of the paired kernel change places: the two blocks of a pair hold 2 x 128 vocabulary entries on
// their accumulator lanes (each loads its own 128-entry W tile, so W still crosses L2 -> SM once) and the
// scored rows are the N columns, N = the row tile padded to 32 (each block loads half of the H tile):
//     D[v][m] = sum_k W[v][k] * H[m][k],   one 256 x N x 16 MMA (cta_group::2) per 16 elements of k.
// At most 31 padded rows are wasted.  Measured against the other two kernels (each alone for seconds, so that
// the power cap has settled, and in short bursts) it wins where they pad most: 33 .. 64 rows (4 .. 5 %) and
// 129 .. 192 rows (4 .. 9 %); with full 128- or 256-row tiles they are 3 .. 9 % faster, so the geometry picks it
// for those two windows only.
//
// Epilogue: a warp owns 32 vocabulary lanes and reads 32 rows (columns) at a time.  It turns that 32 x 32 block
// around through a padded shared-memory tile of its own, after which lane i holds row i's 32 logits and folds
// them into the running state of row chunk*32 + i exactly as the GEMM kernels' epilogue does (no warp-wide
// reductions: those serialise on their latency with one epilogue warp per scheduler).  At the end of the block's
// range the four warps' states fold through the same shared memory and the block writes one partial state per
// row: 2 x splits partial states per row reach the merge kernel.
//
// The ring has as many stages as fit: a stage is the block's 16 KiB W tile plus its half of the H tile.
constexpr int kSwapWBytes = kTileM * kRowBytes;                      // 16 KiB
constexpr int kSwapMaxRowsPerTile = 256;                             // MMA N limit
constexpr int kSwapTmemCols = 512;                                   // 2 accumulators x 256 columns
constexpr int kSwapTurnPitch = 36;                                   // words per lane of a warp's 32 x 32 fp32 block: 16-byte
                                                                     // aligned rows, conflict-free 128-bit stores and column reads
constexpr int kSwapWarpScratchBytes = 32 * kSwapTurnPitch * 4;       // that block; later the warp's 256 row states (4 KiB) for the fold
constexpr int kSwapScratchBytes = 4 * kSwapWarpScratchBytes;
static_assert(kSwapWarpScratchBytes >= kSwapMaxRowsPerTile * 16 && kSwapWarpScratchBytes % 16 == 0, "fold scratch");
constexpr int kSwapRingBytes = 204 * 1024;
constexpr int kSwapMaxStages = 12;
constexpr int kSwapSmemBytes = kSwapRingBytes + 1024 + 512 + kSwapScratchBytes;
static_assert(kSwapSmemBytes <= 227 * 1024, "swapped ring");
static_assert(kSwapMaxStages <= kMaxStages, "barrier arrays");
static_assert(PVF_SWAP_SMALL_MAX_ROWS <= kSwapMaxRowsPerTile && PVF_SWAP_RAGGED_MAX_ROWS <= kSwapMaxRowsPerTile, "one row tile");

__global__ void __launch_bounds__(kThreads, 1)
pvf_score_swap_pair_kernel(const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ WMaps tm_w, const ScoreArgs args)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t tiles_addr = (raw_addr + 1023u) & ~1023u;
    uint8_t *tiles_ptr = smem_raw + (tiles_addr - raw_addr);
    const int n_pad = args.n_pad;                                        // rows per row tile = MMA N (multiple of 32)
    const int n_stages = args.stages;
    const uint32_t h_bytes = (uint32_t)(n_pad / 2) * kRowBytes;          // this block's half of the H tile
    const uint32_t stage_bytes = (uint32_t)kSwapWBytes + h_bytes;
    SharedControl *ctl = reinterpret_cast<SharedControl *>(tiles_ptr + (size_t)n_stages * stage_bytes);
    uint8_t *scratch = reinterpret_cast<uint8_t *>(ctl) + 512;          // one kSwapWarpScratchBytes region per epilogue warp

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_cta_rank();                            // 0: even block (issues the MMAs), 1: its peer
    const int q = blockIdx.x >> 1;                                       // the pair's vocabulary range
    int u0, u1;
    split_range(args.units, args.splits, q, &u0, &u1);                   // granules of 32 entries
    const TileSplit split(u0, u1, kPairUnitsPerTile);
    const int n_tiles = split.n_tiles;
    const int k_steps = args.num_kb;

    if (threadIdx.x == 0) init_pipeline_barriers(ctl, n_stages, 1, 2 * kEpilogueThreads);
    if (warp == 0 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"((unsigned long long)&tm_h) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"((unsigned long long)&tm_w.size[kPairUnitsPerTile - 1]) : "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&ctl->tmem_base)), "r"(kSwapTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after_sync();
    const uint32_t tmem_base = ctl->tmem_base;
    pvf_grid_dependency_wait();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (one per block)
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool alive = true;
            const int row0 = (int)rank * (n_pad / 2);                               // this block's half of the rows
            for (int tile = 0; tile < n_tiles && alive; ++tile) {
                int tu0, tun;
                split.tile(tile, &tu0, &tun);
                const uint32_t bytes = 2u * ((uint32_t)tun * kUnitBytes + h_bytes);                     // both blocks
                const int w_row = tu0 * kPairUnit + (int)rank * tun * kUnit;                            // this block's entries
                for (int step = 0; step < k_steps; ++step) {
                    if (!mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, args.status)) { alive = false; break; }
                    const uint32_t full = smem_u32(&ctl->full[stage]);
                    const uint32_t w_dst = tiles_addr + (uint32_t)stage * stage_bytes;
                    if (rank == 0) mbar_arrive_expect_tx(full, bytes);
                    tma_load_2d_pair(w_dst, &tm_w.size[tun - 1], full, step * kBlockK, w_row);
                    tma_load_2d_pair(w_dst + kSwapWBytes, &tm_h, full, step * kBlockK, row0);
                    if (++stage == n_stages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!alive) {
                const unsigned long long t0 = global_timer_ns();
                while (global_timer_ns() - t0 < 200000ull) {}
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (even block only)
        if (lane == 0 && rank == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool alive = true;
            const uint32_t idesc = instr_desc_bf16_m256(n_pad);
            for (int tile = 0; tile < n_tiles && alive; ++tile) {
                const uint32_t buf = (uint32_t)tile & 1u;
                const uint32_t acc_phase = ((uint32_t)tile >> 1) & 1u;
                if (!mbar_wait(smem_u32(&ctl->acc_empty[buf]), acc_phase ^ 1u, ctl, args.status)) { alive = false; break; }
                tc_fence_after_sync();
                const uint32_t tmem_d = tmem_base + buf * kSwapMaxRowsPerTile;
                for (int step = 0; step < k_steps; ++step) {
                    if (!mbar_wait(smem_u32(&ctl->full[stage]), phase, ctl, args.status)) { alive = false; break; }
                    tc_fence_after_sync();
                    // A ragged vocabulary tile leaves stale bytes on the W tile's last rows: lanes the epilogue skips.
                    const uint32_t w_addr = tiles_addr + (uint32_t)stage * stage_bytes;
                    const uint64_t w_desc = smem_desc_k_major_sw128(w_addr);
                    const uint64_t h_desc = smem_desc_k_major_sw128(w_addr + kSwapWBytes);
#pragma unroll
                    for (int k = 0; k < kBlockK / 16; ++k)
                        tc_mma_bf16_pair(tmem_d, w_desc + (uint64_t)(k * 2), h_desc + (uint64_t)(k * 2), idesc,
                                         (step | k) != 0 ? 1u : 0u);
                    tc_commit_pair(smem_u32(&ctl->empty[stage]));
                    if (++stage == n_stages) { stage = 0; phase ^= 1u; }
                }
                if (alive) tc_commit_pair(smem_u32(&ctl->acc_full[buf]));
            }
            if (!alive) {
                tc_commit_pair_local(smem_u32(&ctl->drain));
                const unsigned long long t0 = global_timer_ns();
                while (!mbar_try_wait(smem_u32(&ctl->drain), 0u) && global_timer_ns() - t0 < kWaitLimitNs) {}
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax epilogue (both blocks)
        const int quad = warp & 3;                                       // tensor-memory lanes quad*32 .. quad*32+31
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        const int n_chunks = n_pad >> 5;                                 // 32-row column groups
        const int e_thread = quad * 32 + lane;
        float *turn = reinterpret_cast<float *>(scratch + quad * kSwapWarpScratchBytes);          // [32 lanes][kSwapTurnPitch]
        float4 *fold_mine = reinterpret_cast<float4 *>(scratch + quad * kSwapWarpScratchBytes);   // [256 rows], after the sweep
        bool alive = true;
        RowState st[kSwapMaxRowsPerTile / 32];                           // lane i: state of row chunk*32 + i
#pragma unroll
        for (int c = 0; c < kSwapMaxRowsPerTile / 32; ++c) { st[c].m = -INFINITY; st[c].s = 0.f; st[c].t = 0.f; st[c].arg = kNoArg; }
        for (int tile = 0; tile < n_tiles && alive; ++tile) {
            int tu0, tun;
            split.tile(tile, &tu0, &tun);
            const uint32_t buf = (uint32_t)tile & 1u;
            const uint32_t acc_phase = ((uint32_t)tile >> 1) & 1u;
            if (!mbar_wait(smem_u32(&ctl->acc_full[buf]), acc_phase, ctl, args.status)) { alive = false; break; }
            tc_fence_after_sync();
            const int block_v0 = tu0 * kPairUnit + (int)rank * tun * kUnit;         // vocabulary id on this block's lane 0
            const int block_end = min(block_v0 + tun * kUnit, args.V);
            const int warp_v0 = block_v0 + quad * 32;
            const int n_real = min(32, block_end - warp_v0);                        // vocabulary entries on this warp's lanes
            if (n_real > 0) {                                                        // warp-uniform
#pragma unroll
                for (int c = 0; c < kSwapMaxRowsPerTile / 32; ++c) {
                    if (c < n_chunks) {                                              // block-uniform
                        uint32_t lo[16], hi[16];
                        const uint32_t col = lane_addr + buf * kSwapMaxRowsPerTile + c * 32;
                        tmem_ld16(col, lo);
                        tmem_ld16(col + 16, hi);
                        tmem_ld_wait();
                        uint4 *mine = reinterpret_cast<uint4 *>(turn + lane * kSwapTurnPitch);       // lane = vocabulary entry
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            mine[j] = make_uint4(lo[4 * j], lo[4 * j + 1], lo[4 * j + 2], lo[4 * j + 3]);
                            mine[4 + j] = make_uint4(hi[4 * j], hi[4 * j + 1], hi[4 * j + 2], hi[4 * j + 3]);
                        }
                        __syncwarp();
#pragma unroll
                        for (int half = 0; half < 2; ++half) {                       // lane = row, 16 vocabulary entries at a time
                            const int n = n_real - half * 16;
                            if (n > 0) {
                                uint32_t x[16];
#pragma unroll
                                for (int l = 0; l < 16; ++l) x[l] = __float_as_uint(turn[(half * 16 + l) * kSwapTurnPitch + lane]);
                                if (n >= 16) fold16<true>(st[c], x, warp_v0 + half * 16, 16);
                                else fold16<false>(st[c], x, warp_v0 + half * 16, n);
                            }
                        }
                        __syncwarp();
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive_even_block(smem_u32(&ctl->acc_empty[buf]));
        }
        // Fold the block's four warps and write the block's partial state of every row.  Every epilogue thread
        // reaches the barrier, aborting or not.
        if (alive) {
#pragma unroll
            for (int c = 0; c < kSwapMaxRowsPerTile / 32; ++c)
                if (c < n_chunks)
                    fold_mine[c * 32 + lane] = make_float4(st[c].m, st[c].s, st[c].t, __int_as_float(st[c].arg));
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kEpilogueThreads) : "memory");
        if (alive && !ctl->abort_flag) {
            for (int row = e_thread; row < args.M; row += kEpilogueThreads) {
                float4 acc = reinterpret_cast<const float4 *>(scratch)[row];
#pragma unroll
                for (int o = 1; o < 4; ++o)
                    state_merge(acc, reinterpret_cast<const float4 *>(scratch + o * kSwapWarpScratchBytes)[row]);
                args.partials[(size_t)row * args.parts + 2 * q + (int)rank] = acc;
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();
    pvf_launch_dependents();
    if (warp == 1) {
        tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kSwapTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------------- merge kernel
// One warp per row: combines the row's `splits` partial states (ascending vocabulary ranges) in
// fp64 and writes token, confidence, entropy and planning-vocabulary membership.
__global__ void __launch_bounds__(256)
pvf_score_merge_kernel(const float4 *__restrict__ partials, int M, int splits, int vocab,
                       const uint32_t *__restrict__ plan_bitmap, int32_t *__restrict__ tok,
                       float *__restrict__ conf, float *__restrict__ ent, uint8_t *__restrict__ in_plan)
{
    pvf_launch_dependents();
    pvf_grid_dependency_wait();
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= M) return;
    const float4 *p = partials + (size_t)row * splits;
    // lane-local pass: only the max and its lowest id
    float m = -INFINITY;
    int arg = kNoArg;
    for (int i = lane; i < splits; i += 32) {
        const float4 v = p[i];
        const int a = __float_as_int(v.w);
        if (a != kNoArg && (v.x > m || (v.x == m && a < arg))) { m = v.x; arg = a; }
    }
    for (int o = 16; o > 0; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
        const int a2 = __shfl_xor_sync(0xffffffffu, arg, o);
        if (m2 > m || (m2 == m && a2 < arg)) { m = m2; arg = a2; }
    }
    // rescale every partial to the global max and add; a partial's sum leaves out its own max's term (1)
    double s = 0.0, t = 0.0;
    for (int i = lane; i < splits; i += 32) {
        const float4 v = p[i];
        if (__float_as_int(v.w) != kNoArg) {
            const double d = (double)v.x - (double)m;
            const double c = exp(d);
            const double total = 1.0 + (double)v.y;
            s += total * c;
            t += ((double)v.z + d * total) * c;
        }
    }
    for (int o = 16; o > 0; o >>= 1) {
        s += __shfl_xor_sync(0xffffffffu, s, o);
        t += __shfl_xor_sync(0xffffffffu, t, o);
    }
    if (lane == 0) {
        // A row of non-finite logits never sets a maximum: its outputs are unspecified, but the token stays a
        // valid id and the bitmap lookup in bounds.
        if ((unsigned)arg >= (unsigned)vocab) arg = 0;
        tok[row] = arg;
        conf[row] = (float)(1.0 / s);
        if (ent) ent[row] = (float)(log(s) - t / s);
        if (in_plan) in_plan[row] = (uint8_t)((plan_bitmap[arg >> 5] >> (arg & 31)) & 1u);
    }
}

// ---------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// bf16 matrix [rows][cols] row-major, box = box_rows x 64 columns, 128-byte swizzle, zero fill outside.
// 256-byte L2 promotion: a 128-byte box row pulls its neighbour into L2 as well, which the next k-panel reads
// (measured on the weight stream: 5.8 TB/s with it, 4.9 TB/s with 128-byte or no promotion).
int make_tensor_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return PVF_ERR_CUDA;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)kBlockK, box_rows};
    cuuint32_t elem[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, elem,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? PVF_OK : PVF_ERR_CUDA;
}

int make_w_maps(CUtensorMap *levels, const void *w_head, int vocab, int hidden)
{
    for (int l = 0; l < kWBoxSizes; ++l) {
        const int rc = make_tensor_map(&levels[l], w_head, (uint64_t)vocab, (uint64_t)hidden, (uint32_t)(kUnit * (l + 1)));
        if (rc != PVF_OK) return rc;
    }
    return PVF_OK;
}

int raise_shared_memory_limits()
{
    if (cudaFuncSetAttribute(pvf_score_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kStreamSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(pvf_score_gemm_kernel<GeneralCfg>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             GeneralCfg::kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(pvf_score_gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kPairSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(pvf_score_swap_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kSwapSmemBytes) != cudaSuccess)
        return PVF_ERR_CUDA;
    return PVF_OK;
}

// Launches the GEMM kernel (shape chosen by the geometry) and the merge kernel on `s`.
int launch_score(const pvf_score_geometry &g, const void *hidden, int M, int V, int D, const CUtensorMap *w_levels,
                 float4 *partials, int32_t *status, const uint32_t *plan_bitmap, int32_t *tok, float *conf, float *ent,
                 uint8_t *in_plan, cudaStream_t s, cudaEvent_t ev_start, cudaEvent_t ev_stop)
{
    CUtensorMap tm_h;
    int rc = make_tensor_map(&tm_h, hidden, (uint64_t)M, (uint64_t)D, (uint32_t)g.a_rows);
    if (rc != PVF_OK) return rc;
    WMaps maps;
    for (int l = 0; l < kWBoxSizes; ++l) maps.size[l] = w_levels[l];

    ScoreArgs a;
    a.M = M; a.V = V; a.D = D;
    a.num_kb = (D + kBlockK - 1) / kBlockK;
    a.units = g.units;
    a.m_tiles = g.m_tiles; a.mb = g.mb; a.splits = g.splits; a.waves = g.waves;
    a.a_rows = g.a_rows;
    a.n_pad = g.n_pad; a.stages = g.stages; a.parts = g.parts;
    a.partials = partials;
    a.status = status;
    const bool timed = ev_start && ev_stop;
    if (timed && cudaEventRecord(ev_start, s) != cudaSuccess) return PVF_ERR_CUDA;
    cudaError_t e;
    if (g.swapped)
        e = pvf_launch_cluster2(pvf_score_swap_pair_kernel, dim3(g.ctas), dim3(kThreads), kSwapSmemBytes, s, tm_h, maps, a);
    else if (g.paired)
        e = pvf_launch_cluster2(pvf_score_gemm_pair_kernel, dim3(g.ctas), dim3(kThreads), kPairSmemBytes, s, tm_h, maps, a);
    else if (g.streaming)
        e = pvf_launch(pvf_score_stream_kernel, dim3(g.ctas), dim3(kStreamThreads), kStreamSmemBytes, s, tm_h, maps, a);
    else
        e = pvf_launch(pvf_score_gemm_kernel<GeneralCfg>, dim3(g.ctas), dim3(kThreads), GeneralCfg::kSmemBytes, s, tm_h, maps, a);
    if (e != cudaSuccess) return PVF_ERR_CUDA;
    if (timed && cudaEventRecord(ev_stop, s) != cudaSuccess) return PVF_ERR_CUDA;
    const int warps_per_block = 8;
    e = pvf_launch(pvf_score_merge_kernel, dim3((M + warps_per_block - 1) / warps_per_block), dim3(warps_per_block * 32), 0, s,
                   (const float4 *)partials, M, g.parts, V, plan_bitmap, tok, conf, ent, in_plan);
    return e == cudaSuccess ? PVF_OK : PVF_ERR_CUDA;
}

}  // namespace

namespace {

// Work split of one kernel shape: `workers` blocks (or pairs of blocks) share m_tiles row tiles of tile_rows
// rows; mb tiles are in flight at once, each swept by `splits` workers over disjoint vocabulary ranges.
// Modelled cost of a choice = waves * (max(MMA time of one worker's range, one pass over W) + a fixed cost
// per wave); the fixed cost (1.5 passes over W) was fitted to measured launches of 13 k and 32 k rows.
struct SplitPlan {
    int m_tiles, units, mb, splits, waves;
    double cost;
};

SplitPlan plan_split(int M, int V, int D, int workers, int tile_rows, int unit, int max_concurrent)
{
    SplitPlan p;
    p.m_tiles = (M + tile_rows - 1) / tile_rows;
    p.units = (V + unit - 1) / unit;
    p.mb = p.splits = p.waves = 0;
    p.cost = 0.0;
    const double flops_per_sm = 1.0e13, hbm = 6.0e12;
    for (int waves = 1; waves <= p.m_tiles; ++waves) {
        const int mb = (p.m_tiles + waves - 1) / waves;
        if (mb > workers || mb > max_concurrent) continue;
        if ((p.m_tiles + mb - 1) / mb != waves) continue;          // same mb already seen with fewer waves
        int splits = workers / mb;
        if (splits > p.units) splits = p.units;
        const int units_per_worker = (p.units + splits - 1) / splits;
        const double t_mma = (double)units_per_worker * unit * kTileM * 2.0 * D / flops_per_sm;   // per SM
        const double t_hbm = 2.0 * V * (double)D / hbm;
        const double cost = waves * ((t_mma > t_hbm ? t_mma : t_hbm) + 1.5 * t_hbm);
        if (p.waves == 0 || cost < p.cost * 0.999) {
            p.cost = cost; p.waves = waves; p.mb = mb; p.splits = splits;
        }
    }
    return p;
}

}  // namespace

pvf_score_geometry pvf_score_geometry_for(int M, int V, int D, int n_sm)
{
    pvf_score_geometry g;
    const int tiles128 = (M + kTileM - 1) / kTileM;
    g.streaming = (tiles128 == 1 && M <= kStreamRows) ? 1 : 0;
    g.a_rows = tiles128 == 1 ? ((M + 7) / 8) * 8 : kTileM;
    SplitPlan p = plan_split(M, V, D, n_sm, kTileM, kUnit, kMaxConcurrentTiles);
    g.paired = 0;
    if (tiles128 >= PVF_PAIR_MIN_TILES && M <= PVF_PAIR_MAX_ROWS && n_sm >= 2) {
        // The paired kernel works on 256-row tiles, granules of 32 vocabulary entries and pairs of SMs.  It
        // feeds the tensor cores better (measured: +8 .. +29 % from 129 to 8192 rows); it loses where pairs
        // and 256-row tiles divide the work less evenly, and in long launches the power cap, not the operand
        // feed, sets the pace (16 k rows and more: the single-block kernel is 4 .. 6 % faster).
        const SplitPlan pp = plan_split(M, V, D, n_sm / 2, 2 * kTileM, kPairUnit, kMaxConcurrentTiles / 2);
        if (pp.waves > 0 && pp.cost <= 1.05 * p.cost) { p = pp; g.paired = 1; }
    }
    g.swapped = 0; g.n_pad = 0; g.stages = 0;
    if (n_sm >= 2 && ((M > kStreamRows && M <= PVF_SWAP_SMALL_MAX_ROWS) || (M > kTileM && M <= PVF_SWAP_RAGGED_MAX_ROWS))) {
        // Swapped paired kernel: one row tile padded to a multiple of 32 rows (the MMA's N), every pair of SMs
        // sweeps one vocabulary range.  Chosen where the other kernels would pad the rows most (see the kernel).
        g.swapped = 1; g.paired = 0;
        g.n_pad = ((M + 31) / 32) * 32;
        g.a_rows = g.n_pad / 2;
        const int stage_bytes = kSwapWBytes + (g.n_pad / 2) * kRowBytes;
        g.stages = kSwapRingBytes / stage_bytes < kSwapMaxStages ? kSwapRingBytes / stage_bytes : kSwapMaxStages;
        p.m_tiles = 1; p.mb = 1; p.waves = 1;
        p.units = (V + kPairUnit - 1) / kPairUnit;
        p.splits = n_sm / 2 < p.units ? n_sm / 2 : p.units;
    }
    g.m_tiles = p.m_tiles; g.units = p.units;
    g.mb = p.mb; g.splits = p.splits; g.waves = p.waves;
    g.ctas = g.mb * g.splits * ((g.paired || g.swapped) ? 2 : 1);
    g.parts = g.splits * (g.swapped ? 2 : 1);
    return g;
}

size_t pvf_score_partials_bytes(const pvf_shape *shape, int n_sm)
{
    size_t worst = 0;
    const int max_tiles = (shape->max_rows + kTileM - 1) / kTileM;
    // Within one kernel choice and row-tile count the need grows with the rows, so it peaks at the upper end of
    // every 128-row step and of the swapped paired kernel's two windows.
    for (int t = 1; t <= max_tiles + 2; ++t) {
        int rows = t * kTileM;
        if (t == max_tiles + 1) rows = PVF_SWAP_SMALL_MAX_ROWS;
        if (t == max_tiles + 2) rows = PVF_SWAP_RAGGED_MAX_ROWS;
        if (rows > shape->max_rows) rows = shape->max_rows;
        if (rows <= 0) continue;
        const pvf_score_geometry g = pvf_score_geometry_for(rows, shape->vocab, shape->hidden, n_sm);
        const size_t need = (size_t)rows * g.parts * sizeof(float4);
        worst = need > worst ? need : worst;
    }
    return worst;
}

int pvf_score_init(pvf_ctx *ctx)
{
    const int rc = make_w_maps(ctx->tm_w, ctx->w_head, ctx->shape.vocab, ctx->shape.hidden);
    if (rc != PVF_OK) return rc;
    return raise_shared_memory_limits();
}

extern "C" {

int pvf_set_score_events(pvf_ctx *ctx, void *start, void *stop)
{
    if (!ctx || ((start == nullptr) != (stop == nullptr))) return PVF_ERR_INVALID;
    ctx->ev_start = (cudaEvent_t)start;
    ctx->ev_stop = (cudaEvent_t)stop;
    return PVF_OK;
}

int pvf_score_plan(pvf_ctx *ctx, int32_t M, int32_t *ctas, int32_t *splits, int32_t *waves, int32_t *launches)
{
    if (!ctx || M < 0 || M > ctx->shape.max_rows) return PVF_ERR_INVALID;
    const pvf_score_geometry g = pvf_score_geometry_for(M, ctx->shape.vocab, ctx->shape.hidden, ctx->n_sm);
    if (ctas) *ctas = g.ctas;
    if (splits) *splits = g.splits;
    if (waves) *waves = g.waves;
    if (launches) *launches = M > 0 ? 2 : 0;
    return PVF_OK;
}

int pvf_score_plan_for_shape(int32_t vocab, int32_t hidden, int32_t n_sm, int32_t M, int32_t *ctas, int32_t *splits,
                             int32_t *waves, int32_t *kernel, int32_t *row_tiles, int32_t *tiles_per_wave)
{
    if (vocab <= 0 || hidden <= 0 || n_sm <= 0 || M <= 0) return PVF_ERR_INVALID;
    const pvf_score_geometry g = pvf_score_geometry_for(M, vocab, hidden, n_sm);
    if (ctas) *ctas = g.ctas;
    if (splits) *splits = g.splits;
    if (waves) *waves = g.waves;
    if (kernel) *kernel = g.streaming ? 0 : (g.swapped ? 3 : (g.paired ? 2 : 1));
    if (row_tiles) *row_tiles = g.m_tiles;
    if (tiles_per_wave) *tiles_per_wave = g.mb;
    return PVF_OK;
}

const char *pvf_score_kernel_name(pvf_ctx *ctx, int32_t M)
{
    if (!ctx || M <= 0 || M > ctx->shape.max_rows) return nullptr;
    const pvf_score_geometry g = pvf_score_geometry_for(M, ctx->shape.vocab, ctx->shape.hidden, ctx->n_sm);
    return g.streaming ? "pvf_score_stream_kernel"
                       : (g.swapped ? "pvf_score_swap_pair_kernel" : (g.paired ? "pvf_score_gemm_pair_kernel" : "pvf_score_gemm_kernel"));
}

int pvf_score(pvf_ctx *ctx, const void *hidden, int32_t M,
              int32_t *tok, float *conf, float *ent, uint8_t *in_plan, void *stream)
{
    if (!ctx || M < 0 || M > ctx->shape.max_rows) return PVF_ERR_INVALID;
    if (M == 0) return PVF_OK;
    if (!hidden || !tok || !conf) return PVF_ERR_INVALID;
    if (((uintptr_t)hidden & 15) != 0) return PVF_ERR_ALIGN;
    const int V = ctx->shape.vocab, D = ctx->shape.hidden;
    const pvf_score_geometry g = pvf_score_geometry_for(M, V, D, ctx->n_sm);
    if ((size_t)M * g.parts * sizeof(float4) > ctx->partials_bytes) return PVF_ERR_WORKSPACE;
    return launch_score(g, hidden, M, V, D, ctx->tm_w, ctx->partials, &ctx->words->status, ctx->plan_bitmap, tok, conf,
                        ent, in_plan, (cudaStream_t)stream, ctx->ev_start, ctx->ev_stop);
}

}  // extern "C"

// ---------------------------------------------------------------------------------- pvf_score_static
// Scoring for callers that cannot allocate: the per-range softmax states (the only scratch the scoring
// kernels need) live in a fixed array inside the library image instead of a caller-provided workspace.
namespace {

constexpr int kStaticMaxRows = PVF_STATIC_MAX_ROWS;
constexpr int kStaticMaxSms = 256;                              // head-room over today's 148 SMs
constexpr size_t kStaticHeaderBytes = 256;                      // status word, padded
constexpr size_t kStaticPartialsBytes = (size_t)kTileM * kStaticMaxSms * sizeof(float4);
constexpr int kStaticMaxDevices = 64;

// Every GPU that loads this library holds these 512.25 KiB until the process exits.
static __device__ __align__(256) unsigned char pvf_static_scratch[kStaticHeaderBytes + kStaticPartialsBytes];

struct StaticDeviceState {
    bool ready;
    int n_sm;
    unsigned char *scratch;     // device address of pvf_static_scratch on that GPU
};
StaticDeviceState g_static_state[kStaticMaxDevices];

// Once per device, with that device current: resolve the array's device address (its name is only a
// host-side handle here) and raise the GEMM kernels' shared-memory limit.
int static_device_state(StaticDeviceState **out)
{
    int device = 0, cc = 0, n_sm = 0;
    if (cudaGetDevice(&device) != cudaSuccess) return PVF_ERR_CUDA;
    if (device < 0 || device >= kStaticMaxDevices) return PVF_ERR_UNSUPPORTED;
    StaticDeviceState *st = &g_static_state[device];
    if (!st->ready) {
        if (cudaDeviceGetAttribute(&cc, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
            cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
            return PVF_ERR_CUDA;
        if (cc != 10 || n_sm > kStaticMaxSms) return PVF_ERR_UNSUPPORTED;
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, pvf_static_scratch) != cudaSuccess || !ptr) return PVF_ERR_CUDA;
        if (raise_shared_memory_limits() != PVF_OK) return PVF_ERR_CUDA;
        st->scratch = (unsigned char *)ptr;
        st->n_sm = n_sm;
        st->ready = true;
    }
    *out = st;
    return PVF_OK;
}

}  // namespace

extern "C" {

int pvf_score_static(const void *w_head, int32_t vocab, int32_t hidden_size, const void *hidden, int32_t M,
                     const uint32_t *plan_bitmap, int32_t *tok, float *conf, float *ent, uint8_t *in_plan,
                     void *stream)
{
    if (vocab <= 0 || hidden_size <= 0 || M < 0) return PVF_ERR_INVALID;
    if (M > kStaticMaxRows) return PVF_ERR_TOO_LARGE;
    if (M == 0) return PVF_OK;
    if (!w_head || !hidden || !tok || !conf || (in_plan && !plan_bitmap)) return PVF_ERR_INVALID;
    if (hidden_size % 8 != 0 || ((uintptr_t)w_head & 15) != 0 || ((uintptr_t)hidden & 15) != 0) return PVF_ERR_ALIGN;
    StaticDeviceState *st = nullptr;
    int rc = static_device_state(&st);
    if (rc != PVF_OK) return rc;
    const pvf_score_geometry g = pvf_score_geometry_for(M, vocab, hidden_size, st->n_sm);
    if ((size_t)M * g.parts * sizeof(float4) > kStaticPartialsBytes) return PVF_ERR_TOO_LARGE;

    CUtensorMap w_levels[kWBoxSizes];
    if ((rc = make_w_maps(w_levels, w_head, vocab, hidden_size)) != PVF_OK) return rc;

    cudaStream_t s = (cudaStream_t)stream;
    int32_t *status = (int32_t *)st->scratch;
    float4 *partials = (float4 *)(st->scratch + kStaticHeaderBytes);
    // The array keeps the previous call's contents.  The status word must start at zero; the partial
    // states need no clearing: the GEMM kernel writes every (row, range) entry the merge kernel reads.
    if (cudaMemsetAsync(status, 0, sizeof(int32_t), s) != cudaSuccess) return PVF_ERR_CUDA;
    return launch_score(g, hidden, M, vocab, hidden_size, w_levels, partials, status, plan_bitmap, tok, conf, ent,
                        in_plan, s, nullptr, nullptr);
}

int pvf_score_static_status(int32_t *status)
{
    if (!status) return PVF_ERR_INVALID;
    StaticDeviceState *st = nullptr;
    int rc = static_device_state(&st);
    if (rc != PVF_OK) return rc;
    if (cudaMemcpy(status, st->scratch, sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess) return PVF_ERR_CUDA;
    return PVF_OK;
}

}  // extern "C"
