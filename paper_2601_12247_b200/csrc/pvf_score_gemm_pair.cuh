// pvf_score_gemm_pair_kernel: two thread blocks (cta_group::2) per 256-row tile.
// (A part of pvf_score.cu's translation unit; see that file for the overview.)
#pragma once
#include "pvf_score_common.cuh"

namespace {

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
__device__ __forceinline__ void tma_load_2d_pair_hint(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4}], [%2], %5;"
        ::"r"(dst), "l"((unsigned long long)map), "r"(bar & kPeerBitMask), "r"(x), "r"(y), "l"(policy) : "memory");
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

// Work of pair `pair` in wave w: its 256-row tile, its vocabulary range (granules of 32) and the index q of that
// range among the tile's.  Every wave but a partial last one has args.mb tiles in flight, each swept by args.splits
// pairs; a partial last wave has args.mb_last tiles and args.splits_last (more) pairs per tile, so that the pairs
// are all busy there too.  False: the pair has nothing to do in this wave.
__device__ __forceinline__ bool pair_wave_work(const ScoreArgs &args, int pair, int w, int *s_tile, int *q, int *u0, int *u1)
{
    const bool last = args.mb_last > 0 && w == args.waves - 1;
    const int mb = last ? args.mb_last : args.mb, splits = last ? args.splits_last : args.splits;
    *q = pair / mb;
    *s_tile = w * args.mb + pair % mb;
    if (*q >= splits || *s_tile >= args.m_tiles) return false;
    split_range(args.units, splits, *q, u0, u1);
    return true;
}

// Wave boundary.  The blocks that sweep one vocabulary range for different row tiles stream the same W tiles, and
// W crosses HBM once per wave only while they stay close together (what one block fetched, the others find in L2).
// Over several waves they drift apart -- measured: 1356 TFLOP/s at 2 waves, 1150 at 17 -- so every block's producer
// thread pauses at the start of each wave until all blocks of the grid have got there: 1373 .. 1385 TFLOP/s at any
// number of waves.  The pause only lines the blocks up; nothing depends on it.  It therefore ends by itself after
// kWaveWaitLimitNs (a fraction of a wave) and the block goes on alone: no block ever needs another one to be resident
// or to make progress, and a profiler that serialises blocks merely loses the alignment.
constexpr unsigned long long kWaveWaitLimitNs = 2000000ull;
__device__ __forceinline__ void wave_boundary(uint32_t *arrivals, unsigned target)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(arrivals) : "memory");
    const unsigned long long t0 = global_timer_ns();
    for (;;) {
        unsigned seen;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(arrivals) : "memory");
        if (seen >= target || global_timer_ns() - t0 > kWaveWaitLimitNs) return;
        __nanosleep(256);
    }
}

// Before the grid-dependency wait of a launch of one wave (W is read once): the producer arms the first ring of
// stages and starts this block's half of their W tiles, then asks the W boxes that follow into L2.  W is a constant
// of the context -- nothing earlier in the stream can change it -- so the weight stream of this launch starts on
// every SM the previous launch has left while the rest of it, and the decision kernel between the two, still run.
// Returns the number of stages started; pair_produce then only adds their hidden-state tiles.
constexpr int kPairL2PrefetchSteps = 16;
__device__ __forceinline__ int pair_prefetch_w(const ScoreArgs &args, const WMaps &tm_w, SharedControl *ctl, uint32_t tiles_addr,
                                               int pair, uint32_t rank, int k_steps, ArmedStages &armed)
{
    int s_tile, q, u0, u1;
    if (!pair_wave_work(args, pair, 0, &s_tile, &q, &u0, &u1)) return 0;
    const TileSplit split(u0, u1, kPairUnitsPerTile, 0);
    const uint64_t w_policy = w_evict_first_policy();
    int started = 0, ahead = 0;
    for (int tile = 0; tile < split.n_tiles && (started < kPairStages || ahead < kPairL2PrefetchSteps); ++tile) {
        int tu0, tun;
        split.tile(tile, &tu0, &tun);
        const uint32_t bytes = 2u * ((uint32_t)kPairABytes + (uint32_t)tun * kUnitBytes);
        const int w_row = tu0 * kPairUnit + (int)rank * tun * kUnit;
        for (int step = 0; step < k_steps && (started < kPairStages || ahead < kPairL2PrefetchSteps); ++step) {
            if (started < kPairStages) {
                const uint32_t full = smem_u32(&ctl->full[started]);
                if (rank == 0) { mbar_arrive_expect_tx(full, bytes); armed.note(started, 0u); }
                tma_load_2d_pair_hint(tiles_addr + started * kPairStageBytes + kPairABytes, &tm_w.size[tun - 1], full, step * kBlockK, w_row,
                                      w_policy);
                ++started;
            } else {
                tma_prefetch_l2_2d(&tm_w.size[tun - 1], step * kBlockK, w_row, w_policy);
                ++ahead;
            }
        }
    }
    return started;
}

// The TMA producer's loop (one thread per block).  kReadOnce: W is read exactly once by the launch (evict-first hint).
// `started` stages (of wave 0) are armed and have their W tiles on the way already (pair_prefetch_w).
template <bool kReadOnce>
__device__ __forceinline__ void pair_produce(const ScoreArgs &args, const CUtensorMap &tm_h, const WMaps &tm_w, SharedControl *ctl,
                                             uint32_t tiles_addr, int pair, uint32_t rank, int k_steps, int started, ArmedStages armed)
{
    int stage = 0;
    uint32_t phase = 0;
    int issued = 0;
    const uint64_t w_policy = kReadOnce ? w_evict_first_policy() : 0ull;
    bool alive = true;
    for (int w = 0; w < args.waves && alive; ++w) {
        if (w > 0 && args.wave_sync) wave_boundary(args.wave_sync, (unsigned)w * gridDim.x);
        int s_tile, q, u0, u1;
        if (!pair_wave_work(args, pair, w, &s_tile, &q, &u0, &u1)) continue;
        const TileSplit split(u0, u1, kPairUnitsPerTile, 0);
        const int n_tiles = split.n_tiles;
        const int row0 = s_tile * 2 * kTileM + (int)rank * kTileM;          // this block's rows
        for (int tile = 0; tile < n_tiles && alive; ++tile) {
            int tu0, tun;
            split.tile(tile, &tu0, &tun);
            const uint32_t bytes = 2u * ((uint32_t)kPairABytes + (uint32_t)tun * kUnitBytes);   // both blocks
            const int w_row = tu0 * kPairUnit + (int)rank * tun * kUnit;                        // this block's half
            for (int step = 0; step < k_steps; ++step, ++issued) {
                const uint32_t full = smem_u32(&ctl->full[stage]);
                const uint32_t a_dst = tiles_addr + stage * kPairStageBytes;
                if (issued < started) {                                      // armed, W half on its way: the H tile is left
                    tma_load_2d_pair(a_dst, &tm_h, full, step * kBlockK, row0);
                } else {
                    if (!mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, args.status)) { alive = false; break; }
                    if (rank == 0) { mbar_arrive_expect_tx(full, bytes); armed.note(stage, phase); }
                    tma_load_2d_pair(a_dst, &tm_h, full, step * kBlockK, row0);
                    if (kReadOnce) tma_load_2d_pair_hint(a_dst + kPairABytes, &tm_w.size[tun - 1], full, step * kBlockK, w_row, w_policy);
                    else tma_load_2d_pair(a_dst + kPairABytes, &tm_w.size[tun - 1], full, step * kBlockK, w_row);
                }
                if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
            }
        }
    }
    if (alive && args.wave_sync && args.waves > 1 && atomicAdd(args.wave_sync + 1, 1u) == gridDim.x - 1) {
        args.wave_sync[0] = 0;                                               // every block is past its last boundary:
        args.wave_sync[1] = 0;                                               // rearm the counters for the next launch
    }
    if (!alive) {
        // Abort: the copies in flight land before the pair leaves.  The even block's full[] barriers count
        // both blocks' bytes, so it waits (bounded) on every stage it armed; the odd block has no barrier
        // of its own to wait on and gives its copies a fixed time (the closing cluster barrier holds both
        // blocks until the slower one is through).
        if (rank == 0) drain_armed_stages(ctl, armed, kPairStages);
        else {
            const unsigned long long t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) {}
        }
    }
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
    ArmedStages armed;                                                   // even block: it arms full[]
    int started = 0;
    if (args.w_once) {
        pvf_launch_dependents();                                         // one wave: the next launch may move in as this one leaves
        if (threadIdx.x == 0) started = pair_prefetch_w(args, tm_w, ctl, tiles_addr, pair, rank, k_steps, armed);
    }
    pvf_grid_dependency_wait();
    LaunchClock launch_clock;
    launch_clock.begin();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (one per block)
        if (lane == 0) {
            if (args.w_once) pair_produce<true>(args, tm_h, tm_w, ctl, tiles_addr, pair, rank, k_steps, started, armed);
            else pair_produce<false>(args, tm_h, tm_w, ctl, tiles_addr, pair, rank, k_steps, 0, armed);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (even block only)
        if (lane == 0 && rank == 0) {
            int stage = 0;
            uint32_t phase = 0;
            uint32_t tile_count = 0;
            bool alive = true;
            for (int w = 0; w < args.waves && alive; ++w) {
                int s_tile, q, u0, u1;
                if (!pair_wave_work(args, pair, w, &s_tile, &q, &u0, &u1)) continue;
                const TileSplit split(u0, u1, kPairUnitsPerTile, 0);
                const int n_tiles = split.n_tiles;
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
            int s_tile, q, u0, u1;
            if (!pair_wave_work(args, pair, w, &s_tile, &q, &u0, &u1)) continue;
            const TileSplit split(u0, u1, kPairUnitsPerTile, 0);
            const int n_tiles = split.n_tiles;
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
            if (alive && row < args.M) {
                float4 *row_parts = args.partials + (size_t)row * args.parts;
                row_parts[q] = make_float4(st.m, st.s, st.t, __int_as_float(st.arg));
                // a row's slots beyond its wave's ranges (the other kind of wave has more) hold empty states
                const int splits = (args.mb_last > 0 && w == args.waves - 1) ? args.splits_last : args.splits;
                if (q == 0)
                    for (int e = splits; e < args.parts; ++e) row_parts[e] = make_float4(-INFINITY, 0.f, 0.f, __int_as_float(kNoArg));
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                                                  // neither block leaves while the other may still signal it
    launch_clock.end(args.clock_acc);
    if (!args.w_once) pvf_launch_dependents();                           // several waves: the next kernel could only wait beside this one
    if (warp == 1) {
        tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kPairTmemCols) : "memory");
    }
}

}  // namespace
