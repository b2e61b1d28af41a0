// pvf_score_swap_pair_kernel: vocabulary on the lanes of a cta_group::2 accumulator, rows on its columns.
// (A part of pvf_score.cu's translation unit; see that file for the overview.)
#pragma once
#include "pvf_score_common.cuh"
#include "pvf_score_gemm_pair.cuh"
#include "pvf_score_stream.cuh"

namespace {

// ---------------------------------------------------------------------------------- swapped paired kernel
// A few dozen to a few hundred rows: the launch sits at the ridge, where HBM, the L2 -> SM feed, the tensor pipe
// and the power cap all matter, and 128- or 256-row MMAs over a ragged row count waste tensor work (and with it
// clock).  Here the operands of the paired kernel change places: the two blocks of a pair hold 2 x 128 vocabulary
// entries on their accumulator lanes (each loads its own 128-entry W tile, so W still crosses L2 -> SM once) and
// the scored rows are the N columns, padded to a multiple of 32 (each block loads half of the H rows):
//     D[v][m] = sum_k W[v][k] * H[m][k],   one 256 x N x 16 MMA (cta_group::2) per 16 elements of k.
// Up to 256 rows are one column group and two accumulators alternate.  257 .. 512 rows are two column groups
// (256 + the rest: two MMAs per k-step on the same W tile) in ONE accumulator that fills tensor memory, so the
// epilogue of a vocabulary tile and the MMAs of the next no longer overlap -- still better than sweeping W
// through the SMs once per 128- or 256-row tile, which is what bounds the other kernels there (their L2 -> SM
// traffic is 2.3 x this kernel's at 288 rows).
// Measured against the other kernels (each alone for seconds, so that the power cap has settled, and in short
// bursts) it wins where they pad most or sweep W twice: 33 .. 64 rows (4 .. 5 %), 129 .. 192 rows (4 .. 9 %) and
// 257 .. 448 rows (17 % at 257, 7 % at 448); with full 128-, 256- or 512-row tiles they are as fast or 3 .. 9 %
// faster, so the geometry picks it for those three windows only.
//
// The MMA-issuing thread is the most latency-sensitive part: a data-dependent branch between the MMAs of a
// k-step (one loop serving one or two column groups) cost 17 .. 33 % of the whole launch; the two cases are
// separate loops.
//
// Epilogue: one warp per quadrant of 32 vocabulary lanes up to 256 rows, kSwapWideWarps above, taking the
// groups of 32 rows (columns) in turn.  A warp turns its 32 x 32 block
// around through a padded shared-memory tile of its own, after which lane i holds row i's 32 logits and folds
// them into the running state of row chunk*32 + i exactly as the GEMM kernels' epilogue does (no warp-wide
// reductions: those serialise on their latency with one epilogue warp per scheduler).  At the end of the block's
// range the four warps' states fold through the same shared memory and the block writes one partial state per
// row: 2 x splits partial states per row reach the merge kernel.
//
// The ring has as many stages as fit: a stage is the block's 16 KiB W tile plus its half of the H tile.
constexpr int kSwapWBytes = kTileM * kRowBytes;                      // 16 KiB
constexpr int kSwapGroupCols = 256;                                  // MMA N limit: columns (rows of H) per MMA
constexpr int kSwapMaxRows = 512;                                    // two column groups fill tensor memory
constexpr int kSwapTmemCols = 512;                                   // two accumulators of up to 256 columns, or one of up to 512
constexpr int kSwapEpilogueWarps = 4 * kSwapWideWarps;          // at most; one per tensor-memory lane quadrant works on up to
                                                                     // 256 rows, kSwapWideWarps (taking row chunks in turn) above
constexpr int kSwapEpilogueThreads = kSwapEpilogueWarps * 32;
constexpr int kSwapThreads = 64 + kSwapEpilogueThreads;              // producer warp, MMA warp, epilogue warps
constexpr int kSwapTurnPitch = 33;                                   // words per lane of a warp's 32 x 32 fp32 block (conflict-free both ways)
constexpr int kSwapWarpScratchBytes = 32 * kSwapTurnPitch * 4;       // that block, one per epilogue warp
// Scratch of one quadrant = its warps' blocks; at the end it holds the quadrant's row states (16 bytes per row).
__host__ __device__ constexpr int swap_warps_per_quad(int n_pad) { return n_pad > kSwapGroupCols ? kSwapWideWarps : 1; }
__host__ __device__ constexpr int swap_quad_scratch_bytes(int n_pad) { return swap_warps_per_quad(n_pad) * kSwapWarpScratchBytes; }
constexpr int kSwapMaxStages = 12;
constexpr int kSwapSmemBytes = 227 * 1024;                           // everything: alignment slack, ring, control block, scratch
static_assert(swap_quad_scratch_bytes(kSwapMaxRows) >= kSwapMaxRows * 16 && swap_quad_scratch_bytes(kSwapGroupCols) >= kSwapGroupCols * 16 &&
              kSwapWarpScratchBytes % 16 == 0, "fold scratch");
static_assert(kSwapMaxStages <= kMaxStages, "barrier arrays");
static_assert(kSwapSmallMaxRows <= kSwapGroupCols && kSwapRaggedMaxRows <= kSwapGroupCols &&
              kSwapWideMaxRows <= kSwapMaxRows, "row limits");

__host__ __device__ constexpr int swap_stage_bytes(int n_pad) { return kSwapWBytes + (n_pad / 2) * kRowBytes; }
// Pipeline stages that fit beside the control block and the epilogue's scratch.
inline int swap_stages(int n_pad)
{
    const int ring = kSwapSmemBytes - 1024 - 512 - 4 * swap_quad_scratch_bytes(n_pad);
    const int n = ring / swap_stage_bytes(n_pad);
    return n < kSwapMaxStages ? n : kSwapMaxStages;
}

// The producer's and the MMA thread's loops, once for one column group (kWide = false) and once for two: these
// two threads set the pace of the kernel, and a run-time choice inside their loops costs more than it looks.
struct SwapLoopArgs {
    uint32_t tiles_addr, stage_bytes, h0_bytes, h1_bytes, tmem_base;
    int n0, n1, n_stages, n_tiles, k_steps, n_bufs;
    uint32_t rank;
};

// Before the grid-dependency wait (W is a constant of the context, see the paired GEMM kernel's pair_prefetch_w): arm
// the first ring of stages, start this block's W tiles of them, ask the boxes that follow into L2.  Returns the
// number of stages started; swap_produce then only adds their hidden-state tiles.
constexpr int kSwapL2PrefetchSteps = 16;
__device__ __forceinline__ int swap_prefetch_w(const SwapLoopArgs &a, const TileSplit &split, SharedControl *ctl, const WMaps &tm_w,
                                               bool wide, ArmedStages &armed)
{
    const uint64_t w_policy = w_evict_first_policy();
    int started = 0, ahead = 0;
    for (int tile = 0; tile < a.n_tiles && (started < a.n_stages || ahead < kSwapL2PrefetchSteps); ++tile) {
        int tu0, tun;
        split.tile(tile, &tu0, &tun);
        const uint32_t bytes = 2u * ((uint32_t)tun * kUnitBytes + a.h0_bytes + (wide ? a.h1_bytes : 0u));
        const int w_row = tu0 * kPairUnit + (int)a.rank * tun * kUnit;
        for (int step = 0; step < a.k_steps && (started < a.n_stages || ahead < kSwapL2PrefetchSteps); ++step) {
            if (started < a.n_stages) {
                const uint32_t full = smem_u32(&ctl->full[started]);
                if (a.rank == 0) { mbar_arrive_expect_tx(full, bytes); armed.note(started, 0u); }
                tma_load_2d_pair_hint(a.tiles_addr + (uint32_t)started * a.stage_bytes, &tm_w.size[tun - 1], full, step * kBlockK, w_row,
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

template <bool kWide>
__device__ __forceinline__ void swap_produce(const SwapLoopArgs &a, const TileSplit &split, SharedControl *ctl,
                                             const CUtensorMap *tm_h, const CUtensorMap *tm_h1, const WMaps &tm_w,
                                             int32_t *status, int started, ArmedStages armed)
{
    int stage = 0;
    uint32_t phase = 0;
    int issued = 0;
    bool alive = true;
    const uint64_t w_policy = w_evict_first_policy();            // one wave, one row tile: W is read once
    const int row0 = (int)a.rank * (a.n0 / 2);                                      // this block's half of each group's rows
    const int row1 = a.n0 + (int)a.rank * (a.n1 / 2);
    for (int tile = 0; tile < a.n_tiles && alive; ++tile) {
        int tu0, tun;
        split.tile(tile, &tu0, &tun);
        const uint32_t bytes = 2u * ((uint32_t)tun * kUnitBytes + a.h0_bytes + (kWide ? a.h1_bytes : 0u));   // both blocks
        const int w_row = tu0 * kPairUnit + (int)a.rank * tun * kUnit;                                        // this block's entries
        for (int step = 0; step < a.k_steps; ++step, ++issued) {
            const uint32_t full = smem_u32(&ctl->full[stage]);
            const uint32_t w_dst = a.tiles_addr + (uint32_t)stage * a.stage_bytes;
            if (issued >= started) {                                                // else: armed, W tile on its way already
                if (!mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, status)) { alive = false; break; }
                if (a.rank == 0) { mbar_arrive_expect_tx(full, bytes); armed.note(stage, phase); }
                tma_load_2d_pair_hint(w_dst, &tm_w.size[tun - 1], full, step * kBlockK, w_row, w_policy);
            }
            tma_load_2d_pair(w_dst + kSwapWBytes, tm_h, full, step * kBlockK, row0);
            if (kWide) tma_load_2d_pair(w_dst + kSwapWBytes + a.h0_bytes, tm_h1, full, step * kBlockK, row1);
            if (++stage == a.n_stages) { stage = 0; phase ^= 1u; }
        }
    }
    if (!alive) {
        // Abort: the copies in flight land before the pair leaves (see the paired GEMM kernel: the even block waits,
        // bounded, on the barriers it armed; the odd block gives its copies a fixed time).
        if (a.rank == 0) drain_armed_stages(ctl, armed, a.n_stages);
        else {
            const unsigned long long t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) {}
        }
    }
}

template <bool kWide>
__device__ __forceinline__ void swap_issue(const SwapLoopArgs &a, SharedControl *ctl, int32_t *status)
{
    int stage = 0;
    uint32_t phase = 0;
    bool alive = true;
    const uint32_t idesc0 = instr_desc_bf16_m256(a.n0);
    const uint32_t idesc1 = instr_desc_bf16_m256(kWide ? a.n1 : a.n0);
    for (int tile = 0; tile < a.n_tiles && alive; ++tile) {
        const uint32_t buf = kWide ? 0u : ((uint32_t)tile & 1u);                    // one accumulator when wide, else two alternate
        const uint32_t acc_phase = (kWide ? (uint32_t)tile : ((uint32_t)tile >> 1)) & 1u;
        if (!mbar_wait(smem_u32(&ctl->acc_empty[buf]), acc_phase ^ 1u, ctl, status)) { alive = false; break; }
        tc_fence_after_sync();
        const uint32_t tmem_d = a.tmem_base + buf * kSwapGroupCols;
        for (int step = 0; step < a.k_steps; ++step) {
            if (!mbar_wait(smem_u32(&ctl->full[stage]), phase, ctl, status)) { alive = false; break; }
            tc_fence_after_sync();
            // A ragged vocabulary tile leaves stale bytes on the W tile's last rows: lanes the epilogue skips.
            const uint32_t w_addr = a.tiles_addr + (uint32_t)stage * a.stage_bytes;
            const uint64_t w_desc = smem_desc_k_major_sw128(w_addr);
            const uint64_t h0_desc = smem_desc_k_major_sw128(w_addr + kSwapWBytes);
            if (!kWide) {
#pragma unroll
                for (int k = 0; k < kBlockK / 16; ++k)
                    tc_mma_bf16_pair(tmem_d, w_desc + (uint64_t)(k * 2), h0_desc + (uint64_t)(k * 2), idesc0,
                                     (step | k) != 0 ? 1u : 0u);
            } else {                                             // columns 256 .. : the second group of rows, same W tile
                const uint64_t h1_desc = smem_desc_k_major_sw128(w_addr + kSwapWBytes + a.h0_bytes);
#pragma unroll
                for (int k = 0; k < kBlockK / 16; ++k) {
                    tc_mma_bf16_pair(tmem_d, w_desc + (uint64_t)(k * 2), h0_desc + (uint64_t)(k * 2), idesc0,
                                     (step | k) != 0 ? 1u : 0u);
                    tc_mma_bf16_pair(a.tmem_base + kSwapGroupCols, w_desc + (uint64_t)(k * 2), h1_desc + (uint64_t)(k * 2),
                                     idesc1, (step | k) != 0 ? 1u : 0u);
                }
            }
            tc_commit_pair(smem_u32(&ctl->empty[stage]));
            if (++stage == a.n_stages) { stage = 0; phase ^= 1u; }
        }
        if (alive) tc_commit_pair(smem_u32(&ctl->acc_full[buf]));
    }
    if (!alive) {
        tc_commit_pair_local(smem_u32(&ctl->drain));
        const unsigned long long t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&ctl->drain), 0u) && global_timer_ns() - t0 < kWaitLimitNs) {}
    }
}

__global__ void __launch_bounds__(kSwapThreads, 1)
pvf_score_swap_pair_kernel(const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ CUtensorMap tm_h1,
                           const __grid_constant__ WMaps tm_w, const ScoreArgs args)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw_addr = smem_u32(smem_raw);
    const uint32_t tiles_addr = (raw_addr + 1023u) & ~1023u;
    uint8_t *tiles_ptr = smem_raw + (tiles_addr - raw_addr);
    const int n_pad = args.n_pad;                                        // padded rows = accumulator columns (multiple of 32)
    const int n0 = min(n_pad, kSwapGroupCols), n1 = n_pad - n0;          // columns of the first and the second MMA of a k-step
    const int n_bufs = n1 > 0 ? 1 : 2;                                   // accumulators: two alternate while they fit
    const int n_stages = args.stages;
    const uint32_t h0_bytes = (uint32_t)(n0 / 2) * kRowBytes;            // this block's half of each column group's H rows
    const uint32_t h1_bytes = (uint32_t)(n1 / 2) * kRowBytes;
    const uint32_t stage_bytes = (uint32_t)kSwapWBytes + h0_bytes + h1_bytes;
    SharedControl *ctl = reinterpret_cast<SharedControl *>(tiles_ptr + (size_t)n_stages * stage_bytes);
    uint8_t *scratch = reinterpret_cast<uint8_t *>(ctl) + 512;          // four quadrants' scratch
    const int warps_per_quad = swap_warps_per_quad(n_pad);
    const int quad_scratch = swap_quad_scratch_bytes(n_pad);
    const int epilogue_threads = 128 * warps_per_quad;                   // warps 2 .. 5, and 6 .. 9 above 256 rows

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_cta_rank();                            // 0: even block (issues the MMAs), 1: its peer
    const int q = blockIdx.x >> 1;                                       // the pair's vocabulary range
    int u0, u1;
    split_range(args.units, args.splits, q, &u0, &u1);                   // granules of 32 entries
    const TileSplit split(u0, u1, kPairUnitsPerTile, 0);
    const int n_tiles = split.n_tiles;
    const int k_steps = args.num_kb;

    if (threadIdx.x == 0) init_pipeline_barriers(ctl, n_stages, 1, 2 * epilogue_threads);
    if (warp == 0 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"((unsigned long long)&tm_h) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"((unsigned long long)&tm_h1) : "memory");
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
    SwapLoopArgs la;
    la.tiles_addr = tiles_addr; la.stage_bytes = stage_bytes; la.h0_bytes = h0_bytes; la.h1_bytes = h1_bytes;
    la.tmem_base = tmem_base; la.n0 = n0; la.n1 = n1; la.n_stages = n_stages; la.n_tiles = n_tiles; la.k_steps = k_steps;
    la.n_bufs = n_bufs; la.rank = rank;
    pvf_launch_dependents();                                             // one wave: the next launch may move in as this one leaves
    ArmedStages armed;                                                   // even block: it arms full[]
    int started = 0;
    if (threadIdx.x == 0) started = swap_prefetch_w(la, split, ctl, tm_w, n1 != 0, armed);
    pvf_grid_dependency_wait();
    LaunchClock launch_clock;
    launch_clock.begin();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (one per block)
        if (lane == 0) {
            if (n1 == 0) swap_produce<false>(la, split, ctl, &tm_h, &tm_h1, tm_w, args.status, started, armed);
            else swap_produce<true>(la, split, ctl, &tm_h, &tm_h1, tm_w, args.status, started, armed);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (even block only)
        if (lane == 0 && rank == 0) {
            if (n1 == 0) swap_issue<false>(la, ctl, args.status);
            else swap_issue<true>(la, ctl, args.status);
        }
    } else if (warp < 2 + 4 * warps_per_quad) {
        // ------------------------------------------------------------------ softmax epilogue (both blocks)
        const int quad = warp & 3;                                       // tensor-memory lanes quad*32 .. quad*32+31
        const int half = (warp - 2) >> 2;                                // which of the quadrant's warps: takes row chunks
                                                                         // half, half + warps_per_quad, ...
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        const int n_chunks = n_pad >> 5;                                 // 32-row column groups
        const int e_thread = (int)threadIdx.x - 64;                      // 0 .. 255
        float *turn = reinterpret_cast<float *>(scratch + quad * quad_scratch + half * kSwapWarpScratchBytes);
        float4 *fold_quad = reinterpret_cast<float4 *>(scratch + quad * quad_scratch);   // [n_pad rows], after the sweep
        bool alive = true;
        RowState st[kSwapMaxRows / 64];                                  // st[i], lane l: state of row (warps_per_quad i + half) * 32 + l
#pragma unroll
        for (int i = 0; i < kSwapMaxRows / 64; ++i) { st[i].m = -INFINITY; st[i].s = 0.f; st[i].t = 0.f; st[i].arg = kNoArg; }
        for (int tile = 0; tile < n_tiles && alive; ++tile) {
            int tu0, tun;
            split.tile(tile, &tu0, &tun);
            const uint32_t buf = n_bufs == 2 ? ((uint32_t)tile & 1u) : 0u;
            const uint32_t acc_phase = (n_bufs == 2 ? ((uint32_t)tile >> 1) : (uint32_t)tile) & 1u;
            if (!mbar_wait(smem_u32(&ctl->acc_full[buf]), acc_phase, ctl, args.status)) { alive = false; break; }
            tc_fence_after_sync();
            const int block_v0 = tu0 * kPairUnit + (int)rank * tun * kUnit;         // vocabulary id on this block's lane 0
            const int block_end = min(block_v0 + tun * kUnit, args.V);
            const int warp_v0 = block_v0 + quad * 32;
            const int n_real = min(32, block_end - warp_v0);                        // vocabulary entries on this warp's lanes
            if (n_real > 0) {                                                        // warp-uniform
#pragma unroll
                for (int i = 0; i < kSwapMaxRows / 64; ++i) {
                    const int c = warps_per_quad * i + half;
                    if (c < n_chunks) {                                              // warp-uniform
                        uint32_t lo[16], hi[16];
                        const uint32_t col = lane_addr + buf * kSwapGroupCols + c * 32;       // column = row: group 1 starts at 256
                        tmem_ld16(col, lo);
                        tmem_ld16(col + 16, hi);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 16; ++j) {                               // lane = vocabulary entry, j = row
                            turn[lane * kSwapTurnPitch + j] = __uint_as_float(lo[j]);
                            turn[lane * kSwapTurnPitch + 16 + j] = __uint_as_float(hi[j]);
                        }
                        __syncwarp();
#pragma unroll
                        for (int part = 0; part < 2; ++part) {                       // lane = row, 16 vocabulary entries at a time
                            const int n = n_real - part * 16;
                            if (n > 0) {
                                uint32_t x[16];
#pragma unroll
                                for (int l = 0; l < 16; ++l) x[l] = __float_as_uint(turn[(part * 16 + l) * kSwapTurnPitch + lane]);
                                if (n >= 16) fold16<true>(st[i], x, warp_v0 + part * 16, 16);
                                else fold16<false>(st[i], x, warp_v0 + part * 16, n);
                            }
                        }
                        __syncwarp();
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive_even_block(smem_u32(&ctl->acc_empty[buf]));
        }
        // Fold the block's four quadrants and write the block's partial state of every row.  The row states
        // reuse the turn tiles, so every warp must have left its last tile first.  Every epilogue thread reaches
        // the barriers, aborting or not.
        asm volatile("bar.sync 1, %0;" ::"r"(epilogue_threads) : "memory");
        if (alive) {
#pragma unroll
            for (int i = 0; i < kSwapMaxRows / 64; ++i) {
                const int c = warps_per_quad * i + half;
                if (c < n_chunks)
                    fold_quad[c * 32 + lane] = make_float4(st[i].m, st[i].s, st[i].t, __int_as_float(st[i].arg));
            }
        }
        asm volatile("bar.sync 1, %0;" ::"r"(epilogue_threads) : "memory");
        if (alive && !ctl->abort_flag) {
            for (int row = e_thread; row < args.M; row += epilogue_threads) {
                float4 acc = reinterpret_cast<const float4 *>(scratch)[row];
#pragma unroll
                for (int o = 1; o < 4; ++o)
                    pvf_state_merge(acc, reinterpret_cast<const float4 *>(scratch + o * quad_scratch)[row]);
                args.partials[(size_t)row * args.parts + 2 * q + (int)rank] = acc;
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();
    launch_clock.end(args.clock_acc);
    if (warp == 1) {
        tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kSwapTmemCols) : "memory");
    }
}

}  // namespace
