// pvf_score_swap_pair_kernel: vocabulary on the lanes of a cta_group::2 accumulator, rows on its columns.
// (A part of pvf_score.cu's translation unit; see that file for the overview.)
#pragma once
#include "pvf_score_common.cuh"
#include "pvf_score_gemm_pair.cuh"
#include "pvf_score_stream.cuh"

namespace {

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

}  // namespace
