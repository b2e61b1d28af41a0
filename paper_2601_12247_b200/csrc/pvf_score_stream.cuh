// pvf_score_stream_kernel: at most 32 rows, vocabulary on the accumulator lanes.
// (A part of pvf_score.cu's translation unit; see that file for the overview.)
#pragma once
#include "pvf_score_common.cuh"

namespace {

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
constexpr int kStreamStages = 6;
constexpr int kStreamTileN = 256;                                   // vocabulary entries per W tile (two 128-lane slices)
constexpr int kStreamUnitsPerTile = kStreamTileN / kUnit;
constexpr int kStreamHBytes = kStreamRows * kRowBytes;              // 4 KiB
constexpr int kStreamWBytes = kStreamTileN * kRowBytes;             // 32 KiB
constexpr int kStreamStageBytes = kStreamHBytes + kStreamWBytes;
constexpr int kStreamTmemCols = 128;                                // 2 buffers x 2 slices x 32 columns
constexpr int kStreamControlBytes = 512;
constexpr int kStreamL2PrefetchSteps = 16;                          // W boxes (up to 32 KB each) asked into L2 before the wait
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
    const TileSplit split(u0, u1, kStreamUnitsPerTile, widest_range(args.units, args.splits));
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
    pvf_launch_dependents();

    // W is a constant of the context: nothing the kernels before this one in the stream do can change it.  The
    // producer therefore starts the W tiles of the first ring of stages BEFORE the grid-dependency wait (the hidden
    // states, which the predecessor may still be writing, follow after it): the weight stream of this launch starts
    // on every SM the previous launch has left, while its slowest blocks and the decision kernel between the two
    // launches are still running.  The ring holds 192 KB of the block's 7 MB; the SM would then idle until the wait
    // returns (the spread of the previous launch's block ends plus the decision kernel: 15 .. 20 us), so the W boxes
    // that follow are asked into L2 (a hint, evict-first like the loads themselves), where the loads after the wait
    // find them.
    ArmedStages armed;
    int prefetched = 0;
    if (threadIdx.x == 0) {
        const uint64_t w_policy = w_evict_first_policy();
        int ahead = 0;                                               // W boxes asked into L2 beyond the ring
        for (int tile = 0; tile < n_tiles && (prefetched < kStreamStages || ahead < kStreamL2PrefetchSteps); ++tile) {
            int tu0, tun;
            split.tile(tile, &tu0, &tun);
            const uint32_t bytes = (uint32_t)args.a_rows * kRowBytes + (uint32_t)tun * kUnitBytes;
            for (int step = 0; step < k_steps && (prefetched < kStreamStages || ahead < kStreamL2PrefetchSteps); ++step) {
                if (prefetched < kStreamStages) {
                    const uint32_t full = smem_u32(&ctl->full[prefetched]);
                    mbar_arrive_expect_tx(full, bytes);              // the stage's H panel and W tile
                    armed.note(prefetched, 0u);
                    load_w_tile<true>(tiles_addr + prefetched * kStreamStageBytes + kStreamHBytes, tm_w, full, step * kBlockK, tu0,
                                      tun, w_policy);
                    ++prefetched;
                } else {
                    tma_prefetch_l2_2d(&tm_w.size[tun - 1], step * kBlockK, tu0 * kUnit, w_policy);
                    ++ahead;
                }
            }
        }
    }
    pvf_grid_dependency_wait();
    LaunchClock launch_clock;
    launch_clock.begin();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int issued = 0;
            const uint64_t w_policy = w_evict_first_policy();         // one wave, one row tile: W is read once
            bool alive = true;
            for (int tile = 0; tile < n_tiles && alive; ++tile) {
                int tu0, tun;
                split.tile(tile, &tu0, &tun);
                const uint32_t bytes = (uint32_t)args.a_rows * kRowBytes + (uint32_t)tun * kUnitBytes;
                for (int step = 0; step < k_steps; ++step, ++issued) {
                    const uint32_t full = smem_u32(&ctl->full[stage]);
                    const uint32_t h_dst = tiles_addr + stage * kStreamStageBytes;
                    if (issued < prefetched) {                           // armed, W tile on its way: the H panel is left
                        tma_load_2d(h_dst, &tm_h, full, step * kBlockK, 0);
                    } else {
                        if (!mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, ctl, args.status)) { alive = false; break; }
                        mbar_arrive_expect_tx(full, bytes);
                        armed.note(stage, phase);
                        tma_load_2d(h_dst, &tm_h, full, step * kBlockK, 0);
                        load_w_tile<true>(h_dst + kStreamHBytes, tm_w, full, step * kBlockK, tu0, tun, w_policy);
                    }
                    if (++stage == kStreamStages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!alive) drain_armed_stages(ctl, armed, kStreamStages);
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
            for (int l = 0; l < 32; ++l) pvf_state_merge(acc, scratch[row * kTileM + part * 32 + l]);
            for (int o = 1; o < 4; o <<= 1) {
                float4 other;
                other.x = __shfl_xor_sync(0xffffffffu, acc.x, o);
                other.y = __shfl_xor_sync(0xffffffffu, acc.y, o);
                other.z = __shfl_xor_sync(0xffffffffu, acc.z, o);
                other.w = __shfl_xor_sync(0xffffffffu, acc.w, o);
                pvf_state_merge(acc, other);
            }
            if (part == 0 && row < args.M) args.partials[(size_t)row * args.splits + q] = acc;
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    launch_clock.end(args.clock_acc);
    if (warp == 1) {
        tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kStreamTmemCols) : "memory");
    }
}

}  // namespace
