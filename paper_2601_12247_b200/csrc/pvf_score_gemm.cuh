// pvf_score_gemm_kernel: rows on the accumulator lanes, one thread block per (row tile, vocabulary range).
// (A part of pvf_score.cu's translation unit; see that file for the overview.)
#pragma once
#include "pvf_score_common.cuh"

namespace {

// ---------------------------------------------------------------------------------- GEMM kernel
// The TMA producer's loop (one thread).  kReadOnce: W is read exactly once by the launch (evict-first hint).
template <class Cfg, bool kReadOnce>
__device__ __forceinline__ void gemm_produce(const ScoreArgs &args, const CUtensorMap &tm_h, const WMaps &tm_w, SharedControl *ctl,
                                             const TileSplit &split, uint32_t tiles_addr, int mt_local, int k_steps)
{
    constexpr int kStages = Cfg::kStages;
    constexpr int kPanels = Cfg::kPanels;
    const int n_tiles = split.n_tiles;
    int stage = 0;
    uint32_t phase = 0;
    ArmedStages armed;
    const uint64_t w_policy = kReadOnce ? w_evict_first_policy() : 0ull;
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
                armed.note(stage, phase);
                for (int p = 0; p < np; ++p) {
                    const int x = (kb0 + p) * kBlockK;
                    tma_load_2d(a_base + p * Cfg::kAPanelBytes, &tm_h, full, x, m_tile * kTileM);
                    load_w_tile<kReadOnce>(b_base + p * Cfg::kBPanelBytes, tm_w, full, x, tu0, tun, w_policy);
                }
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
        }
    }
    // Abort: let every copy this thread started land before the block's memory is released.
    if (!alive) drain_armed_stages(ctl, armed, kStages);
}

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
    const TileSplit split(u0, u1, kUnitsPerTile, 0);
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
    LaunchClock launch_clock;
    launch_clock.begin();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            if (args.w_once) gemm_produce<Cfg, true>(args, tm_h, tm_w, ctl, split, tiles_addr, mt_local, k_steps);
            else gemm_produce<Cfg, false>(args, tm_h, tm_w, ctl, split, tiles_addr, mt_local, k_steps);
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
    launch_clock.end(args.clock_acc);
    pvf_launch_dependents();
    if (warp == 1) {
        tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(Cfg::kTmemCols) : "memory");
    }
}

}  // namespace
