// pvf_score: LM-head projection fused with a streaming softmax (sm_100a).
//
//   logits[m][v] = sum_k H[m][k] * W[v][k]      bf16 operands, fp32 accumulation in tensor memory
//   per row m:     top-1 token, its probability, the entropy of softmax(logits[m][:])
//
// The logits never leave the SM.  Scored rows sit on the 128 lanes of a tcgen05 accumulator, the
// vocabulary on its columns, so one epilogue thread owns one row and keeps that row's running
// softmax state (max, argmax, sum e^{x-max}, sum (x-max) e^{x-max}) in registers while the thread
// block sweeps a contiguous vocabulary range.  Each (row, range) pair leaves one 16-byte partial
// state; the kernel that follows on the stream merges the partial states of a row: the small merge
// kernel of pvf_score, or the head of the step kernels (pvf_draft_step: merge + commit + select in one
// launch; pvf_verify_step: merge + verify), which then write token, confidence, entropy and planning-
// vocabulary membership themselves.
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
// padding, and 257 .. 448 rows, where they sweep W through the SMs twice or more, take the paired kernel
// with swapped operands (pvf_score_swap_pair_kernel).
//
// Work split.  Rows form tiles of 128, the vocabulary granules of 16 entries.  `mb` row tiles are
// in flight at once, each swept by `splits` blocks over disjoint vocabulary ranges (mb * splits
// <= number of SMs); blocks that share a range stream the same W tiles at the same time, so W is
// read from HBM once per wave, and the wave's H tiles stay L2-resident.
//
// Every wait on an mbarrier is bounded: when one runs out the block records PVF_ERR_TIMEOUT in
// the status word, raises a block-wide abort flag, drains its outstanding copies and MMAs with
// bounded waits, frees its tensor memory and returns.
// The kernels live in pvf_score_*.cuh (one file each, all part of this translation unit); this file holds the
// merge kernel, the host-side work split and the entry points.  (Merging in the projection kernel's own tail, by the
// block that finishes last, was built and measured: that code runs once per launch on instructions the weight
// stream has long pushed out of L2, and cost 9 .. 30 us per call against 4 us for a kernel whose blocks are resident
// and waiting -- programmatic dependent launch -- before the projection ends.)
#include <mutex>

#include "pvf_score_common.cuh"
#include "pvf_score_gemm.cuh"
#include "pvf_score_gemm_pair.cuh"
#include "pvf_score_stream.cuh"
#include "pvf_score_swap_pair.cuh"

namespace {

// ---------------------------------------------------------------------------------- merge kernel
// Combines the rows' partial states and writes token, confidence, entropy and planning-vocabulary membership.
constexpr int kMergeKernelThreads = 128;
__global__ void __launch_bounds__(kMergeKernelThreads, 1)
pvf_score_merge_kernel(const float4 *__restrict__ partials, int M, int parts, int vocab,
                       const uint32_t *__restrict__ plan_bitmap, int32_t *__restrict__ tok,
                       float *__restrict__ conf, float *__restrict__ ent, uint8_t *__restrict__ in_plan)
{
    pvf_launch_dependents();
    pvf_grid_dependency_wait();
    const int warps_per_block = kMergeKernelThreads / 32;
    pvf_merge_rows(partials, parts, vocab, plan_bitmap, 0, M, (int)blockIdx.x * warps_per_block + (int)(threadIdx.x >> 5),
                   (int)gridDim.x * warps_per_block, tok, conf, ent, in_plan);
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

// Launches the projection kernel (shape chosen by the geometry) on `s`: it leaves g.parts partial states per row.
int launch_projection(const pvf_score_geometry &g, const void *hidden, int M, int V, int D, const CUtensorMap *w_levels,
                      float4 *partials, int32_t *status, uint32_t *wave_sync, unsigned long long *clock_acc, cudaStream_t s,
                      cudaEvent_t ev_start, cudaEvent_t ev_stop)
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
    a.mb_last = g.mb_last; a.splits_last = g.splits_last;
    a.a_rows = g.a_rows;
    a.n_pad = g.n_pad; a.stages = g.stages; a.parts = g.parts;
    a.w_once = (g.waves == 1 && g.mb == 1) ? 1 : 0;
    a.partials = partials;
    a.status = status;
    a.wave_sync = (g.paired && g.waves > 1) ? wave_sync : nullptr;
    a.clock_acc = clock_acc;
    const bool timed = ev_start && ev_stop;
    if (timed && cudaEventRecord(ev_start, s) != cudaSuccess) return PVF_ERR_CUDA;
    cudaError_t e;
    if (g.swapped) {
        CUtensorMap tm_h1 = tm_h;                                   // rows 256 .. of H: the second column group, if any
        if (g.n_pad > kSwapGroupCols &&
            (rc = make_tensor_map(&tm_h1, hidden, (uint64_t)M, (uint64_t)D, (uint32_t)((g.n_pad - kSwapGroupCols) / 2))) != PVF_OK)
            return rc;
        e = pvf_launch_cluster2(pvf_score_swap_pair_kernel, dim3(g.ctas), dim3(64 + 128 * swap_warps_per_quad(g.n_pad)), kSwapSmemBytes, s, tm_h, tm_h1, maps, a);
    }
    else if (g.paired)
        e = pvf_launch_cluster2(pvf_score_gemm_pair_kernel, dim3(g.ctas), dim3(kThreads), kPairSmemBytes, s, tm_h, maps, a);
    else if (g.streaming)
        e = pvf_launch(pvf_score_stream_kernel, dim3(g.ctas), dim3(kStreamThreads), kStreamSmemBytes, s, tm_h, maps, a);
    else
        e = pvf_launch(pvf_score_gemm_kernel<GeneralCfg>, dim3(g.ctas), dim3(kThreads), GeneralCfg::kSmemBytes, s, tm_h, maps, a);
    if (e != cudaSuccess) return PVF_ERR_CUDA;
    if (timed && cudaEventRecord(ev_stop, s) != cudaSuccess) return PVF_ERR_CUDA;
    return PVF_OK;
}

// The merge kernel of pvf_score on `s`.
int launch_merge(const float4 *partials, int M, int parts, int V, const uint32_t *plan_bitmap, int32_t *tok, float *conf,
                 float *ent, uint8_t *in_plan, cudaStream_t s)
{
    // one turn of a warp covers kMergeRowsInFlight groups of 32 / g rows (g lanes per row)
    int g = 1;
    while (g < parts && g < 32) g <<= 1;
    const int rows_per_turn = (32 / g) * kMergeRowsInFlight, warps_per_block = kMergeKernelThreads / 32;
    const int turns = (M + rows_per_turn - 1) / rows_per_turn;
    int blocks = (turns + warps_per_block - 1) / warps_per_block;
    blocks = blocks > 1184 ? 1184 : blocks;                            // the warps stride over the rows beyond that
    const cudaError_t e = pvf_launch(pvf_score_merge_kernel, dim3(blocks), dim3(kMergeKernelThreads), 0, s, partials, M, parts, V,
                                     plan_bitmap, tok, conf, ent, in_plan);
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
    int mb_last, splits_last;          // paired kernel only: a partial last wave split over more pairs per tile
    double cost;
};

SplitPlan plan_split(int M, int V, int D, int workers, int tile_rows, int unit, int max_concurrent)
{
    SplitPlan p;
    p.m_tiles = (M + tile_rows - 1) / tile_rows;
    p.units = (V + unit - 1) / unit;
    p.mb = p.splits = p.waves = p.mb_last = p.splits_last = 0;
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

// Work split of the paired kernel: 256-row tiles, granules of 32 vocabulary entries, `pairs` pairs of SMs.  Every
// full wave has mb tiles in flight, each swept by `splits` pairs (mb * splits <= pairs); what is left of the tiles
// makes a last wave of mb_last tiles, each swept by splits_last = pairs / mb_last pairs, so that no pair sits out a
// whole sweep because the tile count is not a multiple of mb.  The hidden states of a wave (mb tiles, re-read from L2
// once per vocabulary tile) must stay L2-resident beside the weight stream, which bounds mb: measured at 32768 and
// 103042 rows with budgets of 30 / 40 / 52 / 64 / 80 MB (6 / 4 / 3 / 3 / 2 pairs per tile): 1382 / 1386 / 1378 / 1381 /
// 1346 and 1373 / 1391 / 1367 / 1362 / 1307 TFLOP/s under the power cap.  Cost as in plan_split.
constexpr long long kMaxWaveHiddenBytes = 40ll << 20;

SplitPlan plan_pair_split(int M, int V, int D, int pairs)
{
    SplitPlan p;
    p.m_tiles = (M + 2 * kTileM - 1) / (2 * kTileM);
    p.units = (V + kPairUnit - 1) / kPairUnit;
    p.mb = p.splits = p.waves = p.mb_last = p.splits_last = 0;
    p.cost = 0.0;
    const double flops_per_sm = 1.0e13, hbm = 6.0e12;
    const double t_unit = (double)kPairUnit * kTileM * 2.0 * D / flops_per_sm, t_hbm = 2.0 * V * (double)D / hbm;
    for (int splits = 1; splits <= pairs && splits <= p.units; ++splits) {
        int mb = pairs / splits;
        if (mb > p.m_tiles) mb = p.m_tiles;
        if ((long long)mb * 2 * kTileM * D * 2 > kMaxWaveHiddenBytes && mb > 1) continue;
        const int full = p.m_tiles / mb, rest = p.m_tiles % mb;
        int splits_last = 0;
        if (rest > 0) {
            splits_last = pairs / rest;
            if (splits_last > p.units) splits_last = p.units;
        }
        const int waves = full + (rest > 0 ? 1 : 0);
        const double t_full = (double)((p.units + splits - 1) / splits) * t_unit;
        const double t_rest = rest > 0 ? (double)((p.units + splits_last - 1) / splits_last) * t_unit : 0.0;
        const double cost = full * ((t_full > t_hbm ? t_full : t_hbm) + 1.5 * t_hbm) +
                            (rest > 0 ? (t_rest > t_hbm ? t_rest : t_hbm) + 1.5 * t_hbm : 0.0);
        if (p.waves == 0 || cost < p.cost * 0.999) {
            p.cost = cost; p.waves = waves; p.mb = mb; p.splits = splits;
            p.mb_last = rest; p.splits_last = splits_last;
        }
    }
    return p;
}

}  // namespace

pvf_score_geometry pvf_score_geometry_for(int M, int V, int D, int n_sm, bool allow_swapped)
{
    pvf_score_geometry g;
    const int tiles128 = (M + kTileM - 1) / kTileM;
    g.streaming = (tiles128 == 1 && M <= kStreamRows) ? 1 : 0;
    g.a_rows = tiles128 == 1 ? ((M + 7) / 8) * 8 : kTileM;
    SplitPlan p = plan_split(M, V, D, n_sm, kTileM, kUnit, kMaxConcurrentTiles);
    g.paired = 0;
    if (tiles128 >= kPairMinTiles && n_sm >= 2) {
        // The paired kernel works on 256-row tiles, granules of 32 vocabulary entries and pairs of SMs: each SM
        // pulls a third less through L2 per MMA cycle, which is what bounds the single-block kernel (and costs
        // power: under the cap the paired kernel does the same work at a lower clock).
        const SplitPlan pp = plan_pair_split(M, V, D, n_sm / 2);
        if (pp.waves > 0) { p = pp; g.paired = 1; }
    }
    g.swapped = 0; g.n_pad = 0; g.stages = 0;
    if (allow_swapped && n_sm >= 2 && ((M > kStreamRows && M <= kSwapSmallMaxRows) || (M > kTileM && M <= kSwapRaggedMaxRows) ||
                      (M > kSwapGroupCols && M <= kSwapWideMaxRows))) {
        // Swapped paired kernel: all rows, padded to a multiple of 32, are accumulator columns; every pair of SMs
        // sweeps one vocabulary range.  Chosen where the other kernels pad the rows most or sweep W twice (see the kernel).
        g.swapped = 1; g.paired = 0;
        g.n_pad = ((M + 31) / 32) * 32;
        g.a_rows = (g.n_pad < kSwapGroupCols ? g.n_pad : kSwapGroupCols) / 2;     // H box of the first column group
        g.stages = swap_stages(g.n_pad);
        p.m_tiles = 1; p.mb = 1; p.waves = 1;
        p.units = (V + kPairUnit - 1) / kPairUnit;
        p.splits = n_sm / 2 < p.units ? n_sm / 2 : p.units;
    }
    g.m_tiles = p.m_tiles; g.units = p.units;
    g.mb = p.mb; g.splits = p.splits; g.waves = p.waves;
    g.mb_last = g.paired ? p.mb_last : 0; g.splits_last = g.paired ? p.splits_last : 0;
    int workers = g.mb * g.splits;
    if (g.mb_last * g.splits_last > workers) workers = g.mb_last * g.splits_last;
    g.ctas = workers * ((g.paired || g.swapped) ? 2 : 1);
    g.parts = (g.splits_last > g.splits ? g.splits_last : g.splits) * (g.swapped ? 2 : 1);
    return g;
}

size_t pvf_score_partials_bytes(const pvf_shape *shape, int n_sm)
{
    size_t worst = 0;
    const int max_tiles = (shape->max_rows + kTileM - 1) / kTileM;
    // Within one kernel choice and row-tile count the need grows with the rows, so it peaks at the upper end of
    // every 128-row step and of the swapped paired kernel's two windows.
    for (int t = 1; t <= max_tiles + 3; ++t) {
        int rows = t * kTileM;
        if (t == max_tiles + 1) rows = kSwapSmallMaxRows;
        if (t == max_tiles + 2) rows = kSwapRaggedMaxRows;
        if (t == max_tiles + 3) rows = kSwapWideMaxRows;
        if (rows > shape->max_rows) rows = shape->max_rows;
        if (rows <= 0) continue;
        const pvf_score_geometry g = pvf_score_geometry_for(rows, shape->vocab, shape->hidden, n_sm);
        const size_t need = (size_t)rows * g.parts * sizeof(float4);
        worst = need > worst ? need : worst;
    }
    return worst;
}

int pvf_score_partials(pvf_ctx *ctx, const void *hidden, int32_t M, int *parts, int clock_slot, void *stream)
{
    if (!ctx || !parts || M <= 0 || M > ctx->shape.max_rows || !hidden) return PVF_ERR_INVALID;
    if (((uintptr_t)hidden & 15) != 0) return PVF_ERR_ALIGN;
    const int V = ctx->shape.vocab, D = ctx->shape.hidden;
    const pvf_score_geometry g = pvf_score_geometry_for(M, V, D, ctx->n_sm);
    if ((size_t)M * g.parts * sizeof(float4) > ctx->partials_bytes) return PVF_ERR_WORKSPACE;
    *parts = g.parts;
    return launch_projection(g, hidden, M, V, D, ctx->tm_w, ctx->partials, &ctx->words->status, &ctx->words->wave_arrivals,
                             ctx->words->clock_acc[clock_slot ? 1 : 0], (cudaStream_t)stream, ctx->ev_start, ctx->ev_stop);
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

int pvf_score_clock(pvf_ctx *ctx, int32_t pass, double *ms, double *sm_mhz, int64_t *launches)
{
    if (!ctx || pass < 0 || pass > 1) return PVF_ERR_INVALID;
    unsigned long long acc[3] = {0, 0, 0};
    if (cudaDeviceSynchronize() != cudaSuccess ||
        cudaMemcpy(acc, ctx->words->clock_acc[pass], sizeof acc, cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemset(ctx->words->clock_acc[pass], 0, sizeof acc) != cudaSuccess)
        return PVF_ERR_CUDA;
    if (ms) *ms = acc[2] ? (double)acc[0] * 1e-6 / (double)acc[2] : 0.0;
    if (sm_mhz) *sm_mhz = acc[0] ? (double)acc[1] * 1e3 / (double)acc[0] : 0.0;
    if (launches) *launches = (int64_t)acc[2];
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
                             int32_t *waves, int32_t *kernel, int32_t *row_tiles, int32_t *tiles_per_wave,
                             int32_t *last_wave_tiles, int32_t *last_wave_splits)
{
    if (vocab <= 0 || hidden <= 0 || n_sm <= 0 || M <= 0) return PVF_ERR_INVALID;
    const pvf_score_geometry g = pvf_score_geometry_for(M, vocab, hidden, n_sm);
    if (ctas) *ctas = g.ctas;
    if (splits) *splits = g.splits;
    if (waves) *waves = g.waves;
    if (kernel) *kernel = g.streaming ? 0 : (g.swapped ? 3 : (g.paired ? 2 : 1));
    if (row_tiles) *row_tiles = g.m_tiles;
    if (tiles_per_wave) *tiles_per_wave = g.mb;
    if (last_wave_tiles) *last_wave_tiles = g.mb_last;
    if (last_wave_splits) *last_wave_splits = g.splits_last;
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
    int parts = 0;
    const int rc = pvf_score_partials(ctx, hidden, M, &parts, 0, stream);
    if (rc != PVF_OK) return rc;
    return launch_merge(ctx->partials, M, parts, ctx->shape.vocab, ctx->plan_bitmap, tok, conf, ent, in_plan, (cudaStream_t)stream);
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

// Every GPU that loads this library holds these 512.25 KiB until the process exits: a 256-byte header (the status
// word), then 128 x 256 partial softmax states.
static __device__ __align__(256) unsigned char pvf_static_scratch[kStaticHeaderBytes + kStaticPartialsBytes];

struct StaticDeviceState {
    bool ready;
    int n_sm;
    unsigned char *scratch;     // device address of pvf_static_scratch on that GPU
};
StaticDeviceState g_static_state[kStaticMaxDevices];
std::mutex g_static_mutex;          // guards the set-up below: first calls may come from several host threads

// Once per device, with that device current: resolve the array's device address (its name is only a
// host-side handle here) and raise the GEMM kernels' shared-memory limit.
int static_device_state(StaticDeviceState **out)
{
    int device = 0, cc = 0, n_sm = 0;
    if (cudaGetDevice(&device) != cudaSuccess) return PVF_ERR_CUDA;
    if (device < 0 || device >= kStaticMaxDevices) return PVF_ERR_UNSUPPORTED;
    StaticDeviceState *st = &g_static_state[device];
    std::lock_guard<std::mutex> lock(g_static_mutex);
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
    pvf_score_geometry g = pvf_score_geometry_for(M, vocab, hidden_size, st->n_sm);
    if ((size_t)M * g.parts * sizeof(float4) > kStaticPartialsBytes)       // the array is sized for one state per row and SM:
        g = pvf_score_geometry_for(M, vocab, hidden_size, st->n_sm, false); // above 221 rows the swapped kernel's two do not fit
    if ((size_t)M * g.parts * sizeof(float4) > kStaticPartialsBytes) return PVF_ERR_TOO_LARGE;

    CUtensorMap w_levels[kWBoxSizes];
    if ((rc = make_w_maps(w_levels, w_head, vocab, hidden_size)) != PVF_OK) return rc;

    cudaStream_t s = (cudaStream_t)stream;
    int32_t *status = (int32_t *)st->scratch;
    float4 *partials = (float4 *)(st->scratch + kStaticHeaderBytes);
    // The array keeps the previous call's contents.  The status word must start at zero; the partial
    // states need no clearing: the projection kernel writes every (row, range) entry the merge kernel reads.
    if (cudaMemsetAsync(status, 0, sizeof(int32_t), s) != cudaSuccess) return PVF_ERR_CUDA;
    if ((rc = launch_projection(g, hidden, M, vocab, hidden_size, w_levels, partials, status, nullptr, nullptr, s, nullptr, nullptr)) != PVF_OK) return rc;
    return launch_merge(partials, M, g.parts, vocab, plan_bitmap, tok, conf, ent, in_plan, s);
}

int pvf_score_static_status(int32_t *status)
{
    if (!status) return PVF_ERR_INVALID;
    StaticDeviceState *st = nullptr;
    int rc = static_device_state(&st);
    if (rc != PVF_OK) return rc;
    if (cudaDeviceSynchronize() != cudaSuccess ||       // every stream of the device, non-blocking ones included
        cudaMemcpy(status, st->scratch, sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess)
        return PVF_ERR_CUDA;
    return PVF_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------- self-test of the bounded wait
// Not part of the C interface (not declared in pvf.h): exercises, in its harmless form, the path every kernel takes
// when a wait runs out.  One small block initialises an mbarrier that nothing ever arrives on and waits on it with
// the projection kernels' own bounded wait and a caller-given limit; no copy, no MMA and no tensor memory is in
// flight.  The wait gives up, the status word receives PVF_ERR_TIMEOUT, the kernel returns and the context stays usable.
namespace {

__global__ void __launch_bounds__(64)
pvf_wait_expiry_kernel(int32_t *status, unsigned long long limit_ns, int32_t *gave_up)
{
    __shared__ SharedControl ctl;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&ctl.full[0]), 1);
        ctl.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bool ok = true;
    if (threadIdx.x == 0) ok = mbar_wait_slow(smem_u32(&ctl.full[0]), 0u, &ctl, status, limit_ns);     // runs out
    __syncthreads();
    if (threadIdx.x == 32) ok = mbar_wait_slow(smem_u32(&ctl.full[0]), 0u, &ctl, status, limit_ns);    // sees the abort flag
    if ((threadIdx.x == 0 || threadIdx.x == 32) && !ok) atomicAdd(gave_up, 1);
}

}  // namespace

extern "C" int pvf_selftest_wait_expiry(pvf_ctx *ctx, uint64_t limit_ns, int32_t *gave_up, void *stream)
{
    if (!ctx || !gave_up || limit_ns == 0 || limit_ns > 100000000ull) return PVF_ERR_INVALID;   // at most 0.1 s
    pvf_wait_expiry_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(&ctx->words->status, (unsigned long long)limit_ns, gave_up);
    return cudaGetLastError() == cudaSuccess ? PVF_OK : PVF_ERR_CUDA;
}
