// Internal declarations shared by the translation units of libpvf (not part of the C interface).
#ifndef PVF_INTERNAL_H_
#define PVF_INTERNAL_H_

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "pvf.h"

#define PVF_MAX_BUDGET_LIMIT 64
#define PVF_W_BOX_SIZES 16

// Device scalars at the head of the workspace.
struct pvf_device_words {
    int32_t  status;        // PVF_OK or PVF_ERR_TIMEOUT, written by kernels
    uint32_t select_ticket; // blocks of pvf_select_drafts that have finished; reset by the last one
    uint32_t working_ticket; // the same for pvf_working_set
    uint32_t wave_arrivals; // paired projection kernel: blocks that have reached a wave boundary (all waves of a launch)
    uint32_t wave_done;     //    blocks that are past their last wave boundary; the last one clears both
    uint32_t pad0[3];
    // SM clock of the projection launches, measured on the device (pvf_score_clock): per slot (0: pvf_score and the
    // draft pass, 1: the verification pass) the sums over launches of block 0's wall time (ns, %globaltimer) and of its
    // SM cycles (clock64), and the number of launches.
    unsigned long long clock_acc[2][3];
    uint32_t pad[44];
};

struct pvf_ctx {
    pvf_shape shape;
    int device;
    int n_sm;
    const void *w_head;
    uint8_t *workspace;
    size_t workspace_bytes;
    pvf_device_words *words;
    uint32_t *plan_bitmap;  // ceil(V/32) words, bit v set iff v in P^plan
    uint32_t *seq_tickets;  // one arrival counter per sequence (step kernels; zero between launches)
    size_t seq_tickets_bytes;
    float4 *partials;       // [rows][splits] per-range softmax states of pvf_score
    size_t partials_bytes;
    CUtensorMap tm_w[PVF_W_BOX_SIZES];   // W as [V][D], boxes of 16 * (i + 1) rows x 64 columns, 128-byte swizzle
    cudaEvent_t ev_start, ev_stop;   // optional timing hook around the GEMM kernel
    uint8_t *staging;                // optional device staging of the host-buffer entry points
    size_t staging_bytes;
    uint8_t *bounce;                 // optional pinned host mirror of the staging's small arrays (one copy per direction)
    int32_t host_rows, host_seqs, host_budget;   // shape of the draft half the staging currently holds
    bool host_active;
};

// Work split of pvf_score for M rows on n_sm SMs (see pvf_score.cu).
struct pvf_score_geometry {
    int m_tiles;     // ceil(M / 128) row tiles
    int units;       // ceil(V / 16): vocabulary granules
    int mb;          // row tiles processed concurrently (one wave)
    int splits;      // vocabulary ranges per row tile = partial states per row
    int waves;       // ceil(m_tiles / mb)
    int ctas;        // mb * splits
    int a_rows;      // rows of the hidden-state TMA box
    int streaming;   // 1: at most 32 rows, handled by the swapped-operand streaming kernel
    int paired;      // 1: more than 128 rows, handled by the paired (cta_group::2) kernel; then m_tiles counts
                     //    256-row tiles, units granules of 32 entries, mb / splits pairs of blocks
    int swapped;     // 1: handled by the swapped paired kernel; m_tiles counts row tiles of n_pad rows, units
                     //    granules of 32 entries, mb / splits pairs of blocks
    int n_pad;       // swapped: rows per row tile (multiple of 32, at most 256)
    int stages;      // swapped: pipeline stages that fit the shared-memory ring
    int parts;       // partial states per row handed to the merge kernel (splits, or 2 * splits when swapped; the
                     //    larger of splits and splits_last when the last wave is split differently)
    int mb_last;     // paired: row tiles of the last wave when it is a partial one (else 0), each swept by
    int splits_last; //    splits_last pairs, so that the pairs are all busy in that wave too
};
// allow_swapped = false leaves the swapped paired kernel (which writes twice as many partial states per row) out.
pvf_score_geometry pvf_score_geometry_for(int M, int V, int D, int n_sm, bool allow_swapped = true);
size_t pvf_score_partials_bytes(const pvf_shape *shape, int n_sm);
int pvf_score_init(pvf_ctx *ctx);   // tensor maps of W, kernel attributes
// The projection half of pvf_score alone: launches the kernel that leaves `*parts` partial softmax states per row in
// ctx->partials (row stride *parts); the caller's next kernel on the stream merges them (pvf_merge_rows).
int pvf_score_partials(pvf_ctx *ctx, const void *hidden, int32_t M, int *parts, int clock_slot, void *stream);

// Programmatic dependent launch.  Every kernel of the library is launched with pvf_launch and runs
//     <set-up>; pvf_launch_dependents(); pvf_grid_dependency_wait();
// before it reads anything an earlier kernel may have written, or writes anything, on every thread.  The wait returns
// once the kernel before it in the stream has completed and its writes are visible, so stream order is kept; what
// overlaps is the launch latency and set-up of a kernel with the tail of its predecessor.  Two departures, both in
// the projection kernels: (1) their set-up includes reads of W -- the LM-head weights are a constant of the context,
// which no kernel in the stream writes -- so in launches of one wave the first tiles of W are on their way, and
// further ones asked into L2, before the wait; (2) launches of several waves let their dependents in at their end
// only, since all those could do earlier is wait beside blocks that run for milliseconds.
#ifdef __CUDACC__
__device__ __forceinline__ void pvf_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pvf_grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline cudaError_t pvf_launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                     Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// The same for a kernel whose blocks form clusters of two along x (grid.x even).
template <typename... KArgs, typename... Args>
static inline cudaError_t pvf_launch_cluster2(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                              cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// Partial softmax state of a row over a vocabulary range, as the projection kernels leave it (one float4):
//   x = the range's maximum logit m        y = sum of e^{x_v - m} over the range EXCEPT the entry holding the maximum
//   z = sum of (x_v - m) e^{x_v - m}       w = bits of the lowest token id attaining m (kPvfNoArg: empty state)
// Keeping the maximum's own term (1.0) out of y keeps the small terms of a peaked row above the rounding unit.
#ifdef __CUDACC__
constexpr int kPvfNoArg = 0x7fffffff;

__device__ __forceinline__ float pvf_fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// a <- a merged with b (two states over disjoint vocabulary sets).  The larger max stays outside the sum; the
// other state's max joins it as an ordinary term.  Equal maxima: the lower token id wins.  Branch-free, so that
// independent merges interleave: the loser's distance below the winner is clamped (an empty state sits at -inf and
// comes in with weight e^-inf = 0; two empty states give an empty state).
__device__ __forceinline__ void pvf_state_merge(float4 &a, const float4 b)
{
    constexpr float kLog2e = 1.4426950408889634f;
    const int ia = __float_as_int(a.w), ib = __float_as_int(b.w);
    const bool a_wins = a.x > b.x || (a.x == b.x && ia <= ib);
    const float wm = a_wins ? a.x : b.x, wy = a_wins ? a.y : b.y, wz = a_wins ? a.z : b.z, ww = a_wins ? a.w : b.w;
    const float lm = a_wins ? b.x : a.x, ly = a_wins ? b.y : a.y, lz = a_wins ? b.z : a.z;
    const float d = fmaxf(lm - wm, -1.0e30f);           // <= 0; fmaxf also turns (-inf) - (-inf) into the clamp
    const float c = pvf_fast_exp2(d * kLog2e);
    const float total = ly + 1.f;
    a.x = wm;
    a.y = fmaf(total, c, wy);
    a.z = fmaf(fmaf(d, total, lz), c, wz);
    a.w = ww;
}

// Final merge of rows [row_begin, row_end) by the warps of a block, or of a grid of such blocks (all threads call it;
// `warp` / `n_warps` = this warp's index among the warps that share the row range).  A row's `parts` partial states
// are folded by g = min(32, parts rounded up to a power of two) neighbouring lanes -- lane l takes states l, l + g,
// ... five at a time, folds them pairwise, then the lanes fold pairwise: an order fixed by `parts` alone, so results
// are identical from run to run -- and the row's first lane writes token, confidence = 1 / (1 + y), entropy = ln(1 + y) - z / (1 + y) and
// planning-vocabulary membership (Section 3: y^, p, H; Section 4.1: y^ in P^plan).  ent and in_plan may be NULL.
// A warp works on kMergeRowsInFlight groups of 32 / g rows at once and fetches up to kMergeStatesInFlight states per
// lane and row before it merges any (the merge is a chain of memory round trips otherwise).  No shared memory and
// few registers: the kernels that run this are launched while the projection kernel, which fills an SM's shared
// memory and two thirds of its registers, is still running, and their blocks must fit beside its blocks to be
// resident (and past their set-up) by the time it ends.
constexpr int kMergeRowsInFlight = 2;
constexpr int kMergeStatesInFlight = 5;
__device__ __forceinline__ void pvf_merge_rows(const float4 *__restrict__ partials, int parts, int vocab,
                                               const uint32_t *__restrict__ plan_bitmap, int row_begin, int row_end,
                                               int warp, int n_warps, int32_t *tok, float *conf, float *ent, uint8_t *in_plan)
{
    int g = 1;
    while (g < parts && g < 32) g <<= 1;
    const int lane = threadIdx.x & 31;
    const int gl = lane & (g - 1), sub = lane / g;              // lane within its row, row within the warp's pass
    const int rows_per_pass = 32 / g;
    const int rows_per_turn = rows_per_pass * kMergeRowsInFlight;
    const float4 none = make_float4(-INFINITY, 0.f, 0.f, __int_as_float(kPvfNoArg));
#pragma unroll 1
    for (int row0 = row_begin + warp * rows_per_turn; row0 < row_end; row0 += n_warps * rows_per_turn) {
        float4 acc[kMergeRowsInFlight];
#pragma unroll
        for (int r = 0; r < kMergeRowsInFlight; ++r) acc[r] = none;
#pragma unroll 1
        for (int i0 = gl; i0 < parts; i0 += g * kMergeStatesInFlight) {
            float4 v[kMergeRowsInFlight][kMergeStatesInFlight];
#pragma unroll
            for (int r = 0; r < kMergeRowsInFlight; ++r) {
                const int row = row0 + r * rows_per_pass + sub;
#pragma unroll
                for (int k = 0; k < kMergeStatesInFlight; ++k)
                    v[r][k] = (row < row_end && i0 + k * g < parts) ? __ldg(partials + (size_t)row * parts + i0 + k * g) : none;
            }
            // The states a lane holds are folded pairwise -- (0 1)(2 3), then the pairs, then the fifth -- and the rows
            // side by side: a merge is a chain of some sixty dependent instructions, and with two warps per
            // scheduler nothing else hides their latency.
            static_assert(kMergeStatesInFlight == 5, "the fold below is written out for five states");
#pragma unroll
            for (int r = 0; r < kMergeRowsInFlight; ++r) {
                pvf_state_merge(v[r][0], v[r][1]);
                pvf_state_merge(v[r][2], v[r][3]);
            }
#pragma unroll
            for (int r = 0; r < kMergeRowsInFlight; ++r) pvf_state_merge(v[r][0], v[r][2]);
#pragma unroll
            for (int r = 0; r < kMergeRowsInFlight; ++r) pvf_state_merge(v[r][0], v[r][4]);
#pragma unroll
            for (int r = 0; r < kMergeRowsInFlight; ++r) pvf_state_merge(acc[r], v[r][0]);
        }
#pragma unroll 1
        for (int o = 1; o < g; o <<= 1) {                       // lane l absorbs lane l + o of its row
            float4 other[kMergeRowsInFlight];
#pragma unroll
            for (int r = 0; r < kMergeRowsInFlight; ++r) {
                other[r].x = __shfl_down_sync(0xffffffffu, acc[r].x, o, g);
                other[r].y = __shfl_down_sync(0xffffffffu, acc[r].y, o, g);
                other[r].z = __shfl_down_sync(0xffffffffu, acc[r].z, o, g);
                other[r].w = __shfl_down_sync(0xffffffffu, acc[r].w, o, g);
            }
            if ((gl & (2 * o - 1)) == 0) {
#pragma unroll
                for (int r = 0; r < kMergeRowsInFlight; ++r) pvf_state_merge(acc[r], other[r]);
            }
        }
#pragma unroll
        for (int r = 0; r < kMergeRowsInFlight; ++r) {
            const int row = row0 + r * rows_per_pass + sub;
            if (gl == 0 && row < row_end) {
                // A row of non-finite logits never sets a maximum: its outputs are unspecified, but the token stays a
                // valid id and the bitmap lookup in bounds.
                int arg = __float_as_int(acc[r].w);
                if ((unsigned)arg >= (unsigned)vocab) arg = 0;
                const float norm = 1.f + acc[r].y;              // the maximum's own term is the 1
                const float inv = 1.f / norm;
                tok[row] = arg;
                conf[row] = inv;
                if (ent) ent[row] = __logf(norm) - acc[r].z * inv;
                if (in_plan) in_plan[row] = (uint8_t)((plan_bitmap[arg >> 5] >> (arg & 31)) & 1u);
            }
        }
    }
}
#endif

// Block-wide helpers of the one-block-per-sequence kernels (256 threads; `scratch` holds one entry per warp).
#ifdef __CUDACC__
constexpr int kPvfBlockThreads = 256;
constexpr int kPvfBlockWarps = kPvfBlockThreads / 32;

__device__ __forceinline__ int pvf_block_sum(int v, int *scratch)
{
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();                               // scratch may still be read from a previous call
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    int t = 0;
#pragma unroll
    for (int w = 0; w < kPvfBlockWarps; ++w) t += scratch[w];
    return t;
}

__device__ __forceinline__ int pvf_block_min(int v, int *scratch)
{
    for (int o = 16; o > 0; o >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    int t = scratch[0];
#pragma unroll
    for (int w = 1; w < kPvfBlockWarps; ++w) t = min(t, scratch[w]);
    return t;
}

// Exclusive prefix of a 0/1 flag over the block, in thread order; *total gets the block's count.
__device__ __forceinline__ int pvf_block_rank(bool flag, int *scratch, int *total)
{
    const unsigned ballot = __ballot_sync(0xffffffffu, flag);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) scratch[warp] = __popc(ballot);
    __syncthreads();
    int before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < kPvfBlockWarps; ++w) {
        const int c = scratch[w];
        if (w < warp) before += c;
        all += c;
    }
    *total = all;
    return before + __popc(ballot & ((1u << lane) - 1u));
}
#endif

static inline size_t pvf_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

#endif
