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
    uint32_t pad[61];
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
    int parts;       // partial states per row handed to the merge kernel (splits, or 2 * splits when swapped)
};
// allow_swapped = false leaves the swapped paired kernel (which writes twice as many partial states per row) out.
pvf_score_geometry pvf_score_geometry_for(int M, int V, int D, int n_sm, bool allow_swapped = true);
size_t pvf_score_partials_bytes(const pvf_shape *shape, int n_sm);
int pvf_score_init(pvf_ctx *ctx);   // tensor maps of W, kernel attributes

// Programmatic dependent launch.  Every kernel of the library is launched with pvf_launch and runs
//     <set-up that touches no global memory>; pvf_launch_dependents(); pvf_grid_dependency_wait();
// before its first global access, on every thread.  The wait returns once the kernel before it in
// the stream has completed and its writes are visible, so stream order is kept; what overlaps is the
// launch latency and set-up of a kernel with the tail of its predecessor.
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
