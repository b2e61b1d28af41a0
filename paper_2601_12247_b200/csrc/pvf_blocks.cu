// pvf_working_set: which canvas positions the next decoding step scores.
//
// Semi-autoregressive block order (Appendix A.1): the active block k_t of a sequence is its first block
// that still holds a mask.  Early cross-block revelation (Appendix, Eq. 4): when at most N_s masks are
// left in the active block, the whole next block joins the working index set B_t.  The scored rows are
// the masked positions of B_t in ascending order, sequence after sequence.
//
// Two small kernels, one thread block per sequence: the first counts each sequence's rows and the last
// block to finish turns the counts into offsets; the second writes the rows.  Both recompute the
// sequence's range from the canvas, so nothing but the offsets passes between them.
#include "pvf_internal.h"

namespace {

constexpr int kThreads = kPvfBlockThreads;
constexpr int kWarps = kPvfBlockWarps;

// Position range [lo, hi) that holds B_t of one sequence (empty when the sequence is finished), and
// whether the next block was revealed.  Every thread of the block returns the same values.
__device__ __forceinline__ void working_range(const int32_t *__restrict__ yb, int L, int S, int n_sparse, int mask_id,
                                              int *scratch, int *lo, int *hi, int *expanded)
{
    int first = L;
    for (int i = threadIdx.x; i < L; i += kThreads)
        if (yb[i] == mask_id) { first = i; break; }            // a thread's positions ascend
    first = pvf_block_min(first, scratch);
    if (first >= L) { *lo = 0; *hi = 0; *expanded = 0; return; }
    const int k = first / S;                                   // k_t, 0-based
    const int b0 = k * S, b1 = min(b0 + S, L);
    int n_active = 0;                                          // |M_t^active|
    for (int i = b0 + threadIdx.x; i < b1; i += kThreads) n_active += yb[i] == mask_id ? 1 : 0;
    n_active = pvf_block_sum(n_active, scratch);
    const int reveal = (n_active <= n_sparse && b1 < L) ? 1 : 0;
    *lo = b0;
    *hi = reveal ? min(b1 + S, L) : b1;                        // B_t = M_active, or M_active + I_{k_t+1}
    *expanded = reveal;
}

__global__ void __launch_bounds__(kThreads)
pvf_working_count_kernel(const int32_t *__restrict__ y, int n_seq, int L, int S, int n_sparse, int mask_id,
                         int32_t *__restrict__ seg_off, uint8_t *__restrict__ expanded, unsigned *ticket)
{
    __shared__ int s_int[kWarps];
    __shared__ int s_last;
    pvf_launch_dependents();
    pvf_grid_dependency_wait();
    const int b = blockIdx.x;
    const int32_t *yb = y + (size_t)b * L;
    int lo, hi, ex;
    working_range(yb, L, S, n_sparse, mask_id, s_int, &lo, &hi, &ex);
    int n = 0;
    for (int i = lo + threadIdx.x; i < hi; i += kThreads) n += yb[i] == mask_id ? 1 : 0;
    n = pvf_block_sum(n, s_int);
    if (threadIdx.x == 0) {
        seg_off[b + 1] = n;                                    // a count for now
        if (expanded) expanded[b] = (uint8_t)ex;
    }
    // The last block to finish turns the counts into offsets (in place).
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(ticket, 1u) == (unsigned)(n_seq - 1)) ? 1 : 0;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (threadIdx.x < 32) {
        volatile int32_t *vs = seg_off;
        int running = 0;
        for (int c0 = 0; c0 < n_seq; c0 += 32) {
            const int s = c0 + threadIdx.x;
            const int rows = s < n_seq ? vs[s + 1] : 0;
            int incl = rows;
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, incl, o);
                if ((int)threadIdx.x >= o) incl += t;
            }
            __syncwarp();                                      // every count of this chunk is read before any is overwritten
            if (s < n_seq) vs[s + 1] = running + incl;
            running += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (threadIdx.x == 0) {
            vs[0] = 0;
            *ticket = 0;
        }
    }
}

__global__ void __launch_bounds__(kThreads)
pvf_working_fill_kernel(const int32_t *__restrict__ y, int L, int S, int n_sparse, int mask_id,
                        const int32_t *__restrict__ seg_off, int32_t *__restrict__ row_pos,
                        int32_t *__restrict__ row_seq, uint8_t *__restrict__ active)
{
    __shared__ int s_int[kWarps];
    pvf_launch_dependents();
    pvf_grid_dependency_wait();
    const int b = blockIdx.x;
    const int32_t *yb = y + (size_t)b * L;
    int lo, hi, ex;
    working_range(yb, L, S, n_sparse, mask_id, s_int, &lo, &hi, &ex);
    int out = seg_off[b];
    for (int c0 = lo; c0 < hi; c0 += kThreads) {               // block-uniform trip count
        const int i = c0 + threadIdx.x;
        const bool masked = i < hi && yb[i] == mask_id;
        int all;
        const int rank = pvf_block_rank(masked, s_int, &all);
        if (masked) {
            const int m = out + rank;
            row_pos[m] = i;
            if (row_seq) row_seq[m] = b;
            if (active) active[m] = 1;
        }
        out += all;
    }
}

}  // namespace

extern "C" int pvf_working_set(pvf_ctx *ctx, const int32_t *y, int32_t n_seq, int32_t L, int32_t block,
                               int32_t n_sparse, int32_t mask_id, int32_t *seg_off, int32_t *row_pos,
                               int32_t *row_seq, uint8_t *active, uint8_t *expanded, int32_t rows_capacity,
                               void *stream)
{
    if (!ctx || n_seq < 0 || n_seq > ctx->shape.max_seqs || L <= 0 || block <= 0 || n_sparse < 0 || rows_capacity < 0)
        return PVF_ERR_INVALID;
    if (n_seq == 0) return PVF_OK;
    if (!y || !seg_off || !row_pos) return PVF_ERR_INVALID;
    const long long per_seq = 2LL * block < L ? 2LL * block : L;          // |B_t| never exceeds two blocks
    if ((long long)rows_capacity < per_seq * n_seq) return PVF_ERR_INVALID;
    cudaStream_t s = (cudaStream_t)stream;
    if (pvf_launch(pvf_working_count_kernel, dim3(n_seq), dim3(kThreads), 0, s, y, n_seq, L, block, n_sparse, mask_id,
                   seg_off, expanded, &ctx->words->working_ticket) != cudaSuccess)
        return PVF_ERR_CUDA;
    if (pvf_launch(pvf_working_fill_kernel, dim3(n_seq), dim3(kThreads), 0, s, y, L, block, n_sparse, mask_id,
                   (const int32_t *)seg_off, row_pos, row_seq, active) != cudaSuccess)
        return PVF_ERR_CUDA;
    return PVF_OK;
}
