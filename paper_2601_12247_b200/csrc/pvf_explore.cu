// pvf_explore_commit: the appendix's exploration variants ("Planning tokens beyond high-confidence
// decoding").  After the high-confidence commits, every sequence commits exactly one more token whose
// confidence lies in the closed bin [tau_plan_lo, tau_plan_hi]: drawn uniformly from all eligible rows
// (Random), or from the eligible rows whose top-1 token is in P^plan, falling back to all eligible rows
// when there is none (Planning).  The uniform number of each sequence is an input.
// One thread block per sequence; rows of a sequence ascend in position.
#include "pvf_internal.h"

namespace {

constexpr int kThreads = kPvfBlockThreads;
constexpr int kWarps = kPvfBlockWarps;

__global__ void __launch_bounds__(kThreads)
pvf_explore_kernel(const int32_t *__restrict__ seg_off, const int32_t *__restrict__ row_pos,
                   const uint8_t *__restrict__ active, const int32_t *__restrict__ tok,
                   const float *__restrict__ conf, const uint8_t *__restrict__ in_plan,
                   const float *__restrict__ u, float tau_lo, float tau_hi, int planning,
                   uint8_t *__restrict__ commit, int32_t *__restrict__ explore_row, int32_t *__restrict__ y, int L)
{
    __shared__ int s_int[kWarps];
    pvf_launch_dependents();
    pvf_grid_dependency_wait();
    const int b = blockIdx.x;
    const int r0 = seg_off[b], r1 = seg_off[b + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // sizes of the bin and of its planning subset
    int n_all = 0, n_plan = 0;
    for (int m = r0 + threadIdx.x; m < r1; m += kThreads) {
        const float p = conf[m];
        const bool el = (active ? active[m] != 0 : true) && !commit[m] && p >= tau_lo && p <= tau_hi;
        n_all += el ? 1 : 0;
        n_plan += (el && planning && in_plan[m]) ? 1 : 0;
    }
    n_all = pvf_block_sum(n_all, s_int);
    n_plan = pvf_block_sum(n_plan, s_int);
    const bool use_plan = planning && n_plan > 0;
    const int n = use_plan ? n_plan : n_all;
    if (n == 0) {
        if (threadIdx.x == 0) explore_row[b] = -1;
        return;
    }
    int target = (int)(u[b] * (float)n);                       // floor(u * n), fp32 product
    target = target < 0 ? 0 : (target > n - 1 ? n - 1 : target);
    // the target-th row of the chosen set, in position order
    int seen = 0;
    for (int c0 = r0; c0 < r1; c0 += kThreads) {               // block-uniform trip count
        const int m = c0 + threadIdx.x;
        bool in_set = false;
        if (m < r1) {
            const float p = conf[m];
            in_set = (active ? active[m] != 0 : true) && !commit[m] && p >= tau_lo && p <= tau_hi &&
                     (!use_plan || in_plan[m]);
        }
        const unsigned ballot = __ballot_sync(0xffffffffu, in_set);
        __syncthreads();
        if (lane == 0) s_int[warp] = __popc(ballot);
        __syncthreads();
        int before = 0, all = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const int c = s_int[w];
            if (w < warp) before += c;
            all += c;
        }
        const int rank = seen + before + __popc(ballot & ((1u << lane) - 1u));
        // every row's eligibility was read above; only the chosen row is written, after the barrier
        __syncthreads();
        if (in_set && rank == target) {
            commit[m] = 1;
            explore_row[b] = m;
            if (y) y[(size_t)b * L + row_pos[m]] = tok[m];
        }
        seen += all;
        if (seen > target) break;                              // block-uniform
    }
}

}  // namespace

extern "C" int pvf_explore_commit(pvf_ctx *ctx, const pvf_params *params, int32_t mode, int32_t M, int32_t n_seq,
                                  const int32_t *seg_off, const int32_t *row_pos, const uint8_t *active,
                                  const int32_t *tok, const float *conf, const uint8_t *in_plan,
                                  const float *u, uint8_t *commit, int32_t *explore_row, int32_t *y, int32_t L,
                                  void *stream)
{
    if (!ctx || !params || M < 0 || n_seq < 0 || M > ctx->shape.max_rows || n_seq > ctx->shape.max_seqs ||
        (mode != PVF_EXPLORE_RANDOM && mode != PVF_EXPLORE_PLANNING))
        return PVF_ERR_INVALID;
    if (n_seq == 0) return M == 0 ? PVF_OK : PVF_ERR_INVALID;
    if (!seg_off || !conf || !u || !commit || !explore_row || (mode == PVF_EXPLORE_PLANNING && !in_plan) ||
        (y && (!row_pos || !tok || L <= 0)))
        return PVF_ERR_INVALID;
    const cudaError_t e = pvf_launch(pvf_explore_kernel, dim3(n_seq), dim3(kThreads), 0, (cudaStream_t)stream,
                                     seg_off, row_pos, active, tok, conf, in_plan, u, params->tau_plan_lo,
                                     params->tau_plan_hi, mode == PVF_EXPLORE_PLANNING ? 1 : 0, commit, explore_row, y, L);
    return e == cudaSuccess ? PVF_OK : PVF_ERR_CUDA;
}
