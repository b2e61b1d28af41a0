// Decision kernels of one PVF step: base commit, draft proposal, acceptance check.
// One thread block per sequence; rows of a sequence are contiguous and sorted by position.
// All reductions are warp shuffles plus one shared-memory hop; every result is deterministic.
#include "pvf_internal.h"

namespace {

constexpr int kThreads = kPvfBlockThreads;
constexpr int kWarps = kPvfBlockWarps;

__device__ __forceinline__ unsigned long long block_max(unsigned long long v, unsigned long long *scratch)
{
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long u = __shfl_xor_sync(0xffffffffu, v, o);
        v = u > v ? u : v;
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    unsigned long long t = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) t = scratch[w] > t ? scratch[w] : t;
    return t;
}

// Sort key of a candidate: larger confidence first, then the lower position (rows of a sequence
// ascend in position).  Confidences are non-negative floats, so their bit patterns order like the
// values.  Never 0 for a real candidate.
__device__ __forceinline__ unsigned long long cand_key(float conf, int rel_row)
{
    return ((unsigned long long)__float_as_uint(conf) << 32) | (unsigned long long)(0xffffffffu - (unsigned)rel_row);
}

// ------------------------------------------------------------------------------------ commit
__global__ void __launch_bounds__(kThreads)
pvf_commit_kernel(const int32_t *__restrict__ seg_off, const int32_t *__restrict__ row_pos,
                  const uint8_t *__restrict__ active, const int32_t *__restrict__ tok,
                  const float *__restrict__ conf, float tau_high, int force_progress,
                  uint8_t *__restrict__ commit, int32_t *__restrict__ n_commit,
                  int32_t *__restrict__ y, int L)
{
    __shared__ int s_int[kWarps];
    __shared__ unsigned long long s_key[kWarps];
    pvf_launch_dependents();
    pvf_grid_dependency_wait();
    const int b = blockIdx.x;
    const int r0 = seg_off[b], r1 = seg_off[b + 1];
    int count = 0;
    unsigned long long best = 0;
    for (int m = r0 + threadIdx.x; m < r1; m += kThreads) {
        const bool act = active ? active[m] != 0 : true;
        const float p = conf[m];
        const bool c = act && p >= tau_high;                       // S_base: p >= tau_high
        commit[m] = c ? 1 : 0;
        if (c) {
            ++count;
            if (y) y[(size_t)b * L + row_pos[m]] = tok[m];         // z_base
        }
        if (act) {
            const unsigned long long k = cand_key(p, m - r0);
            best = k > best ? k : best;
        }
    }
    int total = pvf_block_sum(count, s_int);
    if (force_progress && total == 0) {
        best = block_max(best, s_key);
        if (best != 0) {
            if (threadIdx.x == 0) {
                const int m = r0 + (int)(0xffffffffu - (unsigned)(best & 0xffffffffull));
                commit[m] = 1;
                if (y) y[(size_t)b * L + row_pos[m]] = tok[m];
            }
            total = 1;
        }
    }
    if (threadIdx.x == 0 && n_commit) n_commit[b] = total;
}

// ------------------------------------------------------------------------------------ select
__global__ void __launch_bounds__(kThreads)
pvf_select_kernel(int n_seq, const int32_t *__restrict__ seg_off, const uint8_t *__restrict__ active,
                  const float *__restrict__ conf, const uint8_t *__restrict__ in_plan,
                  const uint8_t *__restrict__ commit, float tau_lo, float tau_hi, float tau_ar, int K,
                  int any_token, int ar_fallback, int32_t *__restrict__ draft_rows, int32_t *__restrict__ n_drafts,
                  uint8_t *__restrict__ route, int32_t *__restrict__ rem_rows,
                  int32_t *__restrict__ rem_off, int32_t *__restrict__ v_off, unsigned *ticket)
{
    __shared__ int s_int[kWarps];
    __shared__ unsigned long long s_key[kWarps];
    __shared__ int s_last;
    pvf_launch_dependents();
    pvf_grid_dependency_wait();
    const int b = blockIdx.x;
    const int r0 = seg_off[b], r1 = seg_off[b + 1];

    // R_b starts after the remaining rows of all earlier sequences: count them directly.
    int before = 0;
    for (int m = threadIdx.x; m < r0; m += kThreads)
        before += ((active ? active[m] != 0 : true) && !commit[m]) ? 1 : 0;
    const int rem_base = pvf_block_sum(before, s_int);

    // R_b in position order, and the number of planning candidates.
    int n_rem = 0, n_plan = 0;
    for (int c0 = r0; c0 < r1; c0 += kThreads) {
        const int m = c0 + threadIdx.x;
        bool rem = false, plan = false;
        if (m < r1) {
            rem = (active ? active[m] != 0 : true) && !commit[m];
            const float p = conf[m];
            plan = rem && (any_token || in_plan[m]) && p >= tau_lo && p < tau_hi;  // P_t^plan
        }
        int chunk_total;
        const int rank = pvf_block_rank(rem, s_int, &chunk_total);
        if (rem) rem_rows[rem_base + n_rem + rank] = m;
        n_rem += chunk_total;
        n_plan += plan ? 1 : 0;
    }
    n_plan = pvf_block_sum(n_plan, s_int);

    int kt = 0, rt = 0;
    if (K > 0 && n_plan > 0) {
        // TopK by confidence: round j picks the largest key below the previous winner's.
        kt = n_plan < K ? n_plan : K;
        rt = 1;
        unsigned long long last = ~0ull;
        for (int j = 0; j < kt; ++j) {
            unsigned long long best = 0;
            for (int m = r0 + threadIdx.x; m < r1; m += kThreads) {
                const float p = conf[m];
                const bool plan = (active ? active[m] != 0 : true) && !commit[m] && (any_token || in_plan[m]) &&
                                  p >= tau_lo && p < tau_hi;
                if (plan) {
                    const unsigned long long k = cand_key(p, m - r0);
                    if (k < last && k > best) best = k;
                }
            }
            last = block_max(best, s_key);
            if (threadIdx.x == 0)
                draft_rows[(size_t)b * K + j] = r0 + (int)(0xffffffffu - (unsigned)(last & 0xffffffffull));
        }
    } else if (K > 0 && ar_fallback) {
        // AR fallback: leftmost rows of R_b with p >= tau_AR^l, at most K of them.
        for (int c0 = r0; c0 < r1 && kt < K; c0 += kThreads) {
            const int m = c0 + threadIdx.x;
            const bool ok = m < r1 && (active ? active[m] != 0 : true) && !commit[m] && conf[m] >= tau_ar;
            int chunk_total;
            const int rank = pvf_block_rank(ok, s_int, &chunk_total);
            if (ok && kt + rank < K) draft_rows[(size_t)b * K + kt + rank] = m;
            kt += chunk_total;
        }
        kt = kt < K ? kt : K;
        rt = kt > 0 ? 2 : 0;
    }
    for (int j = kt + threadIdx.x; j < K; j += kThreads) draft_rows[(size_t)b * K + j] = -1;
    if (threadIdx.x == 0) {
        n_drafts[b] = kt;
        route[b] = (uint8_t)rt;
        rem_off[b] = rem_base;
        if (b == n_seq - 1) rem_off[n_seq] = rem_base + n_rem;
    }

    // The last block to finish turns the per-sequence counts into verification-pass offsets.
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = (atomicAdd(ticket, 1u) == (unsigned)(n_seq - 1)) ? 1 : 0;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (threadIdx.x < 32) {
        const volatile int32_t *vd = n_drafts;
        const volatile int32_t *vr = rem_off;
        int running = 0;
        for (int c0 = 0; c0 < n_seq; c0 += 32) {
            const int s = c0 + threadIdx.x;
            int rows = 0;
            if (s < n_seq) {
                const int d = vd[s];
                rows = d > 0 ? (1 + d) * (vr[s + 1] - vr[s]) : 0;
            }
            int incl = rows;
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, incl, o);
                if ((int)threadIdx.x >= o) incl += t;
            }
            if (s < n_seq) v_off[s] = running + incl - rows;
            running += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (threadIdx.x == 0) {
            v_off[n_seq] = running;
            *ticket = 0;
        }
    }
}

// ------------------------------------------------------------------------------------ verify
__global__ void __launch_bounds__(kThreads)
pvf_verify_kernel(const int32_t *__restrict__ seg_off, const int32_t *__restrict__ row_pos,
                  const int32_t *__restrict__ rem_rows, const int32_t *__restrict__ rem_off,
                  const int32_t *__restrict__ v_off, const int32_t *__restrict__ draft_rows,
                  const int32_t *__restrict__ n_drafts, const uint8_t *__restrict__ route,
                  const int32_t *__restrict__ tok, const int32_t *__restrict__ tok_v,
                  const float *__restrict__ conf_v, const uint8_t *__restrict__ commit,
                  float tau_high, int K, int exclude_self,
                  uint8_t *__restrict__ accept, int32_t *__restrict__ choice,
                  uint8_t *__restrict__ final_commit, int32_t *__restrict__ y, int L)
{
    __shared__ int s_ridx[PVF_MAX_BUDGET_LIMIT];      // index of draft j inside R_b
    __shared__ int s_acc[PVF_MAX_BUDGET_LIMIT];
    __shared__ double s_c[PVF_MAX_BUDGET_LIMIT];
    __shared__ int s_choice;
    pvf_launch_dependents();
    pvf_grid_dependency_wait();
    const int b = blockIdx.x;
    const int r0 = seg_off[b], r1 = seg_off[b + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int kt = n_drafts[b];
    const int rt = route[b];
    const int nR = rem_off[b + 1] - rem_off[b];
    const int32_t *rem = rem_rows + rem_off[b];
    const int32_t *drafts = draft_rows + (size_t)b * K;
    const int base = v_off[b];

    for (int m = r0 + threadIdx.x; m < r1; m += kThreads) final_commit[m] = commit[m];
    for (int j = threadIdx.x; j < K; j += kThreads) { accept[(size_t)b * K + j] = 0; s_acc[j] = 0; s_c[j] = 0.0; }
    if (threadIdx.x == 0) s_choice = 0;
    __syncthreads();

    if (kt > 0 && rt != 0) {
        // position of every draft inside R_b
        for (int j = warp; j < kt; j += kWarps) {
            const int d = drafts[j];
            int found = -1;
            for (int r = lane; r < nR; r += 32)
                if (rem[r] == d) found = r;
            for (int o = 16; o > 0; o >>= 1) {
                const int t = __shfl_xor_sync(0xffffffffu, found, o);
                found = t > found ? t : found;
            }
            if (lane == 0) s_ridx[j] = found;
        }
        __syncthreads();

        if (rt == 1) {
            // Filter 1 (impact-set agreement) and C_total of every planning branch, one warp each.
            for (int j = warp; j < kt; j += kWarps) {
                const int rj = s_ridx[j];
                const int32_t *tb = tok_v + base, *tj = tok_v + base + (size_t)(j + 1) * nR;
                const float *cb = conf_v + base, *cj = conf_v + base + (size_t)(j + 1) * nR;
                int n_imp = 0, n_bad = 0;
                double c_total = 0.0;
                for (int r = lane; r < nR; r += 32) {
                    const bool imp = cb[r] >= tau_high && !(exclude_self && r == rj);   // S_impact
                    n_imp += imp ? 1 : 0;
                    n_bad += (imp && tj[r] != tb[r]) ? 1 : 0;
                    if (r != rj) c_total += (double)cj[r];       // positions still masked in branch j
                }
                for (int o = 16; o > 0; o >>= 1) {
                    n_imp += __shfl_xor_sync(0xffffffffu, n_imp, o);
                    n_bad += __shfl_xor_sync(0xffffffffu, n_bad, o);
                    c_total += __shfl_xor_sync(0xffffffffu, c_total, o);
                }
                if (lane == 0) {
                    s_acc[j] = (n_imp > 0 && n_bad == 0) ? 1 : 0;                       // A_t^j
                    s_c[j] = c_total;
                }
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                int best = 0;
                double best_c = 0.0;
                for (int j = 0; j < kt; ++j)
                    if (s_acc[j] && (best == 0 || s_c[j] > best_c)) { best = j + 1; best_c = s_c[j]; }
                s_choice = best;                                                        // j*
            }
        } else {
            // AR verification: branch k is verified iff fills 1..k keep their drafted token under it.
            for (int k = threadIdx.x + 1; k <= kt; k += kThreads) {
                const int32_t *tk = tok_v + base + (size_t)k * nR;
                bool ok = true;
                for (int r = 0; r < k; ++r) ok = ok && s_ridx[r] >= 0 && (tk[s_ridx[r]] == tok[drafts[r]]);
                s_acc[k - 1] = ok ? 1 : 0;
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                int best = 0;
                for (int k = 1; k <= kt; ++k)
                    if (s_acc[k - 1]) best = k;                                         // k* = max K^AR
                s_choice = best;
            }
        }
        __syncthreads();
        for (int j = threadIdx.x; j < kt; j += kThreads) accept[(size_t)b * K + j] = (uint8_t)s_acc[j];
        const int ch = s_choice;
        if (rt == 1) {
            if (ch > 0 && threadIdx.x == 0) final_commit[drafts[ch - 1]] = 1;
        } else {
            for (int r = threadIdx.x; r < ch; r += kThreads) final_commit[drafts[r]] = 1;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) choice[b] = s_choice;
    if (y)
        for (int m = r0 + threadIdx.x; m < r1; m += kThreads)
            if (final_commit[m]) y[(size_t)b * L + row_pos[m]] = tok[m];
}

bool params_ok(const pvf_ctx *ctx, const pvf_params *p, int32_t M, int32_t n_seq)
{
    return ctx && p && M >= 0 && n_seq >= 0 && M <= ctx->shape.max_rows && n_seq <= ctx->shape.max_seqs &&
           p->budget >= 0 && p->budget <= ctx->shape.max_budget;
}

int launch_result(cudaError_t e)
{
    return e == cudaSuccess ? PVF_OK : PVF_ERR_CUDA;
}

}  // namespace

extern "C" {

int pvf_commit(pvf_ctx *ctx, const pvf_params *params, int32_t M, int32_t n_seq,
               const int32_t *seg_off, const int32_t *row_pos, const uint8_t *active,
               const int32_t *tok, const float *conf,
               uint8_t *commit, int32_t *n_commit, int32_t *y, int32_t L, void *stream)
{
    if (!params_ok(ctx, params, M, n_seq)) return PVF_ERR_INVALID;
    if (n_seq == 0) return M == 0 ? PVF_OK : PVF_ERR_INVALID;
    if (!seg_off || !conf || !commit || (M > 0 && y && (!row_pos || !tok || L <= 0))) return PVF_ERR_INVALID;
    return launch_result(pvf_launch(pvf_commit_kernel, dim3(n_seq), dim3(kThreads), 0, (cudaStream_t)stream,
                                    seg_off, row_pos, active, tok, conf, params->tau_high,
                                    (params->flags & PVF_FORCE_PROGRESS) ? 1 : 0, commit, n_commit, y, L));
}

int pvf_select_drafts(pvf_ctx *ctx, const pvf_params *params, int32_t M, int32_t n_seq,
                      const int32_t *seg_off, const int32_t *row_pos, const uint8_t *active,
                      const int32_t *tok, const float *conf, const uint8_t *in_plan,
                      const uint8_t *commit,
                      int32_t *draft_rows, int32_t *n_drafts, uint8_t *route,
                      int32_t *rem_rows, int32_t *rem_off, int32_t *v_off, void *stream)
{
    (void)row_pos; (void)tok;
    if (!params_ok(ctx, params, M, n_seq)) return PVF_ERR_INVALID;
    if (n_seq == 0) return M == 0 ? PVF_OK : PVF_ERR_INVALID;
    const int any_token = (params->flags & PVF_SELECT_ANY_TOKEN) ? 1 : 0;
    if (!seg_off || !conf || (!in_plan && !any_token) || !commit || !n_drafts || !route || !rem_off || !v_off ||
        (params->budget > 0 && !draft_rows) || (M > 0 && !rem_rows))
        return PVF_ERR_INVALID;
    return launch_result(pvf_launch(pvf_select_kernel, dim3(n_seq), dim3(kThreads), 0, (cudaStream_t)stream,
                                    n_seq, seg_off, active, conf, in_plan, commit, params->tau_plan_lo,
                                    params->tau_plan_hi, params->tau_ar_lo, params->budget, any_token,
                                    (params->flags & PVF_NO_AR_FALLBACK) ? 0 : 1, draft_rows, n_drafts,
                                    route, rem_rows, rem_off, v_off, &ctx->words->select_ticket));
}

int pvf_verify(pvf_ctx *ctx, const pvf_params *params, int32_t M, int32_t n_seq,
               const int32_t *seg_off, const int32_t *row_pos,
               const int32_t *rem_rows, const int32_t *rem_off, const int32_t *v_off,
               const int32_t *draft_rows, const int32_t *n_drafts, const uint8_t *route,
               const int32_t *tok, const int32_t *tok_v, const float *conf_v, const uint8_t *commit,
               uint8_t *accept, int32_t *choice, uint8_t *final_commit,
               int32_t *y, int32_t L, void *stream)
{
    if (!params_ok(ctx, params, M, n_seq)) return PVF_ERR_INVALID;
    if (n_seq == 0) return M == 0 ? PVF_OK : PVF_ERR_INVALID;
    if (!seg_off || !rem_off || !v_off || !n_drafts || !route || !commit || !choice || !final_commit ||
        (params->budget > 0 && (!draft_rows || !accept)) ||
        (M > 0 && !tok) || (y && (!row_pos || L <= 0)))
        return PVF_ERR_INVALID;
    return launch_result(pvf_launch(pvf_verify_kernel, dim3(n_seq), dim3(kThreads), 0, (cudaStream_t)stream,
                                    seg_off, row_pos, rem_rows, rem_off, v_off, draft_rows, n_drafts, route, tok,
                                    tok_v, conf_v, commit, params->tau_high, params->budget,
                                    (params->flags & PVF_EXCLUDE_SELF_FROM_IMPACT) ? 1 : 0, accept, choice,
                                    final_commit, y, L));
}

}  // extern "C"
