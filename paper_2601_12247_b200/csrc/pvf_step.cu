// Decision kernels of one PVF step: base commit, draft proposal, acceptance check.
// One thread block per sequence; rows of a sequence are contiguous and sorted by position.
// All reductions are warp shuffles plus one shared-memory hop; every result is deterministic.
//
// The step entry points run two kernels of this file right behind the projection kernel of pvf_score, with the
// merge of its partial softmax states as their first phase:
//     pvf_draft_kernel            merge (the sequence's own rows) + base commit + draft proposal
//     pvf_verify_kernel<true>     merge (the sequence's rows of the verification pass) + acceptance check
// so that a step is four launches.  These kernels keep to a few dozen registers and about a kilobyte of shared memory.
// Measured with %globaltimer stamps: a block of theirs becomes resident on the first SM that a block of the running
// projection leaves, some ten microseconds before its grid-dependency wait returns, and the block of the NEXT
// projection that takes over that SM (it starts fetching weights before its own wait) must fit beside it -- a
// projection block fills an SM's shared memory and two thirds of its registers.  A version that staged the merge
// through 96 KB of shared memory, or held 20 states per thread in registers, was 4 .. 6 us per step slower.  Pointers
// that one phase of a kernel writes and a later phase reads carry no __restrict__ / read-only qualifier in the shared
// device functions.
#include "pvf_internal.h"

namespace {

constexpr int kThreads = kPvfBlockThreads;
constexpr int kWarps = kPvfBlockWarps;
constexpr int kOffsetCache = 256;         // sequence offsets the packing step keeps in shared memory (the step kernels
                                          // must fit beside a projection block that fills an SM's shared memory)

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

// Shared memory of a block of the commit / select kernels.
struct StepShared {
    int s_int[kWarps];
    unsigned long long s_key[kWarps];
    int s_last;
    int s_off[kOffsetCache + 1];
};

// ------------------------------------------------------------------------------------ merge (first phase)
// Final merge of rows row_begin .. row_end-1 by the block's warps.
__device__ __forceinline__ void merge_rows_block(const float4 *__restrict__ partials, int parts, int vocab,
                                                 const uint32_t *__restrict__ plan_bitmap, int row_begin, int row_end,
                                                 int32_t *tok, float *conf, float *ent, uint8_t *in_plan)
{
    pvf_merge_rows(partials, parts, vocab, plan_bitmap, row_begin, row_end, (int)(threadIdx.x >> 5), kWarps, tok, conf, ent, in_plan);
}

// The merge phase of a step kernel that gives every sequence `share` blocks: block c of the sequence merges the c-th
// slice of rows [row_begin, row_end); the block that arrives last on the sequence's ticket (no waiting) goes on to
// the decisions, the others are done.  Returns true in the block that goes on.
__device__ __forceinline__ bool merge_phase(const float4 *__restrict__ partials, int parts, int vocab,
                                            const uint32_t *__restrict__ plan_bitmap, int row_begin, int row_end, int c, int share,
                                            unsigned *seq_ticket, int32_t *tok, float *conf, float *ent, uint8_t *in_plan, int *s_flag)
{
    const int n = row_end - row_begin;
    const int lo = row_begin + (int)((long long)n * c / share), hi = row_begin + (int)((long long)n * (c + 1) / share);
    merge_rows_block(partials, parts, vocab, plan_bitmap, lo, hi, tok, conf, ent, in_plan);
    if (share == 1) {
        __syncthreads();                               // the rows' scores (global memory) before the decisions read them
        return true;
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const int last = atomicAdd(seq_ticket, 1u) == (unsigned)(share - 1) ? 1 : 0;
        if (last) *seq_ticket = 0;
        *s_flag = last;
    }
    __syncthreads();
    if (!*s_flag) return false;
    __threadfence();
    return true;
}

// ------------------------------------------------------------------------------------ commit
// Base set and base branch of sequence b (one block).
__device__ __forceinline__ void commit_block(int b, const int32_t *__restrict__ seg_off, const int32_t *__restrict__ row_pos,
                                             const uint8_t *__restrict__ active, const int32_t *tok, const float *conf,
                                             float tau_high, int force_progress, uint8_t *commit, int32_t *__restrict__ n_commit,
                                             int32_t *__restrict__ y, int L, StepShared *sh)
{
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
    int total = pvf_block_sum(count, sh->s_int);
    if (force_progress && total == 0) {
        best = block_max(best, sh->s_key);
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
// Draft proposal of sequence b (one block).  No block depends on another: R_b is first written where the sequence's
// own rows start (rem_rows[seg_off[b] ..], it cannot be longer than they are) and its length left in rem_off[b + 1];
// the block that finishes last (an arrival ticket, no waiting) turns the lengths into the offsets rem_off and v_off
// and packs the lists to the front of rem_rows.
__device__ __forceinline__ void select_block(int b, int n_seq, const int32_t *__restrict__ seg_off, const uint8_t *__restrict__ active,
                                             const float *conf, const uint8_t *in_plan, const uint8_t *commit,
                                             float tau_lo, float tau_hi, float tau_ar, int K, int any_token, int ar_fallback,
                                             int32_t *__restrict__ draft_rows, int32_t *n_drafts, uint8_t *__restrict__ route,
                                             int32_t *rem_rows, int32_t *rem_off, int32_t *__restrict__ v_off, unsigned *ticket,
                                             StepShared *sh)
{
    const int r0 = seg_off[b], r1 = seg_off[b + 1];

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
        const int rank = pvf_block_rank(rem, sh->s_int, &chunk_total);
        if (rem) rem_rows[r0 + n_rem + rank] = m;
        n_rem += chunk_total;
        n_plan += plan ? 1 : 0;
    }
    n_plan = pvf_block_sum(n_plan, sh->s_int);

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
            last = block_max(best, sh->s_key);
            if (threadIdx.x == 0)
                draft_rows[(size_t)b * K + j] = r0 + (int)(0xffffffffu - (unsigned)(last & 0xffffffffull));
        }
    } else if (K > 0 && ar_fallback) {
        // AR fallback: leftmost rows of R_b with p >= tau_AR^l, at most K of them.
        for (int c0 = r0; c0 < r1 && kt < K; c0 += kThreads) {
            const int m = c0 + threadIdx.x;
            const bool ok = m < r1 && (active ? active[m] != 0 : true) && !commit[m] && conf[m] >= tau_ar;
            int chunk_total;
            const int rank = pvf_block_rank(ok, sh->s_int, &chunk_total);
            if (ok && kt + rank < K) draft_rows[(size_t)b * K + kt + rank] = m;
            kt += chunk_total;
        }
        kt = kt < K ? kt : K;
        rt = kt > 0 ? 2 : 0;
    }
    for (int j = kt + threadIdx.x; j < K; j += kThreads) draft_rows[(size_t)b * K + j] = -1;
    if (n_seq == 1 && r0 == 0) {
        // One sequence: its list is where it belongs and the offsets are its lengths -- no ticket, no fences, no
        // packing (four dependent round trips to L2, 3 .. 4 us of a batch-1 step).
        if (threadIdx.x == 0) {
            n_drafts[0] = kt;
            route[0] = (uint8_t)rt;
            rem_off[0] = 0;
            rem_off[1] = n_rem;
            v_off[0] = 0;
            v_off[1] = kt > 0 ? (1 + kt) * n_rem : 0;
        }
        return;
    }
    if (threadIdx.x == 0) {
        n_drafts[b] = kt;
        route[b] = (uint8_t)rt;
        rem_off[b + 1] = n_rem;                                   // a length for now
    }

    // The last block to finish turns the per-sequence lengths into offsets and packs the lists.
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) sh->s_last = (atomicAdd(ticket, 1u) == (unsigned)(n_seq - 1)) ? 1 : 0;
    __syncthreads();
    if (!sh->s_last) return;
    __threadfence();
    if (threadIdx.x < 32) {
        const volatile int32_t *vd = n_drafts;
        volatile int32_t *vr = rem_off;
        int run_rem = 0, run_v = 0;
        if (threadIdx.x == 0) vr[0] = 0;
        for (int c0 = 0; c0 < n_seq; c0 += 32) {
            const int s = c0 + threadIdx.x;
            int len = 0, rows = 0;
            if (s < n_seq) {
                len = vr[s + 1];
                const int d = vd[s];
                rows = d > 0 ? (1 + d) * len : 0;
            }
            int incl_len = len, incl_rows = rows;
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, incl_len, o);
                const int u = __shfl_up_sync(0xffffffffu, incl_rows, o);
                if ((int)threadIdx.x >= o) { incl_len += t; incl_rows += u; }
            }
            if (s < n_seq) {
                vr[s + 1] = run_rem + incl_len;                   // each entry is read and rewritten by the same lane
                v_off[s] = run_v + incl_rows - rows;
            }
            run_rem += __shfl_sync(0xffffffffu, incl_len, 31);
            run_v += __shfl_sync(0xffffffffu, incl_rows, 31);
        }
        if (threadIdx.x == 0) {
            v_off[n_seq] = run_v;
            *ticket = 0;
        }
    }
    __syncthreads();

    // Pack: element e of the concatenated lists sits at seg_off[b] + (e - rem_off[b]) and belongs at e.  It never
    // moves to the right, and elements are taken in ascending chunks (read, barrier, write), so a write can only
    // land on entries that were moved earlier or belong to the same chunk.
    const volatile int32_t *off = rem_off;
    const int total = off[n_seq];
    if (total == seg_off[n_seq]) return;                          // every row remains: the lists are in place already
    const bool cached = n_seq <= kOffsetCache;
    if (cached) {
        for (int s = threadIdx.x; s <= n_seq; s += kThreads) sh->s_off[s] = off[s];
        __syncthreads();
    }
    for (int e0 = 0; e0 < total; e0 += kThreads) {
        const int e = e0 + threadIdx.x;
        int value = 0;
        if (e < total) {
            int lo = 0, hi = n_seq - 1;                           // the sequence q with rem_off[q] <= e < rem_off[q + 1]
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                const int end = cached ? sh->s_off[mid + 1] : off[mid + 1];
                if (end > e) hi = mid; else lo = mid + 1;
            }
            const int start = cached ? sh->s_off[lo] : off[lo];
            value = __ldcg(rem_rows + seg_off[lo] + (e - start));
        }
        __syncthreads();
        if (e < total) rem_rows[e] = value;
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kThreads, 1)
pvf_commit_kernel(const int32_t *__restrict__ seg_off, const int32_t *__restrict__ row_pos,
                  const uint8_t *__restrict__ active, const int32_t *__restrict__ tok,
                  const float *__restrict__ conf, float tau_high, int force_progress,
                  uint8_t *__restrict__ commit, int32_t *__restrict__ n_commit,
                  int32_t *__restrict__ y, int L)
{
    __shared__ StepShared sh;
    pvf_launch_dependents();
    pvf_grid_dependency_wait();
    commit_block(blockIdx.x, seg_off, row_pos, active, tok, conf, tau_high, force_progress, commit, n_commit, y, L, &sh);
}

__global__ void __launch_bounds__(kThreads, 1)
pvf_select_kernel(int n_seq, const int32_t *__restrict__ seg_off, const uint8_t *__restrict__ active,
                  const float *__restrict__ conf, const uint8_t *__restrict__ in_plan,
                  const uint8_t *__restrict__ commit, float tau_lo, float tau_hi, float tau_ar, int K,
                  int any_token, int ar_fallback, int32_t *__restrict__ draft_rows, int32_t *n_drafts,
                  uint8_t *__restrict__ route, int32_t *rem_rows, int32_t *rem_off, int32_t *__restrict__ v_off,
                  unsigned *ticket)
{
    __shared__ StepShared sh;
    pvf_launch_dependents();
    pvf_grid_dependency_wait();
    select_block(blockIdx.x, n_seq, seg_off, active, conf, in_plan, commit, tau_lo, tau_hi, tau_ar, K, any_token, ar_fallback,
                 draft_rows, n_drafts, route, rem_rows, rem_off, v_off, ticket, &sh);
}

// Base commit and draft proposal of a sequence in one launch.
__global__ void __launch_bounds__(kThreads, 1)
pvf_commit_select_kernel(int n_seq, const int32_t *__restrict__ seg_off, const int32_t *__restrict__ row_pos,
                         const uint8_t *__restrict__ active, const int32_t *__restrict__ tok,
                         const float *__restrict__ conf, const uint8_t *__restrict__ in_plan, float tau_high,
                         int force_progress, float tau_lo, float tau_hi, float tau_ar, int K, int any_token, int ar_fallback,
                         uint8_t *commit, int32_t *__restrict__ n_commit, int32_t *__restrict__ y, int L,
                         int32_t *__restrict__ draft_rows, int32_t *n_drafts, uint8_t *__restrict__ route,
                         int32_t *rem_rows, int32_t *rem_off, int32_t *__restrict__ v_off, unsigned *ticket)
{
    __shared__ StepShared sh;
    pvf_launch_dependents();
    pvf_grid_dependency_wait();
    commit_block(blockIdx.x, seg_off, row_pos, active, tok, conf, tau_high, force_progress, commit, n_commit, y, L, &sh);
    __syncthreads();                                   // this block's commit flags (global memory) before select reads them
    select_block(blockIdx.x, n_seq, seg_off, active, conf, in_plan, commit, tau_lo, tau_hi, tau_ar, K, any_token, ar_fallback,
                 draft_rows, n_drafts, route, rem_rows, rem_off, v_off, ticket, &sh);
}

// The draft half of a step behind the projection kernel: final merge of the sequence's rows (token, confidence,
// entropy, planning-vocabulary membership), base commit, draft proposal.
__global__ void __launch_bounds__(kThreads, 3)          // at most 80 registers: see the note at the top of the file
pvf_draft_kernel(const float4 *__restrict__ partials, int parts, int vocab, const uint32_t *__restrict__ plan_bitmap,
                 int n_seq, const int32_t *__restrict__ seg_off, const int32_t *__restrict__ row_pos,
                 const uint8_t *__restrict__ active, int32_t *tok, float *conf, float *ent, uint8_t *in_plan,
                 float tau_high, int force_progress, float tau_lo, float tau_hi, float tau_ar, int K, int any_token,
                 int ar_fallback, uint8_t *commit, int32_t *__restrict__ n_commit, int32_t *__restrict__ y, int L,
                 int32_t *__restrict__ draft_rows, int32_t *n_drafts, uint8_t *__restrict__ route,
                 int32_t *rem_rows, int32_t *rem_off, int32_t *__restrict__ v_off, unsigned *ticket,
                 int share, unsigned *seq_tickets)
{
    __shared__ StepShared sh;
    pvf_launch_dependents();
    pvf_grid_dependency_wait();
    const int b = (int)blockIdx.x / share;
    if (!merge_phase(partials, parts, vocab, plan_bitmap, seg_off[b], seg_off[b + 1], (int)blockIdx.x % share, share,
                     seq_tickets + b, tok, conf, ent, in_plan, &sh.s_last))
        return;
    commit_block(b, seg_off, row_pos, active, tok, conf, tau_high, force_progress, commit, n_commit, y, L, &sh);
    __syncthreads();
    select_block(b, n_seq, seg_off, active, conf, in_plan, commit, tau_lo, tau_hi, tau_ar, K, any_token, ar_fallback,
                 draft_rows, n_drafts, route, rem_rows, rem_off, v_off, ticket, &sh);
}

// ------------------------------------------------------------------------------------ verify
// kMerge: the kernel runs right behind the projection kernel of the verification pass and first merges the partial
// states of the sequence's verification rows v_off[b] .. v_off[b+1]-1 (tok_v, conf_v and, if asked for, ent_v are
// then outputs).
template <bool kMerge>
__global__ void __launch_bounds__(kThreads, 3)          // at most 80 registers
pvf_verify_kernel(const float4 *__restrict__ partials, int parts, int vocab,
                  const int32_t *__restrict__ seg_off, const int32_t *__restrict__ row_pos,
                  const int32_t *__restrict__ rem_rows, const int32_t *__restrict__ rem_off,
                  const int32_t *__restrict__ v_off, const int32_t *__restrict__ draft_rows,
                  const int32_t *__restrict__ n_drafts, const uint8_t *__restrict__ route,
                  const int32_t *__restrict__ tok, int32_t *tok_v_out, float *conf_v_out, float *ent_v_out,
                  const uint8_t *__restrict__ commit,
                  float tau_high, int K, int exclude_self,
                  uint8_t *__restrict__ accept, int32_t *__restrict__ choice,
                  uint8_t *final_commit, int32_t *__restrict__ y, int L, int share, unsigned *seq_tickets)
{
    __shared__ int s_ridx[PVF_MAX_BUDGET_LIMIT];      // index of draft j inside R_b
    __shared__ int s_acc[PVF_MAX_BUDGET_LIMIT];
    __shared__ double s_c[PVF_MAX_BUDGET_LIMIT];
    __shared__ int s_choice;
    pvf_launch_dependents();
    pvf_grid_dependency_wait();
    const int b = kMerge ? (int)blockIdx.x / share : (int)blockIdx.x;
    if (kMerge && !merge_phase(partials, parts, vocab, nullptr, v_off[b], v_off[b + 1], (int)blockIdx.x % share, share,
                               seq_tickets + b, tok_v_out, conf_v_out, ent_v_out, nullptr, &s_choice))
        return;
    const int32_t *tok_v = tok_v_out;
    const float *conf_v = conf_v_out;
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

// Blocks per sequence of a step kernel's merge phase: enough that a block merges a few dozen rows of `parts` states
// (the decisions then run in one of them).
int merge_share(int32_t rows, int32_t n_seq, int parts)
{
    const long long states_per_seq = (long long)rows * parts / (n_seq > 0 ? n_seq : 1);
    long long share = states_per_seq / 1024;           // 1024 states = 8 rows of 128 parts, a row per warp: one turn of the merge
                                                       // (measured against 4096: 0.3 - 1 % of a batch-1 step, nothing elsewhere)
    if (share < 1) share = 1;
    if (share > 16) share = 16;
    return (int)share;
}

bool select_args_ok(const pvf_params *params, int32_t M, const int32_t *seg_off, const float *conf, const uint8_t *in_plan,
                    const uint8_t *commit, const int32_t *draft_rows, const int32_t *n_drafts, const uint8_t *route,
                    const int32_t *rem_rows, const int32_t *rem_off, const int32_t *v_off)
{
    const bool any_token = (params->flags & PVF_SELECT_ANY_TOKEN) != 0;
    return seg_off && conf && (in_plan || any_token) && commit && n_drafts && route && rem_off && v_off &&
           (params->budget == 0 || draft_rows) && (M == 0 || rem_rows);
}

bool verify_args_ok(const pvf_params *params, int32_t M, const int32_t *seg_off, const int32_t *row_pos,
                    const int32_t *rem_off, const int32_t *v_off, const int32_t *draft_rows, const int32_t *n_drafts,
                    const uint8_t *route, const int32_t *tok, const uint8_t *commit, const uint8_t *accept,
                    const int32_t *choice, const uint8_t *final_commit, const int32_t *y, int32_t L)
{
    return seg_off && rem_off && v_off && n_drafts && route && commit && choice && final_commit &&
           (params->budget == 0 || (draft_rows && accept)) && (M == 0 || tok) && (!y || (row_pos && L > 0));
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
    if (!select_args_ok(params, M, seg_off, conf, in_plan, commit, draft_rows, n_drafts, route, rem_rows, rem_off, v_off))
        return PVF_ERR_INVALID;
    return launch_result(pvf_launch(pvf_select_kernel, dim3(n_seq), dim3(kThreads), 0, (cudaStream_t)stream,
                                    n_seq, seg_off, active, conf, in_plan, commit, params->tau_plan_lo,
                                    params->tau_plan_hi, params->tau_ar_lo, params->budget,
                                    (params->flags & PVF_SELECT_ANY_TOKEN) ? 1 : 0,
                                    (params->flags & PVF_NO_AR_FALLBACK) ? 0 : 1, draft_rows, n_drafts,
                                    route, rem_rows, rem_off, v_off, &ctx->words->select_ticket));
}

int pvf_commit_select(pvf_ctx *ctx, const pvf_params *params, int32_t M, int32_t n_seq,
                      const int32_t *seg_off, const int32_t *row_pos, const uint8_t *active,
                      const int32_t *tok, const float *conf, const uint8_t *in_plan,
                      uint8_t *commit, int32_t *n_commit, int32_t *y, int32_t L,
                      int32_t *draft_rows, int32_t *n_drafts, uint8_t *route,
                      int32_t *rem_rows, int32_t *rem_off, int32_t *v_off, void *stream)
{
    if (!params_ok(ctx, params, M, n_seq)) return PVF_ERR_INVALID;
    if (n_seq == 0) return M == 0 ? PVF_OK : PVF_ERR_INVALID;
    if ((M > 0 && y && (!row_pos || !tok || L <= 0)) ||
        !select_args_ok(params, M, seg_off, conf, in_plan, commit, draft_rows, n_drafts, route, rem_rows, rem_off, v_off))
        return PVF_ERR_INVALID;
    return launch_result(pvf_launch(pvf_commit_select_kernel, dim3(n_seq), dim3(kThreads), 0, (cudaStream_t)stream,
                                    n_seq, seg_off, row_pos, active, tok, conf, in_plan, params->tau_high,
                                    (params->flags & PVF_FORCE_PROGRESS) ? 1 : 0, params->tau_plan_lo, params->tau_plan_hi,
                                    params->tau_ar_lo, params->budget, (params->flags & PVF_SELECT_ANY_TOKEN) ? 1 : 0,
                                    (params->flags & PVF_NO_AR_FALLBACK) ? 0 : 1, commit, n_commit, y, L, draft_rows,
                                    n_drafts, route, rem_rows, rem_off, v_off, &ctx->words->select_ticket));
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
    if (!verify_args_ok(params, M, seg_off, row_pos, rem_off, v_off, draft_rows, n_drafts, route, tok, commit, accept, choice,
                        final_commit, y, L))
        return PVF_ERR_INVALID;
    return launch_result(pvf_launch(pvf_verify_kernel<false>, dim3(n_seq), dim3(kThreads), 0, (cudaStream_t)stream,
                                    (const float4 *)nullptr, 0, 0, seg_off, row_pos, rem_rows, rem_off, v_off, draft_rows,
                                    n_drafts, route, tok, const_cast<int32_t *>(tok_v), const_cast<float *>(conf_v),
                                    (float *)nullptr, commit, params->tau_high, params->budget,
                                    (params->flags & PVF_EXCLUDE_SELF_FROM_IMPACT) ? 1 : 0, accept, choice,
                                    final_commit, y, L, 1, (unsigned *)nullptr));
}

int pvf_draft_step(pvf_ctx *ctx, const pvf_params *params, const void *hidden, int32_t M, int32_t n_seq,
                   const int32_t *seg_off, const int32_t *row_pos, const uint8_t *active,
                   int32_t *tok, float *conf, float *ent, uint8_t *in_plan,
                   uint8_t *commit, int32_t *n_commit, int32_t *y, int32_t L,
                   int32_t *draft_rows, int32_t *n_drafts, uint8_t *route,
                   int32_t *rem_rows, int32_t *rem_off, int32_t *v_off, void *stream)
{
    if (!params_ok(ctx, params, M, n_seq)) return PVF_ERR_INVALID;
    if (n_seq == 0) return M == 0 ? PVF_OK : PVF_ERR_INVALID;
    if ((M > 0 && (!hidden || !tok)) || (M > 0 && y && (!row_pos || L <= 0)) ||
        !select_args_ok(params, M, seg_off, conf, in_plan, commit, draft_rows, n_drafts, route, rem_rows, rem_off, v_off))
        return PVF_ERR_INVALID;
    int parts = 0;
    if (M > 0) {
        const int rc = pvf_score_partials(ctx, hidden, M, &parts, 0, stream);
        if (rc != PVF_OK) return rc;
    }
    const int share = merge_share(M, n_seq, parts);
    return launch_result(pvf_launch(pvf_draft_kernel, dim3(n_seq * share), dim3(kThreads), 0, (cudaStream_t)stream,
                                    (const float4 *)ctx->partials, parts, ctx->shape.vocab, (const uint32_t *)ctx->plan_bitmap,
                                    n_seq, seg_off, row_pos, active, tok, conf, ent, in_plan, params->tau_high,
                                    (params->flags & PVF_FORCE_PROGRESS) ? 1 : 0, params->tau_plan_lo, params->tau_plan_hi,
                                    params->tau_ar_lo, params->budget, (params->flags & PVF_SELECT_ANY_TOKEN) ? 1 : 0,
                                    (params->flags & PVF_NO_AR_FALLBACK) ? 0 : 1, commit, n_commit, y, L, draft_rows,
                                    n_drafts, route, rem_rows, rem_off, v_off, &ctx->words->select_ticket, share,
                                    ctx->seq_tickets));
}

int pvf_verify_step(pvf_ctx *ctx, const pvf_params *params, const void *hidden_v, int32_t Mv, int32_t M, int32_t n_seq,
                    const int32_t *seg_off, const int32_t *row_pos,
                    const int32_t *rem_rows, const int32_t *rem_off, const int32_t *v_off,
                    const int32_t *draft_rows, const int32_t *n_drafts, const uint8_t *route,
                    const int32_t *tok, const uint8_t *commit,
                    int32_t *tok_v, float *conf_v, float *ent_v,
                    uint8_t *accept, int32_t *choice, uint8_t *final_commit, int32_t *y, int32_t L, void *stream)
{
    if (!params_ok(ctx, params, M, n_seq) || Mv < 0 || Mv > ctx->shape.max_rows) return PVF_ERR_INVALID;
    if (n_seq == 0) return (M == 0 && Mv == 0) ? PVF_OK : PVF_ERR_INVALID;
    if ((Mv > 0 && (!hidden_v || !tok_v || !conf_v)) ||
        !verify_args_ok(params, M, seg_off, row_pos, rem_off, v_off, draft_rows, n_drafts, route, tok, commit, accept, choice,
                        final_commit, y, L))
        return PVF_ERR_INVALID;
    int parts = 0;
    if (Mv > 0) {
        const int rc = pvf_score_partials(ctx, hidden_v, Mv, &parts, 1, stream);
        if (rc != PVF_OK) return rc;
        const int share = merge_share(Mv, n_seq, parts);
        return launch_result(pvf_launch(pvf_verify_kernel<true>, dim3(n_seq * share), dim3(kThreads), 0, (cudaStream_t)stream,
                                        (const float4 *)ctx->partials, parts, ctx->shape.vocab, seg_off, row_pos, rem_rows, rem_off,
                                        v_off, draft_rows, n_drafts, route, tok, tok_v, conf_v, ent_v, commit, params->tau_high,
                                        params->budget, (params->flags & PVF_EXCLUDE_SELF_FROM_IMPACT) ? 1 : 0, accept, choice,
                                        final_commit, y, L, share, ctx->seq_tickets));
    }
    return launch_result(pvf_launch(pvf_verify_kernel<false>, dim3(n_seq), dim3(kThreads), 0, (cudaStream_t)stream,
                                    (const float4 *)nullptr, 0, 0, seg_off, row_pos, rem_rows, rem_off, v_off, draft_rows,
                                    n_drafts, route, tok, tok_v, conf_v, (float *)nullptr, commit, params->tau_high,
                                    params->budget, (params->flags & PVF_EXCLUDE_SELF_FROM_IMPACT) ? 1 : 0, accept, choice,
                                    final_commit, y, L, 1, (unsigned *)nullptr));
}

}  // extern "C"
