// Offline construction of the planning-token vocabulary: verified information gain of every measured
// candidate, per-token statistics, and the filtering rule (Section 3, "Verified information gain";
// Appendix, "Planning Token Set Construction").
//
// A calibration step is a decode step whose candidates are chosen with PVF_SELECT_ANY_TOKEN |
// PVF_NO_AR_FALLBACK over the calibration band; pvf_verify gives their acceptance A_j, and
// pvf_calib_accumulate adds each candidate's event to the statistics of its token.  The sums are
// integers (the gain in units of 2^-32 nat), so they do not depend on the order of the atomic adds.
#include "pvf_internal.h"

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr double kVigScale = 4294967296.0;      // 2^32

__global__ void __launch_bounds__(kThreads)
pvf_calib_accumulate_kernel(const int32_t *__restrict__ rem_rows, const int32_t *__restrict__ rem_off,
                            const int32_t *__restrict__ v_off, const int32_t *__restrict__ draft_rows,
                            const int32_t *__restrict__ n_drafts, const uint8_t *__restrict__ route,
                            const int32_t *__restrict__ tok, const float *__restrict__ conf_v,
                            const float *__restrict__ ent_v, const uint8_t *__restrict__ accept,
                            float tau_high, int K, int exclude_self,
                            int32_t *__restrict__ n_v, int32_t *__restrict__ m_v, int32_t *__restrict__ sum_a,
                            long long *__restrict__ sum_vig_q32, double *__restrict__ vig_out)
{
    pvf_launch_dependents();
    pvf_grid_dependency_wait();
    const int b = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int kt = route[b] == 1 ? n_drafts[b] : 0;            // only planning-route candidates are events
    const int nR = rem_off[b + 1] - rem_off[b];
    const int32_t *rem = rem_rows + rem_off[b];
    const int32_t *drafts = draft_rows + (size_t)b * K;
    const int base = v_off[b];
    if (vig_out)
        for (int j = kt + threadIdx.x; j < K; j += kThreads) vig_out[(size_t)b * K + j] = 0.0;
    for (int j = warp; j < kt; j += kWarps) {
        const int d = drafts[j];
        int rj = -1;
        for (int r = lane; r < nR; r += 32)
            if (rem[r] == d) rj = r;
        for (int o = 16; o > 0; o >>= 1) rj = max(rj, __shfl_xor_sync(0xffffffffu, rj, o));
        const float *hb = ent_v + base, *hj = ent_v + base + (size_t)(j + 1) * nR;
        int n_imp = 0;
        double d_sum = 0.0;
        for (int r = lane; r < nR; r += 32) {
            n_imp += (conf_v[base + r] >= tau_high && !(exclude_self && r == rj)) ? 1 : 0;   // S_impact
            if (r != rj) d_sum += (double)hb[r] - (double)hj[r];                             // d_i over R_t^j
        }
        for (int o = 16; o > 0; o >>= 1) {
            n_imp += __shfl_xor_sync(0xffffffffu, n_imp, o);
            d_sum += __shfl_xor_sync(0xffffffffu, d_sum, o);
        }
        if (lane == 0) {
            const int a = accept[(size_t)b * K + j] ? 1 : 0;                                 // A_t^j
            const double d_h = nR > 1 ? d_sum / (double)(nR - 1) : 0.0;                      // empty region: 0
            const double vig = a ? d_h : 0.0;
            const int v = tok[d];
            atomicAdd(&n_v[v], 1);
            if (n_imp > 0) atomicAdd(&m_v[v], 1);
            if (a) {
                atomicAdd(&sum_a[v], 1);
                atomicAdd(reinterpret_cast<unsigned long long *>(&sum_vig_q32[v]),
                          (unsigned long long)__double2ll_rn(vig * kVigScale));
            }
            if (vig_out) vig_out[(size_t)b * K + j] = vig;
        }
    }
}

// One thread per token, one bitmap word per warp.
__global__ void __launch_bounds__(kThreads)
pvf_calib_filter_kernel(int V, const int32_t *__restrict__ n_v, const int32_t *__restrict__ m_v,
                        const int32_t *__restrict__ sum_a, const long long *__restrict__ sum_vig_q32,
                        int n_min, int m_min, float rho_ver, float gamma_vig,
                        uint32_t *__restrict__ bitmap, int32_t *__restrict__ n_plan)
{
    pvf_launch_dependents();
    pvf_grid_dependency_wait();
    const int v = blockIdx.x * kThreads + threadIdx.x;
    bool keep = false;
    if (v < V) {
        const int n = n_v[v], m = m_v[v];
        if (n >= n_min && m >= m_min && n > 0) {
            const double r_ver = m > 0 ? (double)sum_a[v] / (double)m : 0.0;
            const double vig_hat = ((double)sum_vig_q32[v] / kVigScale) / (double)n;
            keep = r_ver >= (double)rho_ver && vig_hat >= (double)gamma_vig;
        }
    }
    const unsigned word = __ballot_sync(0xffffffffu, keep);
    if ((threadIdx.x & 31) == 0 && (v >> 5) < (V + 31) / 32) {
        bitmap[v >> 5] = word;
        if (word && n_plan) atomicAdd(n_plan, __popc(word));
    }
}

}  // namespace

extern "C" {

void pvf_default_calib_params(pvf_calib_params *out)
{
    if (!out) return;
    out->tau_cal_lo = 0.15f;
    out->tau_cal_hi = 0.25f;
    out->n_min = 50;
    out->m_min = 20;
    out->rho_ver = 0.9f;
    out->gamma_vig = 0.03f;
}

int pvf_calib_accumulate(pvf_ctx *ctx, const pvf_params *params, int32_t n_seq,
                         const int32_t *rem_rows, const int32_t *rem_off, const int32_t *v_off,
                         const int32_t *draft_rows, const int32_t *n_drafts, const uint8_t *route,
                         const int32_t *tok, const float *conf_v, const float *ent_v, const uint8_t *accept,
                         int32_t *n_v, int32_t *m_v, int32_t *sum_a, int64_t *sum_vig_q32, double *vig_out,
                         void *stream)
{
    if (!ctx || !params || n_seq < 0 || n_seq > ctx->shape.max_seqs || params->budget < 0 ||
        params->budget > ctx->shape.max_budget)
        return PVF_ERR_INVALID;
    if (n_seq == 0 || params->budget == 0) return PVF_OK;
    if (!rem_off || !v_off || !draft_rows || !n_drafts || !route || !tok || !accept || !n_v || !m_v || !sum_a ||
        !sum_vig_q32)
        return PVF_ERR_INVALID;
    const cudaError_t e = pvf_launch(pvf_calib_accumulate_kernel, dim3(n_seq), dim3(kThreads), 0, (cudaStream_t)stream,
                                     rem_rows, rem_off, v_off, draft_rows, n_drafts, route, tok, conf_v, ent_v, accept,
                                     params->tau_high, params->budget,
                                     (params->flags & PVF_EXCLUDE_SELF_FROM_IMPACT) ? 1 : 0, n_v, m_v, sum_a,
                                     reinterpret_cast<long long *>(sum_vig_q32), vig_out);
    return e == cudaSuccess ? PVF_OK : PVF_ERR_CUDA;
}

int pvf_calib_filter(pvf_ctx *ctx, const pvf_calib_params *cal, const int32_t *n_v, const int32_t *m_v,
                     const int32_t *sum_a, const int64_t *sum_vig_q32, uint32_t *plan_bitmap, int32_t *n_plan,
                     void *stream)
{
    if (!ctx || !cal || !n_v || !m_v || !sum_a || !sum_vig_q32 || !plan_bitmap) return PVF_ERR_INVALID;
    const int V = ctx->shape.vocab;
    cudaStream_t s = (cudaStream_t)stream;
    if (n_plan && cudaMemsetAsync(n_plan, 0, sizeof(int32_t), s) != cudaSuccess) return PVF_ERR_CUDA;
    const int words = (V + 31) / 32;
    const int blocks = (words * 32 + kThreads - 1) / kThreads;
    const cudaError_t e = pvf_launch(pvf_calib_filter_kernel, dim3(blocks), dim3(kThreads), 0, s, V, n_v, m_v, sum_a,
                                     reinterpret_cast<const long long *>(sum_vig_q32), cal->n_min, cal->m_min,
                                     cal->rho_ver, cal->gamma_vig, plan_bitmap, n_plan);
    return e == cudaSuccess ? PVF_OK : PVF_ERR_CUDA;
}

int pvf_set_plan_bitmap(pvf_ctx *ctx, const uint32_t *plan_bitmap, void *stream)
{
    if (!ctx || !plan_bitmap) return PVF_ERR_INVALID;
    const size_t bytes = ((size_t)ctx->shape.vocab + 31) / 32 * 4;
    if (cudaMemcpyAsync(ctx->plan_bitmap, plan_bitmap, bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)stream) != cudaSuccess)
        return PVF_ERR_CUDA;
    return PVF_OK;
}

}  // extern "C"
