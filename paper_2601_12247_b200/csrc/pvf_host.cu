// Host-buffer variants of the step calls (pvf_draft_step, pvf_verify_step): inputs and outputs live in host
// memory, the library stages them through a caller-provided device buffer with cudaMemcpyAsync and
// synchronises the stream before returning.  The arithmetic is the device entry points'; nothing is
// computed on the host.
#include <string.h>

#include "pvf_internal.h"

namespace {

// Device staging of one step.  The hidden states come first (room for max_rows); everything else is packed for
// the sizes of the step at hand, in three groups that each travel as ONE copy when a pinned bounce buffer is
// attached:  inputs (seg_off, row_pos, active)  |  draft outputs (tok .. v_off)  |  verify outputs (accept .. conf_v).
struct StagingLayout {
    size_t hidden, seg_off, row_pos, active, in_end, tok, conf, ent, in_plan, commit, n_commit, draft_rows, n_drafts,
        route, rem_rows, rem_off, v_off, draft_end, accept, choice, final_commit, tok_v, conf_v, total;
};

StagingLayout staging_layout(const pvf_shape *s, size_t R, size_t B, size_t K, size_t Rv)
{
    StagingLayout l;
    size_t off = 0;
    if (K == 0) K = 1;
    auto take = [&](size_t bytes) { size_t o = off; off = pvf_align_up(off + bytes, 256); return o; };
    l.hidden = take((size_t)s->max_rows * (size_t)s->hidden * 2);
    l.seg_off = take((B + 1) * 4);
    l.row_pos = take(R * 4);
    l.active = take(R);
    l.in_end = off;
    l.tok = take(R * 4);
    l.conf = take(R * 4);
    l.ent = take(R * 4);
    l.in_plan = take(R);
    l.commit = take(R);
    l.n_commit = take(B * 4);
    l.draft_rows = take(B * K * 4);
    l.n_drafts = take(B * 4);
    l.route = take(B);
    l.rem_rows = take(R * 4 + 4);
    l.rem_off = take((B + 1) * 4);
    l.v_off = take((B + 1) * 4);
    l.draft_end = off;
    l.accept = take(B * K);
    l.choice = take(B * 4);
    l.final_commit = take(R);
    l.tok_v = take(Rv * 4);
    l.conf_v = take(Rv * 4);
    l.total = off;
    return l;
}

StagingLayout staging_layout_max(const pvf_shape *s)
{
    return staging_layout(s, (size_t)s->max_rows, (size_t)s->max_seqs, (size_t)s->max_budget, (size_t)s->max_rows);
}

bool h2d(void *dst, const void *src, size_t n, cudaStream_t s)
{
    return n == 0 || cudaMemcpyAsync(dst, src, n, cudaMemcpyHostToDevice, s) == cudaSuccess;
}
bool d2h(void *dst, const void *src, size_t n, cudaStream_t s)
{
    return n == 0 || !dst || cudaMemcpyAsync(dst, src, n, cudaMemcpyDeviceToHost, s) == cudaSuccess;
}
void put(uint8_t *bounce, size_t off, const void *src, size_t n) { if (src && n) memcpy(bounce + off, src, n); }
void get(void *dst, const uint8_t *bounce, size_t off, size_t n) { if (dst && n) memcpy(dst, bounce + off, n); }

}  // namespace

extern "C" {

size_t pvf_host_staging_bytes(const pvf_shape *shape)
{
    if (!shape || shape->vocab <= 0 || shape->hidden <= 0 || shape->max_rows < 0 || shape->max_seqs < 0 ||
        shape->max_budget < 0)
        return 0;
    return staging_layout_max(shape).total;
}

size_t pvf_host_bounce_bytes(const pvf_shape *shape)
{
    if (!shape || shape->vocab <= 0 || shape->hidden <= 0 || shape->max_rows < 0 || shape->max_seqs < 0 ||
        shape->max_budget < 0)
        return 0;
    const StagingLayout l = staging_layout_max(shape);
    return l.total - l.seg_off;
}

int pvf_attach_host_bounce(pvf_ctx *ctx, void *pinned_host, size_t bytes)
{
    if (!ctx) return PVF_ERR_INVALID;
    if (!pinned_host) { ctx->bounce = nullptr; return PVF_OK; }
    const StagingLayout l = staging_layout_max(&ctx->shape);
    if (bytes < l.total - l.seg_off) return PVF_ERR_WORKSPACE;
    ctx->bounce = (uint8_t *)pinned_host;
    return PVF_OK;
}

int pvf_attach_host_staging(pvf_ctx *ctx, void *staging, size_t bytes)
{
    if (!ctx) return PVF_ERR_INVALID;
    if (!staging) { ctx->staging = nullptr; ctx->staging_bytes = 0; return PVF_OK; }
    if (((uintptr_t)staging & 255) != 0 || bytes < staging_layout_max(&ctx->shape).total) return PVF_ERR_WORKSPACE;
    ctx->staging = (uint8_t *)staging;
    ctx->staging_bytes = bytes;
    ctx->host_rows = 0;
    ctx->host_seqs = 0;
    return PVF_OK;
}

int pvf_draft_step_host(pvf_ctx *ctx, const pvf_params *params, const void *hidden_host, int32_t M, int32_t n_seq,
                        const int32_t *seg_off_host, const int32_t *row_pos_host, const uint8_t *active_host,
                        int32_t *tok_host, float *conf_host, float *ent_host, uint8_t *in_plan_host,
                        uint8_t *commit_host, int32_t *draft_rows_host, int32_t *n_drafts_host, uint8_t *route_host,
                        int32_t *rem_rows_host, int32_t *rem_off_host, int32_t *v_off_host, void *stream)
{
    if (!ctx || !params || M < 0 || n_seq < 0 || M > ctx->shape.max_rows || n_seq > ctx->shape.max_seqs ||
        params->budget < 0 || params->budget > ctx->shape.max_budget)
        return PVF_ERR_INVALID;
    if (!ctx->staging) return PVF_ERR_WORKSPACE;
    if (M == 0 || n_seq == 0) { ctx->host_rows = 0; ctx->host_seqs = 0; return (M == 0) ? PVF_OK : PVF_ERR_INVALID; }
    if (!hidden_host || !seg_off_host || !row_pos_host) return PVF_ERR_INVALID;
    const StagingLayout l = staging_layout(&ctx->shape, (size_t)M, (size_t)n_seq, (size_t)params->budget, 0);
    uint8_t *g = ctx->staging;
    // the bounce buffer mirrors the device staging from seg_off on
    uint8_t *hb = ctx->bounce ? (uint8_t *)((uintptr_t)ctx->bounce - l.seg_off) : nullptr;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t K = (size_t)params->budget;
    const uint8_t *active_dev = active_host ? g + l.active : nullptr;
    if (!h2d(g + l.hidden, hidden_host, (size_t)M * ctx->shape.hidden * 2, s)) return PVF_ERR_CUDA;
    if (hb) {
        put(hb, l.seg_off, seg_off_host, ((size_t)n_seq + 1) * 4);
        put(hb, l.row_pos, row_pos_host, (size_t)M * 4);
        put(hb, l.active, active_host, (size_t)M);
        if (!h2d(g + l.seg_off, hb + l.seg_off, l.in_end - l.seg_off, s)) return PVF_ERR_CUDA;
    } else if (!h2d(g + l.seg_off, seg_off_host, ((size_t)n_seq + 1) * 4, s) ||
               !h2d(g + l.row_pos, row_pos_host, (size_t)M * 4, s) ||
               (active_host && !h2d(g + l.active, active_host, (size_t)M, s)))
        return PVF_ERR_CUDA;
    int rc = pvf_draft_step(ctx, params, g + l.hidden, M, n_seq, (const int32_t *)(g + l.seg_off), (const int32_t *)(g + l.row_pos),
                            active_dev, (int32_t *)(g + l.tok), (float *)(g + l.conf), (float *)(g + l.ent), g + l.in_plan,
                            g + l.commit, (int32_t *)(g + l.n_commit), nullptr, 0, (int32_t *)(g + l.draft_rows),
                            (int32_t *)(g + l.n_drafts), g + l.route, (int32_t *)(g + l.rem_rows), (int32_t *)(g + l.rem_off),
                            (int32_t *)(g + l.v_off), stream);
    if (rc != PVF_OK) return rc;
    if (hb) {
        if (!d2h(hb + l.tok, g + l.tok, l.draft_end - l.tok, s) || cudaStreamSynchronize(s) != cudaSuccess) return PVF_ERR_CUDA;
        get(tok_host, hb, l.tok, (size_t)M * 4);
        get(conf_host, hb, l.conf, (size_t)M * 4);
        get(ent_host, hb, l.ent, (size_t)M * 4);
        get(in_plan_host, hb, l.in_plan, (size_t)M);
        get(commit_host, hb, l.commit, (size_t)M);
        get(draft_rows_host, hb, l.draft_rows, (size_t)n_seq * K * 4);
        get(n_drafts_host, hb, l.n_drafts, (size_t)n_seq * 4);
        get(route_host, hb, l.route, (size_t)n_seq);
        get(rem_rows_host, hb, l.rem_rows, (size_t)M * 4);
        get(rem_off_host, hb, l.rem_off, ((size_t)n_seq + 1) * 4);
        get(v_off_host, hb, l.v_off, ((size_t)n_seq + 1) * 4);
    } else {
        const bool ok = d2h(tok_host, g + l.tok, (size_t)M * 4, s) && d2h(conf_host, g + l.conf, (size_t)M * 4, s) &&
                        d2h(ent_host, g + l.ent, (size_t)M * 4, s) && d2h(in_plan_host, g + l.in_plan, (size_t)M, s) &&
                        d2h(commit_host, g + l.commit, (size_t)M, s) &&
                        d2h(draft_rows_host, g + l.draft_rows, (size_t)n_seq * K * 4, s) &&
                        d2h(n_drafts_host, g + l.n_drafts, (size_t)n_seq * 4, s) && d2h(route_host, g + l.route, (size_t)n_seq, s) &&
                        d2h(rem_rows_host, g + l.rem_rows, (size_t)M * 4, s) &&
                        d2h(rem_off_host, g + l.rem_off, ((size_t)n_seq + 1) * 4, s) &&
                        d2h(v_off_host, g + l.v_off, ((size_t)n_seq + 1) * 4, s);
        if (!ok || cudaStreamSynchronize(s) != cudaSuccess) return PVF_ERR_CUDA;
    }
    ctx->host_rows = M;
    ctx->host_seqs = n_seq;
    ctx->host_budget = params->budget;
    ctx->host_active = active_host != nullptr;
    return PVF_OK;
}

int pvf_verify_step_host(pvf_ctx *ctx, const pvf_params *params, const void *hidden_v_host, int32_t Mv,
                         int32_t *tok_v_host, float *conf_v_host, uint8_t *accept_host, int32_t *choice_host,
                         uint8_t *final_commit_host, void *stream)
{
    if (!ctx || !params || Mv < 0 || Mv > ctx->shape.max_rows) return PVF_ERR_INVALID;
    if (!ctx->staging) return PVF_ERR_WORKSPACE;
    const int32_t M = ctx->host_rows, n_seq = ctx->host_seqs;
    if (M <= 0 || n_seq <= 0 || params->budget != ctx->host_budget) return PVF_ERR_INVALID;   // no draft half to continue
    if (Mv > 0 && !hidden_v_host) return PVF_ERR_INVALID;
    const StagingLayout l = staging_layout(&ctx->shape, (size_t)M, (size_t)n_seq, (size_t)params->budget, (size_t)Mv);
    uint8_t *g = ctx->staging;
    uint8_t *hb = ctx->bounce ? (uint8_t *)((uintptr_t)ctx->bounce - l.seg_off) : nullptr;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t K = (size_t)params->budget;
    if (!h2d(g + l.hidden, hidden_v_host, (size_t)Mv * ctx->shape.hidden * 2, s)) return PVF_ERR_CUDA;
    int rc = pvf_verify_step(ctx, params, g + l.hidden, Mv, M, n_seq, (const int32_t *)(g + l.seg_off),
                             (const int32_t *)(g + l.row_pos), (const int32_t *)(g + l.rem_rows), (const int32_t *)(g + l.rem_off),
                             (const int32_t *)(g + l.v_off), (const int32_t *)(g + l.draft_rows), (const int32_t *)(g + l.n_drafts),
                             g + l.route, (const int32_t *)(g + l.tok), g + l.commit, (int32_t *)(g + l.tok_v),
                             (float *)(g + l.conf_v), nullptr, g + l.accept, (int32_t *)(g + l.choice), g + l.final_commit,
                             nullptr, 0, stream);
    if (rc != PVF_OK) return rc;
    if (hb) {
        if (!d2h(hb + l.accept, g + l.accept, l.total - l.accept, s) || cudaStreamSynchronize(s) != cudaSuccess) return PVF_ERR_CUDA;
        get(accept_host, hb, l.accept, (size_t)n_seq * K);
        get(choice_host, hb, l.choice, (size_t)n_seq * 4);
        get(final_commit_host, hb, l.final_commit, (size_t)M);
        get(tok_v_host, hb, l.tok_v, (size_t)Mv * 4);
        get(conf_v_host, hb, l.conf_v, (size_t)Mv * 4);
    } else {
        const bool ok = d2h(tok_v_host, g + l.tok_v, (size_t)Mv * 4, s) && d2h(conf_v_host, g + l.conf_v, (size_t)Mv * 4, s) &&
                        d2h(accept_host, g + l.accept, (size_t)n_seq * K, s) && d2h(choice_host, g + l.choice, (size_t)n_seq * 4, s) &&
                        d2h(final_commit_host, g + l.final_commit, (size_t)M, s);
        if (!ok || cudaStreamSynchronize(s) != cudaSuccess) return PVF_ERR_CUDA;
    }
    return PVF_OK;
}

}  // extern "C"
