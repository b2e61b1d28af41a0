// Context management of libpvf: workspace layout, planning-vocabulary bitmap, status word.
#include <new>
#include <vector>

#include "pvf_internal.h"

namespace {

struct Layout {
    size_t words_off, bitmap_off, seq_tickets_off, partials_off, total;
    size_t bitmap_bytes, seq_tickets_bytes, partials_bytes;
};

bool shape_ok(const pvf_shape *s)
{
    return s && s->vocab > 0 && s->hidden > 0 && s->max_rows >= 0 && s->max_seqs >= 0 &&
           s->max_budget >= 0 && s->max_budget <= PVF_MAX_BUDGET_LIMIT;
}

Layout layout_for(const pvf_shape *s, int n_sm)
{
    Layout l;
    l.words_off = 0;
    l.bitmap_off = pvf_align_up(sizeof(pvf_device_words), 256);
    l.bitmap_bytes = pvf_align_up(((size_t)s->vocab + 31) / 32 * 4, 256);
    l.seq_tickets_off = l.bitmap_off + l.bitmap_bytes;
    l.seq_tickets_bytes = pvf_align_up(((size_t)s->max_seqs + 1) * sizeof(uint32_t), 256);
    l.partials_off = l.seq_tickets_off + l.seq_tickets_bytes;
    l.partials_bytes = pvf_align_up(pvf_score_partials_bytes(s, n_sm), 256);
    l.total = l.partials_off + l.partials_bytes;
    return l;
}

int current_sm_count(int *device, int *n_sm, int *cc_major)
{
    if (cudaGetDevice(device) != cudaSuccess) return PVF_ERR_CUDA;
    if (cudaDeviceGetAttribute(n_sm, cudaDevAttrMultiProcessorCount, *device) != cudaSuccess) return PVF_ERR_CUDA;
    if (cudaDeviceGetAttribute(cc_major, cudaDevAttrComputeCapabilityMajor, *device) != cudaSuccess) return PVF_ERR_CUDA;
    return PVF_OK;
}

}  // namespace

extern "C" {

void pvf_default_params(pvf_params *out)
{
    if (!out) return;
    out->tau_high = 0.9f;
    out->tau_plan_lo = 0.2f;
    out->tau_plan_hi = 0.65f;
    out->tau_ar_lo = 0.1f;
    out->budget = 3;
    out->flags = 0;
}

const char *pvf_strerror(int code)
{
    switch (code) {
        case PVF_OK: return "ok";
        case PVF_ERR_INVALID: return "invalid argument";
        case PVF_ERR_ALIGN: return "pointer or pitch not aligned";
        case PVF_ERR_UNSUPPORTED: return "unsupported device or shape";
        case PVF_ERR_CUDA: return "CUDA call failed";
        case PVF_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
        case PVF_ERR_WORKSPACE: return "workspace too small or misaligned";
        case PVF_ERR_TOO_LARGE: return "more rows than the built-in scratch array of pvf_score_static holds";
        default: return "unknown error";
    }
}

size_t pvf_workspace_bytes(const pvf_shape *shape)
{
    if (!shape_ok(shape)) return 0;
    int device, n_sm, cc;
    if (current_sm_count(&device, &n_sm, &cc) != PVF_OK) return 0;
    return layout_for(shape, n_sm).total;
}

int pvf_create(pvf_ctx **out, const pvf_shape *shape, const void *w_head,
               const int32_t *plan_ids_host, int32_t n_plan, void *workspace, size_t workspace_bytes)
{
    if (!out) return PVF_ERR_INVALID;
    *out = nullptr;
    if (!shape_ok(shape) || !w_head || !workspace || n_plan < 0 || (n_plan > 0 && !plan_ids_host))
        return PVF_ERR_INVALID;
    if (shape->hidden % 8 != 0 || ((uintptr_t)w_head & 15) != 0) return PVF_ERR_ALIGN;
    for (int32_t i = 0; i < n_plan; ++i)
        if (plan_ids_host[i] < 0 || plan_ids_host[i] >= shape->vocab) return PVF_ERR_INVALID;
    int device, n_sm, cc;
    int rc = current_sm_count(&device, &n_sm, &cc);
    if (rc != PVF_OK) return rc;
    if (cc != 10) return PVF_ERR_UNSUPPORTED;
    Layout l = layout_for(shape, n_sm);
    if (((uintptr_t)workspace & 255) != 0 || workspace_bytes < l.total) return PVF_ERR_WORKSPACE;

    pvf_ctx *ctx = new (std::nothrow) pvf_ctx();
    if (!ctx) return PVF_ERR_INVALID;
    ctx->shape = *shape;
    ctx->device = device;
    ctx->n_sm = n_sm;
    ctx->w_head = w_head;
    ctx->workspace = (uint8_t *)workspace;
    ctx->workspace_bytes = workspace_bytes;
    ctx->words = (pvf_device_words *)(ctx->workspace + l.words_off);
    ctx->plan_bitmap = (uint32_t *)(ctx->workspace + l.bitmap_off);
    ctx->seq_tickets = (uint32_t *)(ctx->workspace + l.seq_tickets_off);
    ctx->seq_tickets_bytes = l.seq_tickets_bytes;
    ctx->partials = (float4 *)(ctx->workspace + l.partials_off);
    ctx->partials_bytes = l.partials_bytes;
    ctx->ev_start = nullptr;
    ctx->ev_stop = nullptr;
    ctx->staging = nullptr;
    ctx->staging_bytes = 0;
    ctx->bounce = nullptr;
    ctx->host_rows = ctx->host_seqs = ctx->host_budget = 0;
    ctx->host_active = false;

    std::vector<uint32_t> bitmap(l.bitmap_bytes / 4, 0u);
    for (int32_t i = 0; i < n_plan; ++i) bitmap[plan_ids_host[i] >> 5] |= 1u << (plan_ids_host[i] & 31);
    bool ok = cudaMemset(ctx->words, 0, sizeof(pvf_device_words)) == cudaSuccess &&
              cudaMemset(ctx->seq_tickets, 0, l.seq_tickets_bytes) == cudaSuccess &&
              cudaMemcpy(ctx->plan_bitmap, bitmap.data(), l.bitmap_bytes, cudaMemcpyHostToDevice) == cudaSuccess &&
              cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) { delete ctx; return PVF_ERR_CUDA; }
    rc = pvf_score_init(ctx);
    if (rc != PVF_OK) { delete ctx; return rc; }
    *out = ctx;
    return PVF_OK;
}

int pvf_destroy(pvf_ctx *ctx)
{
    delete ctx;
    return PVF_OK;
}

int pvf_last_status(pvf_ctx *ctx, int32_t *status)
{
    if (!ctx || !status) return PVF_ERR_INVALID;
    int32_t host = 0;
    // Every stream of the device, non-blocking ones included: a copy on the legacy default stream alone would
    // not wait for kernels launched on those.
    if (cudaDeviceSynchronize() != cudaSuccess) return PVF_ERR_CUDA;
    if (cudaMemcpy(&host, &ctx->words->status, sizeof host, cudaMemcpyDeviceToHost) != cudaSuccess) return PVF_ERR_CUDA;
    if (host != 0) {
        // A kernel gave up: clear the word (and the arrival tickets, which count whole blocks and so stay whole).
        if (cudaMemset(&ctx->words->status, 0, sizeof(int32_t)) != cudaSuccess ||
            cudaMemset(&ctx->words->select_ticket, 0, 4 * sizeof(uint32_t)) != cudaSuccess ||
            cudaMemset(ctx->seq_tickets, 0, ctx->seq_tickets_bytes) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess)
            return PVF_ERR_CUDA;
    }
    *status = host;
    return PVF_OK;
}

}  // extern "C"
