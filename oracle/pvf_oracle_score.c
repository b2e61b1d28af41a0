/*
 * CPU oracle for the PVF vocabulary pass -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain fp64 restatement of what one scored row means in the paper:
 *   - the model's distribution at a masked position is softmax over the vocabulary of the
 *     LM-head logits x_v = sum_k h[k] * W[v][k]                      (Section 2, reverse process)
 *   - top prediction   y^ = argmax_v P(y = v)                        (Section 2 / Section 3)
 *   - confidence       p  = P(y = y^) = max_v P(y = v)               (Section 3, definition of p_t^i)
 *   - entropy          H  = -sum_v P(v) ln P(v)   (natural log)      (Section 3, H_i(z))
 *   - eligibility      y^ in P^plan                                  (Section 4.1)
 *
 * It is written as the definition: the whole logit row is materialised, then max, then the
 * normaliser, then the entropy sum.  No streaming, no tiling, no reduced precision.  bf16 inputs
 * are widened exactly to double; the logit is the fp64 dot product of those values.
 * Ties in the argmax go to the lowest vocabulary id (the paper does not say).
 *
 * The only parallelism is an OpenMP loop over vocabulary entries of one row.
 * Nothing here is shared with, or called by, the CUDA library.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_double(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int pvf_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Logits of one row: x[v] = sum_k h[k] * W[v][k], fp64. */
void pvf_oracle_logits_row(const uint16_t *W, const uint16_t *h_bits, int64_t V, int64_t D, double *x)
{
    double *h = (double *)malloc((size_t)D * sizeof(double));
    for (int64_t k = 0; k < D; ++k) h[k] = bf16_to_double(h_bits[k]);
#pragma omp parallel for schedule(static)
    for (int64_t v = 0; v < V; ++v) {
        const uint16_t *w = W + v * D;
        double acc = 0.0;
        for (int64_t k = 0; k < D; ++k) acc += h[k] * bf16_to_double(w[k]);
        x[v] = acc;
    }
    free(h);
}

/*
 * Softmax statistics of one materialised logit row (two passes after the max).
 * gap = largest logit minus the largest logit at any other vocabulary id (0 when the maximum
 * is attained twice); callers use it to list near-tie rows.
 */
void pvf_oracle_row_stats(const double *x, int64_t V, int32_t *tok, double *conf, double *ent, double *gap)
{
    int64_t arg = 0;
    double mx = x[0];
    for (int64_t v = 1; v < V; ++v)
        if (x[v] > mx) { mx = x[v]; arg = v; }          /* strict: lowest id wins ties */
    double second = -INFINITY;
    for (int64_t v = 0; v < V; ++v)
        if (v != arg && x[v] > second) second = x[v];
    double Z = 0.0;
    for (int64_t v = 0; v < V; ++v) Z += exp(x[v] - mx);
    double Hs = 0.0;
    for (int64_t v = 0; v < V; ++v) {
        double q = exp(x[v] - mx) / Z;
        if (q > 0.0) Hs -= q * log(q);
    }
    *tok = (int32_t)arg;
    *conf = 1.0 / Z;                                    /* P(y^) = e^0 / Z */
    *ent = Hs;
    *gap = (V > 1) ? (mx - second) : INFINITY;
}

/*
 * Score M rows.  plan_member[v] != 0 iff v is in the planning vocabulary (may be NULL).
 * logits_out, when not NULL, receives the full [M][V] logit matrix (tiny cases only).
 */
int pvf_oracle_score(const uint16_t *W, const uint16_t *H, int64_t M, int64_t V, int64_t D,
                     const uint8_t *plan_member, int32_t *tok, double *conf, double *ent,
                     double *gap, uint8_t *in_plan, double *logits_out)
{
    if (M < 0 || V <= 0 || D <= 0) return -1;
    double *x = (double *)malloc((size_t)V * sizeof(double));
    if (!x) return -2;
    for (int64_t m = 0; m < M; ++m) {
        pvf_oracle_logits_row(W, H + m * D, V, D, x);
        pvf_oracle_row_stats(x, V, &tok[m], &conf[m], &ent[m], &gap[m]);
        if (in_plan) in_plan[m] = (plan_member && plan_member[tok[m]]) ? 1 : 0;
        if (logits_out) memcpy(logits_out + m * V, x, (size_t)V * sizeof(double));
    }
    free(x);
    return 0;
}
