/*
 * pvf.h -- C interface of the B200 (sm_100a) Plan-Verify-Fill vocabulary pass.
 *
 * One decode step of PVF (Algorithm 1 of the paper) as four device-side calls:
 *
 *   pvf_score          hidden states of the masked positions -> top-1 token, confidence, entropy,
 *                      planning-vocabulary membership (LM-head GEMM fused with a streaming softmax;
 *                      logits never reach global memory)
 *   pvf_commit         confidence-threshold base set S_base and base branch z_base
 *   pvf_select_drafts  planning candidates P_t^plan -> top-K drafts, else the AR fallback list
 *   pvf_verify         impact-set acceptance A_t^j, branch choice by C_total, AR k*, final commit
 *
 * and, around the step:
 *
 *   pvf_working_set        rows of the next step from the canvas (block order, early cross-block revelation)
 *   pvf_explore_commit     the appendix's Random / Planning exploration variants
 *   pvf_calib_accumulate, pvf_calib_filter, pvf_set_plan_bitmap
 *                          offline construction of the planning-token vocabulary
 *   pvf_commit_select      pvf_commit + pvf_select_drafts in one launch
 *   pvf_draft_step, pvf_verify_step                the step as two calls of two launches each, device buffers
 *   pvf_draft_step_host, pvf_verify_step_host      the same with host buffers
 *   pvf_score_static       scoring without a context, for callers that must not allocate
 *
 * Conventions common to all calls
 *   - Every data pointer is a DEVICE pointer owned by the caller unless it is marked "host".  The
 *     library never frees caller memory and keeps no pointer beyond a call, except the LM-head
 *     weight and the workspace handed to pvf_create, which must outlive the context.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = the legacy default
 *     stream); they never synchronise and never read device results on the host.
 *   - Return value: PVF_OK or a negative PVF_ERR_* code.  On an argument error nothing is launched.
 *     Nothing is printed, thrown or aborted.
 *   - Kernels bound every internal wait; a wait that runs out stores PVF_ERR_TIMEOUT in the
 *     context's device status word (read it with pvf_last_status after synchronising).
 *   - Token ids, positions and row indices are int32; masks and flags uint8 (0/1); confidences and
 *     entropies float32; hidden states and weights bf16 (the usual 16-bit layout), row-major.
 *   - Rows.  The M scored rows ("masked positions") are grouped by sequence: rows of sequence b are
 *     seg_off[b] .. seg_off[b+1]-1 (seg_off has n_seq+1 entries, seg_off[0] = 0, seg_off[n_seq] = M),
 *     sorted by ascending canvas position row_pos[m].  active[m] != 0 says the position belongs to the
 *     working block B_t (NULL = every row is active).  M = 0 and n_seq = 0 are valid no-ops.
 *   - Calls on one context share its workspace: they must not overlap on the GPU (use one stream, or
 *     order them with events).  Different contexts are independent.
 *   - There is no CPU fallback: every call needs a device of compute capability 10.0.
 */
#ifndef PVF_H_
#define PVF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pvf_ctx pvf_ctx;

enum {
    PVF_OK = 0,
    PVF_ERR_INVALID = -1,     /* NULL required pointer, negative size, size above the context's limits */
    PVF_ERR_ALIGN = -2,       /* weight / hidden pointer not 16-byte aligned, hidden size not a multiple of 8 */
    PVF_ERR_UNSUPPORTED = -3, /* device is not sm_100, or a shape outside what the kernels handle */
    PVF_ERR_CUDA = -4,        /* a CUDA runtime or driver call failed */
    PVF_ERR_TIMEOUT = -5,     /* (status word only) a bounded wait inside a kernel ran out */
    PVF_ERR_WORKSPACE = -6,   /* workspace too small or not 256-byte aligned */
    PVF_ERR_TOO_LARGE = -7    /* pvf_score_static only: more rows than its built-in scratch array holds */
};

/* Limits of a context.  max_rows bounds M of every call, max_seqs bounds n_seq, max_budget bounds K. */
typedef struct {
    int32_t vocab;      /* V: rows of the LM-head weight */
    int32_t hidden;     /* D: multiple of 8 */
    int32_t max_rows;
    int32_t max_seqs;
    int32_t max_budget;
} pvf_shape;

#define PVF_FORCE_PROGRESS            1u  /* a sequence with active rows but an empty base set commits its
                                             single most confident active row (lowest position on ties) */
#define PVF_EXCLUDE_SELF_FROM_IMPACT  2u  /* leave draft j's own position out of the impact set of branch j */
#define PVF_SELECT_ANY_TOKEN          4u  /* pvf_select_drafts: drop the "top-1 token in P^plan" condition */
#define PVF_NO_AR_FALLBACK            8u  /* pvf_select_drafts: no AR route when there is no planning candidate.
                                             Both together, with the band set to the calibration band, select the
                                             calibration candidates C_t^cal (Appendix, planning-token set
                                             construction), at most `budget` per sequence, most confident first */

/* Thresholds of the step.  Names follow the paper: tau_high (Section 2), the planning band
 * [tau_plan_lo, tau_plan_hi) (Section 4.1), tau_ar_lo (Section 4.3), budget = K drafts per sequence. */
typedef struct {
    float    tau_high;
    float    tau_plan_lo;
    float    tau_plan_hi;
    float    tau_ar_lo;
    int32_t  budget;
    uint32_t flags;
} pvf_params;

/* The paper's printed defaults: tau_high = 0.9, K = 3 (Section 5.1); planning band (0.2, 0.65) and
 * tau_AR^l = 0.1 (Table 5, GSM8K / MMLU-Pro rows); flags = 0. */
void pvf_default_params(pvf_params *out);

const char *pvf_strerror(int code);

/* Bytes of device workspace a context of this shape needs (0 on an invalid shape).  Needs a
 * current CUDA device (the layout depends on its SM count). */
size_t pvf_workspace_bytes(const pvf_shape *shape);

/*
 * Create a context.
 *   w_head          device, bf16 [vocab][hidden] row-major, 16-byte aligned: the LM head.  Kept, and treated as
 *                   constant until pvf_destroy: the scoring kernels start reading it before the work queued
 *                   ahead of them on their stream has completed.  To change the weights, synchronise the
 *                   streams that use the context first, then write them (or create a new context).
 *   plan_ids_host   HOST, n_plan token ids of the planning vocabulary P^plan (Section 3; any order,
 *                   duplicates allowed, each in [0, vocab)).  Copied into a device bitmap during the
 *                   call (this call synchronises the device once).
 *   workspace       device, >= pvf_workspace_bytes(shape) bytes, 256-byte aligned.  Kept.
 * The context belongs to the CUDA device that is current during the call.
 */
int pvf_create(pvf_ctx **out, const pvf_shape *shape, const void *w_head,
               const int32_t *plan_ids_host, int32_t n_plan, void *workspace, size_t workspace_bytes);
int pvf_destroy(pvf_ctx *ctx);

/* Copies the device status word to *status (PVF_OK or PVF_ERR_TIMEOUT) and clears it.  Synchronises the whole
 * device first (cudaDeviceSynchronize: streams created non-blocking included).  Results of a call that timed
 * out are undefined. */
int pvf_last_status(pvf_ctx *ctx, int32_t *status);

/*
 * Launch geometry pvf_score would use for M rows; any pointer may be NULL.
 *   ctas        thread blocks of the projection kernel      splits   vocabulary ranges per row tile
 *   waves       passes over the weight matrix               launches kernels launched per call (the projection
 *                                                                    kernel and the merge of the ranges' states)
 */
int pvf_score_plan(pvf_ctx *ctx, int32_t M, int32_t *ctas, int32_t *splits, int32_t *waves, int32_t *launches);

/* The same plan from shapes alone (no context, no device): n_sm = number of SMs to plan for.  `kernel` (may be
 * NULL) receives 0 for the streaming kernel, 1 for the 128-row GEMM kernel, 2 for the paired kernel, 3 for the paired
 * kernel with swapped operands; `row_tiles` the number of row tiles (256 rows in the paired kernel, one tile of up
 * to 512 rows in the swapped paired kernel, else 128) and `tiles_per_wave` how many are in flight.  For kernels 2
 * and 3 `splits` counts pairs of thread blocks.  The paired kernel's last wave may hold fewer tiles than the others
 * and split each over more pairs: `last_wave_tiles` (0: every wave is full) and `last_wave_splits`. */
int pvf_score_plan_for_shape(int32_t vocab, int32_t hidden, int32_t n_sm, int32_t M, int32_t *ctas, int32_t *splits,
                             int32_t *waves, int32_t *kernel, int32_t *row_tiles, int32_t *tiles_per_wave,
                             int32_t *last_wave_tiles, int32_t *last_wave_splits);

/* Name of the projection kernel pvf_score launches for M rows (for profiler filters and reports):
 * "pvf_score_stream_kernel" up to 32 rows (vocabulary on the accumulator lanes, rows on its columns),
 * "pvf_score_swap_pair_kernel" for 33 .. 64, 129 .. 192 and 257 .. 448 rows (the same layout, two thread blocks per
 * vocabulary tile), "pvf_score_gemm_kernel" for 65 .. 128 rows and "pvf_score_gemm_pair_kernel" otherwise (rows on the
 * lanes).
 * NULL on an invalid argument. */
const char *pvf_score_kernel_name(pvf_ctx *ctx, int32_t M);

/*
 * Timing hook for benchmarks.  While both events (cudaEvent_t passed as void*) are non-NULL, every
 * pvf_score call records `start` immediately before and `stop` immediately after its GEMM kernel on
 * the call's stream, so the kernel can be timed alone inside a longer step.  NULL, NULL switches it
 * off (the default).  The events stay owned by the caller.
 */
int pvf_set_score_events(pvf_ctx *ctx, void *start, void *stop);

/*
 * SM clock of the projection launches, measured on the device.  Every projection kernel's first block adds its own
 * run time (nanoseconds) and SM cycle count to sums kept in the workspace; this call synchronises the device, returns
 * the averages since the last call and clears the sums.  pass 0 = pvf_score and pvf_draft_step, 1 = pvf_verify_step.
 *   ms        mean run time of the first block (close to the kernel's duration)       (may be NULL)
 *   sm_mhz    cycles / time: the clock the launches really ran at under the power cap  (may be NULL)
 *   launches  launches counted                                                          (may be NULL)
 * ms * sm_mhz * 1000 = SM cycles per launch: what separates a kernel's efficiency from the clock it was given.
 */
int pvf_score_clock(pvf_ctx *ctx, int32_t pass, double *ms, double *sm_mhz, int64_t *launches);

/*
 * pvf_score -- the vocabulary pass of one forward (Section 2 "confidence-based parallel decoding";
 * Section 3, definitions of y^_t^i, p_t^i and H_i; Section 4.1, "y^ in P^plan").
 *
 *   hidden   [M][hidden] bf16, 16-byte aligned: final hidden state of each scored position.
 * For each row m with logits x_v = sum_k hidden[m][k] * w_head[v][k] (bf16 products, fp32 accumulation)
 * and q = softmax(x):
 *   tok[m]     = argmax_v x_v, the lowest id on ties            conf[m] = q[tok[m]]
 *   ent[m]     = -sum_v q_v ln q_v  (nats)                      in_plan[m] = tok[m] in P^plan
 * ent and in_plan may be NULL.  Non-finite hidden values leave that row's outputs unspecified;
 * the call still terminates and stays in bounds.
 */
int pvf_score(pvf_ctx *ctx, const void *hidden, int32_t M,
              int32_t *tok, float *conf, float *ent, uint8_t *in_plan, void *stream);

/*
 * pvf_commit -- base set and base branch (Section 2, threshold rule; Section 3, S_base and z_base).
 *   commit[m]   = active[m] && conf[m] >= tau_high     (plus the forced row, see PVF_FORCE_PROGRESS)
 *   n_commit[b] = committed rows of sequence b                                   (may be NULL)
 *   y           canvas [n_seq][L] in/out or NULL: y[b][row_pos[m]] = tok[m] at committed rows, every
 *               other entry untouched (committed positions are never re-masked).
 */
int pvf_commit(pvf_ctx *ctx, const pvf_params *params, int32_t M, int32_t n_seq,
               const int32_t *seg_off, const int32_t *row_pos, const uint8_t *active,
               const int32_t *tok, const float *conf,
               uint8_t *commit, int32_t *n_commit, int32_t *y, int32_t L, void *stream);

/*
 * pvf_select_drafts -- draft proposal (Section 4.1 planning candidates and TopK; Section 4.3 AR
 * candidate construction; Algorithm 1, route switch).
 * Per sequence b, with R_b = its rows that are active and not in `commit`, in position order:
 *   planning candidates = rows of R_b with in_plan != 0 and tau_plan_lo <= conf < tau_plan_hi
 *     (in_plan is ignored, and may be NULL, under PVF_SELECT_ANY_TOKEN);
 *   if there are any (and budget > 0): the K_t = min(budget, count) most confident, ties to the lower
 *     position, written in rank order; route = 1.
 *   otherwise: the first <= budget rows of R_b with conf >= tau_ar_lo, in position order; route = 2,
 *     or route = 0 when there is none (always route = 0 under PVF_NO_AR_FALLBACK).
 * Outputs
 *   draft_rows [n_seq][budget]  row indices, -1 padded         n_drafts [n_seq]
 *   route      [n_seq]          0 none, 1 planning, 2 AR
 *   rem_rows   [<= M]           R_b of every sequence, concatenated   rem_off [n_seq+1]
 *   v_off      [n_seq+1]        row offsets of the verification pass: sequence b owns
 *                               (1 + n_drafts[b]) * |R_b| rows if it has drafts, else none.
 */
int pvf_select_drafts(pvf_ctx *ctx, const pvf_params *params, int32_t M, int32_t n_seq,
                      const int32_t *seg_off, const int32_t *row_pos, const uint8_t *active,
                      const int32_t *tok, const float *conf, const uint8_t *in_plan,
                      const uint8_t *commit,
                      int32_t *draft_rows, int32_t *n_drafts, uint8_t *route,
                      int32_t *rem_rows, int32_t *rem_off, int32_t *v_off, void *stream);

/*
 * pvf_commit_select -- pvf_commit followed by pvf_select_drafts in ONE launch (Sections 2, 3, 4.1 and 4.3 as
 * in those two calls; arguments, outputs and results are theirs, bit for bit).  One thread block per sequence
 * takes the base set and then proposes the drafts from it.
 */
int pvf_commit_select(pvf_ctx *ctx, const pvf_params *params, int32_t M, int32_t n_seq,
                      const int32_t *seg_off, const int32_t *row_pos, const uint8_t *active,
                      const int32_t *tok, const float *conf, const uint8_t *in_plan,
                      uint8_t *commit, int32_t *n_commit, int32_t *y, int32_t L,
                      int32_t *draft_rows, int32_t *n_drafts, uint8_t *route,
                      int32_t *rem_rows, int32_t *rem_off, int32_t *v_off, void *stream);

/*
 * pvf_verify -- acceptance check and final commit (Eq. 1 impact set, Eq. 3 verified compatibility,
 * Section 4.2 Filter 1 and Filter 2, Section 4.3 AR verification and selection).
 *   tok_v, conf_v   pvf_score outputs of the verification pass, rows [b][c][r]: index
 *                   v_off[b] + c * |R_b| + r; c = 0 is the base branch, c = j the branch that adds draft
 *                   j (planning) or the first j fills (AR); r indexes rem_rows of sequence b.
 *   tok             tokens of the draft pass (the drafted tokens).
 * Planning route: S_impact = {r : conf_v[base][r] >= tau_high}; accept[b][j-1] = S_impact non-empty and
 *   tok_v[j][r] == tok_v[base][r] on all of it; C_j = sum over r != draft j of conf_v[j][r] (fp64, in row
 *   order); choice[b] = the accepted j with the largest C_j (lowest j on ties), 0 if none.
 * AR route: accept[b][k-1] = for all r <= k: tok_v[k][row of fill r] == tok[fill r];
 *   choice[b] = largest accepted k, 0 if none.
 * final_commit = commit, plus draft `choice` (planning) or fills 1..choice (AR).  y as in pvf_commit,
 * written at every final_commit row.  accept entries beyond n_drafts[b] are 0.  tok_v, conf_v and
 * rem_rows are only read for sequences that have drafts (they may be NULL when v_off[n_seq] = 0).
 */
int pvf_verify(pvf_ctx *ctx, const pvf_params *params, int32_t M, int32_t n_seq,
               const int32_t *seg_off, const int32_t *row_pos,
               const int32_t *rem_rows, const int32_t *rem_off, const int32_t *v_off,
               const int32_t *draft_rows, const int32_t *n_drafts, const uint8_t *route,
               const int32_t *tok, const int32_t *tok_v, const float *conf_v, const uint8_t *commit,
               uint8_t *accept, int32_t *choice, uint8_t *final_commit,
               int32_t *y, int32_t L, void *stream);

/*
 * One decoding iteration of Algorithm 1 as two calls around the model's verification forward, on device
 * buffers, two kernel launches each: the projection kernel of pvf_score, and one kernel that first merges the
 * projection's per-vocabulary-range softmax states (what pvf_score's own small second kernel does) and then
 * takes the decisions -- results equal to the calls they combine, bit for bit.
 *   pvf_draft_step    = pvf_score(hidden) + pvf_commit + pvf_select_drafts: scores of the draft pass (tok, conf,
 *                     in_plan [M]; ent [M] or NULL), base set, drafts, and the row layout (rem_rows, rem_off,
 *                     v_off) of the verification pass.  seg_off[n_seq] must equal M: every scored row belongs
 *                     to a sequence (the rows are merged sequence by sequence).
 *   pvf_verify_step   = pvf_score(hidden_v) + pvf_verify: scores of the verification rows (tok_v, conf_v [Mv];
 *                     ent_v [Mv] or NULL), acceptance, branch choice, final commit.  Mv must equal the draft
 *                     half's v_off[n_seq] (a device value the caller reads back to size the forward pass).
 * Other arguments as in the calls they combine; asynchronous on `stream` like them.
 */
int pvf_draft_step(pvf_ctx *ctx, const pvf_params *params, const void *hidden, int32_t M, int32_t n_seq,
                   const int32_t *seg_off, const int32_t *row_pos, const uint8_t *active,
                   int32_t *tok, float *conf, float *ent, uint8_t *in_plan,
                   uint8_t *commit, int32_t *n_commit, int32_t *y, int32_t L,
                   int32_t *draft_rows, int32_t *n_drafts, uint8_t *route,
                   int32_t *rem_rows, int32_t *rem_off, int32_t *v_off, void *stream);
int pvf_verify_step(pvf_ctx *ctx, const pvf_params *params, const void *hidden_v, int32_t Mv, int32_t M, int32_t n_seq,
                    const int32_t *seg_off, const int32_t *row_pos,
                    const int32_t *rem_rows, const int32_t *rem_off, const int32_t *v_off,
                    const int32_t *draft_rows, const int32_t *n_drafts, const uint8_t *route,
                    const int32_t *tok, const uint8_t *commit,
                    int32_t *tok_v, float *conf_v, float *ent_v,
                    uint8_t *accept, int32_t *choice, uint8_t *final_commit, int32_t *y, int32_t L, void *stream);

/*
 * pvf_explore_commit -- the exploration variants of the appendix ("Planning tokens beyond high-confidence
 * decoding", the Random / Planning ablation): after pvf_commit, every sequence commits exactly one more token
 * from the CLOSED confidence bin [tau_plan_lo, tau_plan_hi] (no verification pass).
 *   eligible rows: active, not in `commit`, tau_plan_lo <= conf <= tau_plan_hi
 *   PVF_EXPLORE_RANDOM    one eligible row, drawn uniformly
 *   PVF_EXPLORE_PLANNING  one eligible row whose top-1 token is in P^plan (in_plan != 0), drawn uniformly;
 *                         the Random rule when there is none
 *   u [n_seq]             the draws: u[b] in [0, 1) picks row floor(u[b] * n) of the n rows of the chosen set in
 *                         position order (fp32 product, clamped to n - 1); the caller owns the random numbers
 * commit is updated in place (the chosen row set to 1), explore_row[b] receives the row or -1 when the bin is
 * empty, y as in pvf_commit.  The Static baseline of the paper's tables (one most confident token per step)
 * is pvf_commit with tau_high above 1 and PVF_FORCE_PROGRESS.
 */
#define PVF_EXPLORE_RANDOM   0
#define PVF_EXPLORE_PLANNING 1
int pvf_explore_commit(pvf_ctx *ctx, const pvf_params *params, int32_t mode, int32_t M, int32_t n_seq,
                       const int32_t *seg_off, const int32_t *row_pos, const uint8_t *active,
                       const int32_t *tok, const float *conf, const uint8_t *in_plan,
                       const float *u, uint8_t *commit, int32_t *explore_row, int32_t *y, int32_t L,
                       void *stream);

/*
 * Offline construction of the planning-token vocabulary (Section 3, "Verified information gain" and
 * "Planning-token vocabulary"; Appendix, "Planning Token Set Construction").
 *
 * A calibration step is a decode step on the calibration data with candidates chosen by
 * pvf_select_drafts under PVF_SELECT_ANY_TOKEN | PVF_NO_AR_FALLBACK and the band [tau_cal_lo, tau_cal_hi):
 * pvf_score (with entropies) on the verification pass, pvf_verify for the acceptance A_j, then
 *
 * pvf_calib_accumulate -- one event per candidate j of every sequence on the planning route, for the
 * token v = tok[draft row j]:
 *     dH_j  = mean over the remaining rows r != draft j of  ent_v[base][r] - ent_v[j][r]   (0 if there is none)
 *     VIG_j = accept[b][j] * dH_j
 *     n_v[v] += 1;   m_v[v] += (S_impact non-empty);   sum_a[v] += accept[b][j];
 *     sum_vig_q32[v] += round(VIG_j * 2^32)      (integer sums: independent of the order of accumulation)
 *   conf_v, ent_v   pvf_score outputs of the verification pass, rows as in pvf_verify
 *   accept          pvf_verify's output for the same step
 *   n_v, m_v, sum_a [vocab] int32 and sum_vig_q32 [vocab] int64: caller-owned, zeroed by the caller before the
 *                   first step, accumulated across steps
 *   vig_out         [n_seq][budget] VIG_j of this step (0 beyond n_drafts), or NULL
 *
 * pvf_calib_filter -- the filtering rule: bit v of plan_bitmap (ceil(vocab/32) words, fully overwritten) is set
 * iff n_v >= n_min, m_v >= m_min, sum_a/m_v >= rho_ver (0 when m_v = 0) and (sum_vig_q32 / 2^32)/n_v >= gamma_vig;
 * *n_plan (may be NULL) receives the number of kept tokens.
 *
 * pvf_set_plan_bitmap -- makes such a device bitmap the context's planning vocabulary P^plan (device-to-device
 * copy on `stream`).
 *
 * pvf_default_calib_params: the paper's printed calibration band [0.15, 0.25) and thresholds n_min = 50,
 * m_min = 20, rho_ver = 0.9, gamma_vig = 0.03.
 */
typedef struct {
    float   tau_cal_lo, tau_cal_hi;
    int32_t n_min, m_min;
    float   rho_ver, gamma_vig;
} pvf_calib_params;
void pvf_default_calib_params(pvf_calib_params *out);
int pvf_calib_accumulate(pvf_ctx *ctx, const pvf_params *params, int32_t n_seq,
                         const int32_t *rem_rows, const int32_t *rem_off, const int32_t *v_off,
                         const int32_t *draft_rows, const int32_t *n_drafts, const uint8_t *route,
                         const int32_t *tok, const float *conf_v, const float *ent_v, const uint8_t *accept,
                         int32_t *n_v, int32_t *m_v, int32_t *sum_a, int64_t *sum_vig_q32, double *vig_out,
                         void *stream);
int pvf_calib_filter(pvf_ctx *ctx, const pvf_calib_params *cal, const int32_t *n_v, const int32_t *m_v,
                     const int32_t *sum_a, const int64_t *sum_vig_q32, uint32_t *plan_bitmap, int32_t *n_plan,
                     void *stream);
int pvf_set_plan_bitmap(pvf_ctx *ctx, const uint32_t *plan_bitmap, void *stream);

/*
 * pvf_working_set -- the rows of the next step, from the canvas (Appendix A.1, semi-autoregressive block
 * order; Appendix "Planning-Guided Early Cross-Block Revelation", Eq. 4).
 *   y          [n_seq][L] canvas, mask_id marks a masked position; block = S tokens per block (the last
 *              block is shorter when S does not divide L).
 * Per sequence: k_t = the first block that holds a mask, M_active = its masked positions; the working index
 * set B_t is M_active, plus the whole index range of block k_t + 1 when |M_active| <= n_sparse (N_s) and
 * that block exists.  The rows are the masked positions of B_t, ascending; n_sparse = 0 is strict block order.
 * Outputs
 *   seg_off   [n_seq+1]   row offsets per sequence; seg_off[n_seq] = M, the number of rows (read it back to
 *                         size the forward pass and the pvf_score call)
 *   row_pos   [M]         canvas position of each row          row_seq [M]  its sequence       (may be NULL)
 *   active    [M]         1 for every row written (all of them lie in B_t)                     (may be NULL)
 *   expanded  [n_seq]     1 where the next block was revealed                                  (may be NULL)
 * rows_capacity = entries available in row_pos / row_seq / active; at least n_seq * min(2 * block, L), else
 * PVF_ERR_INVALID and nothing is launched.  A finished sequence owns no rows.
 */
int pvf_working_set(pvf_ctx *ctx, const int32_t *y, int32_t n_seq, int32_t L, int32_t block,
                    int32_t n_sparse, int32_t mask_id, int32_t *seg_off, int32_t *row_pos,
                    int32_t *row_seq, uint8_t *active, uint8_t *expanded, int32_t rows_capacity,
                    void *stream);

/*
 * Host-buffer variants of the step (Algorithm 1, one decoding iteration split at the model's
 * verification forward).  Every array argument is a HOST pointer (pinned memory makes the copies
 * asynchronous); the library copies inputs into a device staging buffer, runs the device entry points
 * above on `stream`, copies the results back and synchronises the stream before returning.  Output
 * pointers may be NULL (that result is not copied back).
 *
 *   pvf_host_staging_bytes   bytes of device staging a context of this shape needs (about
 *                            max_rows * (2 * hidden + 40) bytes)
 *   pvf_attach_host_staging  hand the context a 256-byte-aligned device buffer of that size (kept until
 *                            replaced; NULL detaches).  Without it the two calls return PVF_ERR_WORKSPACE.
 *   pvf_host_bounce_bytes    bytes of PINNED HOST memory for the optional bounce buffer of this shape
 *   pvf_attach_host_bounce   hand the context such a buffer (kept until replaced; NULL detaches).  With it, the
 *                            small input arrays travel as one host-to-device copy and all outputs of a call as
 *                            one device-to-host copy into the buffer, from which they are copied to the output
 *                            pointers (which then need not be pinned); without it every array is copied on its own.
 *   pvf_draft_step_host      pvf_draft_step on hidden_host[M][hidden]; outputs as there.  The device copies
 *                            stay in the staging buffer.
 *   pvf_verify_step_host     pvf_verify_step on hidden_v_host[Mv][hidden], continuing the draft
 *                            half most recently run on this context (same budget); Mv must equal that
 *                            half's v_off[n_seq].
 */
size_t pvf_host_staging_bytes(const pvf_shape *shape);
int pvf_attach_host_staging(pvf_ctx *ctx, void *staging, size_t bytes);
size_t pvf_host_bounce_bytes(const pvf_shape *shape);
int pvf_attach_host_bounce(pvf_ctx *ctx, void *pinned_host, size_t bytes);
int pvf_draft_step_host(pvf_ctx *ctx, const pvf_params *params, const void *hidden_host, int32_t M, int32_t n_seq,
                        const int32_t *seg_off_host, const int32_t *row_pos_host, const uint8_t *active_host,
                        int32_t *tok_host, float *conf_host, float *ent_host, uint8_t *in_plan_host,
                        uint8_t *commit_host, int32_t *draft_rows_host, int32_t *n_drafts_host, uint8_t *route_host,
                        int32_t *rem_rows_host, int32_t *rem_off_host, int32_t *v_off_host, void *stream);
int pvf_verify_step_host(pvf_ctx *ctx, const pvf_params *params, const void *hidden_v_host, int32_t Mv,
                         int32_t *tok_v_host, float *conf_v_host, uint8_t *accept_host, int32_t *choice_host,
                         uint8_t *final_commit_host, void *stream);

/*
 * pvf_score_static -- pvf_score for callers that must not allocate.  (The paper has no counterpart: this
 * is a packaging variant of pvf_score: same arithmetic, the same kernels.)
 *
 * Some callers of this library cannot call cudaMalloc at the point where they score: code that runs
 * inside a memory-pool or arena discipline where every device byte is accounted for up front, plugins
 * loaded into a host process that forbids allocation after start-up, and latency-critical serving loops
 * where an allocation (and the implicit device synchronisation it can cause) is not acceptable.  pvf_score
 * asks such callers for a workspace through pvf_create; this entry point needs neither a context nor a
 * workspace.  Its scratch memory -- the per-vocabulary-range softmax states that the projection kernel writes
 * and the merge kernel reads, and a status word -- is a fixed 512.25 KiB array inside the library image.  Every GPU that loads
 * the library holds that array until the process exits, whether or not this function is ever called.
 * (The array holds one state per row and SM.  Where pvf_score would pick the kernel that leaves two, and they
 * do not fit -- more than 221 rows -- this entry point takes the kernel pvf_score uses outside that window:
 * same arithmetic, results equal within the accumulation order.)
 *
 *   w_head       device, bf16 [vocab][hidden_size] row-major, 16-byte aligned; not written by work still queued
 *                on the stream when the call is made (the kernels start reading it before that work is done)
 *   hidden       device, bf16 [M][hidden_size], 16-byte aligned; hidden_size a multiple of 8
 *   M            at most PVF_STATIC_MAX_ROWS; larger M returns PVF_ERR_TOO_LARGE and launches nothing
 *   plan_bitmap  device, ceil(vocab/32) words, bit v set iff token v is in P^plan; may be NULL when
 *                in_plan is NULL
 *   tok, conf, ent, in_plan   outputs as in pvf_score (ent and in_plan may be NULL)
 *
 * The call itself allocates nothing: no cudaMalloc / cudaFree, no allocating library routine; it
 * encodes its tensor maps on the host, clears one status word with cudaMemsetAsync and launches the two
 * scoring kernels on `stream`.  The first call on each device additionally looks up the array's device
 * address and raises the scoring kernels' shared-memory limit (this also makes the CUDA runtime load the
 * kernels); make that first call with the device current and before any stream capture begins.  That set-up
 * is guarded by a lock, so several host threads may make their first calls at the same time.
 *
 * All calls on a device share the one array, and it keeps the last call's contents.  Only the status word
 * has to start from zero and the call clears it; the softmax states are fully rewritten before they are
 * read.  Two calls that overlap on the GPU (different streams without an ordering between them, or two
 * threads) race on the array and give wrong results: serialise them.
 *
 * pvf_score_static_status copies the status word of the current device to *status (PVF_OK or
 * PVF_ERR_TIMEOUT of the most recent call); it synchronises the device.
 */
#define PVF_STATIC_MAX_ROWS 1024
int pvf_score_static(const void *w_head, int32_t vocab, int32_t hidden_size, const void *hidden, int32_t M,
                     const uint32_t *plan_bitmap, int32_t *tok, float *conf, float *ent, uint8_t *in_plan,
                     void *stream);
int pvf_score_static_status(int32_t *status);

#ifdef __cplusplus
}
#endif
#endif /* PVF_H_ */
