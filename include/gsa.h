/*
 * gsa.h -- C ABI of the B200 (sm_100a) forward path of Gated Sparse Attention.
 *
 * Three stages and their fusion, named after the paper's notation:
 *   gsa_indexer_scores         gated lightning indexer                     (Eq. 7)
 *   gsa_adaptive_topk          adaptive budget k_t and top-k_t selection   (Eq. 8, Eq. 4)
 *   gsa_sparse_gated_attn_fwd  value gate G2, sparse softmax attention over
 *                              S_t, output gate G1                         (Eq. 9, 11, 12, 10)
 *   gsa_forward                all of the above for a whole batch          (Sec. 3.2, Eq. 6 pipeline)
 * The steps either side of the path and its training side:
 *   gsa_project, gsa_output_projection     the projections that feed / follow the path (text below Eq. 7,
 *                                          Eq. 9, Eq. 10, Sec. 2.1)
 *   gsa_sparse_gated_attn_fwd_lse, gsa_sparse_gated_attn_bwd
 *                                          the attention stage for training and its backward pass
 *   gsa_attn_probs_mean, gsa_indexer_kl_bwd   the indexer's loss and its derivatives (Sec. 5.1, Eq. 13-14)
 *   gsa_vbar_update                        the running mean of the score variance of Eq. 8
 *
 * Conventions common to every call
 *   - Every data pointer is DEVICE memory owned by the caller, 16-byte aligned and
 *     contiguous in the stated layout, unless the argument says "host".
 *   - The library allocates no memory and never synchronises the device (except
 *     gsa_forward_host, gsa_device_status and gsa_select_fallback_rows, which wait for
 *     `stream`).  Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is
 *     the legacy default stream).
 *   - No data is kept between calls.  The only state the library holds is process-wide
 *     and set explicitly: the launch counter, the debug / tuning knobs
 *     (gsa_debug_set_indexer_path, gsa_debug_set_attn_range_keys, gsa_debug_set_wait_limit)
 *     and the profiling hooks (gsa_profile_set_events, gsa_profile_set_timeline).  A knob
 *     changes the launch plan -- and with gsa_debug_set_attn_range_keys the workspace
 *     size -- of every later call on every host thread; set them before the calls they are
 *     meant for, not concurrently with them.
 *   - Return value: GSA_OK or a negative gsa_status.  Argument errors are detected on
 *     the host before anything is launched.  Conditions only the device can see are
 *     recorded in a status word at the start of the workspace; read it with
 *     gsa_device_status: a bounded wait that ran out inside a tensor-core pipeline
 *     (every device-side wait has a limit of about a second; the kernel then stops issuing
 *     work, lets what it issued complete, frees what it holds and returns), or an index
 *     set handed to an attention / backward / loss call with an entry outside [0, Lk) or a
 *     budget outside [0, k_max].  Such an entry never becomes an address: budgets are
 *     clamped, a position used for a gather is clamped into the tensor, an entry that
 *     would be scattered is skipped; the results of that row are then meaningless.
 *   - bf16 tensors are passed as void*; fp32 accumulation everywhere; outputs are
 *     rounded to bf16 once (round to nearest even).
 *   - Query t (0-based, of Lq) may look at keys s = 0 .. Lk-Lq+t ("visible keys",
 *     n_t = Lk-Lq+t+1).  Prefill is Lq == Lk; decode is Lq == 1 over an Lk-token cache.
 *
 * Supported shapes: d_h in {64, 128}; dI in {32, 64}; HI in {1, 2, 4, 8};
 * n_h / n_kv in {1, 2, 4, 8}; n_kv in {1, 2, 4, 8}; k_max <= 4096; 1 <= Lq <= Lk < 2^24.
 */
#ifndef GSA_H_
#define GSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GSA_OK = 0,
    GSA_ERR_INVALID_ARG = -1,      /* NULL / misaligned pointer, inconsistent sizes          */
    GSA_ERR_UNSUPPORTED_SHAPE = -2,/* a shape outside the list above                         */
    GSA_ERR_WORKSPACE = -3,        /* workspace missing or smaller than gsa_workspace_bytes  */
    GSA_ERR_CUDA = -4,             /* a CUDA runtime / driver call failed                    */
    GSA_ERR_DEVICE_TIMEOUT = -5,   /* a bounded device-side wait expired (see device status) */
    GSA_ERR_STATIC_SCRATCH = -6,   /* problem larger than the built-in scratch array of the
                                      allocation-free entry point                            */
    GSA_ERR_INDEX_RANGE = -7       /* a kernel met an index set entry outside [0, Lk) or a budget
                                      outside [0, k_max] (see device status)                 */
} gsa_status;

/* Hyper-parameters (Table 1 of the paper) plus the call's geometry. */
typedef struct gsa_params {
    int32_t B;          /* batch                                                             */
    int32_t Lq, Lk;     /* query positions, key positions per batch element                  */
    int32_t n_h;        /* query heads                                                       */
    int32_t n_kv;       /* key/value heads; head h uses KV head h / (n_h / n_kv)             */
    int32_t d_h;        /* head dimension d_k                                                */
    int32_t HI;         /* indexer heads H^I                                                 */
    int32_t dI;         /* indexer dimension d^I                                             */
    int32_t k_base;     /* base selection budget                                             */
    int32_t k_min;      /* budget bounds, 1 <= k_min <= k_max                                */
    int32_t k_max;
    int32_t k_mode;     /* 0: Eq. 8 as printed, k ~ Var/Vbar.  1: the direction the paper's
                           prose describes, k ~ Vbar/Var (Var = 0 gives k_max).
                           2: fixed k = k_base
                           3: every visible key (needs k_max >= Lk): the dense fallback for
                              short contexts, where the indexer costs more than it saves
                              (Sec. 8); gsa_forward then runs no indexer and no selection
                              (qI, kI, w may be NULL) and the layer is dense gated attention */
    float v_bar;        /* Vbar of Eq. 8: caller-owned running mean of score variance, > 0   */
    float sm_scale;     /* softmax scale of Eq. 11; <= 0 means 1/sqrt(d_h)                   */
    int32_t q_begin;    /* per-stage calls process query rows q_begin <= t < q_end of every  */
    int32_t q_end;      /* batch element; q_end <= 0 means Lq.  gsa_forward ignores both.    */
    int32_t act;        /* indexer activation: 0 = sigmoid (Eq. 7, GSA); 1 = ReLU (Eq. 3, the
                           lightning indexer GSA starts from; scores are then unbounded above) */
} gsa_params_t;

/*
 * Bytes of device workspace gsa_forward (and the per-stage calls) need for `p`.
 * `slab_rows` is the number of query rows whose fp32 score rows gsa_forward keeps
 * resident at a time (0 = library default: about 4 GiB of score rows, at least 32 rows).
 * Host call; writes *bytes.
 */
int gsa_workspace_bytes(const gsa_params_t *p, int32_t slab_rows, size_t *bytes);

/*
 * Gated lightning indexer, Eq. 7:
 *     I[t,s] = sum_j w[t,j] * sigmoid(qI[t,j,:] . kI[s,:] + bI[j]),   s visible to t
 *   (p->act == 1: max(., 0) in place of the sigmoid, Eq. 3).
 *   qI     [B, Lq, HI, dI] bf16        kI  [B, Lk, dI] bf16 (one key shared by all heads)
 *   w      [B, Lq, HI]     fp32, the already-activated head weights sigmoid(h_t W^Iw_j)
 *   bI     [HI] fp32 or NULL (= zeros)
 *   scores fp32; the row of (b, t) starts at scores[((b * R) + (t - q_begin)) * row_stride]
 *          with R = q_end - q_begin and row_stride >= Lk, a multiple of 4.  Entries beyond
 *          the row's visible keys are left unwritten.
 *   ws     workspace (device status word lives at its start); ws_bytes >= 256.
 */
int gsa_indexer_scores(const gsa_params_t *p, const void *qI, const void *kI, const float *w,
                       const float *bI, float *scores, int64_t row_stride, void *ws,
                       size_t ws_bytes, void *stream);

/*
 * Upstream projections of the layer (text below Eq. 7; Eq. 9; Eq. 10) as one tensor-core GEMM:
 *     q^I_j = h W^Iq_j,   k^I = h W^Ik,   w_j = sigmoid(h W^Iw_j),   g1 logits = h W^g_O,   g2 logits = h W^g_V.
 * Needs Lq == Lk (one hidden state per position).  The outputs are exactly the inputs of gsa_forward.
 *   H      [B * Lk, d_model] bf16 hidden states, d_model a multiple of 8
 *   Wt     [gsa_project_columns(p), d_model] bf16: the weight matrices transposed and stacked, one
 *          row of d_model per output column, in the order q^I (HI*dI rows; head-major), k^I (dI),
 *          head weights (8 rows, the first HI used), g1 (n_h*d_h), g2 (n_kv*d_h)
 *   qI [B,Lk,HI,dI], kI [B,Lk,dI], g1_logits [B,Lk,n_h,d_h], g2_logits [B,Lk,n_kv,d_h] bf16 (fp32
 *   accumulation, rounded once); w [B,Lk,HI] fp32, after the sigmoid
 *   ws     workspace, ws_bytes >= 256 (device status word)
 */
int gsa_project_columns(const gsa_params_t *p, int32_t *columns);
int gsa_project(const gsa_params_t *p, int32_t d_model, const void *H, const void *Wt, void *qI, void *kI,
                float *w, void *g1_logits, void *g2_logits, void *ws, size_t ws_bytes, void *stream);

/*
 * Output projection (Sec. 2.1: the heads are concatenated and projected by W_O):
 *     u[token, :] = out[token, :, :] (n_h * d_h values) * W_O,    the same tensor-core GEMM kernel.
 *   attn_out [B, Lq, n_h, d_h] bf16 (the `out` of gsa_forward);  Wo_t [d_model, n_h*d_h] bf16 (W_O
 *   transposed: one row per output column);  u [B, Lq, d_model] bf16;  d_model a multiple of 8
 *   ws     workspace, ws_bytes >= 256 (device status word)
 */
int gsa_output_projection(const gsa_params_t *p, int32_t d_model, const void *attn_out, const void *Wo_t,
                          void *u, void *ws, size_t ws_bytes, void *stream);

/*
 * Backward of sparse gated attention: Eq. 9, 11, 12 and 10 differentiated for rows [q_begin, q_end)
 * with the index sets held fixed (top-k selection has no derivative; Sec. 5.1 trains the indexer with
 * its own loss).  With out = o * sigmoid(g1), o = sum_j a_j v'_j, a = softmax_j(sm_scale * q.k_j) over
 * j in S_t and v' = V * sigmoid(g2), and dout the derivative of the loss with respect to `out`:
 *     dg1 = dout * o * sigmoid'(g1),        do = dout * sigmoid(g1),
 *     dz_j = a_j (do.v'_j - sum_i a_i do.v'_i),   dQ = sm_scale * sum_j dz_j k_j,
 *     dK[s] = sm_scale * sum over (t, h, j: s_j = s) of dz_j q,    dv'[s] = sum of a_j do,
 *     dV = dv' * sigmoid(g2),   dg2 = dv' * V * sigmoid'(g2).
 *   Q, K, V, g1_logits, g2_logits, idx, kt   as given to gsa_sparse_gated_attn_fwd (g2_logits required)
 *   out    [B, Lq, n_h, d_h] bf16: what the forward call wrote (rows of the range are read)
 *   dout   [B, Lq, n_h, d_h] bf16 (rows of the range are read)
 *   dQ, dg1  [B, Lq, n_h, d_h] bf16: rows of the range are written, other rows are left alone
 *   dK, dV, dg2  [B, Lk, n_kv, d_h] bf16: every element is written; sums over the rows of the range,
 *          accumulated in fp32 (in an order that depends on scheduling) and rounded once
 *   pbar   [B, R, k_max] fp32 or NULL: the target of the indexer's loss (what gsa_attn_probs_mean writes,
 *          see below), which this call's second sweep has at hand: one call instead of two
 *   lse    [B, Lq, n_h] fp32 or NULL: what gsa_sparse_gated_attn_fwd_lse saved for the same inputs; with it
 *          the sweep over S_t that recomputes the softmax statistics is skipped
 *   ws     workspace of gsa_attn_bwd_workspace_bytes(p) bytes (depends on q_begin / q_end): status word,
 *          V', dout * sigmoid(g1), softmax statistics, and the index sets inverted (key -> query rows)
 * Returns GSA_ERR_WORKSPACE if ws is too small; nothing is launched on an argument error.
 */
int gsa_attn_bwd_workspace_bytes(const gsa_params_t *p, size_t *bytes);
int gsa_sparse_gated_attn_bwd(const gsa_params_t *p, const void *Q, const void *K, const void *V,
                              const void *g1_logits, const void *g2_logits, const int32_t *idx,
                              const int32_t *kt, const void *out, const void *dout, void *dQ, void *dK,
                              void *dV, void *dg1, void *dg2, float *pbar, const float *lse, void *ws,
                              size_t ws_bytes, void *stream);

/*
 * The indexer's sparse-phase loss (Sec. 5.1, Eq. 14) for rows [q_begin, q_end):
 *     loss_t = sum_{j in S_t} pbar[t, j] * (log pbar[t, j] - log q_j),     q = softmax_j I[t, s_j],
 * I from Eq. 7 (or Eq. 3 with act = 1), with 0 log 0 = 0.  The target is a constant of the loss.
 *
 * gsa_attn_probs_mean writes the target: Eq. 11 gives one attention distribution over S_t per head and the
 * indexer score has no head index, so pbar[t, j] is their mean over the n_h heads (the paper says "the
 * softmax attention" without naming the reduction over heads).
 *   Q, K, idx, kt   as given to gsa_sparse_gated_attn_fwd
 *   pbar   [B, R, k_max] fp32: entry j belongs to key idx[.., j]; entries past kt are 0
 *   ws     workspace, ws_bytes >= 256 (device status word)
 *
 * gsa_indexer_kl_bwd computes the loss per row and the derivatives of the sum of the rows' losses:
 *     dI_j = q_j * sum_i pbar_i - pbar_j,    with x_ij = q^I_i . k^I_{s_j} + b_i and f = sigmoid (or ReLU):
 *     dw_i = sum_j dI_j f(x_ij),   dx_ij = dI_j w_i f'(x_ij),   dq^I_i = sum_j dx_ij k^I_{s_j},
 *     dk^I[s] = sum over (t, i, j: s_j = s) of dx_ij q^I_i,      db_i = sum over (t, j) of dx_ij.
 *   qI, kI, w, bI   as given to gsa_indexer_scores (bI may be NULL); w is the weight after its sigmoid,
 *                   dw the derivative with respect to that value
 *   pbar   [B, R, k_max] fp32 (any non-negative target works; it need not sum to 1)
 *   loss   [B, R] fp32
 *   dqI    [B, Lq, HI, dI] bf16 and dw [B, Lq, HI] fp32: rows of the range are written
 *   dkI    [B, Lk, dI] bf16: every element is written (fp32 sums, order depends on scheduling, rounded once)
 *   dbI    [HI] fp32 or NULL (fp32 atomics: order depends on scheduling)
 *   ws     workspace of gsa_indexer_kl_workspace_bytes(p) bytes: status word and the fp32 sums of dk^I
 */
int gsa_attn_probs_mean(const gsa_params_t *p, const void *Q, const void *K, const int32_t *idx,
                        const int32_t *kt, float *pbar, void *ws, size_t ws_bytes, void *stream);
int gsa_indexer_kl_workspace_bytes(const gsa_params_t *p, size_t *bytes);
int gsa_indexer_kl_bwd(const gsa_params_t *p, const void *qI, const void *kI, const float *w, const float *bI,
                       const int32_t *idx, const int32_t *kt, const float *pbar, float *loss, void *dqI,
                       void *dkI, float *dw, float *dbI, void *ws, size_t ws_bytes, void *stream);

/*
 * Running mean of the score variance: the normaliser v_bar of Eq. 8 is an exponential moving average of
 * the score variance across the batch.  The paper gives neither momentum nor start value: both are the
 * caller's.
 *     mean_var = mean of var[0 .. n),      v_bar <- momentum * v_bar + (1 - momentum) * mean_var
 *   var       n fp32 row variances on the device (the `var` output of gsa_forward / gsa_adaptive_topk)
 *   v_bar     one fp32 on the device, read and written; copy it into gsa_params_t.v_bar for the next step
 *   mean_var  one fp32 on the device or NULL
 *   momentum  in [0, 1]
 * The sum is taken in fp64 in a fixed order: the result does not depend on scheduling.
 */
int gsa_vbar_update(const float *var, int64_t n, float momentum, float *v_bar, float *mean_var, void *stream);

/*
 * Adaptive sparsity controller, Eq. 8 then Eq. 4, one row at a time:
 *     Var_t = population variance of the n_t visible scores (accumulated in fp64),
 *     k_t   = clamp(floor(k_base * Var_t / v_bar), k_min, k_max)   (k_mode 0),
 *     S_t   = the min(k_t, n_t) positions with the largest scores; equal scores are
 *             ordered by position, lower first.
 *   scores as written by gsa_indexer_scores (same q_begin / q_end / row_stride)
 *   idx    [B, R, k_max] int32: S_t in ascending position order, then -1
 *   kt     [B, R] int32: |S_t| = min(k_t, n_t)
 *   var    [B, R] fp32 or NULL: Var_t (for the caller's running mean)
 *   ws     optional (may be NULL); with >= 256 bytes the fallback-row counter is kept at its head
 */
int gsa_adaptive_topk(const gsa_params_t *p, const float *scores, int64_t row_stride,
                      int32_t *idx, int32_t *kt, float *var, void *ws, size_t ws_bytes,
                      void *stream);

/*
 * Sparse gated attention, Eq. 9, 11, 12, 10, for query rows q_begin..q_end:
 *     V'[s]   = V[s] * sigmoid(g2[s])                       (elementwise, G2)
 *     A[t,s]  = softmax over s in S_t of  sm_scale * Q[t,h,:] . K[s,g(h),:]
 *     out[t,h,:] = (sum_s A[t,s] V'[s,g(h),:]) * sigmoid(g1[t,h,:])   (G1)
 *   Q, g1_logits [B, Lq, n_h, d_h] bf16;  K, V, g2_logits [B, Lk, n_kv, d_h] bf16
 *   g2_logits may be NULL: V is then taken as already gated.
 *   idx [B, R, k_max], kt [B, R] as written by gsa_adaptive_topk (R = q_end - q_begin)
 *       A row with kt = 0 (an empty S_t; gsa_adaptive_topk never writes one) has an empty sum: its
 *       out row is written as zeros.
 *   out [B, Lq, n_h, d_h] bf16 (rows outside q_begin..q_end untouched)
 *   ws  workspace of at least gsa_attn_workspace_bytes(p, 0) bytes (status word, the fp32
 *       online-softmax state that is carried between key ranges or merged across parallel
 *       segments).  With gsa_attn_workspace_bytes(p, 1) bytes there is room for the gated values as
 *       well and G2 runs as one streaming pre-pass when that is cheaper than gating the gathered
 *       rows; otherwise the g2 rows are gathered with K and V.
 */
int gsa_attn_workspace_bytes(const gsa_params_t *p, int32_t with_value_gate_prepass, size_t *bytes);
int gsa_sparse_gated_attn_fwd(const gsa_params_t *p, const void *Q, const void *K, const void *V,
                              const void *g1_logits, const void *g2_logits, const int32_t *idx,
                              const int32_t *kt, void *out, void *ws, size_t ws_bytes,
                              void *stream);

/*
 * The value gate on its own, Eq. 9:  V_gated = bf16(V * sigmoid(g2_logits)), elementwise over n_elems
 * bf16 values (a multiple of 8; three distinct device buffers, 16-byte aligned).
 * What gsa_forward runs as its pre-pass; exposed for callers that gate their own shard of the values
 * before exchanging them (context-parallel prefill) and then pass g2_logits = NULL.
 */
int gsa_value_gate(const void *V, const void *g2_logits, void *V_gated, int64_t n_elems, void *stream);

/*
 * The same call for training: also saves the softmax statistics the backward pass needs,
 *     lse[b, t, h] = log sum_{j in S_t} exp(sm_scale * q_h . k_j)      (natural logarithm, fp32),
 * for rows [q_begin, q_end) of [B, Lq, n_h]; gsa_sparse_gated_attn_bwd takes them back.
 */
int gsa_sparse_gated_attn_fwd_lse(const gsa_params_t *p, const void *Q, const void *K, const void *V,
                                  const void *g1_logits, const void *g2_logits, const int32_t *idx,
                                  const int32_t *kt, void *out, float *lse, void *ws, size_t ws_bytes,
                                  void *stream);

/*
 * gsa_sparse_gated_attn_fwd for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a deployment variant of the call above, same arithmetic, same kernels.)
 *
 * Who needs it: code that runs inside a fixed, pre-reserved memory budget, in a latency-critical
 * or callback context, or under a host allocator that must not be entered from the GPU-driving
 * thread cannot call cudaMalloc (it may block, synchronise the device, or fail) and may have no
 * spare buffer to pass as workspace.  Here the scratch the call needs -- the gated values
 * V' = bf16(V * sigmoid(g2)) of Eq. 9 and the attention kernels' fp32 softmax state -- lives in an
 * array of GSA_STATIC_SCRATCH_BYTES that is part of the library image; every GPU that loads the library holds that array until the process exits.
 * The call and everything below it allocate nothing.
 *
 *   Arguments as gsa_sparse_gated_attn_fwd, without ws; g2_logits must not be NULL.
 *   Limit: B * Lk * n_kv * d_h * 2 + (gsa_attn_workspace_bytes(p, 0) - 256) <= GSA_STATIC_SCRATCH_BYTES
 *   (for example 8192 cache tokens and 1024 query tokens at n_kv = 8, n_h = 16, d_h = 128); larger
 *   problems return GSA_ERR_STATIC_SCRATCH and launch nothing.
 *   The first call on each device looks up the array's device address (one runtime query, made with
 *   that device current); make that first call outside of any stream capture.
 *   All calls on one GPU share the one array: calls that may overlap on the GPU (different streams,
 *   different host threads) race on it -- serialise them.  Each call rewrites every element it
 *   later reads, so no contents carry over from one call to the next.
 */
#define GSA_STATIC_SCRATCH_BYTES (32u << 20)
int gsa_sparse_gated_attn_fwd_static(const gsa_params_t *p, const void *Q, const void *K, const void *V,
                                     const void *g1_logits, const void *g2_logits, const int32_t *idx,
                                     const int32_t *kt, void *out, void *stream);

/*
 * The whole forward path (pipeline of Sec. 3.2): G2, indexer, budget, top-k, sparse
 * attention, G1, for all B * Lq queries.  Score rows are produced and consumed slab by
 * slab inside the workspace and never leave it.
 *   idx_out [B, Lq, k_max] int32 or NULL;  kt_out [B, Lq] int32 or NULL;
 *   var_out [B, Lq] fp32 or NULL.
 *   slab_rows as in gsa_workspace_bytes (must be the value the workspace was sized with).
 */
int gsa_forward(const gsa_params_t *p, const void *Q, const void *K, const void *V,
                const void *qI, const void *kI, const float *w, const float *bI,
                const void *g1_logits, const void *g2_logits, void *out, int32_t *idx_out,
                int32_t *kt_out, float *var_out, int32_t slab_rows, void *ws, size_t ws_bytes,
                void *stream);

/*
 * gsa_forward on HOST buffers (pinned memory recommended): copies the nine inputs to a
 * caller-provided device arena, runs gsa_forward there, copies `out` (and kt_out if
 * not NULL) back and waits for `stream`.  All tensor pointers are host pointers.
 * The large tensors (Q, K, V, gate logits) are copied on a second stream that exists for the
 * duration of the call, under the indexer and the selection, which need only qI, kI and w.
 * `arena` is device memory of at least gsa_forward_host_arena_bytes(p, slab_rows).
 */
int gsa_forward_host_arena_bytes(const gsa_params_t *p, int32_t slab_rows, size_t *bytes);
int gsa_forward_host(const gsa_params_t *p, const void *Q, const void *K, const void *V,
                     const void *qI, const void *kI, const float *w, const float *bI,
                     const void *g1_logits, const void *g2_logits, void *out, int32_t *kt_out,
                     int32_t slab_rows, void *arena, size_t arena_bytes, void *stream);

/*
 * Waits for `stream`, reads the device status word at the start of `ws` into
 * *status_out (host) and returns GSA_OK, GSA_ERR_DEVICE_TIMEOUT (*status_out 1..3: copy producer,
 * MMA issuer, epilogue) or GSA_ERR_INDEX_RANGE (*status_out 6) accordingly.
 * The word is cleared by every call that takes `ws`.  ws == NULL reads the status word of
 * gsa_sparse_gated_attn_fwd_static (it lives in the library's built-in array on the current device).
 */
int gsa_device_status(const void *ws, void *stream, int32_t *status_out);

/*
 * Waits for `stream` and reads how many rows of the last gsa_forward / gsa_adaptive_topk call on `ws`
 * took the selection kernel's whole-row fallback (the sampled candidate threshold misjudged the row:
 * slower, same result).  A diagnostic: a large share means the scores are far from what the sample
 * assumes (for instance sorted by position).
 */
int gsa_select_fallback_rows(const void *ws, void *stream, int32_t *rows_out);

/* Number of kernel launches the library has enqueued so far in this process (host counter). */
int64_t gsa_launch_count(void);

/*
 * Debug knob: 0 = tensor-core (tcgen05) indexer where the shape allows it (default),
 * 1 = plain CUDA-core indexer.  Process-wide; not meant for production use.
 */
void gsa_debug_set_indexer_path(int32_t path);

/*
 * Tuning knob: keys per key range of the sparse-attention gather (default 16384: the K and V' rows of
 * a range then occupy 64 MB of the 126 MB L2 at n_kv * d_h = 1024).  Process-wide; the workspace size
 * depends on it, so set it before gsa_workspace_bytes.
 */
void gsa_debug_set_attn_range_keys(int32_t keys);

/*
 * Test knob for the bounded device-side waits: `cycles` is the limit of every wait in SM clock cycles
 * (<= 0 restores the default of 2^31, about a second).  With withhold_first_copy != 0 the copy producer of
 * each tensor-core kernel (gsa_indexer_scores / gsa_forward on the tcgen05 path, gsa_project,
 * gsa_output_projection) leaves out its first copy, so that the wait for it meets a barrier that nothing
 * completes: the way to see the give-up path work (status word set, kernel returns, context intact).
 * Process-wide; not meant for production use.
 */
void gsa_debug_set_wait_limit(int64_t cycles, int32_t withhold_first_copy);

/*
 * Profiling hook: three cudaEvent_t handles (or NULL to switch off) that every following
 * gsa_forward records on its stream: at entry, after the last indexer/top-k slab (before the
 * sparse-attention launch), and after the sparse-attention launch.  Process-wide; the caller
 * owns the events and reads them after synchronising.
 */
void gsa_profile_set_events(void *ev_begin, void *ev_selected, void *ev_end);

/*
 * Profiling hook with one interval per launch: `events` is an array of `capacity` cudaEvent_t handles
 * (created by the caller, timing enabled).  Every following gsa_forward records events[0] at entry and the
 * next event behind each stage it enqueues, and writes into the HOST arrays stage_out[i] which stage the
 * interval events[i] .. events[i + 1] belongs to (0 indexer, 1 budget + top-k, 2 value gate, 3 range cuts,
 * 4 sparse attention, 5 normalise + output gate) and into *count_out the number of intervals.  The events
 * serialise nothing but cost a little: use it for a profiling step, not inside a timed loop.  NULL / 0
 * switches it off.  Process-wide; the caller owns the events and the arrays and reads them after
 * synchronising.
 */
void gsa_profile_set_timeline(void **events, int32_t capacity, int32_t *stage_out, int32_t *count_out);

/*
 * Rate probes (measurement aids; the paper has no counterpart).  They enqueue one kernel on `stream`; the
 * caller times it with events and divides.
 *   gsa_probe_gather: reads the first piece_bytes of table row row_idx[i] for every i < n_idx with plain
 *     32-byte loads, every thread keeping four loads in flight (2048 threads per SM): n_idx * piece_bytes bytes
 *     gathered.
 *     table: n_rows rows of row_bytes (device, 32-byte aligned; row_bytes a multiple of 32, piece_bytes
 *     32 times a power of two);
 *     row_idx: n_idx int32 on the device (values outside [0, n_rows) are clamped); sink: 4 bytes of device
 *     memory.  A table smaller than the L2 gives the L2's gather rate, a larger one HBM's.
 *   gsa_probe_ex2: every resident thread runs `iters` rounds of eight independent 2^x on the
 *     special-function unit; *ops_out (host) receives the number of 2^x evaluated.  sink: 4 bytes (device).
 */
int gsa_probe_gather(const void *table, int32_t n_rows, int64_t row_bytes, int32_t piece_bytes,
                     const int32_t *row_idx, int64_t n_idx, void *sink, void *stream);
int gsa_probe_ex2(int32_t iters, int64_t *ops_out, void *sink, void *stream);

/* Static string for a gsa_status value. */
const char *gsa_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* GSA_H_ */
