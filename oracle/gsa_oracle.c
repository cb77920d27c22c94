/*
 * CPU oracle for the forward path of Gated Sparse Attention.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain loops, fp64 arithmetic, no blocking, no fusion.
 * It shares no code with the CUDA library and must never be called from the product
 * path: only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Inputs arrive as fp32 arrays holding exactly the bf16 / fp32 values the GPU reads
 * (widening is exact); every sum, exponential and division below is done in double.
 *
 * Steps, in the paper's order:
 *   Eq. 7   gated lightning indexer     I[t,s] = sum_j w[t,j] * sigmoid(q^I[t,j] . k^I[s] + b_j)
 *           (act = 1: the ReLU indexer of Eq. 3 that Eq. 7 replaces, sum_j w[t,j] * max(q^I.k^I + b_j, 0))
 *   Eq. 8   adaptive budget             k_t = clamp(floor(k_base * Var(I[t,:]) / Vbar), k_min, k_max)
 *   Eq. 4   top-k_t selection           S_t = the k_t positions with the largest I[t,s]
 *   Eq. 9   value gate G2               V'[s] = V[s] * sigmoid(g2[s])      (elementwise)
 *   Eq. 11  softmax over S_t            A[t,s] = exp(Q_t.K_s/sqrt(d_k)) / sum_{j in S_t} exp(...)
 *   Eq. 12  aggregation                 O[t] = sum_{s in S_t} A[t,s] V'[s]
 *   Eq. 10  output gate G1              out[t,h] = O[t,h] * sigmoid(g1[t,h]) (elementwise)
 *
 * Readings where the paper is silent (listed with the library's documentation as well):
 *   - query t of Lq sees keys s = 0 .. Lk-Lq+t (causal; decode is Lq = 1);
 *   - Var is the population variance over the visible scores only;
 *   - k_eff = min(k_t, number of visible keys);
 *   - ties in I are broken towards the lower position; S_t is emitted ascending;
 *   - one S_t per query position, shared by all heads (I has no head index);
 *   - k_mode 0 is Eq. 8 as printed; k_mode 1 is the direction the prose describes
 *     (k_base * Vbar / Var; Var = 0 gives k_max); k_mode 2 is a fixed k = k_base;
 *     k_mode 3 selects every visible key (the dense fallback for short contexts, Sec. 8).
 *
 * Pins (tests/test_oracle_pins.py): closed-form sigmoid values on one-hot inputs,
 * the reflection identity I(q)+I(-q)=sum_j w_j, the open range (0, sum w), two-valued
 * rows with known variance, clamp edges, monotonicity per mode, brute-force top-k
 * with exact ties (ReLU variant: positive homogeneity, I(q) - I(-q) linear in q), reduction to
 * library softmax attention when S_t is everything
 * and gates are saturated, single-key and equal-logit closed forms, g1 = -40 -> 0.
 * Training side (end of this file): the backward of Eq. 9-12 and Eq. 10 is pinned by central differences
 * of the forward above, by library autograd on the forward written as masked dense attention, and by the
 * single-key / shift-invariance closed forms; the running mean of the variance by a worked example; the
 * indexer's sparse-phase loss (Eq. 14) and its derivatives by library softmax / KL divergence / autograd, a
 * two-key closed form, the zero of the loss at target = softmax(I), and central differences.
 * Parity unpinned: nothing (every function above has at least one such pin); the
 * absolute values on random data have no printed reference in the paper.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t B, Lq, Lk;
    int32_t n_h, n_kv, d_h;
    int32_t HI, dI;
    int32_t k_base, k_min, k_max;
    int32_t k_mode;
    double v_bar;
    double sm_scale; /* <= 0: 1/sqrt(d_h) */
    int32_t act;     /* 0: sigmoid (Eq. 7), 1: ReLU (Eq. 3) */
} gsa_oracle_params;

static double sigmoid_d(double x) { return 1.0 / (1.0 + exp(-x)); }

int gsa_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* number of keys query t may look at */
int gsa_oracle_visible(const gsa_oracle_params *p, int t) { return p->Lk - p->Lq + t + 1; }

/* ---- Eq. 7 -------------------------------------------------------------- */
/* qI_t: [HI, dI] of this query; kI_b: [Lk, dI] of this batch element; w_t: [HI]. */
void gsa_oracle_score_row(const gsa_oracle_params *p, const float *qI_t, const float *kI_b,
                          const float *w_t, const float *bI, int n_t, double *I_row)
{
    for (int s = 0; s < n_t; ++s) {
        double acc = 0.0;
        for (int j = 0; j < p->HI; ++j) {
            double x = bI ? (double)bI[j] : 0.0;
            for (int c = 0; c < p->dI; ++c)
                x += (double)qI_t[j * p->dI + c] * (double)kI_b[(size_t)s * p->dI + c];
            acc += (double)w_t[j] * (p->act == 1 ? (x > 0.0 ? x : 0.0) : sigmoid_d(x));
        }
        I_row[s] = acc;
    }
}

/* ---- Eq. 8 -------------------------------------------------------------- */
void gsa_oracle_budget(const gsa_oracle_params *p, const double *I_row, int n_t,
                       double *var_out, double *r_out, int32_t *k_t_out, int32_t *k_eff_out)
{
    double mean = 0.0;
    for (int s = 0; s < n_t; ++s) mean += I_row[s];
    mean /= (double)n_t;
    double var = 0.0;
    for (int s = 0; s < n_t; ++s) var += (I_row[s] - mean) * (I_row[s] - mean);
    var /= (double)n_t;

    double r;
    if (p->k_mode == 0)      r = (double)p->k_base * var / p->v_bar;
    else if (p->k_mode == 1) r = var > 0.0 ? (double)p->k_base * p->v_bar / var : INFINITY;
    else if (p->k_mode == 2) r = (double)p->k_base;
    else                     r = INFINITY;            /* k_mode 3: every visible key (k_max >= Lk) */

    double f = floor(r);
    int32_t k;
    if (!(f < (double)p->k_max)) k = p->k_max;          /* also catches +inf */
    else if (f < (double)p->k_min) k = p->k_min;
    else k = (int32_t)f;
    if (var_out) *var_out = var;
    if (r_out) *r_out = r;
    *k_t_out = k;
    *k_eff_out = k < n_t ? k : n_t;
}

/* ---- Eq. 4 -------------------------------------------------------------- */
typedef struct { double score; int32_t pos; } scored_t;

static int by_score_desc_pos_asc(const void *a, const void *b)
{
    const scored_t *x = (const scored_t *)a, *y = (const scored_t *)b;
    if (x->score > y->score) return -1;
    if (x->score < y->score) return 1;
    return (x->pos > y->pos) - (x->pos < y->pos);
}
static int by_int_asc(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/* full sort of the row; the first k_eff entries are S_t; written ascending, rest -1 */
void gsa_oracle_topk(const double *I_row, int n_t, int k_eff, int32_t *idx_out, int k_pad)
{
    scored_t *a = (scored_t *)malloc(sizeof(scored_t) * (size_t)n_t);
    for (int s = 0; s < n_t; ++s) { a[s].score = I_row[s]; a[s].pos = s; }
    qsort(a, (size_t)n_t, sizeof(scored_t), by_score_desc_pos_asc);
    for (int i = 0; i < k_eff; ++i) idx_out[i] = a[i].pos;
    qsort(idx_out, (size_t)k_eff, sizeof(int32_t), by_int_asc);
    for (int i = k_eff; i < k_pad; ++i) idx_out[i] = -1;
    free(a);
}

/* ---- Eq. 9, 11, 12, 10 --------------------------------------------------- */
/* Q_t, g1_t: [n_h, d_h]; K_b, V_b, g2_b: [Lk, n_kv, d_h]; idx: k_eff positions. */
void gsa_oracle_attn_row(const gsa_oracle_params *p, const float *Q_t, const float *K_b,
                         const float *V_b, const float *g1_t, const float *g2_b,
                         const int32_t *idx, int k_eff, double *out_t)
{
    const int d = p->d_h, grp = p->n_h / p->n_kv;
    const double scale = p->sm_scale > 0.0 ? p->sm_scale : 1.0 / sqrt((double)d);
    double *z = (double *)malloc(sizeof(double) * (size_t)(k_eff > 0 ? k_eff : 1));
    for (int h = 0; h < p->n_h; ++h) {
        const int g = h / grp;
        double zmax = -INFINITY;
        for (int i = 0; i < k_eff; ++i) {
            const float *Ks = K_b + ((size_t)idx[i] * p->n_kv + g) * d;
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += (double)Q_t[h * d + c] * (double)Ks[c];
            z[i] = dot * scale;
            if (z[i] > zmax) zmax = z[i];
        }
        double den = 0.0;
        for (int i = 0; i < k_eff; ++i) { z[i] = exp(z[i] - zmax); den += z[i]; }
        for (int c = 0; c < d; ++c) {
            double o = 0.0;
            for (int i = 0; i < k_eff; ++i) {
                const size_t at = ((size_t)idx[i] * p->n_kv + g) * d + c;
                const double vg = (double)V_b[at] * sigmoid_d((double)g2_b[at]);   /* Eq. 9 */
                o += (z[i] / den) * vg;                                             /* Eq. 11-12 */
            }
            out_t[h * d + c] = o * sigmoid_d((double)g1_t[h * d + c]);            /* Eq. 10 */
        }
    }
    free(z);
}

/* ---- upstream projections (text below Eq. 7; Eq. 9; Eq. 10) ---------------- */
/* One token's projections from its hidden state h [d_model]:
 *   q^I_j = h W^Iq_j,  k^I = h W^Ik,  head weight sigmoid(h W^Iw_j),  g1 logits = h W^g_O,  g2 logits = h W^g_V.
 * Wt holds the weight matrices transposed and stacked, one row of d_model per output column, in the
 * order q^I (HI*dI rows), k^I (dI), head weights (8 rows, the first HI used), g1 (n_h*d_h), g2 (n_kv*d_h). */
void gsa_oracle_project_rows(const gsa_oracle_params *p, int d_model, const float *H, const float *Wt,
                             const int32_t *rows_m, int n_rows, double *qI, double *kI, double *w,
                             double *g1, double *g2)
{
    const int nq = p->HI * p->dI, nk = p->dI, ng1 = p->n_h * p->d_h, ng2 = p->n_kv * p->d_h;
    const int o_k = nq, o_w = nq + nk, o_g1 = o_w + 8, o_g2 = o_g1 + ng1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
        const float *h = H + (size_t)rows_m[r] * d_model;
        for (int n = 0; n < o_g2 + ng2; ++n) {
            if (n >= o_w + p->HI && n < o_g1) continue;              /* unused rows of the weight block */
            const float *wt = Wt + (size_t)n * d_model;
            double acc = 0.0;
            for (int c = 0; c < d_model; ++c) acc += (double)h[c] * (double)wt[c];
            if (n < o_k)        qI[(size_t)r * nq + n] = acc;
            else if (n < o_w)   kI[(size_t)r * nk + (n - o_k)] = acc;
            else if (n < o_g1)  w[(size_t)r * p->HI + (n - o_w)] = sigmoid_d(acc);
            else if (n < o_g2)  g1[(size_t)r * ng1 + (n - o_g1)] = acc;
            else                g2[(size_t)r * ng2 + (n - o_g2)] = acc;
        }
    }
}

/* ---- output projection (Sec. 2.1: concatenated heads times W_O) -------------- */
/* u[token, n] = sum_c X[token, c] * Wt[n, c] for the listed tokens; X is the gated attention output
 * with its n_h heads concatenated ([tokens, K]), Wt the transposed weight ([N, K]). */
void gsa_oracle_out_project_rows(int K, int N, const float *X, const float *Wt, const int32_t *rows_m,
                                 int n_rows, double *u)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r)
        for (int n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int c = 0; c < K; ++c)
                acc += (double)X[(size_t)rows_m[r] * K + c] * (double)Wt[(size_t)n * K + c];
            u[(size_t)r * N + n] = acc;
        }
}

/* ---- drivers over a list of (batch, query) rows -------------------------- */

/* scores of the listed rows: out[r, 0..n_t) in a [n_rows, Lk] double array */
void gsa_oracle_scores_rows(const gsa_oracle_params *p, const float *qI, const float *kI,
                            const float *w, const float *bI, const int32_t *rows_b,
                            const int32_t *rows_t, int n_rows, double *scores_out)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
        const int b = rows_b[r], t = rows_t[r];
        const int n_t = gsa_oracle_visible(p, t);
        gsa_oracle_score_row(p, qI + ((size_t)b * p->Lq + t) * p->HI * p->dI,
                             kI + (size_t)b * p->Lk * p->dI, w + ((size_t)b * p->Lq + t) * p->HI,
                             bI, n_t, scores_out + (size_t)r * p->Lk);
    }
}

/* Eq. 8 + Eq. 4 on externally supplied fp32 score rows ("staged" mode): row r of
 * `scores` (stride in floats) belongs to query rows_t[r]. */
void gsa_oracle_select_rows_f32(const gsa_oracle_params *p, const float *scores, int64_t stride,
                                const int32_t *rows_t, int n_rows, int32_t *idx_out,
                                int32_t *kt_out, int32_t *keff_out, double *var_out,
                                double *r_out)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
        const int n_t = gsa_oracle_visible(p, rows_t[r]);
        double *row = (double *)malloc(sizeof(double) * (size_t)n_t);
        for (int s = 0; s < n_t; ++s) row[s] = (double)scores[(size_t)r * stride + s];
        gsa_oracle_budget(p, row, n_t, var_out + r, r_out + r, kt_out + r, keff_out + r);
        gsa_oracle_topk(row, n_t, keff_out[r], idx_out + (size_t)r * p->k_max, p->k_max);
        free(row);
    }
}

/* Eq. 9-12, 10 for the listed rows with given index sets (idx: [n_rows, k_max]) */
void gsa_oracle_attn_rows(const gsa_oracle_params *p, const float *Q, const float *K,
                          const float *V, const float *g1, const float *g2,
                          const int32_t *rows_b, const int32_t *rows_t, int n_rows,
                          const int32_t *idx, const int32_t *keff, double *out)
{
    const size_t qrow = (size_t)p->n_h * p->d_h, kvb = (size_t)p->Lk * p->n_kv * p->d_h;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
        const int b = rows_b[r], t = rows_t[r];
        gsa_oracle_attn_row(p, Q + ((size_t)b * p->Lq + t) * qrow, K + b * kvb, V + b * kvb,
                            g1 + ((size_t)b * p->Lq + t) * qrow, g2 + b * kvb,
                            idx + (size_t)r * p->k_max, keff[r], out + (size_t)r * qrow);
    }
}

/* the whole path, end to end, for the listed rows.  scores_out may be NULL. */
void gsa_oracle_forward_rows(const gsa_oracle_params *p, const float *Q, const float *K,
                             const float *V, const float *qI, const float *kI, const float *w,
                             const float *bI, const float *g1, const float *g2,
                             const int32_t *rows_b, const int32_t *rows_t, int n_rows,
                             double *out, int32_t *idx_out, int32_t *kt_out, int32_t *keff_out,
                             double *var_out, double *r_out, double *scores_out)
{
    const size_t qrow = (size_t)p->n_h * p->d_h, kvb = (size_t)p->Lk * p->n_kv * p->d_h;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
        const int b = rows_b[r], t = rows_t[r];
        const int n_t = gsa_oracle_visible(p, t);
        double *row = scores_out ? scores_out + (size_t)r * p->Lk
                                 : (double *)malloc(sizeof(double) * (size_t)n_t);
        gsa_oracle_score_row(p, qI + ((size_t)b * p->Lq + t) * p->HI * p->dI,
                             kI + (size_t)b * p->Lk * p->dI, w + ((size_t)b * p->Lq + t) * p->HI,
                             bI, n_t, row);
        gsa_oracle_budget(p, row, n_t, var_out + r, r_out + r, kt_out + r, keff_out + r);
        int32_t *idx = idx_out + (size_t)r * p->k_max;
        gsa_oracle_topk(row, n_t, keff_out[r], idx, p->k_max);
        gsa_oracle_attn_row(p, Q + ((size_t)b * p->Lq + t) * qrow, K + b * kvb, V + b * kvb,
                            g1 + ((size_t)b * p->Lq + t) * qrow, g2 + b * kvb, idx, keff_out[r],
                            out + (size_t)r * qrow);
        if (!scores_out) free(row);
    }
}

/* ---- training side of the path --------------------------------------------- */
/* Backward of Eq. 9-12 and Eq. 10 for the listed rows with given index sets: the derivatives of
 *   loss = sum over listed rows of <dout[r], out[r]>
 * with respect to Q, K, V and the two gate logits.  The index sets are constants (top-k selection
 * has no derivative; the indexer is trained by its own loss, Sec. 5.1).  Written from the chain rule
 * on the forward definition, per head h of query row t with KV head g:
 *   v'_j = V[s_j] * sigmoid(g2[s_j])                                   (Eq. 9)
 *   z_j  = scale * q . k_j,   a = softmax_j(z),   o = sum_j a_j v'_j   (Eq. 11-12)
 *   out  = o * sigmoid(g1)                                             (Eq. 10)
 * so, with do = dout * sigmoid(g1):
 *   dg1   = dout * o * sigmoid'(g1)
 *   da_j  = do . v'_j,   dz_j = a_j (da_j - sum_i a_i da_i)
 *   dq    = scale * sum_j dz_j k_j,      dK[s_j] += scale * dz_j q
 *   dv'_j = a_j do  ->  dV[s_j] += dv'_j * sigmoid(g2[s_j]),  dg2[s_j] += dv'_j * V[s_j] * sigmoid'(g2[s_j])
 * dQ, dg1: [n_rows, n_h, d_h]; dK, dV, dg2: [B, Lk, n_kv, d_h], zeroed here, summed over the listed rows.
 * Threads split the KV heads, so no two threads add into the same element. */
void gsa_oracle_attn_bwd_rows(const gsa_oracle_params *p, const float *Q, const float *K,
                              const float *V, const float *g1, const float *g2,
                              const int32_t *rows_b, const int32_t *rows_t, int n_rows,
                              const int32_t *idx, const int32_t *keff, const float *dout,
                              double *dQ, double *dg1, double *dK, double *dV, double *dg2)
{
    const int d = p->d_h, grp = p->n_h / p->n_kv;
    const double scale = p->sm_scale > 0.0 ? p->sm_scale : 1.0 / sqrt((double)d);
    const size_t qrow = (size_t)p->n_h * d, kvb = (size_t)p->Lk * p->n_kv * d;
    memset(dK, 0, sizeof(double) * kvb * (size_t)p->B);
    memset(dV, 0, sizeof(double) * kvb * (size_t)p->B);
    memset(dg2, 0, sizeof(double) * kvb * (size_t)p->B);
#pragma omp parallel for schedule(dynamic, 1)
    for (int g = 0; g < p->n_kv; ++g) {
        double *a = (double *)malloc(sizeof(double) * (size_t)(p->k_max > 0 ? p->k_max : 1));
        double *da = (double *)malloc(sizeof(double) * (size_t)(p->k_max > 0 ? p->k_max : 1));
        double *dov = (double *)malloc(sizeof(double) * (size_t)d);
        for (int r = 0; r < n_rows; ++r) {
            const int b = rows_b[r], t = rows_t[r], ke = keff[r];
            const int32_t *S = idx + (size_t)r * p->k_max;
            for (int h = g * grp; h < (g + 1) * grp; ++h) {
                const float *q = Q + ((size_t)b * p->Lq + t) * qrow + (size_t)h * d;
                const float *gl = g1 + ((size_t)b * p->Lq + t) * qrow + (size_t)h * d;
                const float *dy = dout + (size_t)r * qrow + (size_t)h * d;
                double zmax = -INFINITY, den = 0.0;
                for (int j = 0; j < ke; ++j) {
                    const float *ks = K + b * kvb + ((size_t)S[j] * p->n_kv + g) * d;
                    double dot = 0.0;
                    for (int c = 0; c < d; ++c) dot += (double)q[c] * (double)ks[c];
                    a[j] = dot * scale;
                    if (a[j] > zmax) zmax = a[j];
                }
                for (int j = 0; j < ke; ++j) { a[j] = exp(a[j] - zmax); den += a[j]; }
                for (int j = 0; j < ke; ++j) a[j] /= den;
                /* o, do, dg1 */
                for (int c = 0; c < d; ++c) {
                    double o = 0.0;
                    for (int j = 0; j < ke; ++j) {
                        const size_t at = b * kvb + ((size_t)S[j] * p->n_kv + g) * d + c;
                        o += a[j] * ((double)V[at] * sigmoid_d((double)g2[at]));
                    }
                    const double s1 = sigmoid_d((double)gl[c]);
                    dov[c] = (double)dy[c] * s1;
                    dg1[(size_t)r * qrow + (size_t)h * d + c] = (double)dy[c] * o * s1 * (1.0 - s1);
                }
                /* da_j and the softmax backward */
                double dsum = 0.0;
                for (int j = 0; j < ke; ++j) {
                    double acc = 0.0;
                    for (int c = 0; c < d; ++c) {
                        const size_t at = b * kvb + ((size_t)S[j] * p->n_kv + g) * d + c;
                        acc += dov[c] * ((double)V[at] * sigmoid_d((double)g2[at]));
                    }
                    da[j] = acc;
                    dsum += a[j] * acc;
                }
                for (int c = 0; c < d; ++c) dQ[(size_t)r * qrow + (size_t)h * d + c] = 0.0;
                for (int j = 0; j < ke; ++j) {
                    const double dz = a[j] * (da[j] - dsum);
                    const size_t row = b * kvb + ((size_t)S[j] * p->n_kv + g) * d;
                    for (int c = 0; c < d; ++c) {
                        dQ[(size_t)r * qrow + (size_t)h * d + c] += scale * dz * (double)K[row + c];
                        dK[row + c] += scale * dz * (double)q[c];
                        const double s2 = sigmoid_d((double)g2[row + c]);
                        const double dvg = a[j] * dov[c];
                        dV[row + c] += dvg * s2;
                        dg2[row + c] += dvg * (double)V[row + c] * s2 * (1.0 - s2);
                    }
                }
            }
        }
        free(a); free(da); free(dov);
    }
}

/* Running mean of the score variance (text below Eq. 8: the normaliser of the budget is an exponential
 * moving average of the score variance across the batch).  The paper gives neither the momentum nor the
 * start value: both are the caller's.  mean_var = mean of the n row variances; returns
 * momentum * v_bar + (1 - momentum) * mean_var. */
double gsa_oracle_vbar_update(double v_bar, double momentum, const float *var, int64_t n, double *mean_var)
{
    double s = 0.0;
    for (int64_t i = 0; i < n; ++i) s += (double)var[i];
    const double m = n > 0 ? s / (double)n : 0.0;
    if (mean_var) *mean_var = m;
    return momentum * v_bar + (1.0 - momentum) * m;
}

/* ---- the indexer's sparse-phase loss (Sec. 5.1, Eq. 14) ------------------------ */
/* Target of the loss: the attention distribution on S_t.  Eq. 11 gives one distribution per head; the
 * indexer score has no head index, so the target is their mean over the n_h heads (each sums to 1 over
 * S_t, hence so does the mean).  pbar: [n_rows, k_max], entries past keff are 0. */
void gsa_oracle_attn_probs_mean_rows(const gsa_oracle_params *p, const float *Q, const float *K,
                                     const int32_t *rows_b, const int32_t *rows_t, int n_rows,
                                     const int32_t *idx, const int32_t *keff, double *pbar)
{
    const int d = p->d_h, grp = p->n_h / p->n_kv;
    const double scale = p->sm_scale > 0.0 ? p->sm_scale : 1.0 / sqrt((double)d);
    const size_t qrow = (size_t)p->n_h * d, kvb = (size_t)p->Lk * p->n_kv * d;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
        const int b = rows_b[r], t = rows_t[r], ke = keff[r];
        const int32_t *S = idx + (size_t)r * p->k_max;
        double *out = pbar + (size_t)r * p->k_max;
        double *z = (double *)malloc(sizeof(double) * (size_t)(ke > 0 ? ke : 1));
        for (int j = 0; j < p->k_max; ++j) out[j] = 0.0;
        for (int h = 0; h < p->n_h; ++h) {
            const int g = h / grp;
            const float *q = Q + ((size_t)b * p->Lq + t) * qrow + (size_t)h * d;
            double zmax = -INFINITY, den = 0.0;
            for (int j = 0; j < ke; ++j) {
                const float *ks = K + b * kvb + ((size_t)S[j] * p->n_kv + g) * d;
                double dot = 0.0;
                for (int c = 0; c < d; ++c) dot += (double)q[c] * (double)ks[c];
                z[j] = dot * scale;
                if (z[j] > zmax) zmax = z[j];
            }
            for (int j = 0; j < ke; ++j) { z[j] = exp(z[j] - zmax); den += z[j]; }
            for (int j = 0; j < ke; ++j) out[j] += z[j] / den / (double)p->n_h;
        }
        free(z);
    }
}

/* Eq. 14 for the listed rows, with the target distribution given (a constant: no derivative flows into it):
 *     loss_t = sum_{j in S_t} pbar_j * (log pbar_j - log q_j),   q = softmax_j(I[t, s_j]),   0 log 0 = 0,
 * I from Eq. 7 (or Eq. 3 with act = 1).  Derivatives of sum_t loss_t by the chain rule:
 *     dI_j = q_j * sum_i pbar_i - pbar_j                       (= q_j - pbar_j for a normalised target)
 *     with x_ij = q^I_i . k^I_{s_j} + b_i and f = sigmoid (or ReLU):
 *     dw_i = sum_j dI_j f(x_ij),   dx_ij = dI_j w_i f'(x_ij),
 *     dq^I_i = sum_j dx_ij k^I_{s_j},   dk^I[s_j] += sum_i dx_ij q^I_i,   db_i += sum_j dx_ij.
 * loss: [n_rows]; dqI: [n_rows, HI, dI]; dw: [n_rows, HI]; dkI: [B, Lk, dI] and dbI: [HI], zeroed here and
 * summed over the listed rows.  Rows run one after the other (no two threads add into dkI). */
void gsa_oracle_indexer_kl_rows(const gsa_oracle_params *p, const float *qI, const float *kI,
                                const float *w, const float *bI, const int32_t *rows_b,
                                const int32_t *rows_t, int n_rows, const int32_t *idx,
                                const int32_t *keff, const double *pbar, double *loss, double *dqI,
                                double *dw, double *dkI, double *dbI)
{
    const int H = p->HI, D = p->dI;
    memset(dkI, 0, sizeof(double) * (size_t)p->B * p->Lk * D);
    for (int i = 0; i < H; ++i) dbI[i] = 0.0;
    double *I = (double *)malloc(sizeof(double) * (size_t)(p->k_max > 0 ? p->k_max : 1));
    double *x = (double *)malloc(sizeof(double) * (size_t)(p->k_max > 0 ? p->k_max : 1) * H);
    for (int r = 0; r < n_rows; ++r) {
        const int b = rows_b[r], t = rows_t[r], ke = keff[r];
        const int32_t *S = idx + (size_t)r * p->k_max;
        const double *pb = pbar + (size_t)r * p->k_max;
        const float *q = qI + ((size_t)b * p->Lq + t) * H * D;
        const float *wt = w + ((size_t)b * p->Lq + t) * H;
        double imax = -INFINITY, den = 0.0, psum = 0.0;
        for (int j = 0; j < ke; ++j) {
            const float *k = kI + ((size_t)b * p->Lk + S[j]) * D;
            double acc = 0.0;
            for (int i = 0; i < H; ++i) {
                double v = bI ? (double)bI[i] : 0.0;
                for (int c = 0; c < D; ++c) v += (double)q[i * D + c] * (double)k[c];
                x[(size_t)j * H + i] = v;
                acc += (double)wt[i] * (p->act == 1 ? (v > 0.0 ? v : 0.0) : sigmoid_d(v));
            }
            I[j] = acc;
            if (acc > imax) imax = acc;
            psum += pb[j];
        }
        for (int j = 0; j < ke; ++j) den += exp(I[j] - imax);
        const double logden = imax + log(den);
        double L = 0.0;
        for (int j = 0; j < ke; ++j)
            if (pb[j] > 0.0) L += pb[j] * (log(pb[j]) - (I[j] - logden));
        loss[r] = L;
        for (int i = 0; i < H; ++i) {
            dw[(size_t)r * H + i] = 0.0;
            for (int c = 0; c < D; ++c) dqI[((size_t)r * H + i) * D + c] = 0.0;
        }
        for (int j = 0; j < ke; ++j) {
            const double dI = exp(I[j] - logden) * psum - pb[j];
            const float *k = kI + ((size_t)b * p->Lk + S[j]) * D;
            double *dk = dkI + ((size_t)b * p->Lk + S[j]) * D;
            for (int i = 0; i < H; ++i) {
                const double v = x[(size_t)j * H + i];
                double f, fp;
                if (p->act == 1) { f = v > 0.0 ? v : 0.0; fp = v > 0.0 ? 1.0 : 0.0; }
                else { f = sigmoid_d(v); fp = f * (1.0 - f); }
                dw[(size_t)r * H + i] += dI * f;
                const double dx = dI * (double)wt[i] * fp;
                dbI[i] += dx;
                for (int c = 0; c < D; ++c) {
                    dqI[((size_t)r * H + i) * D + c] += dx * (double)k[c];
                    dk[c] += dx * (double)q[i * D + c];
                }
            }
        }
    }
    free(I); free(x);
}
