// C ABI of the library (declared in include/gsa.h): argument checks, workspace plan,
// the slab loop of gsa_forward, and the host-buffer variant.
#include <math.h>
#include <stdio.h>

#include "gsa_common.cuh"

namespace gsa {

std::atomic<int64_t> g_launches{0};

int sm_count() {
    constexpr int kMaxDevices = 64;
    static std::atomic<int> cache[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
    int n = cache[dev].load(std::memory_order_relaxed);
    if (n <= 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cache[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}
thread_local int32_t* t_dev_status = nullptr;
static int32_t g_indexer_path = 0;
static std::atomic<long long> g_wait_cycles{kSpinCycles};
static std::atomic<int> g_withhold_first_copy{0};

long long wait_limit_cycles() { return g_wait_cycles.load(std::memory_order_relaxed); }
bool withhold_first_copy() { return g_withhold_first_copy.load(std::memory_order_relaxed) != 0; }
static cudaEvent_t g_prof_ev[3] = {nullptr, nullptr, nullptr};

// profiling timeline: the caller's event handles and host arrays; armed only inside gsa_forward
static cudaEvent_t* g_tl_events = nullptr;
static int32_t g_tl_cap = 0;
static int32_t* g_tl_stage = nullptr;
static int32_t* g_tl_count = nullptr;
static bool g_tl_armed = false;

static void timeline_begin(cudaStream_t st) {
    if (!g_tl_events || g_tl_cap < 2) return;
    *g_tl_count = 0;
    g_tl_armed = cudaEventRecord(g_tl_events[0], st) == cudaSuccess;
}
static void timeline_end() { g_tl_armed = false; }

void timeline_mark(int32_t stage, cudaStream_t st) {
    if (!g_tl_armed) return;
    const int32_t n = *g_tl_count;
    if (n + 1 >= g_tl_cap) return;                       // out of events: the rest of the call is not split up
    if (cudaEventRecord(g_tl_events[n + 1], st) != cudaSuccess) return;
    g_tl_stage[n] = stage;
    *g_tl_count = n + 1;
}

cudaError_t launch_indexer_simple(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* qI,
                                  const __nv_bfloat16* kI, const float* w, const float* bI,
                                  float* scores, int64_t row_stride, cudaStream_t st);
bool indexer_tc_supported(const gsa_params_t& p);
cudaError_t launch_indexer_tc(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* qI,
                              const __nv_bfloat16* kI, const float* w, const float* bI,
                              float* scores, int64_t row_stride, int32_t* dev_status,
                              cudaStream_t st);

bool indexer_rows_preferred(const gsa_params_t& p, RowRange rr);
cudaError_t launch_indexer_rows(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* qI,
                                const __nv_bfloat16* kI, const float* w, const float* bI, float* scores,
                                int64_t row_stride, cudaStream_t st);

cudaError_t launch_indexer(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* qI,
                           const __nv_bfloat16* kI, const float* w, const float* bI, float* scores,
                           int64_t row_stride, int32_t* dev_status, cudaStream_t st) {
    // few query rows per sequence (decode): stream the keys once per row instead of filling 32-query tiles
    if (g_indexer_path == 0 && indexer_rows_preferred(p, rr))
        return launch_indexer_rows(p, rr, qI, kI, w, bI, scores, row_stride, st);
    if (g_indexer_path == 0 && indexer_tc_supported(p))
        return launch_indexer_tc(p, rr, qI, kI, w, bI, scores, row_stride, dev_status, st);
    return launch_indexer_simple(p, rr, qI, kI, w, bI, scores, row_stride, st);
}

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool one_of(int v, std::initializer_list<int> l) {
    for (int x : l) if (x == v) return true;
    return false;
}

int check_params(const gsa_params_t* p) {
    if (!p) return GSA_ERR_INVALID_ARG;
    if (p->B < 1 || p->Lq < 1 || p->Lk < p->Lq || p->n_h < 1 || p->n_kv < 1) return GSA_ERR_INVALID_ARG;
    if (p->n_h % p->n_kv != 0) return GSA_ERR_INVALID_ARG;
    if (p->k_min < 1 || p->k_min > p->k_max || p->k_base < 1) return GSA_ERR_INVALID_ARG;
    if (p->k_mode < 0 || p->k_mode > 3) return GSA_ERR_INVALID_ARG;
    if (p->k_mode == 3 && p->k_max < p->Lk) return GSA_ERR_INVALID_ARG;
    if (p->act < 0 || p->act > 1) return GSA_ERR_INVALID_ARG;
    if (p->k_mode < 2 && !(p->v_bar > 0.f)) return GSA_ERR_INVALID_ARG;
    if (!one_of(p->d_h, {64, 128}) || !one_of(p->dI, {32, 64}) || !one_of(p->HI, {1, 2, 4, 8}))
        return GSA_ERR_UNSUPPORTED_SHAPE;
    if (!one_of(p->n_h / p->n_kv, {1, 2, 4, 8}) || !one_of(p->n_kv, {1, 2, 4, 8}))
        return GSA_ERR_UNSUPPORTED_SHAPE;
    if (p->k_max > 4096 || p->Lk >= (1 << 24)) return GSA_ERR_UNSUPPORTED_SHAPE;
    if ((int64_t)p->B * p->Lq >= (1ll << 31)) return GSA_ERR_UNSUPPORTED_SHAPE;
    return GSA_OK;
}

int row_range(const gsa_params_t* p, RowRange* rr) {
    const int qe = p->q_end <= 0 ? p->Lq : p->q_end;
    if (p->q_begin < 0 || p->q_begin >= qe || qe > p->Lq) return GSA_ERR_INVALID_ARG;
    rr->b0 = 0; rr->nb = p->B; rr->q_begin = p->q_begin; rr->R = qe - p->q_begin;
    return GSA_OK;
}

struct WsPlan {
    int64_t row_stride;
    int32_t slab_rows;
    bool prepass;                  // Eq. 9 as a pre-pass (prefill) or inside the gather (decode)
    size_t slab_off, vg_off, idx_off, kt_off, attn_off, total;
};

WsPlan plan_ws(const gsa_params_t& p, int32_t slab_rows) {
    WsPlan w;
    w.row_stride = (int64_t)align_up((size_t)p.Lk, 32);
    const int64_t rows_total = (int64_t)p.B * p.Lq;
    if (slab_rows <= 0) {
        // measured on B200 at L = 128K: per-slab launch and tail costs outweigh L2 residency of the
        // slab, so the default is large (about 4 GiB of score rows: indexer + selection take 45.8 / 41.9 /
        // 40.4 / 39.2 ms with slabs of 1024 / 2048 / 4096 / 8192 rows)
        const int64_t target = 4ll << 30;
        int64_t r = target / (w.row_stride * 4);
        r = r / 32 * 32;
        slab_rows = (int32_t)(r < 32 ? 32 : r);
    }
    if (slab_rows > rows_total) slab_rows = (int32_t)rows_total;
    w.slab_rows = slab_rows;
    // gating the whole V once costs 3 passes over it; gating inside the gather costs one more
    // gathered row per selected key.
    w.prepass = (int64_t)p.Lq * p.k_base > 3ll * p.Lk;
    size_t off = kStatusBytes;
    w.slab_off = off; off += align_up((size_t)slab_rows * w.row_stride * 4, 256);
    w.vg_off = off;   off += w.prepass ? align_up((size_t)p.B * p.Lk * p.n_kv * p.d_h * 2, 256) : 0;
    w.idx_off = off;  off += align_up((size_t)rows_total * p.k_max * 4, 256);
    w.kt_off = off;   off += align_up((size_t)rows_total * 4, 256);
    w.attn_off = off; off += align_up(attn_scratch_bytes(p), 256);
    w.total = off;
    return w;
}

int cuda_rc(cudaError_t e) {
    if (e == cudaSuccess) return GSA_OK;
    fprintf(stderr, "gsa: CUDA error: %s\n", cudaGetErrorString(e));
    return GSA_ERR_CUDA;
}

}  // namespace
}  // namespace gsa

using namespace gsa;
typedef __nv_bfloat16 bf16;

extern "C" {

int gsa_workspace_bytes(const gsa_params_t* p, int32_t slab_rows, size_t* bytes) {
    int rc = check_params(p);
    if (rc) return rc;
    if (!bytes || slab_rows < 0) return GSA_ERR_INVALID_ARG;
    *bytes = plan_ws(*p, slab_rows).total;
    return GSA_OK;
}

int gsa_indexer_scores(const gsa_params_t* p, const void* qI, const void* kI, const float* w,
                       const float* bI, float* scores, int64_t row_stride, void* ws,
                       size_t ws_bytes, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    RowRange rr;
    if ((rc = row_range(p, &rr))) return rc;
    if (!qI || !kI || !w || !scores || !aligned16(qI) || !aligned16(kI) || !aligned16(w) || !aligned16(scores))
        return GSA_ERR_INVALID_ARG;
    if (row_stride < p->Lk || row_stride % 4 != 0) return GSA_ERR_INVALID_ARG;
    if (!ws || ws_bytes < (size_t)kStatusBytes || !aligned16(ws)) return GSA_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    t_dev_status = (int32_t*)ws;
    cudaError_t e = cudaMemsetAsync(ws, 0, kStatusBytes, st);
    if (e != cudaSuccess) return cuda_rc(e);
    return cuda_rc(launch_indexer(*p, rr, (const bf16*)qI, (const bf16*)kI, w, bI, scores, row_stride,
                                  (int32_t*)ws, st));
}

int gsa_project_columns(const gsa_params_t* p, int32_t* columns) {
    int rc = check_params(p);
    if (rc) return rc;
    if (!columns) return GSA_ERR_INVALID_ARG;
    *columns = project_columns(*p);
    return GSA_OK;
}

int gsa_project(const gsa_params_t* p, int32_t d_model, const void* H, const void* Wt, void* qI, void* kI,
                float* w, void* g1_logits, void* g2_logits, void* ws, size_t ws_bytes, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    if (p->Lq != p->Lk) return GSA_ERR_INVALID_ARG;           // one hidden state per position, queries = keys
    if (d_model < 64 || d_model % 8 != 0) return GSA_ERR_UNSUPPORTED_SHAPE;
    if ((int64_t)p->B * p->Lk >= (1ll << 31)) return GSA_ERR_UNSUPPORTED_SHAPE;
    const void* ptrs[] = {H, Wt, qI, kI, w, g1_logits, g2_logits};
    for (const void* q : ptrs) if (!q || !aligned16(q)) return GSA_ERR_INVALID_ARG;
    if (!ws || ws_bytes < (size_t)kStatusBytes || !aligned16(ws)) return GSA_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    t_dev_status = (int32_t*)ws;
    cudaError_t e = cudaMemsetAsync(ws, 0, kStatusBytes, st);
    if (e != cudaSuccess) return cuda_rc(e);
    return cuda_rc(launch_project(*p, d_model, (const bf16*)H, (const bf16*)Wt, (bf16*)qI, (bf16*)kI, w,
                                  (bf16*)g1_logits, (bf16*)g2_logits, (int32_t*)ws, st));
}

int gsa_output_projection(const gsa_params_t* p, int32_t d_model, const void* attn_out, const void* Wo_t, void* u,
                          void* ws, size_t ws_bytes, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    if (d_model < 8 || d_model % 8 != 0) return GSA_ERR_UNSUPPORTED_SHAPE;
    if ((int64_t)p->B * p->Lq >= (1ll << 31)) return GSA_ERR_UNSUPPORTED_SHAPE;
    const void* ptrs[] = {attn_out, Wo_t, u};
    for (const void* q : ptrs) if (!q || !aligned16(q)) return GSA_ERR_INVALID_ARG;
    if (!ws || ws_bytes < (size_t)kStatusBytes || !aligned16(ws)) return GSA_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    t_dev_status = (int32_t*)ws;
    cudaError_t e = cudaMemsetAsync(ws, 0, kStatusBytes, st);
    if (e != cudaSuccess) return cuda_rc(e);
    return cuda_rc(launch_gemm_bf16(p->B * p->Lq, p->n_h * p->d_h, d_model, (const bf16*)attn_out, (const bf16*)Wo_t,
                                    (bf16*)u, (int32_t*)ws, st));
}

int gsa_adaptive_topk(const gsa_params_t* p, const float* scores, int64_t row_stride, int32_t* idx,
                      int32_t* kt, float* var, void* ws, size_t ws_bytes, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    RowRange rr;
    if ((rc = row_range(p, &rr))) return rc;
    if (!scores || !idx || !kt || !aligned16(scores) || !aligned16(idx)) return GSA_ERR_INVALID_ARG;
    if (row_stride < p->Lk || row_stride % 4 != 0) return GSA_ERR_INVALID_ARG;
    IdxLayout il{0, rr.q_begin, rr.R};
    int32_t* fb = nullptr;
    t_dev_status = nullptr;
    if (ws && aligned16(ws) && ws_bytes >= (size_t)kStatusBytes) {
        cudaError_t e = cudaMemsetAsync(ws, 0, kStatusBytes, (cudaStream_t)stream);
        if (e != cudaSuccess) return cuda_rc(e);
        fb = (int32_t*)ws + kStatusFallbackWord;
        t_dev_status = (int32_t*)ws;
    }
    return cuda_rc(launch_select(*p, rr, scores, row_stride, idx, kt, var, il, fb, (cudaStream_t)stream));
}

// workspace of the per-stage attention call: [status][attention scratch][V' (optional)]
static size_t attn_ws_bytes(const gsa_params_t& p, bool with_prepass) {
    size_t n = kStatusBytes + align_up(attn_scratch_bytes(p), 256);
    if (with_prepass) n += align_up((size_t)p.B * p.Lk * p.n_kv * p.d_h * 2, 256);
    return n;
}

// workspace of the backward call: [status][V' bf16][do bf16][lse2 fp32][delta fp32][key-range scratch][inverted index sets]
struct BwdPlan {
    size_t vg_off, dos_off, lse_off, delta_off, range_off, inv_off, total;
};
static BwdPlan plan_bwd_ws(const gsa_params_t& p, int32_t rows_per_batch) {
    BwdPlan w;
    size_t off = kStatusBytes;
    w.vg_off = off;    off += align_up((size_t)p.B * p.Lk * p.n_kv * p.d_h * 2, 256);
    w.dos_off = off;   off += align_up((size_t)p.B * p.Lq * p.n_h * p.d_h * 2, 256);
    w.lse_off = off;   off += align_up((size_t)p.B * p.Lq * p.n_h * 4, 256);
    w.delta_off = off; off += align_up((size_t)p.B * p.Lq * p.n_h * 4, 256);
    w.range_off = off; off += attn_bwd_range_bytes(p);
    w.inv_off = off;   off += attn_bwd_invert_bytes(p, rows_per_batch);
    w.total = off;
    return w;
}

int gsa_attn_bwd_workspace_bytes(const gsa_params_t* p, size_t* bytes) {
    int rc = check_params(p);
    if (rc) return rc;
    RowRange rr;
    if ((rc = row_range(p, &rr))) return rc;
    if (!bytes) return GSA_ERR_INVALID_ARG;
    *bytes = plan_bwd_ws(*p, rr.R).total;
    return GSA_OK;
}

int gsa_sparse_gated_attn_bwd(const gsa_params_t* p, const void* Q, const void* K, const void* V,
                              const void* g1_logits, const void* g2_logits, const int32_t* idx,
                              const int32_t* kt, const void* out, const void* dout, void* dQ, void* dK,
                              void* dV, void* dg1, void* dg2, float* pbar, const float* lse, void* ws,
                              size_t ws_bytes, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    RowRange rr;
    if ((rc = row_range(p, &rr))) return rc;
    if (!attn_bwd_supported(*p)) return GSA_ERR_UNSUPPORTED_SHAPE;
    if ((int64_t)p->B * p->Lk >= (1ll << 31) || (int64_t)p->B * rr.R * p->k_max >= (1ll << 31))
        return GSA_ERR_UNSUPPORTED_SHAPE;
    const void* ptrs[] = {Q, K, V, g1_logits, g2_logits, idx, out, dout, dQ, dK, dV, dg1, dg2};
    for (const void* q : ptrs) if (!q || !aligned16(q)) return GSA_ERR_INVALID_ARG;
    if (!kt || (pbar && !aligned16(pbar)) || (lse && !aligned16(lse))) return GSA_ERR_INVALID_ARG;
    const BwdPlan wp = plan_bwd_ws(*p, rr.R);
    if (!ws || !aligned16(ws) || ws_bytes < wp.total) return GSA_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char* wsb = (char*)ws;
    bf16* Vg = (bf16*)(wsb + wp.vg_off);
    bf16* dOs = (bf16*)(wsb + wp.dos_off);
    float* lse2 = (float*)(wsb + wp.lse_off);
    float* delta = (float*)(wsb + wp.delta_off);
    t_dev_status = (int32_t*)ws;
    cudaError_t e = cudaMemsetAsync(ws, 0, kStatusBytes, st);
    if (e == cudaSuccess)
        e = launch_value_gate((const bf16*)V, (const bf16*)g2_logits, Vg, (int64_t)p->B * p->Lk * p->n_kv * p->d_h, st);
    IdxLayout il{0, rr.q_begin, rr.R};
    if (e == cudaSuccess && pbar) e = cudaMemsetAsync(pbar, 0, (size_t)rr.rows() * p->k_max * 4, st);
    if (e == cudaSuccess)
        e = launch_sparse_attn_bwd(*p, rr, (const bf16*)Q, (const bf16*)K, Vg, (const bf16*)g1_logits,
                                   (const bf16*)out, (const bf16*)dout, idx, kt, il, (bf16*)dQ, (bf16*)dg1,
                                   dOs, lse2, delta, pbar, lse, wsb + wp.range_off, st);
    if (e == cudaSuccess)
        e = launch_sparse_attn_bwd_keys(*p, rr, (const bf16*)Q, dOs, (const bf16*)K, (const bf16*)V, Vg,
                                        (const bf16*)g2_logits, lse2, delta, idx, kt, il, wsb + wp.inv_off,
                                        (bf16*)dK, (bf16*)dV, (bf16*)dg2, st);
    return cuda_rc(e);
}

int gsa_attn_probs_mean(const gsa_params_t* p, const void* Q, const void* K, const int32_t* idx,
                        const int32_t* kt, float* pbar, void* ws, size_t ws_bytes, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    RowRange rr;
    if ((rc = row_range(p, &rr))) return rc;
    if (!attn_bwd_supported(*p)) return GSA_ERR_UNSUPPORTED_SHAPE;
    if (!Q || !K || !idx || !kt || !pbar || !aligned16(Q) || !aligned16(K) || !aligned16(idx) || !aligned16(pbar))
        return GSA_ERR_INVALID_ARG;
    if (!ws || !aligned16(ws) || ws_bytes < (size_t)kStatusBytes) return GSA_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    t_dev_status = (int32_t*)ws;
    cudaError_t e = cudaMemsetAsync(ws, 0, kStatusBytes, st);
    IdxLayout il{0, rr.q_begin, rr.R};
    if (e == cudaSuccess) e = launch_attn_probs_mean(*p, rr, (const bf16*)Q, (const bf16*)K, idx, kt, il, pbar, st);
    return cuda_rc(e);
}

int gsa_indexer_kl_workspace_bytes(const gsa_params_t* p, size_t* bytes) {
    int rc = check_params(p);
    if (rc) return rc;
    if (!bytes) return GSA_ERR_INVALID_ARG;
    *bytes = kStatusBytes + align_up((size_t)p->B * p->Lk * p->dI * 4, 256);
    return GSA_OK;
}

int gsa_indexer_kl_bwd(const gsa_params_t* p, const void* qI, const void* kI, const float* w, const float* bI,
                       const int32_t* idx, const int32_t* kt, const float* pbar, float* loss, void* dqI,
                       void* dkI, float* dw, float* dbI, void* ws, size_t ws_bytes, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    RowRange rr;
    if ((rc = row_range(p, &rr))) return rc;
    const void* ptrs[] = {qI, kI, w, idx, pbar, dqI, dkI};
    for (const void* q : ptrs) if (!q || !aligned16(q)) return GSA_ERR_INVALID_ARG;
    if (!kt || !loss || !dw) return GSA_ERR_INVALID_ARG;
    size_t need = 0;
    gsa_indexer_kl_workspace_bytes(p, &need);
    if (!ws || !aligned16(ws) || ws_bytes < need) return GSA_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    t_dev_status = (int32_t*)ws;
    cudaError_t e = cudaMemsetAsync(ws, 0, kStatusBytes, st);
    IdxLayout il{0, rr.q_begin, rr.R};
    if (e == cudaSuccess)
        e = launch_indexer_kl(*p, rr, (const bf16*)qI, (const bf16*)kI, w, bI, idx, kt, il, pbar, loss, (bf16*)dqI,
                              (bf16*)dkI, dw, dbI, (float*)((char*)ws + kStatusBytes), st);
    return cuda_rc(e);
}

int gsa_vbar_update(const float* var, int64_t n, float momentum, float* v_bar, float* mean_var, void* stream) {
    if (!var || !v_bar || n < 1 || !(momentum >= 0.f && momentum <= 1.f)) return GSA_ERR_INVALID_ARG;
    return cuda_rc(launch_vbar_update(var, n, momentum, v_bar, mean_var, (cudaStream_t)stream));
}

int gsa_value_gate(const void* V, const void* g2_logits, void* V_gated, int64_t n_elems, void* stream) {
    if (!V || !g2_logits || !V_gated || n_elems < 1 || n_elems % 8 != 0) return GSA_ERR_INVALID_ARG;
    if (!aligned16(V) || !aligned16(g2_logits) || !aligned16(V_gated)) return GSA_ERR_INVALID_ARG;
    return cuda_rc(launch_value_gate((const bf16*)V, (const bf16*)g2_logits, (bf16*)V_gated, n_elems, (cudaStream_t)stream));
}

int gsa_attn_workspace_bytes(const gsa_params_t* p, int32_t with_value_gate_prepass, size_t* bytes) {
    int rc = check_params(p);
    if (rc) return rc;
    if (!bytes) return GSA_ERR_INVALID_ARG;
    *bytes = attn_ws_bytes(*p, with_value_gate_prepass != 0);
    return GSA_OK;
}

static int attn_fwd_impl(const gsa_params_t* p, const void* Q, const void* K, const void* V,
                         const void* g1_logits, const void* g2_logits, const int32_t* idx, const int32_t* kt,
                         void* out, float* lse, void* ws, size_t ws_bytes, void* stream) {
    int rc = check_params(p);
    if (rc) return rc;
    RowRange rr;
    if ((rc = row_range(p, &rr))) return rc;
    if (!Q || !K || !V || !g1_logits || !idx || !kt || !out) return GSA_ERR_INVALID_ARG;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(g1_logits) || !aligned16(out) ||
        !aligned16(idx) || (g2_logits && !aligned16(g2_logits)))
        return GSA_ERR_INVALID_ARG;
    if (!ws || !aligned16(ws) || ws_bytes < attn_ws_bytes(*p, false)) return GSA_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    t_dev_status = (int32_t*)ws;
    cudaError_t e0 = cudaMemsetAsync(ws, 0, kStatusBytes, st);
    if (e0 != cudaSuccess) return cuda_rc(e0);
    IdxLayout il{0, rr.q_begin, rr.R};
    char* wsb = (char*)ws;
    void* scratch = wsb + kStatusBytes;
    const bf16* Vuse = (const bf16*)V;
    const bf16* g2use = (const bf16*)g2_logits;
    if (g2_logits) {
        const WsPlan wp = plan_ws(*p, 0);
        // pre-pass when it pays and the caller gave room for V'; otherwise gate the gathered rows
        if (wp.prepass && ws_bytes >= attn_ws_bytes(*p, true)) {
            bf16* Vg = (bf16*)(wsb + attn_ws_bytes(*p, false));
            cudaError_t e = launch_value_gate((const bf16*)V, (const bf16*)g2_logits, Vg,
                                              (int64_t)p->B * p->Lk * p->n_kv * p->d_h, st);
            if (e != cudaSuccess) return cuda_rc(e);
            Vuse = Vg;
            g2use = nullptr;
        }
    }
    return cuda_rc(launch_sparse_attn(*p, rr, (const bf16*)Q, (const bf16*)K, Vuse, (const bf16*)g1_logits,
                                      g2use, idx, kt, il, (bf16*)out, scratch, st, nullptr, lse));
}

int gsa_sparse_gated_attn_fwd(const gsa_params_t* p, const void* Q, const void* K, const void* V,
                              const void* g1_logits, const void* g2_logits, const int32_t* idx,
                              const int32_t* kt, void* out, void* ws, size_t ws_bytes, void* stream) {
    return attn_fwd_impl(p, Q, K, V, g1_logits, g2_logits, idx, kt, out, nullptr, ws, ws_bytes, stream);
}

int gsa_sparse_gated_attn_fwd_lse(const gsa_params_t* p, const void* Q, const void* K, const void* V,
                                  const void* g1_logits, const void* g2_logits, const int32_t* idx,
                                  const int32_t* kt, void* out, float* lse, void* ws, size_t ws_bytes,
                                  void* stream) {
    if (!lse || !aligned16(lse)) return GSA_ERR_INVALID_ARG;
    return attn_fwd_impl(p, Q, K, V, g1_logits, g2_logits, idx, kt, out, lse, ws, ws_bytes, stream);
}

// The whole path.  `kv_ready` (may be NULL) is an event the stream waits for before anything reads
// Q, K, V or the gate logits: the indexer and the selection need only qI, kI and w, so a caller that is
// still copying the large tensors can let those copies run under the first two stages.
static int forward_impl(const gsa_params_t* p, const void* Q, const void* K, const void* V, const void* qI,
                        const void* kI, const float* w, const float* bI, const void* g1_logits,
                        const void* g2_logits, void* out, int32_t* idx_out, int32_t* kt_out, float* var_out,
                        int32_t slab_rows, void* ws, size_t ws_bytes, void* stream, cudaEvent_t kv_ready,
                        AttnProgress* progress) {
    int rc = check_params(p);
    if (rc) return rc;
    const bool dense = p->k_mode == 3;                 // every visible key: no indexer, no selection
    if (!Q || !K || !V || !g1_logits || !out || slab_rows < 0) return GSA_ERR_INVALID_ARG;
    if (!dense && (!qI || !kI || !w)) return GSA_ERR_INVALID_ARG;
    const void* ptrs[] = {Q, K, V, qI, kI, w, g1_logits, g2_logits, out, idx_out, kt_out, var_out};
    for (const void* q : ptrs) if (q && !aligned16(q)) return GSA_ERR_INVALID_ARG;
    const WsPlan wp = plan_ws(*p, slab_rows);
    if (!ws || !aligned16(ws) || ws_bytes < wp.total) return GSA_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char* wsb = (char*)ws;
    t_dev_status = (int32_t*)ws;
    cudaError_t e = cudaMemsetAsync(ws, 0, kStatusBytes, st);
    if (e != cudaSuccess) return cuda_rc(e);

    float* slab = (float*)(wsb + wp.slab_off);
    int32_t* idx = idx_out ? idx_out : (int32_t*)(wsb + wp.idx_off);
    int32_t* kt = kt_out ? kt_out : (int32_t*)(wsb + wp.kt_off);
    const IdxLayout il{0, 0, p->Lq};

    if (g_prof_ev[0]) cudaEventRecord(g_prof_ev[0], st);
    timeline_begin(st);
    struct TimelineGuard { ~TimelineGuard() { timeline_end(); } } timeline_guard;

    // Eq. 7, 8, 4 slab by slab: score rows live only inside the workspace
    if (dense) {
        RowRange all_rows{0, p->B, 0, p->Lq};
        if ((e = launch_all_visible(*p, all_rows, idx, kt, var_out, il, st)) != cudaSuccess) return cuda_rc(e);
    } else if (wp.slab_rows >= p->Lq) {
        const int nb_per = wp.slab_rows / p->Lq;
        for (int b0 = 0; b0 < p->B; b0 += nb_per) {
            RowRange rr{b0, (p->B - b0 < nb_per ? p->B - b0 : nb_per), 0, p->Lq};
            if ((e = launch_indexer(*p, rr, (const bf16*)qI, (const bf16*)kI, w, bI, slab, wp.row_stride,
                                    (int32_t*)ws, st)) != cudaSuccess) return cuda_rc(e);
            timeline_mark(kStageIndexer, st);
            if ((e = launch_select(*p, rr, slab, wp.row_stride, idx, kt, var_out, il, (int32_t*)ws + kStatusFallbackWord, st)) != cudaSuccess)
                return cuda_rc(e);
            timeline_mark(kStageSelect, st);
        }
    } else {
        for (int b = 0; b < p->B; ++b)
            for (int q0 = 0; q0 < p->Lq; q0 += wp.slab_rows) {
                RowRange rr{b, 1, q0, (p->Lq - q0 < wp.slab_rows ? p->Lq - q0 : wp.slab_rows)};
                if ((e = launch_indexer(*p, rr, (const bf16*)qI, (const bf16*)kI, w, bI, slab, wp.row_stride,
                                        (int32_t*)ws, st)) != cudaSuccess) return cuda_rc(e);
                timeline_mark(kStageIndexer, st);
                if ((e = launch_select(*p, rr, slab, wp.row_stride, idx, kt, var_out, il, (int32_t*)ws + kStatusFallbackWord, st)) != cudaSuccess)
                    return cuda_rc(e);
                timeline_mark(kStageSelect, st);
            }
    }

    if (g_prof_ev[1]) cudaEventRecord(g_prof_ev[1], st);
    if (kv_ready && (e = cudaStreamWaitEvent(st, kv_ready, 0)) != cudaSuccess) return cuda_rc(e);
    // Eq. 9: value gate (touches only V, so its place in the order is free; the pipeline of Sec. 3.2 lists it first)
    const bf16* Vuse = (const bf16*)V;
    const bf16* g2use = (const bf16*)g2_logits;
    if (g2_logits && wp.prepass) {
        bf16* Vg = (bf16*)(wsb + wp.vg_off);
        e = launch_value_gate((const bf16*)V, (const bf16*)g2_logits, Vg,
                              (int64_t)p->B * p->Lk * p->n_kv * p->d_h, st);
        if (e != cudaSuccess) return cuda_rc(e);
        timeline_mark(kStageValueGate, st);
        Vuse = Vg;
        g2use = nullptr;
    }
    // Eq. 11, 12, 10 over all rows
    RowRange all{0, p->B, 0, p->Lq};
    e = launch_sparse_attn(*p, all, (const bf16*)Q, (const bf16*)K, Vuse, (const bf16*)g1_logits, g2use, idx,
                           kt, il, (bf16*)out, wsb + wp.attn_off, st, progress);
    if (g_prof_ev[2]) cudaEventRecord(g_prof_ev[2], st);
    return cuda_rc(e);
}

int gsa_forward(const gsa_params_t* p, const void* Q, const void* K, const void* V, const void* qI,
                const void* kI, const float* w, const float* bI, const void* g1_logits,
                const void* g2_logits, void* out, int32_t* idx_out, int32_t* kt_out, float* var_out,
                int32_t slab_rows, void* ws, size_t ws_bytes, void* stream) {
    return forward_impl(p, Q, K, V, qI, kI, w, bI, g1_logits, g2_logits, out, idx_out, kt_out, var_out, slab_rows,
                        ws, ws_bytes, stream, nullptr, nullptr);
}

int gsa_forward_host_arena_bytes(const gsa_params_t* p, int32_t slab_rows, size_t* bytes) {
    int rc = check_params(p);
    if (rc) return rc;
    if (!bytes || slab_rows < 0) return GSA_ERR_INVALID_ARG;
    const size_t q = (size_t)p->B * p->Lq * p->n_h * p->d_h * 2, kv = (size_t)p->B * p->Lk * p->n_kv * p->d_h * 2;
    size_t t = 0;
    t += 3 * align_up(q, 256);                                   // Q, g1, out
    t += 3 * align_up(kv, 256);                                  // K, V, g2
    t += align_up((size_t)p->B * p->Lq * p->HI * p->dI * 2, 256);  // qI
    t += align_up((size_t)p->B * p->Lk * p->dI * 2, 256);          // kI
    t += align_up((size_t)p->B * p->Lq * p->HI * 4, 256);          // w
    t += 256;                                                    // bI
    t += align_up((size_t)p->B * p->Lq * 4, 256);                  // kt
    t += plan_ws(*p, slab_rows).total;
    *bytes = t;
    return GSA_OK;
}

int gsa_forward_host(const gsa_params_t* p, const void* Q, const void* K, const void* V, const void* qI,
                     const void* kI, const float* w, const float* bI, const void* g1_logits,
                     const void* g2_logits, void* out, int32_t* kt_out, int32_t slab_rows, void* arena,
                     size_t arena_bytes, void* stream) {
    size_t need = 0;
    int rc = gsa_forward_host_arena_bytes(p, slab_rows, &need);
    if (rc) return rc;
    if (!Q || !K || !V || !qI || !kI || !w || !g1_logits || !out) return GSA_ERR_INVALID_ARG;
    if (!arena || !aligned16(arena) || arena_bytes < need) return GSA_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t q = (size_t)p->B * p->Lq * p->n_h * p->d_h * 2, kv = (size_t)p->B * p->Lk * p->n_kv * p->d_h * 2;
    const size_t qi = (size_t)p->B * p->Lq * p->HI * p->dI * 2, ki = (size_t)p->B * p->Lk * p->dI * 2;
    const size_t wb = (size_t)p->B * p->Lq * p->HI * 4, ktb = (size_t)p->B * p->Lq * 4;
    char* a = (char*)arena;
    size_t off = 0;
    auto take = [&](size_t bytes) { char* r = a + off; off += align_up(bytes, 256); return r; };
    char *dQ = take(q), *dG1 = take(q), *dOut = take(q), *dK = take(kv), *dV = take(kv), *dG2 = take(kv);
    char *dqI = take(qi), *dkI = take(ki), *dw = take(wb), *dbI = take(256), *dkt = take(ktb);
    char* dws = a + off;
    // The small indexer inputs go first on the caller's stream; the large tensors follow on a second
    // stream and are awaited only before the value gate / attention, so they copy under the indexer and
    // the selection.  (The stream and the two events live for this call only.)
    cudaError_t e;
    cudaStream_t cs = nullptr;
    cudaEvent_t ev_go = nullptr, ev_kv = nullptr;
    if ((e = cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking)) != cudaSuccess) return cuda_rc(e);
    auto cleanup = [&]() {
        if (ev_go) cudaEventDestroy(ev_go);
        if (ev_kv) cudaEventDestroy(ev_kv);
        if (cs) { cudaStreamSynchronize(cs); cudaStreamDestroy(cs); }
    };
#define GSA_TRY(call) if ((e = (call)) != cudaSuccess) { cleanup(); return cuda_rc(e); }
    GSA_TRY(cudaEventCreateWithFlags(&ev_go, cudaEventDisableTiming));
    GSA_TRY(cudaEventCreateWithFlags(&ev_kv, cudaEventDisableTiming));
    GSA_TRY(cudaEventRecord(ev_go, st));                   // earlier work on `st` may still use the arena
    GSA_TRY(cudaStreamWaitEvent(cs, ev_go, 0));
#define GSA_H2D(dst, src, n, s_) GSA_TRY(cudaMemcpyAsync(dst, src, n, cudaMemcpyHostToDevice, s_))
    GSA_H2D(dqI, qI, qi, st); GSA_H2D(dkI, kI, ki, st); GSA_H2D(dw, w, wb, st);
    if (bI) GSA_H2D(dbI, bI, (size_t)p->HI * 4, st);
    GSA_H2D(dV, V, kv, cs);
    if (g2_logits) GSA_H2D(dG2, g2_logits, kv, cs);
    GSA_H2D(dK, K, kv, cs); GSA_H2D(dQ, Q, q, cs); GSA_H2D(dG1, g1_logits, q, cs);
#undef GSA_H2D
    GSA_TRY(cudaEventRecord(ev_kv, cs));
    // output rows become final key range by key range; each block goes back to the host on the copy
    // stream while the later ranges are still being computed
    constexpr int kMaxBlocks = 64;
    cudaEvent_t ev_rows[kMaxBlocks] = {};
    AttnProgress prog;
    prog.events = ev_rows; prog.cap = kMaxBlocks; prog.n = 0;
    for (int i = 0; i < kMaxBlocks; ++i) {
        if ((e = cudaEventCreateWithFlags(&ev_rows[i], cudaEventDisableTiming)) != cudaSuccess) break;
    }
    auto cleanup_rows = [&]() { for (int i = 0; i < kMaxBlocks; ++i) if (ev_rows[i]) cudaEventDestroy(ev_rows[i]); };
    if (e != cudaSuccess) { cleanup_rows(); cleanup(); return cuda_rc(e); }
    rc = forward_impl(p, dQ, dK, dV, dqI, dkI, (const float*)dw, bI ? (const float*)dbI : nullptr, dG1,
                      g2_logits ? dG2 : nullptr, dOut, nullptr, (int32_t*)dkt, nullptr, slab_rows, dws,
                      arena_bytes - off, st, ev_kv, &prog);
    if (rc) { cleanup_rows(); cleanup(); return rc; }
    const size_t row_bytes = (size_t)p->n_h * p->d_h * 2;
    int covered_to = 0;
    for (int i = 0; i < prog.n && e == cudaSuccess; ++i) {
        e = cudaStreamWaitEvent(cs, ev_rows[i], 0);
        for (int b = 0; b < p->B && e == cudaSuccess; ++b) {
            const size_t o = ((size_t)b * p->Lq + prog.t_lo[i]) * row_bytes;
            e = cudaMemcpyAsync((char*)out + o, dOut + o, (size_t)(prog.t_hi[i] - prog.t_lo[i]) * row_bytes,
                                cudaMemcpyDeviceToHost, cs);
        }
        covered_to = prog.t_hi[i];
    }
    if (e == cudaSuccess && covered_to < p->Lq) {
        // (more row blocks than events: the rest goes after the last kernel)
        for (int b = 0; b < p->B && e == cudaSuccess; ++b) {
            const size_t o = ((size_t)b * p->Lq + covered_to) * row_bytes;
            e = cudaMemcpyAsync((char*)out + o, dOut + o, (size_t)(p->Lq - covered_to) * row_bytes,
                                cudaMemcpyDeviceToHost, st);
        }
    }
    if (e == cudaSuccess && kt_out) e = cudaMemcpyAsync(kt_out, dkt, ktb, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(cs);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    cleanup_rows();
    if (e != cudaSuccess) { cleanup(); return cuda_rc(e); }
#undef GSA_TRY
    cleanup();
    int32_t dev = 0;
    return gsa_device_status(dws, stream, &dev);
}

int gsa_device_status(const void* ws, void* stream, int32_t* status_out) {
    if (!ws) {
        // the allocation-free entry point keeps its status word in the library's built-in array
        void* builtin = nullptr;
        cudaError_t e = static_scratch_address(&builtin);
        if (e != cudaSuccess) return cuda_rc(e);
        ws = builtin;
    }
    int32_t v = 0;
    cudaError_t e = cudaMemcpyAsync(&v, ws, sizeof(v), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_rc(e);
    if (status_out) *status_out = v;
    return v == kDevOk ? GSA_OK : (v == kDevBadIndex ? GSA_ERR_INDEX_RANGE : GSA_ERR_DEVICE_TIMEOUT);
}

int gsa_select_fallback_rows(const void* ws, void* stream, int32_t* rows_out) {
    if (!ws || !rows_out) return GSA_ERR_INVALID_ARG;
    int32_t v = 0;
    cudaError_t e = cudaMemcpyAsync(&v, (const int32_t*)ws + kStatusFallbackWord, sizeof(v), cudaMemcpyDeviceToHost,
                                    (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_rc(e);
    *rows_out = v;
    return GSA_OK;
}

int64_t gsa_launch_count(void) { return g_launches.load(); }

void gsa_debug_set_indexer_path(int32_t path) { g_indexer_path = path; }

void gsa_debug_set_attn_range_keys(int32_t keys) { set_attn_range_keys(keys); }

void gsa_debug_set_wait_limit(int64_t cycles, int32_t withhold_first_copy) {
    g_wait_cycles.store(cycles > 0 ? (long long)cycles : kSpinCycles, std::memory_order_relaxed);
    g_withhold_first_copy.store(withhold_first_copy != 0 ? 1 : 0, std::memory_order_relaxed);
}

void gsa_profile_set_timeline(void** events, int32_t capacity, int32_t* stage_out, int32_t* count_out) {
    const bool on = events && stage_out && count_out && capacity >= 2;
    g_tl_events = on ? (cudaEvent_t*)events : nullptr;
    g_tl_cap = on ? capacity : 0;
    g_tl_stage = on ? stage_out : nullptr;
    g_tl_count = on ? count_out : nullptr;
    g_tl_armed = false;
}

void gsa_profile_set_events(void* ev_begin, void* ev_selected, void* ev_end) {
    g_prof_ev[0] = (cudaEvent_t)ev_begin;
    g_prof_ev[1] = (cudaEvent_t)ev_selected;
    g_prof_ev[2] = (cudaEvent_t)ev_end;
}

const char* gsa_status_string(int s) {
    switch (s) {
        case GSA_OK: return "ok";
        case GSA_ERR_INVALID_ARG: return "invalid argument";
        case GSA_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case GSA_ERR_WORKSPACE: return "workspace missing or too small";
        case GSA_ERR_CUDA: return "CUDA error";
        case GSA_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
        case GSA_ERR_INDEX_RANGE: return "an index set entry or a budget was out of range (clamped or skipped on the device)";
        case GSA_ERR_STATIC_SCRATCH: return "problem exceeds the built-in scratch array (GSA_STATIC_SCRATCH_BYTES)";
    }
    return "unknown status";
}

}  // extern "C"
