// Shared declarations of the sm_100a GSA kernels: argument structs, small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "gsa.h"

namespace gsa {

// A contiguous block of work: batch elements b0 .. b0+nb-1, query rows q_begin .. q_begin+R-1
// of each.  Local row index lr = (b - b0) * R + (t - q_begin).
struct RowRange {
    int32_t b0, nb, q_begin, R;
    __host__ __device__ int32_t rows() const { return nb * R; }
};

// Where the index sets of a RowRange live: row (b, t) starts at
// idx + ((b - b_origin) * batch_rows + (t - t_origin)) * k_max, kt likewise without k_max.
struct IdxLayout {
    int32_t b_origin, t_origin, batch_rows;
    __host__ __device__ int64_t row(int32_t b, int32_t t) const {
        return (int64_t)(b - b_origin) * batch_rows + (t - t_origin);
    }
};

constexpr int kStatusBytes = 256;   // head of every workspace: device status word, counters, padding
constexpr int kStatusFallbackWord = 1;   // int32 word: rows on which top-k selection took its whole-row fallback

// device status word values: which bounded wait of a tensor-core pipeline ran out (copy producer, MMA
// issuer, epilogue), or that a kernel met an index set entry / budget outside its range
enum : int32_t { kDevOk = 0, kDevTimeoutTma = 1, kDevTimeoutMma = 2, kDevTimeoutEpi = 3, kDevBadIndex = 6 };

// Status word of the call this host thread is enqueueing: the entry point sets it (the head of the call's
// workspace, or null when the call has none) and the launchers copy it into their kernels' arguments.
extern thread_local int32_t* t_dev_status;

// Limit of every bounded device-side wait, in SM clock cycles (about one second unless the debug knob
// changed it), and the fault-injection switch of the same knob: the copy producers of the tensor-core
// kernels leave out their first copy, so the barrier it would complete is one that nothing sets.
long long wait_limit_cycles();
bool withhold_first_copy();

extern std::atomic<int64_t> g_launches;   // host-side launch counter (any host thread may launch)

// multiprocessors of the current device (cached per device; 148 if the query fails)
int sm_count();

// Profiling timeline (off unless gsa_profile_set_timeline armed one): while gsa_forward enqueues its work,
// every launcher records the next event of the caller's array behind the stage it just enqueued and notes
// which stage the interval that ends there belongs to.
enum : int32_t { kStageIndexer = 0, kStageSelect = 1, kStageValueGate = 2, kStageRangeCuts = 3, kStageAttn = 4,
                 kStageFinalize = 5 };
void timeline_mark(int32_t stage, cudaStream_t st);

// ---- stage launchers (host) ----------------------------------------------------------------
cudaError_t launch_indexer(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* qI,
                           const __nv_bfloat16* kI, const float* w, const float* bI, float* scores,
                           int64_t row_stride, int32_t* dev_status, cudaStream_t st);

cudaError_t launch_select(const gsa_params_t& p, RowRange rr, const float* scores,
                          int64_t row_stride, int32_t* idx, int32_t* kt, float* var,
                          IdxLayout il, int32_t* fallback_rows /*nullable counter*/, cudaStream_t st);

cudaError_t launch_value_gate(const __nv_bfloat16* V, const __nv_bfloat16* g2, __nv_bfloat16* Vg,
                              int64_t n_elems, cudaStream_t st);

// Backward of sparse gated attention.  Query-major half (gsa_attn_bwd.cu): dQ, dg1 for the rows of rr, and
// per (row, head) do = dout * sigmoid(g1), the softmax statistics lse2 and delta for the key-major half
// (gsa_attn_bwd_keys.cu), which inverts the index sets inside invert_ws (attn_bwd_invert_bytes) and writes
// dK, dV, dg2 for every key.
bool attn_bwd_supported(const gsa_params_t& p);
cudaError_t launch_sparse_attn_bwd(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* Q,
                                   const __nv_bfloat16* K, const __nv_bfloat16* Vg, const __nv_bfloat16* g1,
                                   const __nv_bfloat16* out, const __nv_bfloat16* dout, const int32_t* idx,
                                   const int32_t* kt, IdxLayout il, __nv_bfloat16* dQ, __nv_bfloat16* dg1,
                                   __nv_bfloat16* dOs, float* lse2, float* delta, float* pbar,
                                   const float* lse_in /*nullable: the forward's saved statistics*/, void* range_ws,
                                   cudaStream_t st);
size_t attn_bwd_range_bytes(const gsa_params_t& p);      // scratch of the query-major half when Lk spans several key ranges
size_t attn_bwd_invert_bytes(const gsa_params_t& p, int32_t rows_per_batch);
cudaError_t launch_sparse_attn_bwd_keys(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* Q,
                                        const __nv_bfloat16* dOs, const __nv_bfloat16* K, const __nv_bfloat16* V,
                                        const __nv_bfloat16* Vg, const __nv_bfloat16* g2, const float* lse2,
                                        const float* delta, const int32_t* idx, const int32_t* kt, IdxLayout il,
                                        void* invert_ws, __nv_bfloat16* dK, __nv_bfloat16* dV, __nv_bfloat16* dg2,
                                        cudaStream_t st);
// The indexer's sparse-phase loss (gsa_indexer_loss.cu): its target (mean over the heads of the attention
// distribution on S_t; pbar is zeroed inside) and the loss with its derivatives (dkI32: B * Lk * dI floats
// of scratch, zeroed inside; dbI may be null).
cudaError_t launch_attn_probs_mean(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* Q,
                                   const __nv_bfloat16* K, const int32_t* idx, const int32_t* kt, IdxLayout il,
                                   float* pbar, cudaStream_t st);
cudaError_t launch_indexer_kl(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* qI,
                              const __nv_bfloat16* kI, const float* w, const float* bI, const int32_t* idx,
                              const int32_t* kt, IdxLayout il, const float* pbar, float* loss,
                              __nv_bfloat16* dqI, __nv_bfloat16* dkI, float* dw, float* dbI, float* dkI32,
                              cudaStream_t st);
// Running mean of the score variance (gsa_vbar.cu)
cudaError_t launch_vbar_update(const float* var, int64_t n, float momentum, float* v_bar, float* mean_var,
                               cudaStream_t st);

// k_mode 3: S_t = every visible key (idx = 0, 1, ..., kt = number of visible keys, var = 0)
cudaError_t launch_all_visible(const gsa_params_t& p, RowRange rr, int32_t* idx, int32_t* kt, float* var,
                               IdxLayout il, cudaStream_t st);

// Optional progress report of launch_sparse_attn: output rows become final range by range (a query
// row is final once the key range holding its last visible key has been processed).  events[i], which
// the caller created, is recorded when rows t_lo[i] <= t < t_hi[i] of every batch element are final.
struct AttnProgress {
    cudaEvent_t* events;
    int cap;
    int n;
    int32_t t_lo[64], t_hi[64];
};

cudaError_t launch_sparse_attn(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* Q,
                               const __nv_bfloat16* K, const __nv_bfloat16* V,
                               const __nv_bfloat16* g1, const __nv_bfloat16* g2 /*nullable*/,
                               const int32_t* idx, const int32_t* kt, IdxLayout il,
                               __nv_bfloat16* out, void* scratch, cudaStream_t st,
                               AttnProgress* progress = nullptr, float* lse = nullptr);

// bytes of device scratch launch_sparse_attn needs for `p` (softmax state slots, range cuts)
size_t attn_scratch_bytes(const gsa_params_t& p);
// keys per L2-resident key range of the sparse-attention gather (tuning knob)
void set_attn_range_keys(int keys);
int attn_range_keys();

// device address, on the current device, of the library's built-in scratch array (status word at
// its start, then the gated values of the allocation-free entry point)
cudaError_t static_scratch_address(void** ptr);

// upstream projections: C = H * Wt^T routed to q^I, k^I, head weights (sigmoid), g1 and g2 logits
int project_columns(const gsa_params_t& p);
cudaError_t launch_project(const gsa_params_t& p, int d_model, const __nv_bfloat16* H, const __nv_bfloat16* Wt,
                           __nv_bfloat16* qI, __nv_bfloat16* kI, float* w, __nv_bfloat16* g1, __nv_bfloat16* g2,
                           int32_t* dev_status, cudaStream_t st);

cudaError_t launch_gemm_bf16(int M, int K, int N, const __nv_bfloat16* A, const __nv_bfloat16* Bt, __nv_bfloat16* C,
                             int32_t* dev_status, cudaStream_t st);

// ---- device helpers ------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}

// Index sets and budgets come from the caller.  Every kernel that takes them applies the same rule, so that a
// corrupt set cannot take an access out of its tensor: the budget is clamped to [0, k_max]; a position used
// as a gather address is clamped into [0, Lk); an entry that would be scattered to (counters, lists) is
// skipped unless it lies in [0, Lk).
__device__ __forceinline__ int32_t clamp_budget(int32_t kt, int32_t k_max) { return min(max(kt, 0), k_max); }
__device__ __forceinline__ int32_t clamp_pos(int32_t s, int32_t Lk) { return min(max(s, 0), Lk - 1); }
__device__ __forceinline__ bool key_in_range(int32_t s, int32_t Lk) { return (uint32_t)s < (uint32_t)Lk; }
// the same two rules, reporting what they had to correct through the status word (first report wins)
__device__ __forceinline__ void report_bad_index(int32_t* dev_status) {
    if (dev_status) atomicCAS(dev_status, kDevOk, kDevBadIndex);
}
__device__ __forceinline__ int32_t checked_budget(int32_t kt, int32_t k_max, int32_t* dev_status) {
    if (kt < 0 || kt > k_max) report_bad_index(dev_status);
    return clamp_budget(kt, k_max);
}
__device__ __forceinline__ int32_t checked_pos(int32_t s, int32_t Lk, int32_t* dev_status) {
    if (key_in_range(s, Lk)) return s;
    report_bad_index(dev_status);
    return clamp_pos(s, Lk);
}

__device__ __forceinline__ float fast_sigmoid(float x) {
    // 1 / (1 + 2^(-x log2 e)); ex2.approx and rcp.approx are accurate to a few ulp
    float e, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(fminf(-1.4426950408889634f * x, 126.f)));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
    return r;
}

// Sigmoid of a value-gate logit (Eq. 9): 1/2 + 1/2 tanh(x/2), one special-function instruction.
// tanh.approx is good to 2^-11 relative; the gated value is rounded to bf16 (2^-9) right after.
__device__ __forceinline__ float gate_sigmoid(float x) {
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * x));
    return fmaf(0.5f, t, 0.5f);
}

__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(smem_dst), "l"(gsrc));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3,
                                            uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                                  uint32_t& r3, uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// ---- mbarrier (shared-memory barrier objects completed by arrivals and by async-copy bytes) --
constexpr uint32_t kSpinLimit = 1u << 24;        // polls
constexpr long long kSpinCycles = 1ll << 31;     // ~1 s of SM clock: no wait may last longer (default limit)
constexpr uint32_t kDrainPolls = 1u << 20;       // polls granted to a completion that is already on its way

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded wait of at most `limit` cycles; returns false if it gave up (and raises the CTA's abort flag)
// or if another thread of the CTA already had
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long limit) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t_start = clock64();
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 15u) == 15u) {
            if (*abort_flag) return false;
            if (clock64() - t_start > limit) break;
        }
    }
    *abort_flag = 1;
    return false;
}
// Wait of the give-up path, for a completion that is already on its way (a copy or an MMA issued earlier
// completes by itself): bounded by a poll count of its own, whatever the limit that ran out was.
__device__ __forceinline__ bool mbar_drain(uint32_t bar, uint32_t parity) {
    for (uint32_t p = 0; p < kDrainPolls; ++p)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

}  // namespace gsa
