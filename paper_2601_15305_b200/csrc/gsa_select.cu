// Adaptive sparsity controller: per query row, the variance of the visible scores (Eq. 8),
// the budget k_t, and the exact top-k_t positions (Eq. 4) by radix select.
//
// One CTA per row.  The fp32 row is staged in shared memory when it fits (one read of
// global memory); longer rows are re-read from global memory, where the forward pass keeps
// the current slab of rows L2-resident.  Passes over the row:
//   A   fp64 sum / sum of squares (second pass for the centred sum when the row is staged),
//       min and max of the order-preserving integer key
//   B*  histogram of (key - lo) >> shift over the live key range [lo, hi], 4096 bins; the
//       bin holding the k-th largest key becomes the next range.  At most three rounds
//       (32 key bits / 12 bits per round); two when the row spans at most two binades.
//   C   per-warp counts of keys above / equal to the threshold T over contiguous segments
//   D   ordered emission: keys > T, and the first (k - #greater) keys == T by position,
//       written in ascending position order.
// Ties therefore go to the lower position, and the output is unique.
#include "gsa_common.cuh"

namespace gsa {

namespace {

constexpr int kSelThreads = 512;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kBinsLog2 = 12;
constexpr int kBins = 1 << kBinsLog2;
constexpr int kBinsPerThread = kBins / kSelThreads;   // 8

struct SelectArgs {
    const float* scores;
    int64_t row_stride;
    int32_t* idx;
    int32_t* kt;
    float* var;
    RowRange rr;
    IdxLayout il;
    int32_t Lq, Lk;
    int32_t k_base, k_min, k_max, k_mode;
    float v_bar;
    int32_t cache_cap;    // floats of row cache in dynamic shared memory (0: none)
};

// monotone map fp32 -> uint32 (larger float <=> larger key); -0 is folded onto +0
__device__ __forceinline__ uint32_t order_key(float x) {
    uint32_t b = __float_as_uint(x + 0.0f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

struct SelShared {
    uint32_t hist[kBins];
    double red_a[kSelWarps];
    double red_b[kSelWarps];
    uint32_t red_min[kSelWarps];
    uint32_t red_max[kSelWarps];
    uint32_t warp_tot[kSelWarps];
    uint32_t seg_gt[kSelWarps];
    uint32_t seg_eq[kSelWarps];
    uint32_t found_bin;
    uint32_t found_above;
    double bc_a, bc_b;
    uint32_t bc_min, bc_max;
};

template <bool CACHED>
__device__ __forceinline__ float row_at(const float* __restrict__ grow, const float* srow, int i) {
    return CACHED ? srow[i] : __ldg(grow + i);
}

template <bool CACHED>
__global__ void __launch_bounds__(kSelThreads) gsa_select_kernel(const SelectArgs a) {
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    SelShared& sh = *reinterpret_cast<SelShared*>(dyn_smem);
    float* srow = reinterpret_cast<float*>(dyn_smem + ((sizeof(SelShared) + 15) / 16) * 16);

    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int lr = blockIdx.x;
    const int b = a.rr.b0 + lr / a.rr.R;
    const int t = a.rr.q_begin + lr % a.rr.R;
    const int n = a.Lk - a.Lq + t + 1;                       // visible keys
    const float* __restrict__ grow = a.scores + (int64_t)lr * a.row_stride;
    const int64_t orow = a.il.row(b, t);
    int32_t* __restrict__ out_idx = a.idx + orow * a.k_max;

    // ---- pass A: stage the row, fp64 moments, key range -------------------------------------
    double s1 = 0.0, s2 = 0.0;
    uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
    for (int i = tid; i < n; i += kSelThreads) {
        const float x = __ldg(grow + i);
        if (CACHED) srow[i] = x;
        const double xd = (double)x;
        s1 += xd;
        if (!CACHED) s2 += xd * xd;
        const uint32_t k = order_key(x);
        kmin = min(kmin, k);
        kmax = max(kmax, k);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        s1 += __shfl_xor_sync(0xFFFFFFFFu, s1, o);
        s2 += __shfl_xor_sync(0xFFFFFFFFu, s2, o);
        kmin = min(kmin, __shfl_xor_sync(0xFFFFFFFFu, kmin, o));
        kmax = max(kmax, __shfl_xor_sync(0xFFFFFFFFu, kmax, o));
    }
    if (lane == 0) { sh.red_a[wid] = s1; sh.red_b[wid] = s2; sh.red_min[wid] = kmin; sh.red_max[wid] = kmax; }
    __syncthreads();
    if (tid == 0) {
        double ta = 0.0, tb = 0.0;
        uint32_t mn = 0xFFFFFFFFu, mx = 0u;
        for (int i = 0; i < kSelWarps; ++i) {
            ta += sh.red_a[i]; tb += sh.red_b[i];
            mn = min(mn, sh.red_min[i]); mx = max(mx, sh.red_max[i]);
        }
        sh.bc_a = ta; sh.bc_b = tb; sh.bc_min = mn; sh.bc_max = mx;
    }
    __syncthreads();
    const double mean = sh.bc_a / (double)n;
    double var;
    if (CACHED) {
        double c2 = 0.0;
        for (int i = tid; i < n; i += kSelThreads) {
            const double dlt = (double)srow[i] - mean;
            c2 += dlt * dlt;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) c2 += __shfl_xor_sync(0xFFFFFFFFu, c2, o);
        __syncthreads();                       // red_a was read by thread 0 above
        if (lane == 0) sh.red_a[wid] = c2;
        __syncthreads();
        double tc = 0.0;
        for (int i = 0; i < kSelWarps; ++i) tc += sh.red_a[i];
        var = tc / (double)n;
    } else {
        var = sh.bc_b / (double)n - mean * mean;
        if (var < 0.0) var = 0.0;
    }

    // ---- Eq. 8 ------------------------------------------------------------------------------
    double r;
    if (a.k_mode == 0)      r = (double)a.k_base * var / (double)a.v_bar;
    else if (a.k_mode == 1) r = var > 0.0 ? (double)a.k_base * (double)a.v_bar / var : 1e300;
    else                    r = (double)a.k_base;
    const double fl = floor(r);
    int k_t;
    if (!(fl < (double)a.k_max)) k_t = a.k_max;
    else if (fl < (double)a.k_min) k_t = a.k_min;
    else k_t = (int)fl;
    const int k = k_t < n ? k_t : n;
    if (tid == 0) {
        a.kt[orow] = k;
        if (a.var) a.var[orow] = (float)var;
    }

    if (k == n) {                               // everything visible is selected
        for (int i = tid; i < a.k_max; i += kSelThreads) out_idx[i] = i < n ? i : -1;
        return;
    }

    // ---- passes B: narrow [lo, hi] onto the k-th largest key ---------------------------------
    uint32_t lo = sh.bc_min, hi = sh.bc_max;
    uint32_t want = (uint32_t)k;                // rank (1 = largest) wanted inside [lo, hi]
    uint32_t n_above = 0;                       // keys > hi
    while (true) {
        const uint32_t span = hi - lo;          // inclusive range has span + 1 keys
        int shift = 0;
        while (shift < 32 && (span >> shift) >= (uint32_t)kBins) ++shift;
        for (int i = tid; i < kBins; i += kSelThreads) sh.hist[i] = 0u;
        __syncthreads();
        for (int i = tid; i < n; i += kSelThreads) {
            const uint32_t key = order_key(row_at<CACHED>(grow, srow, i));
            if (key >= lo && key <= hi) atomicAdd(&sh.hist[(key - lo) >> shift], 1u);
        }
        __syncthreads();
        // thread `tid` owns bins [8 tid, 8 tid + 8); suffix sums from the top bin down
        uint32_t mine = 0;
#pragma unroll
        for (int j = 0; j < kBinsPerThread; ++j) mine += sh.hist[tid * kBinsPerThread + j];
        uint32_t suf = mine;                    // inclusive suffix over higher lanes
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_down_sync(0xFFFFFFFFu, suf, o);
            if (lane + o < 32) suf += v;
        }
        if (lane == 0) sh.warp_tot[wid] = suf;
        __syncthreads();
        uint32_t above_warp = 0;
        for (int i = wid + 1; i < kSelWarps; ++i) above_warp += sh.warp_tot[i];
        const uint32_t above_mine = above_warp + suf - mine;   // keys in bins above my 8 bins
        if (above_mine < want && want <= above_mine + mine) {
            uint32_t acc = above_mine;
            for (int j = kBinsPerThread - 1; j >= 0; --j) {
                const uint32_t c = sh.hist[tid * kBinsPerThread + j];
                if (want <= acc + c) { sh.found_bin = tid * kBinsPerThread + j; sh.found_above = acc; break; }
                acc += c;
            }
        }
        __syncthreads();
        const uint32_t fb = sh.found_bin, fa = sh.found_above;
        n_above += fa;
        want -= fa;
        const uint32_t nlo = lo + (fb << shift);
        const uint32_t nhi = shift == 0 ? nlo : min(hi, nlo + ((1u << shift) - 1u));
        lo = nlo; hi = nhi;
        if (shift == 0) break;
        __syncthreads();                         // found_* are rewritten next round
    }
    const uint32_t T = lo;                       // the k-th largest key
    const uint32_t need_eq = want;               // how many keys == T are taken (lowest positions)

    // ---- pass C: per-warp segment counts ----------------------------------------------------
    const int seg = ((n + kSelWarps - 1) / kSelWarps + 31) & ~31;
    const int seg_lo = wid * seg, seg_hi = min(n, seg_lo + seg);
    uint32_t cg = 0, ce = 0;
    for (int i = seg_lo + lane; i < seg_hi; i += 32) {
        const uint32_t key = order_key(row_at<CACHED>(grow, srow, i));
        cg += key > T;
        ce += key == T;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        cg += __shfl_xor_sync(0xFFFFFFFFu, cg, o);
        ce += __shfl_xor_sync(0xFFFFFFFFu, ce, o);
    }
    if (lane == 0) { sh.seg_gt[wid] = cg; sh.seg_eq[wid] = ce; }
    __syncthreads();
    uint32_t run_gt = 0, run_eq = 0;
    for (int i = 0; i < wid; ++i) { run_gt += sh.seg_gt[i]; run_eq += sh.seg_eq[i]; }

    // ---- pass D: ordered emission -----------------------------------------------------------
    const uint32_t lt_mask = (1u << lane) - 1u;
    for (int base = seg_lo; base < seg_hi; base += 32) {
        const int i = base + lane;
        uint32_t key = 0;
        const bool in = i < seg_hi;
        if (in) key = order_key(row_at<CACHED>(grow, srow, i));
        const bool gt = in && key > T, eq = in && key == T;
        const uint32_t bg = __ballot_sync(0xFFFFFFFFu, gt), be = __ballot_sync(0xFFFFFFFFu, eq);
        const uint32_t g_before = run_gt + __popc(bg & lt_mask);
        const uint32_t e_before = run_eq + __popc(be & lt_mask);
        if (gt || (eq && e_before < need_eq)) out_idx[g_before + min(e_before, need_eq)] = i;
        run_gt += __popc(bg);
        run_eq += __popc(be);
    }
    for (int i = k + tid; i < a.k_max; i += kSelThreads) out_idx[i] = -1;
}

}  // namespace

cudaError_t launch_select(const gsa_params_t& p, RowRange rr, const float* scores,
                          int64_t row_stride, int32_t* idx, int32_t* kt, float* var, IdxLayout il,
                          cudaStream_t st) {
    if (rr.rows() <= 0) return cudaSuccess;
    SelectArgs a;
    a.scores = scores; a.row_stride = row_stride; a.idx = idx; a.kt = kt; a.var = var;
    a.rr = rr; a.il = il; a.Lq = p.Lq; a.Lk = p.Lk;
    a.k_base = p.k_base; a.k_min = p.k_min; a.k_max = p.k_max; a.k_mode = p.k_mode; a.v_bar = p.v_bar;

    const int n_max = p.Lk - p.Lq + (rr.q_begin + rr.R - 1) + 1;
    const size_t fixed = ((sizeof(SelShared) + 15) / 16) * 16;
    constexpr size_t kMaxSmem = 200 * 1024;
    const size_t want = fixed + (size_t)n_max * sizeof(float);
    cudaError_t e;
    if (want <= kMaxSmem) {
        a.cache_cap = n_max;
        static bool attr_done = false;
        if (!attr_done) {
            e = cudaFuncSetAttribute(gsa_select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)kMaxSmem);
            if (e != cudaSuccess) return e;
            attr_done = true;
        }
        gsa_select_kernel<true><<<rr.rows(), kSelThreads, want, st>>>(a);
    } else {
        a.cache_cap = 0;
        gsa_select_kernel<false><<<rr.rows(), kSelThreads, fixed, st>>>(a);
    }
    ++g_launches;
    return cudaGetLastError();
}

}  // namespace gsa
