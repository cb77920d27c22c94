// Adaptive sparsity controller: per query row, the variance of the visible scores (Eq. 8),
// the budget k_t, and the exact top-k_t positions (Eq. 4).
//
// One CTA per row, one full read of the row:
//   0  a sample of the row (256 chunks of 32 consecutive scores, evenly spread) is histogrammed;
//      it gives a threshold key tau that about 1.3 * min(k_max, n) scores of the row should reach
//      (k_t itself is not known yet: it depends on the variance of the whole row)
//   1  full read, no block-wide barrier: the row is cut into at most 512 chunks (512 scores each, or
//      512 * 2^s for very long rows) that are dealt to the 16 warps round-robin, so each warp sees an
//      even sample of the row.  Loads are fully coalesced float4s; every score goes into fp64 sum and
//      sum of squares; a score that reaches tau (one float compare) is appended, in position order, to
//      the warp's private candidate list in shared memory, and each chunk remembers where its entries
//      start and how many it has.   -> Var, k_t
//   2  on chip: radix rounds over the candidates give the exact threshold key T of the k_t-th largest
//      score and how many keys equal to T are taken; the chunks are then walked in position order
//      (counts per chunk, one block scan, ballot-ordered emission) to write S_t ascending.
// Equal keys go to the lower position, so the output is unique.  If the list overflows or comes out
// shorter than k_t (the sample misjudged the row: huge ties, scores sorted by position, ...) the CTA
// falls back to radix rounds over the whole row in global memory: slower, same result.
#include "gsa_common.cuh"

namespace gsa {

namespace {

constexpr int kSelThreads = 512;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kBinsLog2 = 12;
constexpr int kBins = 1 << kBinsLog2;
constexpr int kBinsPerThread = kBins / kSelThreads;   // 8
constexpr int kListCap = 8192;                        // entries of the candidate list
constexpr int kListPerThread = kListCap / kSelThreads;  // 16
constexpr int kWarpCap = kListCap / kSelWarps;        // entries of one warp's private list: 512
constexpr int kIterElems = 512;                       // scores one warp iteration covers (4 float4 per lane)
constexpr int kMaxChunks = 512;
constexpr int kSampleChunks = 256;                    // sample = 256 chunks of 32 scores
constexpr int kSamplePerThread = kSampleChunks * 32 / kSelThreads;   // 16

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
};

// monotone map fp32 -> uint32 (larger float <=> larger key); -0 is folded onto +0
__device__ __forceinline__ uint32_t order_key(float x) {
    const uint32_t b = __float_as_uint(x + 0.0f);
    return b ^ ((uint32_t)((int32_t)b >> 31) | 0x80000000u);     // negative: all bits flip; else: sign bit set
}

struct SelShared {
    uint32_t hist[kBins];
    uint32_t list_idx[kListCap];
    uint32_t list_key[kListCap];
    double red_a[kSelWarps];
    double red_b[kSelWarps];
    uint32_t red_min[kSelWarps];
    uint32_t red_max[kSelWarps];
    uint32_t warp_tot[2][kSelWarps];
    uint32_t seg_gt[kSelWarps];
    uint32_t seg_eq[kSelWarps];
    uint16_t ch_off[kMaxChunks];      // chunk c: its entries start at list[(c % 16) * kWarpCap + ch_off[c]]
    uint16_t ch_cnt[kMaxChunks];      //          and there are ch_cnt[c] of them
    uint16_t ch_gt[kMaxChunks];       // selected entries of the chunks before c: keys > T ...
    uint16_t ch_eq[kMaxChunks];       // ... and keys == T (before the cut at need_eq)
    uint32_t wl_cnt[kSelWarps];       // live entries of each warp's list
    uint32_t found_bin;
    uint32_t found_above;
    uint32_t overflow;
    double bc_a, bc_b;
    uint32_t bc_min, bc_max;
};


__device__ __forceinline__ void block_minmax(SelShared& sh, uint32_t& kmin, uint32_t& kmax) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        kmin = min(kmin, __shfl_xor_sync(0xFFFFFFFFu, kmin, o));
        kmax = max(kmax, __shfl_xor_sync(0xFFFFFFFFu, kmax, o));
    }
    if (lane == 0) { sh.red_min[wid] = kmin; sh.red_max[wid] = kmax; }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t mn = 0xFFFFFFFFu, mx = 0u;
        for (int i = 0; i < kSelWarps; ++i) { mn = min(mn, sh.red_min[i]); mx = max(mx, sh.red_max[i]); }
        sh.bc_min = mn; sh.bc_max = mx;
    }
    __syncthreads();
    kmin = sh.bc_min; kmax = sh.bc_max;
    __syncthreads();
}

// After a histogram has been filled: the bin holding the `want`-th largest entry (1 = largest) and
// the number of entries in higher bins.  All threads get the result.
__device__ __forceinline__ void find_bin(SelShared& sh, uint32_t want, uint32_t& bin, uint32_t& above) {
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    uint32_t mine = 0;
#pragma unroll
    for (int j = 0; j < kBinsPerThread; ++j) mine += sh.hist[tid * kBinsPerThread + j];
    uint32_t suf = mine;                    // inclusive suffix over higher lanes
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_down_sync(0xFFFFFFFFu, suf, o);
        if (lane + o < 32) suf += v;
    }
    if (lane == 0) sh.warp_tot[0][wid] = suf;
    __syncthreads();
    uint32_t above_warp = 0;
    for (int i = wid + 1; i < kSelWarps; ++i) above_warp += sh.warp_tot[0][i];
    const uint32_t above_mine = above_warp + suf - mine;   // entries in bins above my 8 bins
    if (above_mine < want && want <= above_mine + mine) {
        uint32_t acc = above_mine;
        for (int j = kBinsPerThread - 1; j >= 0; --j) {
            const uint32_t c = sh.hist[tid * kBinsPerThread + j];
            if (want <= acc + c) { sh.found_bin = tid * kBinsPerThread + j; sh.found_above = acc; break; }
            acc += c;
        }
    }
    __syncthreads();
    bin = sh.found_bin;
    above = sh.found_above;
    __syncthreads();
}

// Radix rounds over `count` keys fetched by `key_of(i)`: narrows [lo, hi] onto the want-th largest
// key.  Returns T = that key, need_eq = how many keys == T belong to the top set.
template <class KeyOf>
__device__ __forceinline__ void radix_rounds(SelShared& sh, int count, KeyOf key_of, uint32_t lo, uint32_t hi,
                                             uint32_t want, uint32_t& T, uint32_t& need_eq) {
    const int tid = threadIdx.x;
    while (true) {
        const uint32_t span = hi - lo;          // inclusive range has span + 1 keys
        int shift = 0;
        while (shift < 32 && (span >> shift) >= (uint32_t)kBins) ++shift;
        for (int i = tid; i < kBins; i += kSelThreads) sh.hist[i] = 0u;
        __syncthreads();
        for (int i = tid; i < count; i += kSelThreads) {
            const uint32_t key = key_of(i);
            if (key >= lo && key <= hi) atomicAdd(&sh.hist[(key - lo) >> shift], 1u);
        }
        __syncthreads();
        uint32_t fb, fa;
        find_bin(sh, want, fb, fa);
        want -= fa;
        const uint32_t nlo = lo + (fb << shift);
        const uint32_t nhi = shift == 0 ? nlo : min(hi, nlo + ((1u << shift) - 1u));
        lo = nlo; hi = nhi;
        if (shift == 0) break;
    }
    T = lo;
    need_eq = want;
}

// block-wide exclusive scan of one value per thread; returns the exclusive prefix and the total.
// `slot` alternates 0/1 between consecutive calls so one barrier per call suffices.
__device__ __forceinline__ uint32_t block_excl_scan(SelShared& sh, uint32_t v, int slot, uint32_t& total) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += u;
    }
    if (lane == 31) sh.warp_tot[slot][wid] = inc;
    __syncthreads();
    uint32_t before = 0, tot = 0;
#pragma unroll
    for (int i = 0; i < kSelWarps; ++i) {
        const uint32_t t = sh.warp_tot[slot][i];
        before += i < wid ? t : 0u;
        tot += t;
    }
    total = tot;
    return before + inc - v;
}

__global__ void __launch_bounds__(kSelThreads, 2) gsa_select_kernel(const SelectArgs a) {
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    SelShared& sh = *reinterpret_cast<SelShared*>(dyn_smem);

    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int lr = blockIdx.x;
    const int b = a.rr.b0 + lr / a.rr.R;
    const int t = a.rr.q_begin + lr % a.rr.R;
    const int n = a.Lk - a.Lq + t + 1;                       // visible keys
    const float* __restrict__ grow = a.scores + (int64_t)lr * a.row_stride;
    const int64_t orow = a.il.row(b, t);
    int32_t* __restrict__ out_idx = a.idx + orow * a.k_max;

    if (tid == 0) sh.overflow = 0u;

    // ---- pass 0: candidate threshold from a sample ------------------------------------------
    uint32_t tau = 0u;                                        // every key reaches 0: short rows keep everything
    if (n > kListCap) {
        const int chunks = n >> 5;                            // full chunks of 32
        // sample chunk j of 256 sits at floor(j * chunks / 256): evenly spread over the row
        uint32_t skey[kSamplePerThread];
        uint32_t smin = 0xFFFFFFFFu, smax = 0u;
#pragma unroll
        for (int e = 0; e < kSamplePerThread; ++e) {
            const int j = wid + e * kSelWarps;
            const int c = (int)(((int64_t)j * chunks) >> 8);
            skey[e] = order_key(__ldg(grow + (c << 5) + lane));
            smin = min(smin, skey[e]);
            smax = max(smax, skey[e]);
        }
        block_minmax(sh, smin, smax);
        int shift = 0;
        while (shift < 32 && ((smax - smin) >> shift) >= (uint32_t)kBins) ++shift;
        for (int i = tid; i < kBins; i += kSelThreads) sh.hist[i] = 0u;
        __syncthreads();
#pragma unroll
        for (int e = 0; e < kSamplePerThread; ++e) atomicAdd(&sh.hist[(skey[e] - smin) >> shift], 1u);
        __syncthreads();
        // the sample rank that corresponds to 1.3 * min(k_max, n) + 64 scores of the whole row
        const int k_cap = a.k_max < n ? a.k_max : n;
        const double frac = (1.3 * (double)k_cap + 64.0) / (double)n;
        uint32_t want = (uint32_t)ceil(frac * (double)(kSampleChunks * 32));
        want = max(1u, min(want, (uint32_t)(kSampleChunks * 32)));
        uint32_t fb, fa;
        find_bin(sh, want, fb, fa);
        tau = smin + (fb << shift);                           // lower edge of that bin
    }
    __syncthreads();

    // ---- pass 1: fp64 moments of every score; per-warp ordered lists of the candidates ---------
    // tau as a float: x >= tau_f  <=>  order_key(x) >= tau for every non-NaN x
    // (tau == 0, "keep everything", has no float counterpart: use -inf)
    const float tau_f = tau == 0u ? -INFINITY : __uint_as_float((tau & 0x80000000u) ? (tau & 0x7FFFFFFFu) : ~tau);
    int cshift = 0;                                           // chunk = kIterElems << cshift scores
    while (((int64_t)n + ((int64_t)kIterElems << cshift) - 1) / ((int64_t)kIterElems << cshift) > kMaxChunks) ++cshift;
    const int chunk_elems = kIterElems << cshift;
    const int nchunks = (n + chunk_elems - 1) / chunk_elems;
    double s1 = 0.0, s2 = 0.0;
    uint32_t wcnt = 0;                                        // entries in this warp's list (warp-uniform)
    bool w_over = false;
    uint32_t* const wl_idx = sh.list_idx + wid * kWarpCap;
    uint32_t* const wl_key = sh.list_key + wid * kWarpCap;
    for (int c = wid; c < nchunks; c += kSelWarps) {
        const uint32_t c_start = wcnt;
        const int c_lo = c * chunk_elems, c_hi = min(n, c_lo + chunk_elems);
        for (int i0 = c_lo; i0 < c_hi; i0 += kIterElems) {
            float xs[16];
            if (i0 + kIterElems <= c_hi) {
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const float4 x4 = __ldg(reinterpret_cast<const float4*>(grow + i0) + v * 32 + lane);
                    xs[v * 4] = x4.x; xs[v * 4 + 1] = x4.y; xs[v * 4 + 2] = x4.z; xs[v * 4 + 3] = x4.w;
                }
            } else {
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const int i = i0 + ((e >> 2) * 32 + lane) * 4 + (e & 3);
                    xs[e] = i < c_hi ? __ldg(grow + i) : __int_as_float(0x7FC00000);   // NaN: never a candidate
                }
            }
            uint32_t flags = 0;
            const bool full = i0 + kIterElems <= c_hi;
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const double xd = (double)xs[e];
                if (full || i0 + ((e >> 2) * 32 + lane) * 4 + (e & 3) < c_hi) {
                    s1 += xd;
                    s2 = fma(xd, xd, s2);
                }
                flags |= (xs[e] >= tau_f ? 1u : 0u) << e;
            }
            if (__any_sync(0xFFFFFFFFu, flags != 0u)) {
                // position order inside the iteration is (v, lane, e): one packed scan gives, for each of
                // the four float4 rounds v, how many candidates the lower lanes hold
                uint32_t packed = __popc(flags & 0xFu) | (__popc(flags & 0xF0u) << 8) |
                                  (__popc(flags & 0xF00u) << 16) | (__popc(flags & 0xF000u) << 24);
                uint32_t inc = packed;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, inc, o);
                    if (lane >= o) inc += u;
                }
                const uint32_t tot = __shfl_sync(0xFFFFFFFFu, inc, 31);     // per-v totals, one byte each
                const uint32_t excl = inc - packed;
                const uint32_t iter_total = (tot & 0xFFu) + ((tot >> 8) & 0xFFu) + ((tot >> 16) & 0xFFu) + (tot >> 24);
                if (wcnt + iter_total <= (uint32_t)kWarpCap) {
                    uint32_t vbase = wcnt;
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        uint32_t pos = vbase + ((excl >> (8 * v)) & 0xFFu);
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (flags & (1u << (v * 4 + e))) {
                                // the score is read again (L1) so that xs[] need not stay live
                                const int i = i0 + (v * 32 + lane) * 4 + e;
                                wl_idx[pos] = (uint32_t)i;
                                wl_key[pos] = order_key(__ldg(grow + i));
                                ++pos;
                            }
                        vbase += (tot >> (8 * v)) & 0xFFu;
                    }
                } else {
                    w_over = true;
                }
                wcnt += iter_total;
            }
        }
        if (lane == 0) {
            sh.ch_off[c] = (uint16_t)min(c_start, (uint32_t)kWarpCap);
            sh.ch_cnt[c] = (uint16_t)min(wcnt - c_start, (uint32_t)kWarpCap);
        }
    }
    if (lane == 0) {
        if (w_over) sh.overflow = 1u;
        sh.wl_cnt[wid] = min(wcnt, (uint32_t)kWarpCap);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        s1 += __shfl_xor_sync(0xFFFFFFFFu, s1, o);
        s2 += __shfl_xor_sync(0xFFFFFFFFu, s2, o);
    }
    if (lane == 0) { sh.red_a[wid] = s1; sh.red_b[wid] = s2; }
    __syncthreads();
    if (tid == 0) {
        double ta = 0.0, tb = 0.0;
        for (int i = 0; i < kSelWarps; ++i) { ta += sh.red_a[i]; tb += sh.red_b[i]; }
        sh.bc_a = ta; sh.bc_b = tb;
    }
    __syncthreads();
    const double mean = sh.bc_a / (double)n;
    double var = sh.bc_b / (double)n - mean * mean;
    if (var < 0.0) var = 0.0;
    const bool overflow = sh.overflow != 0u;

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

    int m = 0;                                  // candidates found (all of them listed unless overflow)
    for (int w = 0; w < kSelWarps; ++w) m += (int)sh.wl_cnt[w];
    uint32_t T, need_eq;
    if (!overflow && m >= k) {
        // ---- exact threshold among the candidates (the 16 warp lists, padded to kWarpCap) -------
        // slot i of the padded array belongs to warp i / kWarpCap and is live below that warp's count
        uint32_t cmin = 0xFFFFFFFFu, cmax = 0u;
        for (int i = tid; i < kListCap; i += kSelThreads)
            if ((uint32_t)(i & (kWarpCap - 1)) < sh.wl_cnt[i / kWarpCap]) {
                const uint32_t key = sh.list_key[i];
                cmin = min(cmin, key); cmax = max(cmax, key);
            }
        block_minmax(sh, cmin, cmax);
        // dead slots read as a key outside [cmin, cmax], which no round counts
        const uint32_t dead = cmin > 0u ? cmin - 1u : cmax + 1u;
        radix_rounds(sh, kListCap, [&](int i) -> uint32_t {
            return (uint32_t)(i & (kWarpCap - 1)) < sh.wl_cnt[i / kWarpCap] ? sh.list_key[i] : dead;
        }, cmin, cmax, (uint32_t)k, T, need_eq);

        // ---- emission in position order: chunk by chunk ---------------------------------------
        // (a) per chunk: how many of its entries are above T / equal to T
        for (int c = wid; c < nchunks; c += kSelWarps) {
            const uint32_t off = (uint32_t)(c & (kSelWarps - 1)) * kWarpCap + sh.ch_off[c];
            const int cnt = sh.ch_cnt[c];
            uint32_t g = 0, q = 0;
            for (int j = lane; j < cnt; j += 32) {
                const uint32_t key = sh.list_key[off + j];
                g += key > T;
                q += key == T;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                g += __shfl_xor_sync(0xFFFFFFFFu, g, o);
                q += __shfl_xor_sync(0xFFFFFFFFu, q, o);
            }
            if (lane == 0) { sh.ch_gt[c] = (uint16_t)g; sh.ch_eq[c] = (uint16_t)q; }
        }
        __syncthreads();
        // (b) exclusive prefix over the chunks (thread c owns chunk c)
        {
            const uint32_t mine = tid < nchunks ? (((uint32_t)sh.ch_eq[tid] << 16) | sh.ch_gt[tid]) : 0u;
            uint32_t total;
            const uint32_t before = block_excl_scan(sh, mine, 0, total);
            __syncthreads();
            if (tid < nchunks) { sh.ch_gt[tid] = (uint16_t)(before & 0xFFFFu); sh.ch_eq[tid] = (uint16_t)(before >> 16); }
        }
        __syncthreads();
        // (c) each warp writes its chunks; inside a chunk, ballots give the order
        const uint32_t below = (1u << lane) - 1u;
        for (int c = wid; c < nchunks; c += kSelWarps) {
            const uint32_t off = (uint32_t)(c & (kSelWarps - 1)) * kWarpCap + sh.ch_off[c];
            const int cnt = sh.ch_cnt[c];
            uint32_t run_gt = sh.ch_gt[c], run_eq = sh.ch_eq[c];
            for (int j0 = 0; j0 < cnt; j0 += 32) {
                const int j = j0 + lane;
                const bool in = j < cnt;
                const uint32_t key = in ? sh.list_key[off + j] : 0u;
                const bool gt = in && key > T, eq = in && key == T;
                const uint32_t bg = __ballot_sync(0xFFFFFFFFu, gt), be = __ballot_sync(0xFFFFFFFFu, eq);
                const uint32_t g_before = run_gt + __popc(bg & below);
                const uint32_t e_before = run_eq + __popc(be & below);
                if (gt || (eq && e_before < need_eq))
                    out_idx[g_before + min(e_before, need_eq)] = (int32_t)sh.list_idx[off + j];
                run_gt += __popc(bg);
                run_eq += __popc(be);
            }
        }
    } else {
        // ---- fallback: radix rounds over the whole row, then ordered emission ----------------
        radix_rounds(sh, n, [&](int i) { return order_key(__ldg(grow + i)); }, 0u, 0xFFFFFFFFu,
                     (uint32_t)k, T, need_eq);
        const int seg = ((n + kSelWarps - 1) / kSelWarps + 31) & ~31;
        const int seg_lo = min(n, wid * seg), seg_hi = min(n, seg_lo + seg);
        uint32_t cg = 0, ce = 0;
        for (int i = seg_lo + lane; i < seg_hi; i += 32) {
            const uint32_t key = order_key(__ldg(grow + i));
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
        const uint32_t lt_mask = (1u << lane) - 1u;
        for (int base2 = seg_lo; base2 < seg_hi; base2 += 32) {
            const int i = base2 + lane;
            uint32_t key = 0;
            const bool in = i < seg_hi;
            if (in) key = order_key(__ldg(grow + i));
            const bool gt = in && key > T, eq = in && key == T;
            const uint32_t bg = __ballot_sync(0xFFFFFFFFu, gt), be = __ballot_sync(0xFFFFFFFFu, eq);
            const uint32_t g_before = run_gt + __popc(bg & lt_mask);
            const uint32_t e_before = run_eq + __popc(be & lt_mask);
            if (gt || (eq && e_before < need_eq)) out_idx[g_before + min(e_before, need_eq)] = i;
            run_gt += __popc(bg);
            run_eq += __popc(be);
        }
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

    const size_t smem = ((sizeof(SelShared) + 15) / 16) * 16;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(gsa_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    gsa_select_kernel<<<rr.rows(), kSelThreads, smem, st>>>(a);
    ++g_launches;
    return cudaGetLastError();
}

}  // namespace gsa
