// Adaptive sparsity controller: per query row, the variance of the visible scores (Eq. 8),
// the budget k_t, and the exact top-k_t positions (Eq. 4).
//
// One CTA per row, one full read of the row:
//   0  a sample of the row (256 chunks of 32 consecutive scores, evenly spread) is histogrammed;
//      it gives a threshold key tau that about 1.3 * min(k_max, n) scores of the row should reach
//      (k_t itself is not known yet: it depends on the variance of the whole row)
//   1  full read, no block-wide barrier: the row is cut into at most 512 chunks (128 * 2^s scores each)
//      that are dealt to the 16 warps round-robin, so each warp sees an even sample of the row.  Loads are fully coalesced float4s; every score goes into fp64 sum and
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
constexpr int kListCap = 8192;                        // entries of the candidate lists (all warps)
constexpr int kListPerThread = kListCap / kSelThreads;  // 16
constexpr int kWarpCap = kListCap / kSelWarps;        // entries of one warp's private list: 512
constexpr int kMaxChunks = 512;
constexpr int kSampleChunks = 256;                    // sample = 256 chunks of 32 scores
constexpr int kSamplePerThread = kSampleChunks * 32 / kSelThreads;   // 16

struct SelectArgs {
    const float* scores;
    int64_t row_stride;
    int32_t* idx;
    int32_t* kt;
    float* var;
    int32_t* fallback_rows;
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
    uint16_t list_rel[kListCap];      // candidate position relative to the start of its chunk
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
    uint32_t bc_want;                 // pass 0: sample rank of the candidate threshold
    int32_t bc_k;                     // the row's k_t (Eq. 8), computed by one thread
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

// smallest shift with (span >> shift) < kBins
__device__ __forceinline__ int shift_for(uint32_t span) {
    const int bits = 32 - __clz(span);
    return bits > kBinsLog2 ? bits - kBinsLog2 : 0;
}

// Radix rounds over `count` keys fetched by `key_of(i)`: narrows [lo, hi] onto the want-th largest
// key.  Returns T = that key, need_eq = how many keys == T belong to the top set.
template <class KeyOf>
__device__ __forceinline__ void radix_rounds(SelShared& sh, int count, KeyOf key_of, uint32_t lo, uint32_t hi,
                                             uint32_t want, uint32_t& T, uint32_t& need_eq) {
    const int tid = threadIdx.x;
    while (true) {
        const uint32_t span = hi - lo;          // inclusive range has span + 1 keys
        const int shift = shift_for(span);
        for (int i = tid; i < kBins; i += kSelThreads) sh.hist[i] = 0u;
        __syncthreads();
        for (int i = tid; i < count; i += kSelThreads) {
            const uint32_t key = key_of(i);
            if (key - lo <= span) atomicAdd(&sh.hist[(key - lo) >> shift], 1u);
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

// The same over the 16 per-warp candidate lists: each warp walks its own list (no dead slots).
__device__ __forceinline__ void radix_rounds_lists(SelShared& sh, uint32_t lo, uint32_t hi, uint32_t want,
                                                   uint32_t& T, uint32_t& need_eq) {
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const uint32_t* const wl_key = sh.list_key + wid * kWarpCap;
    const int my_cnt = (int)sh.wl_cnt[wid];
    while (true) {
        const uint32_t span = hi - lo;
        const int shift = shift_for(span);
        for (int i = tid; i < kBins; i += kSelThreads) sh.hist[i] = 0u;
        __syncthreads();
        for (int j = lane; j < my_cnt; j += 32) {
            const uint32_t key = wl_key[j];
            if (key - lo <= span) atomicAdd(&sh.hist[(key - lo) >> shift], 1u);
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

// k_t of Eq. 8 from a variance (shared by the estimate on the sample and the final value)
__device__ __forceinline__ int budget_from_var(const SelectArgs& a, double var, double* r_out) {
    double r;
    if (a.k_mode == 0)      r = (double)a.k_base * var / (double)a.v_bar;
    else if (a.k_mode == 1) r = var > 0.0 ? (double)a.k_base * (double)a.v_bar / var : 1e300;
    else                    r = (double)a.k_base;
    if (r_out) *r_out = r;
    const double fl = floor(r);
    if (!(fl < (double)a.k_max)) return a.k_max;
    if (fl < (double)a.k_min) return a.k_min;
    return (int)fl;
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
    const bool short_row = n <= kListCap;                     // the whole row fits the list: no sampling

    if (tid == 0) sh.overflow = 0u;

    // ---- pass 0 (long rows): candidate threshold from a sample --------------------------------
    // 256 chunks of 32 consecutive scores, evenly spread, give (a) an estimate of the row's variance and
    // with it an upper estimate k_hi of the budget, (b) a key tau that about 1.3 * k_hi scores reach.
    float tau_f = -INFINITY;
    if (!short_row) {
        const int chunks = n >> 5;                            // full chunks of 32
        uint32_t skey[kSamplePerThread];
        uint32_t smin = 0xFFFFFFFFu, smax = 0u;
        float m1 = 0.f, m2 = 0.f;
        float x0 = 0.f;                                       // centre for the sample moments
#pragma unroll
        for (int e = 0; e < kSamplePerThread; ++e) {
            const int j = wid + e * kSelWarps;
            const int c = (int)(((int64_t)j * chunks) >> 8);
            const float x = __ldg(grow + (c << 5) + lane);
            if (e == 0) x0 = __shfl_sync(0xFFFFFFFFu, x, 0);
            const float y = x - x0;
            m1 += y;
            m2 = fmaf(y, y, m2);
            skey[e] = order_key(x);
            smin = min(smin, skey[e]);
            smax = max(smax, skey[e]);
        }
        // per-warp centred moments -> mean and second moment about the warp's own centre; combine in fp64
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            m1 += __shfl_xor_sync(0xFFFFFFFFu, m1, o);
            m2 += __shfl_xor_sync(0xFFFFFFFFu, m2, o);
        }
        if (lane == 0) {
            const double cnt = 32.0 * kSamplePerThread;
            const double mu = (double)x0 + (double)m1 / cnt;
            // sum of squares about zero, reconstructed from the centred sums
            sh.red_a[wid] = mu * cnt;
            sh.red_b[wid] = (double)m2 + 2.0 * (double)x0 * (double)m1 + cnt * (double)x0 * (double)x0;
        }
        block_minmax(sh, smin, smax);                         // (has the barriers that publish red_a / red_b)
        if (tid == 0) {
            double sa = 0.0, sb = 0.0;
            for (int i = 0; i < kSelWarps; ++i) { sa += sh.red_a[i]; sb += sh.red_b[i]; }
            const double scnt = (double)(kSampleChunks * 32);
            double svar = sb / scnt - (sa / scnt) * (sa / scnt);
            if (svar < 0.0) svar = 0.0;
            // budget the sample predicts, widened by 25 % (mode 1: narrowed variance) for the sampling error
            const int k_est = budget_from_var(a, a.k_mode == 1 ? svar / 1.25 : svar * 1.25, nullptr);
            const int k_hi = min(min(k_est + 32, a.k_max), n);
            const double frac = (1.3 * (double)k_hi + 128.0) / (double)n;
            const uint32_t want = (uint32_t)ceil(frac * scnt);
            sh.bc_want = max(1u, min(want, (uint32_t)(kSampleChunks * 32)));
        }
        const int shift = shift_for(smax - smin);
        for (int i = tid; i < kBins; i += kSelThreads) sh.hist[i] = 0u;
        __syncthreads();
#pragma unroll
        for (int e = 0; e < kSamplePerThread; ++e) atomicAdd(&sh.hist[(skey[e] - smin) >> shift], 1u);
        __syncthreads();
        const uint32_t want = sh.bc_want;
        uint32_t fb, fa;
        find_bin(sh, want, fb, fa);
        const uint32_t tau = smin + (fb << shift);            // lower edge of that bin
        // as a float: x >= tau_f  <=>  order_key(x) >= tau for every non-NaN x
        tau_f = __uint_as_float((tau & 0x80000000u) ? (tau & 0x7FFFFFFFu) : ~tau);
    }
    __syncthreads();

    // ---- pass 1: fp64 moments of every score; candidates into lists ----------------------------
    double s1 = 0.0, s2 = 0.0;
    uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;                   // range of the keys that went into the list(s)
    // The row is cut into rounds of 128 consecutive scores (one coalesced float4 load of a warp) and
    // chunks of 2^cshift rounds, at most 512 chunks; chunk c belongs to warp c % 16.
    constexpr int kRound = 128;
    const int n_rounds = (n + kRound - 1) / kRound;
    int cshift = 0;
    while (((n_rounds + (1 << cshift) - 1) >> cshift) > kMaxChunks) ++cshift;
    const int chunk_elems = kRound << cshift;
    const int nchunks = (n_rounds + (1 << cshift) - 1) >> cshift;
    if (short_row) {
        // the list is simply the row, in order
        for (int i = tid; i < n; i += kSelThreads) {
            const float x = __ldg(grow + i);
            const double xd = (double)x;
            s1 += xd;
            s2 = fma(xd, xd, s2);
            const uint32_t key = order_key(x);
            sh.list_key[i] = key;
            kmin = min(kmin, key);
            kmax = max(kmax, key);
        }
    } else {
        const int rpc_mask = (1 << cshift) - 1;               // rounds per chunk - 1
        uint32_t wcnt = 0;                                    // entries in this warp's list (warp-uniform)
        bool w_over = false;
        uint16_t* const wl_rel = sh.list_rel + wid * kWarpCap;
        uint32_t* const wl_key = sh.list_key + wid * kWarpCap;
        // the warp walks its chunks (wid, wid + 16, ...) round by round, four rounds per iteration
        const int my_chunks = wid < nchunks ? (nchunks - wid + kSelWarps - 1) / kSelWarps : 0;
        const int my_rounds = my_chunks << cshift;
        auto round_start = [&](int j) -> int {                // first score of the warp's j-th round
            return (wid + kSelWarps * (j >> cshift)) * chunk_elems + (j & rpc_mask) * kRound;
        };
        for (int j0 = 0; j0 < my_rounds; j0 += 4) {
            int rs[4];
#pragma unroll
            for (int v = 0; v < 4; ++v) rs[v] = j0 + v < my_rounds ? round_start(j0 + v) : n;   // n: nothing there
            uint32_t flags = 0;
            if (rs[3] + kRound <= n && rs[0] + kRound <= n && rs[1] + kRound <= n && rs[2] + kRound <= n) {
                float4 x4[4];
#pragma unroll
                for (int v = 0; v < 4; ++v) x4[v] = __ldg(reinterpret_cast<const float4*>(grow + rs[v]) + lane);
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const float xs[4] = {x4[v].x, x4[v].y, x4[v].z, x4[v].w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const double xd = (double)xs[e];
                        s1 += xd;
                        s2 = fma(xd, xd, s2);
                        flags |= (xs[e] >= tau_f ? 1u : 0u) << (v * 4 + e);
                    }
                }
            } else {
#pragma unroll
                for (int v = 0; v < 4; ++v)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int i = rs[v] + lane * 4 + e;
                        if (i < n) {
                            const float x = __ldg(grow + i);
                            const double xd = (double)x;
                            s1 += xd;
                            s2 = fma(xd, xd, s2);
                            flags |= (x >= tau_f ? 1u : 0u) << (v * 4 + e);
                        }
                    }
            }
            // position order inside the iteration is (round v, lane, e): one packed scan gives, for each of
            // the four rounds, how many candidates the lower lanes hold (bytes: at most 128 per round)
            const uint32_t packed = __popc(flags & 0xFu) | (__popc(flags & 0xF0u) << 8) |
                                    (__popc(flags & 0xF00u) << 16) | (__popc(flags & 0xF000u) << 24);
            uint32_t inc = packed;
            uint32_t t0 = 0, t1 = 0, t2 = 0, t3 = 0;
            if (__any_sync(0xFFFFFFFFu, flags != 0u)) {
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, inc, o);
                    if (lane >= o) inc += u;
                }
                const uint32_t tot = __shfl_sync(0xFFFFFFFFu, inc, 31);
                t0 = tot & 0xFFu; t1 = (tot >> 8) & 0xFFu; t2 = (tot >> 16) & 0xFFu; t3 = tot >> 24;
            }
            const uint32_t excl = inc - packed;
            // entries of the rounds before round v (two 16-bit fields per word)
            const uint32_t base_lo = t0 << 16;                              // rounds 0, 1: 0, t0
            const uint32_t base_hi = ((t0 + t1 + t2) << 16) | (t0 + t1);   // rounds 2, 3
            const uint32_t iter_total = t0 + t1 + t2 + t3;
            if (iter_total != 0u) {
                if (wcnt + iter_total <= (uint32_t)kWarpCap) {
                    uint32_t f = flags;
                    while (f) {                                           // one candidate per pass and lane
                        const int bit = __ffs(f) - 1;
                        f &= f - 1;
                        const int v = bit >> 2;
                        const uint32_t own_before = __popc(flags & ((1u << bit) - 1u) & (0xFu << (v * 4)));
                        const uint32_t base_v = (((v & 2) ? base_hi : base_lo) >> ((v & 1) * 16)) & 0xFFFFu;
                        const uint32_t pos = wcnt + base_v + ((excl >> (8 * v)) & 0xFFu) + own_before;
                        const int rsv = v == 0 ? rs[0] : (v == 1 ? rs[1] : (v == 2 ? rs[2] : rs[3]));
                        const int i = rsv + lane * 4 + (bit & 3);
                        wl_rel[pos] = (uint16_t)(((j0 + v) & rpc_mask) * kRound + lane * 4 + (bit & 3));
                        const uint32_t key = order_key(__ldg(grow + i));  // read again (L1)
                        wl_key[pos] = key;
                        kmin = min(kmin, key);
                        kmax = max(kmax, key);
                    }
                } else {
                    w_over = true;
                }
            }
            // chunk table: where each chunk's entries start in this warp's list and how many there are
            if (lane == 0) {
                const uint32_t tv[4] = {t0, t1, t2, t3};
                uint32_t run = wcnt;
#pragma unroll
                for (int v = 0; v < 4; ++v)
                    if (j0 + v < my_rounds) {
                        const int c = wid + kSelWarps * ((j0 + v) >> cshift);
                        if (((j0 + v) & rpc_mask) == 0) sh.ch_off[c] = (uint16_t)min(run, (uint32_t)kWarpCap);
                        run += tv[v];
                        if (((j0 + v) & rpc_mask) == rpc_mask)
                            sh.ch_cnt[c] = (uint16_t)(min(run, (uint32_t)kWarpCap) - sh.ch_off[c]);
                    }
            }
            wcnt += iter_total;
        }
        if (lane == 0) {
            if (w_over) sh.overflow = 1u;
            sh.wl_cnt[wid] = min(wcnt, (uint32_t)kWarpCap);
        }
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
        const double mean = ta / (double)n;
        double var = tb / (double)n - mean * mean;
        if (var < 0.0) var = 0.0;
        // ---- Eq. 8 ----
        const int k_t = budget_from_var(a, var, nullptr);
        const int kk = k_t < n ? k_t : n;
        sh.bc_k = kk;
        a.kt[orow] = kk;
        if (a.var) a.var[orow] = (float)var;
    }
    block_minmax(sh, kmin, kmax);               // (its barriers also publish bc_k and the lists)
    const int k = sh.bc_k;
    const bool overflow = sh.overflow != 0u;

    if (k == n) {                               // everything visible is selected
        for (int i = tid; i < a.k_max; i += kSelThreads) out_idx[i] = i < n ? i : -1;
        return;
    }

    uint32_t T, need_eq;
    if (short_row) {
        // ---- the row is the list: radix rounds, then one ordered compaction -------------------
        radix_rounds(sh, n, [&](int i) { return sh.list_key[i]; }, kmin, kmax, (uint32_t)k, T, need_eq);
        uint32_t gt = 0, eq = 0;
        const int j0 = tid * kListPerThread;
#pragma unroll
        for (int e = 0; e < kListPerThread; ++e)
            if (j0 + e < n) {
                const uint32_t key = sh.list_key[j0 + e];
                gt += key > T;
                eq += key == T;
            }
        uint32_t total;
        const uint32_t packed = block_excl_scan(sh, (eq << 16) | gt, 0, total);
        uint32_t g_before = packed & 0xFFFFu, e_before = packed >> 16;
#pragma unroll
        for (int e = 0; e < kListPerThread; ++e)
            if (j0 + e < n) {
                const uint32_t key = sh.list_key[j0 + e];
                if (key > T) {
                    out_idx[g_before + min(e_before, need_eq)] = j0 + e;
                    ++g_before;
                } else if (key == T) {
                    if (e_before < need_eq) out_idx[g_before + e_before] = j0 + e;
                    ++e_before;
                }
            }
        for (int i = k + tid; i < a.k_max; i += kSelThreads) out_idx[i] = -1;
        return;
    }

    int m = 0;                                  // candidates found (all of them listed unless overflow)
    for (int w = 0; w < kSelWarps; ++w) m += (int)sh.wl_cnt[w];
    if (!overflow && m >= k) {
        // ---- exact threshold among the candidates (each warp walks its own list) ----------------
        radix_rounds_lists(sh, kmin, kmax, (uint32_t)k, T, need_eq);

        // ---- emission in position order: thread c owns chunk c (a handful of entries, in order) ----
        uint32_t g = 0, q = 0;
        uint32_t off = 0;
        int cnt = 0;
        if (tid < nchunks) {
            off = (uint32_t)(tid & (kSelWarps - 1)) * kWarpCap + sh.ch_off[tid];
            cnt = sh.ch_cnt[tid];
            for (int j = 0; j < cnt; ++j) {
                const uint32_t key = sh.list_key[off + j];
                g += key > T;
                q += key == T;
            }
        }
        uint32_t total;
        const uint32_t before = block_excl_scan(sh, (q << 16) | g, 0, total);
        uint32_t g_before = before & 0xFFFFu, e_before = before >> 16;
        const int c_base = tid * chunk_elems;
        for (int j = 0; j < cnt; ++j) {
            const uint32_t key = sh.list_key[off + j];
            if (key > T) {
                out_idx[g_before + min(e_before, need_eq)] = c_base + (int32_t)sh.list_rel[off + j];
                ++g_before;
            } else if (key == T) {
                if (e_before < need_eq) out_idx[g_before + e_before] = c_base + (int32_t)sh.list_rel[off + j];
                ++e_before;
            }
        }
    } else {
        // ---- fallback: radix rounds over the whole row, then ordered emission ----------------
        if (tid == 0 && a.fallback_rows) atomicAdd(a.fallback_rows, 1);
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
                          int32_t* fallback_rows, cudaStream_t st) {
    if (rr.rows() <= 0) return cudaSuccess;
    SelectArgs a;
    a.scores = scores; a.row_stride = row_stride; a.idx = idx; a.kt = kt; a.var = var;
    a.fallback_rows = fallback_rows;
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
