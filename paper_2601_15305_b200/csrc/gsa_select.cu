// Adaptive sparsity controller: per query row, the variance of the visible scores (Eq. 8),
// the budget k_t, and the exact top-k_t positions (Eq. 4).
//
// One CTA per row, one full read of the row:
//   0  a sample of the row (256 chunks of 32 consecutive scores, evenly spread) is histogrammed;
//      it gives a threshold key tau that about 1.3 * min(k_max, n) scores of the row should reach
//      (k_t itself is not known yet: it depends on the variance of the whole row)
//   1  full read, no block-wide barrier: the row is cut into chunks of 512 consecutive scores that
//      are dealt to the 16 warps round-robin, so each warp sees an even sample of the row.  Loads are
//      fully coalesced float4s, one chunk ahead, turned through shared memory so that a lane holds 16
//      consecutive scores; every score goes into fp64 sum and sum of squares; the position of a score
//      that reaches tau (one float compare) goes into the candidate list in shared memory, with its
//      order key: a warp scan of the lanes' counts orders the chunk's candidates, one shared-memory
//      atomic claims their space, and a table remembers where each chunk's entries start and how many
//      there are.   -> Var, k_t
//   2  on chip: radix rounds over the candidates' keys give the exact threshold key T of the k_t-th
//      largest score and how many keys equal to T are taken.  S_t is then written ascending: if every
//      key equal to T is taken (no tie is cut) and the row has at most 131072 scores, the selected
//      candidates mark their positions in a bitmap and the threads turn stretches of it into positions;
//      otherwise the chunks are walked in position order (counts per thread, one block scan, emission).
// Equal keys go to the lower position, so the output is unique.  If the list overflows or comes out
// shorter than k_t (the sample misjudged the row: huge ties, scores sorted by position, ...) the CTA
// falls back to radix rounds over the whole row in global memory: slower, same result.  Rows of more
// than 2048 chunks (1 Mi scores) always take that path.
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
constexpr int kIter = 512;                            // scores a warp takes per iteration (= one chunk)
constexpr int kMaxChunks = 2048;                      // rows of up to kIter * kMaxChunks = 1 Mi scores are listed
constexpr int kKeysInScan = kListCap - kBins;         // list entries below this get their key during pass 1
static_assert(kListCap - kKeysInScan + kBins == kSelWarps * kIter, "upper half of list_key + hist hold one chunk per warp");
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
    uint32_t list_pos[kListCap];      // candidate positions; the entries of one chunk are consecutive and ascending
    uint32_t list_key[kListCap];      // their order keys; pass 1 stages scores in the upper half and in hist (next member)
    uint32_t hist[kBins];
    double red_a[kSelWarps];
    double red_b[kSelWarps];
    uint32_t red_min[kSelWarps];
    uint32_t red_max[kSelWarps];
    uint32_t warp_tot[2][kSelWarps];
    uint32_t seg_gt[kSelWarps];
    uint32_t seg_eq[kSelWarps];
    uint16_t ch_off[kMaxChunks];      // table chunk c (128 or 512 consecutive scores): its entries start at list[ch_off[c]]
    uint16_t ch_cnt[kMaxChunks];      //          and there are ch_cnt[c] of them
    uint32_t list_total;              // entries handed out so far
    uint32_t found_bin;
    uint32_t found_above;
    uint32_t found_count;             // entries in the found bin
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
    // (no barrier here: every caller passes another barrier before red_* or bc_* are written again)
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
            if (want <= acc + c) { sh.found_bin = tid * kBinsPerThread + j; sh.found_above = acc; sh.found_count = c; break; }
            acc += c;
        }
    }
    __syncthreads();
    bin = sh.found_bin;
    above = sh.found_above;
    // (no barrier here: the histogram is not read after the barrier above, and found_* / warp_tot are next
    // written only after the caller's next barriers)
}

// smallest shift with (span >> shift) < kBins
__device__ __forceinline__ int shift_for(uint32_t span) {
    const int bits = 32 - __clz(span);
    return bits > kBinsLog2 ? bits - kBinsLog2 : 0;
}

// Radix rounds over `count` keys fetched by `key_of(i)`: narrows [lo, hi] onto the want-th largest
// key.  Returns T = that key, need_eq = how many keys == T belong to the top set, eq_total = how many there are.
template <class KeyOf>
__device__ __forceinline__ void radix_rounds(SelShared& sh, int count, KeyOf key_of, uint32_t lo, uint32_t hi,
                                             uint32_t want, uint32_t& T, uint32_t& need_eq, uint32_t& eq_total) {
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
    eq_total = sh.found_count;               // the last round's bins are single keys: all keys equal to T
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
    else if (a.k_mode == 2) r = (double)a.k_base;
    else                    r = 1e300;                          // k_mode 3: everything visible
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
    const int nchunks = (n + kIter - 1) / kIter;              // chunks of 512 consecutive scores (long rows)
    const bool listed = !short_row && nchunks <= kMaxChunks;  // longer rows go straight to the whole-row path
    // the table of list segments has one entry per 128 scores (8 lanes of an iteration) while that fits,
    // else one per 512: finer entries spread the emission over more threads
    const int lpc_shift = nchunks * 4 <= kMaxChunks ? 3 : 5;
    const int lpc = 1 << lpc_shift;                           // lanes per table chunk
    const int ntab = (n + 16 * lpc - 1) / (16 * lpc);         // table chunks of 16 * lpc scores

    if (tid == 0) { sh.overflow = 0u; sh.list_total = 0u; }

    // ---- pass 0 (long rows): candidate threshold from a sample --------------------------------
    // 256 chunks of 32 consecutive scores, evenly spread, give (a) an estimate of the row's variance and
    // with it an upper estimate k_hi of the budget, (b) a key tau that about 1.3 * k_hi scores reach.
    float tau_f = listed ? -INFINITY : INFINITY;              // not listed: nothing is a candidate
    uint32_t tau_key = 0u;                                    // the same threshold as an order key
    if (listed) {
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
        tau_key = tau;
    }
    __syncthreads();

    // ---- pass 1: fp64 moments of every score; candidates into the list -------------------------
    double s1 = 0.0, s2 = 0.0;
    uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;                   // range of the keys that went into the list
    // Long rows are cut into chunks of 512 consecutive scores, dealt to the 16 warps round-robin (chunk c
    // belongs to warp c % 16), one chunk per warp iteration.  Rows with more than kMaxChunks chunks are
    // not listed at all (tau_f = +inf below): they take the whole-row path.
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
        const int my_iters = wid < nchunks ? (nchunks - wid + kSelWarps - 1) / kSelWarps : 0;
        kmin = tau_key;                                       // every listed key reaches the threshold
        bool w_over = false;
        // The 512 scores of an iteration arrive by coalesced 16-byte loads (lane l gets scores 4l..4l+3 of
        // each 128) and are turned, through shared memory, so that lane l holds scores 16l..16l+15: a
        // lane's candidates are then consecutive in position order and one warp scan of the counts places
        // them.  The staging buffer is the upper half of list_key and the histogram behind it (idle during this
        // pass); a candidate's score is read back from it for the order key that goes into the list with the
        // position, as long as the list has not grown into the staging area (entries from kKeysInScan on, rare:
        // they get their keys after the pass).
        // 16-byte slot q (= position / 4) is kept at q ^ ((q >> 3) & 3): no bank conflicts either way.
        float4* const tb = reinterpret_cast<float4*>(sh.list_key + kKeysInScan + wid * kIter);
        const float* const tbf = reinterpret_cast<const float*>(tb);
        const int wslot = lane ^ ((lane >> 3) & 3);
        const int rsw = (lane >> 1) & 3;
        // loads run one iteration ahead
        float4 ld[4];
        if (my_iters > 0 && (wid + 1) * kIter <= n) {
            const float4* const gp = reinterpret_cast<const float4*>(grow + wid * kIter) + lane;
#pragma unroll
            for (int v = 0; v < 4; ++v) ld[v] = __ldg(gp + 32 * v);
        }
        for (int j = 0; j < my_iters; ++j) {
            const int c = wid + kSelWarps * j;                // this iteration's chunk
            const int rs0 = c * kIter;                        // its first score
            uint32_t flags = 0;                               // bit e: score rs0 + 16 lane + e is a candidate
            if (rs0 + kIter <= n) {
                __syncwarp();                                 // the previous iteration's slots have been read
#pragma unroll
                for (int v = 0; v < 4; ++v) tb[wslot + 32 * v] = ld[v];
                __syncwarp();
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float4 xv = tb[4 * lane + (u ^ rsw)];
                    const float xs[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const double xd = (double)xs[e];
                        s1 += xd;
                        s2 = fma(xd, xd, s2);
                        flags |= (xs[e] >= tau_f ? 1u : 0u) << (u * 4 + e);
                    }
                }
            } else {                                          // the row's last, partial chunk
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const int i = rs0 + lane * 16 + e;
                    if (i < n) {
                        const float x = __ldg(grow + i);
                        const double xd = (double)x;
                        s1 += xd;
                        s2 = fma(xd, xd, s2);
                        flags |= (x >= tau_f ? 1u : 0u) << e;
                    }
                }
            }
            // next iteration's loads, issued before the scan and the list stores so that this work covers
            // part of their latency
            if (j + 1 < my_iters && rs0 + (kSelWarps + 1) * kIter <= n) {
                const float4* const gp = reinterpret_cast<const float4*>(grow + rs0 + kSelWarps * kIter) + lane;
#pragma unroll
                for (int v = 0; v < 4; ++v) ld[v] = __ldg(gp + 32 * v);
            }
            const uint32_t cnt = __popc(flags);
            uint32_t inc = cnt;                               // candidates of lanes 0..lane
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, inc, o);
                if (lane >= o) inc += u;
            }
            const uint32_t iter_total = __shfl_sync(0xFFFFFFFFu, inc, 31);
            // the iteration's entries are consecutive in the list: lane 31 claims the space; the last lane
            // of every table chunk (8 or 32 lanes) notes where the chunk's entries start and how many there are
            if (listed) {
                uint32_t base = 0;
                if (lane == 31 && iter_total != 0u) base = atomicAdd(&sh.list_total, iter_total);
                base = __shfl_sync(0xFFFFFFFFu, base, 31);
                const int first = lane & ~(lpc - 1);                        // first lane of this lane's chunk
                uint32_t before = __shfl_sync(0xFFFFFFFFu, inc, first > 0 ? first - 1 : 0);
                if (first == 0) before = 0u;                                // candidates of the chunks before it
                if ((lane & (lpc - 1)) == lpc - 1) {
                    const int tc = (c << (5 - lpc_shift)) + (lane >> lpc_shift);
                    if (tc < ntab) {
                        sh.ch_off[tc] = (uint16_t)min(base + before, (uint32_t)kListCap);
                        sh.ch_cnt[tc] = (uint16_t)(inc - before);
                    }
                }
                if (iter_total != 0u) {
                    if (base + iter_total <= (uint32_t)kListCap) {
                        uint32_t pos = base + inc - cnt;
                        const uint32_t ib = (uint32_t)(rs0 + lane * 16);
                        uint32_t f = flags;
                        while (f) {                           // one candidate per pass and lane
                            sh.list_pos[pos++] = ib + (uint32_t)(__ffs(f) - 1);
                            f &= f - 1;
                        }
                        __syncwarp();
                        // the chunk's order keys, all lanes side by side: the scores are still in the staging area
                        // (slot q = offset / 4, swizzled) or, for the row's partial last chunk, in global memory
                        for (uint32_t q = lane; q < iter_total && base + q < (uint32_t)kKeysInScan; q += 32) {
                            const uint32_t at = sh.list_pos[base + q];
                            float x;
                            if (rs0 + kIter <= n) {
                                const uint32_t off = at - (uint32_t)rs0, slot = off >> 2;
                                x = tbf[4 * (slot ^ ((slot >> 3) & 3)) + (off & 3)];
                            } else {
                                x = __ldg(grow + at);
                            }
                            const uint32_t key = order_key(x);
                            sh.list_key[base + q] = key;
                            kmax = max(kmax, key);
                        }
                    } else {
                        w_over = true;
                    }
                }
            }
        }
        if (w_over && lane == 0) sh.overflow = 1u;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        s1 += __shfl_xor_sync(0xFFFFFFFFu, s1, o);
        s2 += __shfl_xor_sync(0xFFFFFFFFu, s2, o);
    }
    if (lane == 0) { sh.red_a[wid] = s1; sh.red_b[wid] = s2; }
    __syncthreads();
    const int m = listed ? (int)min(sh.list_total, (uint32_t)kListCap) : 0;   // candidates found (all listed unless overflow)
    if (listed && sh.overflow == 0u)                                          // entries that pass 1 left without a key
        for (int q = kKeysInScan + tid; q < m; q += kSelThreads) {
            const uint32_t key = order_key(__ldg(grow + sh.list_pos[q]));
            sh.list_key[q] = key;
            kmax = max(kmax, key);
        }
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

    uint32_t T, need_eq, eq_total;
    if (short_row) {
        // ---- the row is the list: radix rounds, then one ordered compaction -------------------
        radix_rounds(sh, n, [&](int i) { return sh.list_key[i]; }, kmin, kmax, (uint32_t)k, T, need_eq, eq_total);
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

    if (!overflow && m >= k) {
        // ---- exact threshold among the candidates ------------------------------------------------
        radix_rounds(sh, m, [&](int i) { return sh.list_key[i]; }, kmin, kmax, (uint32_t)k, T, need_eq, eq_total);

        if (eq_total == need_eq && n <= kBins * 32) {
            // ---- emission through a bitmap of the row's positions (every key equal to T is taken, so the
            // selected candidates are simply those with key >= T): the candidates mark their positions, all
            // threads side by side, then every thread turns its stretch of the bitmap into ascending positions.
            // The bitmap is the histogram's space: one bit per position, rows of up to 32 * kBins scores.
            const int words = (n + 31) >> 5;
            for (int i = tid; i < words; i += kSelThreads) sh.hist[i] = 0u;
            __syncthreads();
            for (int q = tid; q < m; q += kSelThreads)
                if (sh.list_key[q] >= T) {
                    const uint32_t pos = sh.list_pos[q];
                    atomicOr(&sh.hist[pos >> 5], 1u << (pos & 31u));
                }
            __syncthreads();
            const int wpt = (words + kSelThreads - 1) / kSelThreads;            // 1 .. 8
            const int w_lo = min(words, tid * wpt), w_hi = min(words, w_lo + wpt);
            uint32_t mine = 0;
            for (int w = w_lo; w < w_hi; ++w) mine += __popc(sh.hist[w]);
            uint32_t total;
            uint32_t at = block_excl_scan(sh, mine, 0, total);
            for (int w = w_lo; w < w_hi; ++w) {
                uint32_t bits = sh.hist[w];
                while (bits) {
                    out_idx[at++] = (int32_t)((w << 5) + __ffs(bits) - 1);
                    bits &= bits - 1u;
                }
            }
            for (int i = k + tid; i < a.k_max; i += kSelThreads) out_idx[i] = -1;
            return;
        }

        // ---- emission in position order: thread t owns table chunks t*cpt .. t*cpt + cpt - 1 -------
        const int cpt = (ntab + kSelThreads - 1) / kSelThreads;             // 1 .. 4
        const int c_lo = min(ntab, tid * cpt), c_hi = min(ntab, c_lo + cpt);
        uint32_t g = 0, q = 0;
        for (int c = c_lo; c < c_hi; ++c) {
            const uint32_t off = sh.ch_off[c];
            const int cnt = sh.ch_cnt[c];
            for (int j = 0; j < cnt; ++j) {
                const uint32_t key = sh.list_key[off + j];
                g += key > T;
                q += key == T;
            }
        }
        uint32_t total;
        const uint32_t before = block_excl_scan(sh, (q << 16) | g, 0, total);
        uint32_t g_before = before & 0xFFFFu, e_before = before >> 16;
        for (int c = c_lo; c < c_hi; ++c) {
            const uint32_t off = sh.ch_off[c];
            const int cnt = sh.ch_cnt[c];
            for (int j = 0; j < cnt; ++j) {
                const uint32_t key = sh.list_key[off + j];
                if (key > T) {
                    out_idx[g_before + min(e_before, need_eq)] = (int32_t)sh.list_pos[off + j];
                    ++g_before;
                } else if (key == T) {
                    if (e_before < need_eq) out_idx[g_before + e_before] = (int32_t)sh.list_pos[off + j];
                    ++e_before;
                }
            }
        }
    } else {
        // ---- fallback: radix rounds over the whole row, then ordered emission ----------------
        if (tid == 0 && a.fallback_rows) atomicAdd(a.fallback_rows, 1);
        radix_rounds(sh, n, [&](int i) { return order_key(__ldg(grow + i)); }, 0u, 0xFFFFFFFFu,
                     (uint32_t)k, T, need_eq, eq_total);
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

// k_mode 3 without scores: S_t is every visible key
__global__ void __launch_bounds__(256) gsa_all_visible_kernel(RowRange rr, IdxLayout il, int32_t Lq, int32_t Lk,
                                                              int32_t k_max, int32_t* __restrict__ idx,
                                                              int32_t* __restrict__ kt, float* __restrict__ var) {
    const int lr = blockIdx.x;
    const int b = rr.b0 + lr / rr.R, t = rr.q_begin + lr % rr.R;
    const int n = Lk - Lq + t + 1;
    const int64_t row = il.row(b, t);
    for (int i = threadIdx.x; i < k_max; i += blockDim.x) idx[row * k_max + i] = i < n ? i : -1;
    if (threadIdx.x == 0) {
        kt[row] = n;
        if (var) var[row] = 0.f;
    }
}

}  // namespace

cudaError_t launch_all_visible(const gsa_params_t& p, RowRange rr, int32_t* idx, int32_t* kt, float* var,
                               IdxLayout il, cudaStream_t st) {
    if (rr.rows() <= 0) return cudaSuccess;
    gsa_all_visible_kernel<<<rr.rows(), 256, 0, st>>>(rr, il, p.Lq, p.Lk, p.k_max, idx, kt, var);
    ++g_launches;
    return cudaGetLastError();
}

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
    // (set on every call: the attribute belongs to the current device)
    {
        cudaError_t e = cudaFuncSetAttribute(gsa_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    gsa_select_kernel<<<rr.rows(), kSelThreads, smem, st>>>(a);
    ++g_launches;
    return cudaGetLastError();
}

}  // namespace gsa
