// Backward of sparse gated attention, key-major half: dK, dV, dg2.
//
// dK[s] and dV'[s] are sums over every (query row, head) whose index set holds key s.  Instead of
// scattering fp32 additions from the query side, the index sets are inverted once per call
//     count (one integer atomic per selected pair) -> exclusive scan -> fill (one more integer atomic)
// into, for every key, the list of query rows that selected it; one warp per key then walks its list.
// The index sets are shared by all heads, so a tile of 16 rows is "a few queries x their heads": a
// contiguous block of Q (and of do = dout * sigmoid(g1)), copied into shared memory by 16-byte
// asynchronous copies.  With the KV heads of key s as the N columns (K[s] and V'[s] are contiguous too):
//     S[(t,h), g]   = Q[t,h] . K[s,g]          dP[(t,h), g] = do[t,h] . V'[s,g]      (A: tile via ldmatrix)
//     P = 2^(c S - lse2[t,h]),  dS = P (dP - delta[t,h]),  both zero unless g is the KV head of h
//     dK^T[d, g] += Q^T[d, (t,h)] dS[(t,h), g]   dV'^T[d, g] += do^T[d, (t,h)] P[(t,h), g]  (ldmatrix.trans)
// on the tensor cores (bf16 mma.sync, fp32 accumulation); lse2 and delta come from the query-major
// kernel.  The epilogue applies the value gate's derivative and rounds to bf16 once.  The order of a key's
// list depends on scheduling (integer atomics hand out the slots), so the fp32 sums may differ in the last
// bits from run to run.
// Bound: the gather of Q and do, 2 * n_h * d_h * 2 bytes per selected (query, key) pair.  For more than
// kBwdRangeRows query rows per sequence the rows are cut into ranges whose Q and do (8 KB per row at 16
// heads of 128) fit the L2 with room to spare: the lists are filled range by range, so each list is grouped by range, and the
// work items run range-major, (range, key), so that the warps in flight share one range.  The partial
// sums of a key's ranges then meet in fp32 arrays (one reduction per range and element, not per pair) and
// a streaming post-pass applies the gate's derivative and rounds.
#include "gsa_common.cuh"

namespace gsa {

namespace {

constexpr int kKeyWarps = 4;
constexpr int kBwdRangeRows = 4096;                  // query rows per range: 32 MB of Q and do at 16 x 128 (measured best of 2048 .. 8192)
constexpr int kBwdMaxRanges = 64;
constexpr int kScanThreads = 1024;
constexpr int kScanPerThread = 4;
constexpr int kScanBlock = kScanThreads * kScanPerThread;      // 4096 counters per block
constexpr float kLog2eK = 1.4426950408889634f;

// ---- inverting the index sets -------------------------------------------------------------------------
struct InvArgs {
    const int32_t* idx;
    const int32_t* kt;
    RowRange rr;
    IdxLayout il;
    int32_t Lq, Lk, k_max;
    int32_t* dev_status;          // where a skipped entry is reported (may be null)
};

// one warp per query row: cnt[b * Lk + s] += 1 for every selected s
__global__ void __launch_bounds__(256) gsa_bwd_count_kernel(const InvArgs a, int32_t* __restrict__ cnt) {
    const int lane = threadIdx.x & 31;
    const int64_t lr = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (lr >= a.rr.rows()) return;
    const int b = a.rr.b0 + (int)(lr / a.rr.R), t = a.rr.q_begin + (int)(lr % a.rr.R);
    const int64_t irow = a.il.row(b, t);
    const int ke = clamp_budget(a.kt[irow], a.k_max);
    const int32_t* __restrict__ S = a.idx + irow * a.k_max;
    for (int j = lane; j < ke; j += 32) {
        const int32_t s = S[j];
        if (key_in_range(s, a.Lk)) atomicAdd(cnt + (int64_t)b * a.Lk + s, 1);
        else report_bad_index(a.dev_status);
    }
}

// one warp per query row: the row's number goes into the list of every selected key
__global__ void __launch_bounds__(256) gsa_bwd_fill_kernel(const InvArgs a, int32_t* __restrict__ cur,
                                                           int32_t* __restrict__ rows_of_key) {
    const int lane = threadIdx.x & 31;
    const int64_t lr = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (lr >= a.rr.rows()) return;
    const int b = a.rr.b0 + (int)(lr / a.rr.R), t = a.rr.q_begin + (int)(lr % a.rr.R);
    const int64_t irow = a.il.row(b, t);
    const int ke = clamp_budget(a.kt[irow], a.k_max);
    const int32_t* __restrict__ S = a.idx + irow * a.k_max;
    const int32_t qrow = b * a.Lq + t;
    for (int j = lane; j < ke; j += 32) {
        const int32_t s = S[j];
        if (!key_in_range(s, a.Lk)) continue;             // (the same entries the count skipped)
        const int32_t pos = atomicAdd(cur + (int64_t)b * a.Lk + s, 1);
        rows_of_key[pos] = qrow;
    }
}

__device__ __forceinline__ int32_t block_excl_scan_i32(int32_t v, int32_t* warp_tot, int32_t& total) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    int32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t u = __shfl_up_sync(0xFFFFFFFFu, inc, o);
        if (lane >= o) inc += u;
    }
    if (lane == 31) warp_tot[wid] = inc;
    __syncthreads();
    int32_t before = 0, tot = 0;
    for (int i = 0; i < kScanThreads / 32; ++i) {
        const int32_t w = warp_tot[i];
        before += i < wid ? w : 0;
        tot += w;
    }
    __syncthreads();
    total = tot;
    return before + inc - v;
}

// exclusive scan of n counters in three steps: block sums, scan of the block sums, final offsets
__global__ void __launch_bounds__(kScanThreads) gsa_bwd_scan_sums_kernel(const int32_t* __restrict__ cnt, int64_t n,
                                                                         int32_t* __restrict__ bsum) {
    __shared__ int32_t warp_tot[kScanThreads / 32];
    const int64_t base = (int64_t)blockIdx.x * kScanBlock + threadIdx.x * kScanPerThread;
    int32_t v = 0;
#pragma unroll
    for (int e = 0; e < kScanPerThread; ++e) v += base + e < n ? cnt[base + e] : 0;
    int32_t total;
    block_excl_scan_i32(v, warp_tot, total);
    if (threadIdx.x == 0) bsum[blockIdx.x] = total;
}
__global__ void __launch_bounds__(kScanThreads) gsa_bwd_scan_top_kernel(int32_t* __restrict__ bsum, int nblk) {
    __shared__ int32_t warp_tot[kScanThreads / 32];
    __shared__ int32_t carry;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int c0 = 0; c0 < nblk; c0 += kScanThreads) {             // (one pass up to 1024 blocks = 4 Mi keys)
        const int i = c0 + threadIdx.x;
        const int32_t v = i < nblk ? bsum[i] : 0;
        int32_t total;
        const int32_t ex = block_excl_scan_i32(v, warp_tot, total);
        if (i < nblk) bsum[i] = carry + ex;
        __syncthreads();
        if (threadIdx.x == 0) carry += total;
        __syncthreads();
    }
}
__global__ void __launch_bounds__(kScanThreads) gsa_bwd_scan_final_kernel(const int32_t* __restrict__ cnt, int64_t n,
                                                                          const int32_t* __restrict__ bsum,
                                                                          int32_t* __restrict__ off,
                                                                          int32_t* __restrict__ cur) {
    __shared__ int32_t warp_tot[kScanThreads / 32];
    const int64_t base = (int64_t)blockIdx.x * kScanBlock + threadIdx.x * kScanPerThread;
    int32_t c[kScanPerThread], v = 0;
#pragma unroll
    for (int e = 0; e < kScanPerThread; ++e) { c[e] = base + e < n ? cnt[base + e] : 0; v += c[e]; }
    int32_t total;
    int32_t run = bsum[blockIdx.x] + block_excl_scan_i32(v, warp_tot, total);
#pragma unroll
    for (int e = 0; e < kScanPerThread; ++e) {
        if (base + e < n) { off[base + e] = run; cur[base + e] = run; }
        run += c[e];
    }
}

// ---- the key-major kernel -----------------------------------------------------------------------------
struct KeyArgs {
    const __nv_bfloat16* Q;
    const __nv_bfloat16* dOs;
    const __nv_bfloat16* K;
    const __nv_bfloat16* V;
    const __nv_bfloat16* Vg;
    const __nv_bfloat16* g2;
    const float* lse2;
    const float* delta;
    const int32_t* off;           // key -> first entry of its list
    const int32_t* bnd;           // [n_ranges][n_keys]: one past the key's last entry of range r (and before)
    float* dK32;                  // partial sums meet here when there are several ranges
    float* dV32;
    const int32_t* rows_of_key;
    __nv_bfloat16* dK;
    __nv_bfloat16* dV;
    __nv_bfloat16* dg2;
    int64_t n_keys;               // B * Lk
    int32_t n_h, n_kv, G;
    int32_t HB;                   // heads per tile row block: min(n_h, 16), a power of two
    int32_t hb_shift;             // log2(HB)
    int32_t NHB;                  // head blocks: n_h / HB
    float scale;
};

__device__ __forceinline__ uint32_t movmatrix_tk(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ float ex2_approx_k(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int DH, bool PARTIAL>
__global__ void __launch_bounds__(kKeyWarps * 32) gsa_sparse_attn_bwd_keys_kernel(const KeyArgs a, const int n_ranges) {
    constexpr int ROW = (DH + 8) * 2;                  // bytes of a padded tile row (odd multiple of 16)
    constexpr int TILE16 = 16 * ROW, TILE8 = 8 * ROW;
    constexpr int STAGE = 2 * TILE16;                  // a Q tile and a do tile
    constexpr int WARP_SMEM = 2 * STAGE;               // two stages; the B-operand tiles borrow stage 1 first
    constexpr int KS = DH / 16;
    constexpr int CPR = DH / 8;                        // 16-byte chunks per row
    extern __shared__ __align__(16) unsigned char key_smem[];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gid = lane >> 2, tig = lane & 3;
    const int64_t item = (int64_t)blockIdx.x * kKeyWarps + warp;
    if (item >= a.n_keys * a.NHB * n_ranges) return;   // (no block-wide barrier below)
    // range-major: all keys of query range 0, then range 1, ...
    const int range = (int)(item / (a.n_keys * a.NHB));
    const int64_t key = (item / a.NHB) % a.n_keys;     // b * Lk + s
    const int hb = (int)(item % a.NHB);
    const int beg = range == 0 ? a.off[key] : a.bnd[(int64_t)(range - 1) * a.n_keys + key];
    const int end = a.bnd[(int64_t)range * a.n_keys + key];
    if (PARTIAL && beg == end) return;                 // nothing of this key in this range
    const int h_base = hb * a.HB;                      // first head of the block
    const int g_base = h_base / a.G;                   // its KV head = column 0
    const int n_cols = a.HB / a.G > 0 ? a.HB / a.G : 1;   // KV heads the block's heads map to (<= 8)
    const int TQ = 16 / a.HB;                          // queries per tile

    unsigned char* const ws = key_smem + warp * WARP_SMEM;
    const uint32_t st_s32 = (uint32_t)__cvta_generic_to_shared(ws);       // stage i: Q tile at i * STAGE, do tile after it
    const uint32_t k_s32 = st_s32 + STAGE;
    const uint32_t v_s32 = k_s32 + TILE8;

    // B operands: rows = KV heads g_base .. (zero rows beyond n_cols), K[s] and V'[s]
    {
        const __nv_bfloat16* const krow = a.K + (key * a.n_kv + g_base) * DH;
        const __nv_bfloat16* const vrow = a.Vg + (key * a.n_kv + g_base) * DH;
#pragma unroll
        for (int i = 0; i < 8 * CPR / 32; ++i) {
            const int chunk = i * 32 + lane;
            const int r = chunk / CPR, c = chunk % CPR;
            uint4 kv = make_uint4(0u, 0u, 0u, 0u), vv = kv;
            if (r < n_cols) {
                kv = *reinterpret_cast<const uint4*>(krow + r * DH + c * 8);
                vv = *reinterpret_cast<const uint4*>(vrow + r * DH + c * 8);
            }
            *reinterpret_cast<uint4*>(ws + STAGE + r * ROW + c * 16) = kv;
            *reinterpret_cast<uint4*>(ws + STAGE + TILE8 + r * ROW + c * 16) = vv;
        }
    }
    __syncwarp();
    uint32_t kb[2 * KS], vb[2 * KS];
#pragma unroll
    for (int k2 = 0; k2 < KS / 2; ++k2) {
        const uint32_t o = (lane & 7) * ROW + (lane >> 3) * 16 + k2 * 64;
        ldmatrix_x4(kb[4 * k2], kb[4 * k2 + 1], kb[4 * k2 + 2], kb[4 * k2 + 3], k_s32 + o);
        ldmatrix_x4(vb[4 * k2], vb[4 * k2 + 1], vb[4 * k2 + 2], vb[4 * k2 + 3], v_s32 + o);
    }
    __syncwarp();                                      // stage 1 is free for tiles from here on

    auto tile_times = [&](uint32_t tile_s32, const uint32_t (&bf)[2 * KS], float (&acc)[4]) {
        // two accumulators (even / odd k-steps): half the length of the dependent MMA chain
        float acc2[4] = {0.f, 0.f, 0.f, 0.f};
        acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
        const uint32_t addr = tile_s32 + (lane & 15) * ROW + (lane >> 4) * 16;
#pragma unroll
        for (int ks = 0; ks < KS; ks += 2) {
            uint32_t a0, a1, a2, a3, c0, c1, c2r, c3;
            ldmatrix_x4(a0, a1, a2, a3, addr + ks * 32);
            ldmatrix_x4(c0, c1, c2r, c3, addr + (ks + 1) * 32);
            mma_bf16_16816(acc, a0, a1, a2, a3, bf[2 * ks], bf[2 * ks + 1]);
            mma_bf16_16816(acc2, c0, c1, c2r, c3, bf[2 * ks + 2], bf[2 * ks + 3]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] += acc2[i];
    };

    const float c2 = a.scale * kLog2eK;
    float dk[KS][4], dv[KS][4];
#pragma unroll
    for (int mt = 0; mt < KS; ++mt) {
        dk[mt][0] = dk[mt][1] = dk[mt][2] = dk[mt][3] = 0.f;
        dv[mt][0] = dv[mt][1] = dv[mt][2] = dv[mt][3] = 0.f;
    }
    // tile row r = (query r / HB of the tile, head h_base + r % HB); this lane's rows are gid and gid + 8
    const int q_of_r0 = gid >> a.hb_shift, q_of_r1 = (gid + 8) >> a.hb_shift;
    const int h_r0 = h_base + (gid & (a.HB - 1)), h_r1 = h_base + ((gid + 8) & (a.HB - 1));
    const int col_r0 = h_r0 / a.G - g_base, col_r1 = h_r1 / a.G - g_base;     // the one column that counts

    // tiles are fetched one iteration ahead, together with the statistics of this lane's two rows
    int32_t qr_n0 = 0, qr_n1 = 0;
    float lse_n0 = 0.f, lse_n1 = 0.f, dl_n0 = 0.f, dl_n1 = 0.f;
    auto fetch = [&](int j, int stage) {
        if (j < end) {
            // lanes 0 .. TQ-1 hold the tile's query rows (the last one repeated past the end of the list)
            const int32_t t16 = a.rows_of_key[min(j + (lane & 15), end - 1)];
            const uint32_t q_dst = st_s32 + stage * STAGE, d_dst = q_dst + TILE16;
#pragma unroll
            for (int i = 0; i < 16 * CPR / 32; ++i) {
                const int chunk = i * 32 + lane;
                const int r = chunk / CPR, c = chunk % CPR;
                const int32_t qrow = __shfl_sync(0xFFFFFFFFu, t16, r >> a.hb_shift);
                const size_t at = ((size_t)qrow * a.n_h + h_base + (r & (a.HB - 1))) * DH + c * 8;
                cp_async16(q_dst + r * ROW + c * 16, a.Q + at);
                cp_async16(d_dst + r * ROW + c * 16, a.dOs + at);
            }
            qr_n0 = __shfl_sync(0xFFFFFFFFu, t16, q_of_r0);
            qr_n1 = __shfl_sync(0xFFFFFFFFu, t16, q_of_r1);
            lse_n0 = a.lse2[(size_t)qr_n0 * a.n_h + h_r0];
            lse_n1 = a.lse2[(size_t)qr_n1 * a.n_h + h_r1];
            dl_n0 = a.delta[(size_t)qr_n0 * a.n_h + h_r0];
            dl_n1 = a.delta[(size_t)qr_n1 * a.n_h + h_r1];
        }
        cp_async_commit();                                // (possibly empty: keeps the group count uniform)
    };
    fetch(beg, 0);
    int stage = 0;
    for (int j0 = beg; j0 < end; j0 += TQ, stage ^= 1) {
        const float lse0 = lse_n0, lse1 = lse_n1, dl0 = dl_n0, dl1 = dl_n1;
        const bool v0 = j0 + q_of_r0 < end, v1 = j0 + q_of_r1 < end;
        fetch(j0 + TQ, stage ^ 1);                        // (the other stage was released at the end of the last iteration)
        cp_async_wait<1>();
        __syncwarp();
        const uint32_t q_s32 = st_s32 + stage * STAGE, d_s32 = q_s32 + TILE16;
        float s[4], dp[4], p[4], ds[4];
        tile_times(q_s32, kb, s);
        tile_times(d_s32, vb, dp);
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int col = 2 * tig + e;
            p[e] = (v0 && col == col_r0) ? ex2_approx_k(s[e] * c2 - lse0) : 0.f;
            p[2 + e] = (v1 && col == col_r1) ? ex2_approx_k(s[2 + e] * c2 - lse1) : 0.f;
            ds[e] = p[e] * (dp[e] - dl0);
            ds[2 + e] = p[2 + e] * (dp[2 + e] - dl1);
        }
        const uint32_t bs0 = movmatrix_tk(pack_bf16(ds[0], ds[1])), bs1 = movmatrix_tk(pack_bf16(ds[2], ds[3]));
        const uint32_t bp0 = movmatrix_tk(pack_bf16(p[0], p[1])), bp1 = movmatrix_tk(pack_bf16(p[2], p[3]));
        {
            const int mi = lane >> 3;
            const uint32_t o = ((lane & 7) + (mi >> 1) * 8) * ROW + (mi & 1) * 16;
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                uint32_t a0, a1, a2, a3;
                ldmatrix_x4_trans(a0, a1, a2, a3, q_s32 + o + mt * 32);
                mma_bf16_16816(dk[mt], a0, a1, a2, a3, bs0, bs1);
                ldmatrix_x4_trans(a0, a1, a2, a3, d_s32 + o + mt * 32);
                mma_bf16_16816(dv[mt], a0, a1, a2, a3, bp0, bp1);
            }
        }
        __syncwarp();                                     // this stage is refilled by the next iteration
    }
    cp_async_wait<0>();

    // ---- epilogue: fragment rows are d, columns the KV heads g_base + 2 tig, + 1 ------------------------
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int col = 2 * tig + e;
        if (col < n_cols) {
            const size_t row = (key * a.n_kv + g_base + col) * DH;
#pragma unroll
            for (int mt = 0; mt < KS; ++mt)
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const size_t at = row + mt * 16 + gid + hf * 8;
                    const float dvg = dv[mt][2 * hf + e];
                    if (PARTIAL) {
                        atomicAdd(a.dK32 + at, dk[mt][2 * hf + e] * a.scale);
                        atomicAdd(a.dV32 + at, dvg);
                    } else {
                        const float sg = 1.0f / (1.0f + __expf(-__bfloat162float(a.g2[at])));
                        a.dK[at] = __float2bfloat16(dk[mt][2 * hf + e] * a.scale);
                        a.dV[at] = __float2bfloat16(dvg * sg);
                        a.dg2[at] = __float2bfloat16(dvg * __bfloat162float(a.V[at]) * sg * (1.0f - sg));
                    }
                }
        }
    }
}

// dK = bf16(dK32);  dV = bf16(dV'32 * sigmoid(g2));  dg2 = bf16(dV'32 * V * sigmoid'(g2))
__global__ void __launch_bounds__(256) gsa_attn_bwd_finish_kernel(const float* __restrict__ dK32,
                                                                  const float* __restrict__ dV32,
                                                                  const __nv_bfloat16* __restrict__ V,
                                                                  const __nv_bfloat16* __restrict__ g2,
                                                                  __nv_bfloat16* __restrict__ dK,
                                                                  __nv_bfloat16* __restrict__ dV,
                                                                  __nv_bfloat16* __restrict__ dg2, int64_t n) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x * 4;
    for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4; i < n; i += stride) {
        const float4 k4 = *reinterpret_cast<const float4*>(dK32 + i);
        const float4 v4 = *reinterpret_cast<const float4*>(dV32 + i);
        const uint2 vr = *reinterpret_cast<const uint2*>(V + i);
        const uint2 gr = *reinterpret_cast<const uint2*>(g2 + i);
        const float dk[4] = {k4.x, k4.y, k4.z, k4.w}, dvg[4] = {v4.x, v4.y, v4.z, v4.w};
        const __nv_bfloat16* vv = reinterpret_cast<const __nv_bfloat16*>(&vr);
        const __nv_bfloat16* gg = reinterpret_cast<const __nv_bfloat16*>(&gr);
        __align__(8) __nv_bfloat16 ok[4], ov[4], og[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float sg = 1.0f / (1.0f + __expf(-__bfloat162float(gg[e])));
            ok[e] = __float2bfloat16(dk[e]);
            ov[e] = __float2bfloat16(dvg[e] * sg);
            og[e] = __float2bfloat16(dvg[e] * __bfloat162float(vv[e]) * sg * (1.0f - sg));
        }
        *reinterpret_cast<uint2*>(dK + i) = *reinterpret_cast<const uint2*>(ok);
        *reinterpret_cast<uint2*>(dV + i) = *reinterpret_cast<const uint2*>(ov);
        *reinterpret_cast<uint2*>(dg2 + i) = *reinterpret_cast<const uint2*>(og);
    }
}

template <int DH, bool PARTIAL>
cudaError_t launch_keys_t(const KeyArgs& a, int n_ranges, cudaStream_t st) {
    constexpr int ROW = (DH + 8) * 2;
    constexpr int WARP_SMEM = 4 * 16 * ROW;
    const int smem = kKeyWarps * WARP_SMEM;
    // (set on every call: the attribute belongs to the current device)
    {
        cudaError_t e = cudaFuncSetAttribute(gsa_sparse_attn_bwd_keys_kernel<DH, PARTIAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
    }
    const int64_t items = a.n_keys * a.NHB * n_ranges;
    const int64_t ctas = (items + kKeyWarps - 1) / kKeyWarps;
    gsa_sparse_attn_bwd_keys_kernel<DH, PARTIAL><<<(unsigned)ctas, kKeyWarps * 32, smem, st>>>(a, n_ranges);
    ++g_launches;
    return cudaGetLastError();
}

int bwd_ranges(int32_t rows_per_batch) {
    int n = (rows_per_batch + kBwdRangeRows - 1) / kBwdRangeRows;
    return n < 1 ? 1 : (n > kBwdMaxRanges ? kBwdMaxRanges : n);
}

}  // namespace

// integers the inversion needs: counters, offsets, cursors (n_keys each), block sums, range boundaries, the
// lists; then, with several ranges, the two fp32 arrays the partial sums meet in
size_t attn_bwd_invert_bytes(const gsa_params_t& p, int32_t rows_per_batch) {
    const size_t n_keys = (size_t)p.B * p.Lk;
    const size_t nblk = (n_keys + kScanBlock - 1) / kScanBlock;
    const int n_ranges = bwd_ranges(rows_per_batch);
    const size_t ints = (3 + n_ranges) * n_keys + nblk + (size_t)p.B * rows_per_batch * p.k_max;
    size_t bytes = (ints * 4 + 255) / 256 * 256;
    if (n_ranges > 1) bytes += 2 * ((n_keys * p.n_kv * p.d_h * 4 + 255) / 256 * 256);
    return bytes;
}

cudaError_t launch_sparse_attn_bwd_keys(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* Q,
                                        const __nv_bfloat16* dOs, const __nv_bfloat16* K, const __nv_bfloat16* V,
                                        const __nv_bfloat16* Vg, const __nv_bfloat16* g2, const float* lse2,
                                        const float* delta, const int32_t* idx, const int32_t* kt, IdxLayout il,
                                        void* invert_ws, __nv_bfloat16* dK, __nv_bfloat16* dV, __nv_bfloat16* dg2,
                                        cudaStream_t st) {
    const int64_t n_keys = (int64_t)p.B * p.Lk;
    const int nblk = (int)((n_keys + kScanBlock - 1) / kScanBlock);
    int32_t* cnt = (int32_t*)invert_ws;
    int32_t* off = cnt + n_keys;
    int32_t* cur = off + n_keys;
    const int n_ranges = bwd_ranges(rr.R);
    int32_t* bnd = cur + n_keys;
    int32_t* bsum = bnd + (size_t)n_ranges * n_keys;
    int32_t* rows_of_key = bsum + nblk;
    const size_t ints = (3 + (size_t)n_ranges) * n_keys + nblk + (size_t)p.B * rr.R * p.k_max;
    const size_t n_kv_elems = (size_t)n_keys * p.n_kv * p.d_h;
    float* dK32 = (float*)((char*)invert_ws + (ints * 4 + 255) / 256 * 256);
    float* dV32 = (float*)((char*)dK32 + (n_kv_elems * 4 + 255) / 256 * 256);

    cudaError_t e = cudaMemsetAsync(cnt, 0, (size_t)n_keys * 4, st);
    if (e != cudaSuccess) return e;
    InvArgs ia;
    ia.idx = idx; ia.kt = kt; ia.rr = rr; ia.il = il; ia.Lq = p.Lq; ia.Lk = p.Lk; ia.k_max = p.k_max;
    ia.dev_status = t_dev_status;
    const unsigned row_ctas = (unsigned)((rr.rows() + 7) / 8);
    if (rr.rows() > 0) {
        gsa_bwd_count_kernel<<<row_ctas, 256, 0, st>>>(ia, cnt);
        ++g_launches;
    }
    gsa_bwd_scan_sums_kernel<<<nblk, kScanThreads, 0, st>>>(cnt, n_keys, bsum);
    gsa_bwd_scan_top_kernel<<<1, kScanThreads, 0, st>>>(bsum, nblk);
    gsa_bwd_scan_final_kernel<<<nblk, kScanThreads, 0, st>>>(cnt, n_keys, bsum, off, cur);
    g_launches += 3;
    // the lists are filled range by range (in stream order), so every list is grouped by range; the
    // cursors after range r are the boundaries of range r
    const int range_rows = (rr.R + n_ranges - 1) / n_ranges;
    for (int r = 0; r < n_ranges; ++r) {
        InvArgs ir = ia;
        ir.rr.q_begin = rr.q_begin + r * range_rows;
        ir.rr.R = rr.R - r * range_rows < range_rows ? rr.R - r * range_rows : range_rows;
        if (ir.rr.rows() > 0) {
            gsa_bwd_fill_kernel<<<(unsigned)((ir.rr.rows() + 7) / 8), 256, 0, st>>>(ir, cur, rows_of_key);
            ++g_launches;
        }
        e = cudaMemcpyAsync(bnd + (size_t)r * n_keys, cur, (size_t)n_keys * 4, cudaMemcpyDeviceToDevice, st);
        if (e != cudaSuccess) return e;
    }
    if ((e = cudaGetLastError()) != cudaSuccess) return e;

    KeyArgs a;
    a.Q = Q; a.dOs = dOs; a.K = K; a.V = V; a.Vg = Vg; a.g2 = g2; a.lse2 = lse2; a.delta = delta;
    a.off = off; a.bnd = bnd; a.rows_of_key = rows_of_key; a.dK = dK; a.dV = dV; a.dg2 = dg2;
    a.dK32 = dK32; a.dV32 = dV32;
    a.n_keys = n_keys; a.n_h = p.n_h; a.n_kv = p.n_kv; a.G = p.n_h / p.n_kv;
    a.HB = p.n_h < 16 ? p.n_h : 16;
    a.NHB = p.n_h / a.HB;
    a.hb_shift = 0;
    while ((1 << a.hb_shift) < a.HB) ++a.hb_shift;
    a.scale = p.sm_scale > 0.f ? p.sm_scale : 1.0f / sqrtf((float)p.d_h);
    if (p.d_h != 128 && p.d_h != 64) return cudaErrorInvalidValue;
    if (n_ranges == 1)
        return p.d_h == 128 ? launch_keys_t<128, false>(a, 1, st) : launch_keys_t<64, false>(a, 1, st);
    if ((e = cudaMemsetAsync(dK32, 0, 2 * ((n_kv_elems * 4 + 255) / 256 * 256), st)) != cudaSuccess) return e;
    e = p.d_h == 128 ? launch_keys_t<128, true>(a, n_ranges, st) : launch_keys_t<64, true>(a, n_ranges, st);
    if (e != cudaSuccess) return e;
    {
        const int64_t n_elems = (int64_t)n_kv_elems;
        const int64_t want = (n_elems / 4 + 255) / 256;
        const int blocks = (int)(want < sm_count() * 16 ? want : sm_count() * 16);
        gsa_attn_bwd_finish_kernel<<<blocks, 256, 0, st>>>(dK32, dV32, V, g2, dK, dV, dg2, n_elems);
        ++g_launches;
    }
    return cudaGetLastError();
}

}  // namespace gsa
