// Backward of sparse gated attention (Eq. 9-12 and Eq. 10 differentiated; the index sets S_t are
// constants: top-k selection has no derivative and the indexer is trained by its own loss, Sec. 5.1).
//
// With out = o * sigmoid(g1), o = sum_j a_j v'_j, a = softmax_j(scale * q.k_j), v' = V * sigmoid(g2):
//   do    = dout * sigmoid(g1)
//   dg1   = dout * o * sigmoid'(g1)          = dout * out * (1 - sigmoid(g1))       (o * sigmoid = out)
//   delta = sum_j a_j (do . v'_j) = do . o   = sum_d dout_d * out_d
//   dz_j  = a_j (do . v'_j - delta),   dq = scale * sum_j dz_j k_j,   dK[s_j] += scale * dz_j q
//   dv'_j = a_j do  ->  dV = dv' * sigmoid(g2),   dg2 = dv' * V * sigmoid'(g2)      (post-pass)
// so the saved forward output is all the state the backward needs; the softmax statistics are
// recomputed from K in a first sweep over S_t.
//
// Two kernels, neither with floating-point atomics:
//  * this file, query-major: one warp per (query row, KV head).  Per 16 selected keys the K and V' rows
//    are copied (16-byte asynchronous copies) into a private shared-memory tile, the V' rows go straight
//    from global memory into MMA fragments, and every product runs on the tensor cores (bf16 mma.sync, fp32
//    accumulation) with the keys as M:
//        S^T[key, head] = K . Q^T           (A: tile via ldmatrix)
//        dP^T[key, head] = V' . do^T        (A: 32-byte loads, contraction index in load order)
//        dQ^T[d, head] += K^T . dS^T                                          (A: tile via ldmatrix.trans)
//    A streaming preparation kernel writes dg1, do (bf16) and delta per (row, head) first; this kernel
//    writes dQ and leaves the softmax statistics in the workspace for the other kernel.  When the keys span several L2-sized ranges (as in the forward pass:
//    random 256-byte rows come much faster out of L2 than out of HBM) the work items are (key range, row,
//    KV head), range-major, in two launches: the first leaves each range's softmax statistics, the second
//    combines them, does the gradient sweep over its range's part of S_t (ascending index sets make that a
//    contiguous sub-list) and adds its part of dQ into an fp32 array that a streaming pass rounds;
//  * gsa_attn_bwd_keys.cu, key-major: dK and dV' are sums over every query that selected the key, so the
//    index sets are first inverted (key -> list of query rows) and one warp per key then walks its list.
#include "gsa_common.cuh"

namespace gsa {

namespace {

constexpr int kBwdWarps = 4;
constexpr float kLog2e = 1.4426950408889634f;

struct BwdArgs {
    const __nv_bfloat16* Q;
    const __nv_bfloat16* K;
    const __nv_bfloat16* Vg;      // V' = bf16(V * sigmoid(g2)), as the forward uses it
    const __nv_bfloat16* g1;
    const __nv_bfloat16* out;     // the forward's output
    const __nv_bfloat16* dout;
    const int32_t* idx;
    const int32_t* kt;
    __nv_bfloat16* dQ;
    __nv_bfloat16* dg1;
    __nv_bfloat16* dOs;           // workspace: do = dout * sigmoid(g1), [B, Lq, n_h, d_h]
    float* lse2;                  // workspace: log2-domain log-sum-exp of the scaled logits, [B, Lq, n_h]
    float* delta;                 // workspace: sum_d dout * out, [B, Lq, n_h]
    float* pbar;                  // optional output: mean over the heads of P on S_t, [B, R, k_max], pre-zeroed
    const float* lse_in;          // optional: natural-log softmax statistics saved by the forward pass, [B, Lq, n_h]
    float2* part_ml;              // key ranges: per range (max, sum) of the scaled logits, [n_ranges][B * Lq * n_h]
    float* dq32;                  // key ranges: dQ summed over the ranges, [B, Lq, n_h, d_h], pre-zeroed
    int32_t range_keys, n_ranges;
    const int32_t* cuts;          // key ranges: [B * Lq][n_ranges + 1] first position of each range in the row's index set
    int64_t total_rows;           // B * Lq
    RowRange rr;
    IdxLayout il;
    int32_t Lq, Lk, n_h, n_kv, k_max;
    float scale;
    int32_t* dev_status;          // where an out-of-range index or budget is reported (may be null)
};

__device__ __forceinline__ uint32_t movmatrix_t(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Per (row, head), before the sweeps: do = dout * sigmoid(g1) (bf16), dg1 = dout * out * (1 - sigmoid(g1)),
// delta = sum_d dout * out.  One warp per (row, head).
template <int DH>
__global__ void __launch_bounds__(256) gsa_bwd_prep_kernel(const __nv_bfloat16* __restrict__ g1,
                                                           const __nv_bfloat16* __restrict__ out,
                                                           const __nv_bfloat16* __restrict__ dout,
                                                           __nv_bfloat16* __restrict__ dOs, __nv_bfloat16* __restrict__ dg1,
                                                           float* __restrict__ delta, RowRange rr, int32_t Lq, int32_t n_h) {
    constexpr int EPL = DH / 32;
    const int lane = threadIdx.x & 31;
    const int64_t w = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (w >= (int64_t)rr.rows() * n_h) return;
    const int lr = (int)(w / n_h), h = (int)(w % n_h);
    const int64_t qrow = (int64_t)(rr.b0 + lr / rr.R) * Lq + rr.q_begin + lr % rr.R;
    const int64_t at = (qrow * n_h + h) * DH + lane * EPL;
    float part = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
        const float dy = __bfloat162float(dout[at + e]);
        const float y = __bfloat162float(out[at + e]);
        const float sg = 1.0f / (1.0f + __expf(-__bfloat162float(g1[at + e])));
        dOs[at + e] = __float2bfloat16(dy * sg);
        dg1[at + e] = __float2bfloat16(dy * y * (1.0f - sg));
        part = fmaf(dy, y, part);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, o);
    if (lane == 0) delta[qrow * n_h + h] = part;
}

// first position j of the ascending list S[0 .. n) with S[j] >= x; the whole warp calls it (32 probes a round)
__device__ __forceinline__ int warp_lower_bound(const int32_t* __restrict__ S, int n, int x, int lane) {
    int lo = 0, len = n;
    while (len > 0) {
        const int step = (len + 31) >> 5;
        const int pos = lo + (lane + 1) * step - 1;
        const bool lt = pos < lo + len && S[pos] < x;
        const int c = __popc(__ballot_sync(0xFFFFFFFFu, lt));          // the first c probes are below x
        const int end = lo + len;
        lo += c * step;
        len = min(step - 1, end - lo);
        if (len < 0) len = 0;
    }
    return lo;
}

// cuts[row][c] = first position of the row's ascending index set that lies in key range c (c = n_ranges: the end)
__global__ void __launch_bounds__(256) gsa_bwd_range_cuts_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ kt,
                                                                 int32_t* __restrict__ cuts, RowRange rr, IdxLayout il,
                                                                 int32_t Lq, int32_t k_max, int32_t n_ranges, int32_t range_keys) {
    const int lane = threadIdx.x & 31;
    const int64_t lr = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (lr >= rr.rows()) return;
    const int b = rr.b0 + (int)(lr / rr.R), t = rr.q_begin + (int)(lr % rr.R);
    const int64_t irow = il.row(b, t);
    const int ke = clamp_budget(kt[irow], k_max);
    const int32_t* __restrict__ S = idx + irow * k_max;
    int32_t* const out = cuts + ((int64_t)b * Lq + t) * (n_ranges + 1);
    for (int c = 0; c <= n_ranges; ++c) {
        const int j = c == 0 ? 0 : (c == n_ranges ? ke : warp_lower_bound(S, ke, c * range_keys, lane));
        if (lane == 0) out[c] = j;
    }
}

// MODE 0: one item = (row, KV head), both sweeps over the whole index set.
// MODE 1: one item = (key range, row, KV head): statistics sweep over the range's part of S_t -> part_ml.
// MODE 2: one item = (key range, row, KV head): statistics combined from part_ml, gradient sweep over the
//         range's part, dQ added into dq32; the items of range 0 also write dg1, do, delta and lse2.
template <int DH, int G, int MODE>
__global__ void __launch_bounds__(kBwdWarps * 32, 4) gsa_sparse_attn_bwd_kernel(const BwdArgs a) {
    constexpr int ROW = (DH + 8) * 2;                  // bytes of a padded tile row (odd multiple of 16)
    constexpr int KTILE = 16 * ROW, QTILE = 8 * ROW;
    constexpr int STAGE = KTILE;                       // a K tile (V' rows go straight into MMA fragments)
    constexpr int WARP_SMEM = 2 * STAGE;               // two stages; the Q / do tiles borrow them before the sweeps
    static_assert(2 * QTILE <= WARP_SMEM, "the row's own tiles must fit the two stages");
    constexpr int NC = DH / 32;                        // 16-byte pieces of a head row per lane (register-direct rows)
    constexpr int KS = DH / 16;                        // k-steps of the S^T / dP^T products, m-tiles of dQ^T
    constexpr int EPL = DH / 32;                       // elements of a head row per lane (row staging)
    constexpr int CPR = DH / 8;                        // 16-byte chunks per tile row
    extern __shared__ __align__(16) unsigned char bwd_smem[];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gid = lane >> 2, tig = lane & 3;
    const int64_t item = (int64_t)blockIdx.x * kBwdWarps + warp;
    const int64_t per_range = (int64_t)a.rr.rows() * a.n_kv;
    if (item >= per_range * (MODE == 0 ? 1 : a.n_ranges)) return;     // (no block-wide barrier below)
    const int range = MODE == 0 ? 0 : (int)(item / per_range);       // range-major: the warps in flight share a range
    const int64_t rem = item % per_range;
    // long rows first: late rows have the most keys
    const int lr = a.rr.rows() - 1 - (int)(rem / a.n_kv);
    const int g = (int)(rem % a.n_kv);
    const int b = a.rr.b0 + lr / a.rr.R;
    const int t = a.rr.q_begin + lr % a.rr.R;
    const int64_t qrow = (int64_t)b * a.Lq + t;
    const int64_t irow = a.il.row(b, t);
    const int ke_all = checked_budget(a.kt[irow], a.k_max, a.dev_status);
    const int32_t* __restrict__ S = a.idx + irow * a.k_max;
    // this item's part of the index set: positions [j_lo, ke)
    int j_lo = 0, ke = ke_all;
    if (MODE != 0) {
        const int32_t* const cut = a.cuts + qrow * (a.n_ranges + 1) + range;
        j_lo = cut[0];
        ke = cut[1];
    }
    const bool writes_row = MODE == 0 || (MODE == 2 && range == 0);   // lse2 is written once per row
    if (MODE == 1 && j_lo >= ke) {                     // nothing of the row in this range
        if (lane < G) a.part_ml[((size_t)range * a.total_rows + qrow) * a.n_h + g * G + lane] = make_float2(-INFINITY, 0.f);
        return;
    }
    if (MODE == 2 && j_lo >= ke && !writes_row) return;

    unsigned char* const ws = bwd_smem + warp * WARP_SMEM;
    unsigned char* const q_tile = ws;                   // rows = the group's heads (rows >= G are zero)
    unsigned char* const d_tile = ws + QTILE;
    const uint32_t st_s32 = (uint32_t)__cvta_generic_to_shared(ws);   // stage i: K tile at i * STAGE
    const uint32_t q_s32 = (uint32_t)__cvta_generic_to_shared(q_tile);
    const uint32_t d_s32 = (uint32_t)__cvta_generic_to_shared(d_tile);

    // ---- the row's Q and do = dout * sigmoid(g1) (written by the preparation kernel) staged as tiles ---
#pragma unroll
    for (int hl = 0; hl < 8; ++hl) {
        __nv_bfloat16* qd = reinterpret_cast<__nv_bfloat16*>(q_tile + hl * ROW) + lane * EPL;
        __nv_bfloat16* dd = reinterpret_cast<__nv_bfloat16*>(d_tile + hl * ROW) + lane * EPL;
        const int64_t at = (qrow * a.n_h + (g * G + hl)) * DH + lane * EPL;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            qd[e] = hl < G ? a.Q[at + e] : __float2bfloat16(0.f);
            dd[e] = (hl < G && MODE != 1) ? a.dOs[at + e] : __float2bfloat16(0.f);
        }
    }
    __syncwarp();
    float delta[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) delta[e] = (MODE != 1 && 2 * tig + e < G) ? a.delta[qrow * a.n_h + g * G + 2 * tig + e] : 0.f;

    // B operands of S^T = K Q^T and dP^T = V' do^T: (k = d, n = head), kept for the whole row
    uint32_t qb[2 * KS];
#pragma unroll
    for (int k2 = 0; k2 < KS / 2; ++k2) {
        const uint32_t off = (lane & 7) * ROW + (lane >> 3) * 16 + k2 * 64;
        ldmatrix_x4(qb[4 * k2], qb[4 * k2 + 1], qb[4 * k2 + 2], qb[4 * k2 + 3], q_s32 + off);
    }
    // B operand of dP^T = V' do^T in the order the V' rows are loaded in: lane (gid, tig) brings bytes
    // [(c/2)*128 + tig*32 + (c%2)*16, +16) of the rows of keys gid and gid + 8 straight from global memory
    // into the A fragments, so the contraction index is permuted; do of head gid is read the same way
    uint4 dobd[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c)
        dobd[c] = *reinterpret_cast<const uint4*>(d_tile + gid * ROW + (c >> 1) * 128 + tig * 32 + (c & 1) * 16);
    __syncwarp();                                      // the stages are free for tiles from here on

    const float c2 = a.scale * kLog2e;
    const size_t kv_row = (size_t)a.n_kv * DH;           // elements between consecutive keys
    const __nv_bfloat16* const kbase = a.K + ((size_t)b * a.Lk * a.n_kv + g) * DH;
    const __nv_bfloat16* const vbase = a.Vg + ((size_t)b * a.Lk * a.n_kv + g) * DH;

    // copies the rows of 16 selected keys (positions held by lanes 0..15 of pos16) into a tile
    auto fetch_tile = [&](const __nv_bfloat16* base, uint32_t tile_s32, int32_t pos16) {
#pragma unroll
        for (int i = 0; i < 16 * CPR / 32; ++i) {
            const int chunk = i * 32 + lane;
            const int r = chunk / CPR, c = chunk % CPR;
            const int32_t p = __shfl_sync(0xFFFFFFFFu, pos16, r);
            cp_async16(tile_s32 + r * ROW + c * 16, base + (size_t)p * kv_row + c * 8);
        }
    };
    // S^T (or dP^T) of the staged tile: rows gid, gid + 8 = keys, columns 2 tig, 2 tig + 1 = heads
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

    // ---- sweep 1: softmax statistics per head (log2 domain) ----------------------------------------
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    // tiles are fetched one iteration ahead
    int32_t pos_fetched = 0;                              // positions of the tile fetched last (lanes 0..15)
    auto fetch = [&](int j, int stage) {
        if (j < ke) {
            pos_fetched = checked_pos(S[min(j + (lane & 15), ke - 1)], a.Lk, a.dev_status);
            fetch_tile(kbase, st_s32 + stage * STAGE, pos_fetched);
        }
        cp_async_commit();                                // (possibly empty: keeps the group count uniform)
    };
    // V' rows of 16 keys as A fragments (see dobd above)
    uint4 vb[2 * NC];
    const unsigned char* const vrow0 = reinterpret_cast<const unsigned char*>(vbase) + tig * 32;
    auto load_v = [&](int32_t pos16) {
        const uint32_t p0 = __shfl_sync(0xFFFFFFFFu, pos16, gid), p1 = __shfl_sync(0xFFFFFFFFu, pos16, gid + 8);
        const unsigned char* v0p = vrow0 + (size_t)p0 * kv_row * 2;
        const unsigned char* v1p = vrow0 + (size_t)p1 * kv_row * 2;
#pragma unroll
        for (int c = 0; c < NC; c += 2) {
            asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(vb[c].x), "=r"(vb[c].y), "=r"(vb[c].z), "=r"(vb[c].w), "=r"(vb[c + 1].x),
                           "=r"(vb[c + 1].y), "=r"(vb[c + 1].z), "=r"(vb[c + 1].w)
                         : "l"(v0p + (c >> 1) * 128));
            asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(vb[NC + c].x), "=r"(vb[NC + c].y), "=r"(vb[NC + c].z), "=r"(vb[NC + c].w),
                           "=r"(vb[NC + c + 1].x), "=r"(vb[NC + c + 1].y), "=r"(vb[NC + c + 1].z), "=r"(vb[NC + c + 1].w)
                         : "l"(v1p + (c >> 1) * 128));
        }
    };
    if (MODE != 2 && !a.lse_in) {
    fetch(j_lo, 0);
    for (int j0 = j_lo, stage = 0; j0 < ke; j0 += 16, stage ^= 1) {
        fetch(j0 + 16, stage ^ 1);
        cp_async_wait<1>();
        __syncwarp();
        float s[4];
        tile_times(st_s32 + stage * STAGE, qb, s);
        const bool v0 = j0 + gid < ke, v1 = j0 + gid + 8 < ke;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const float x0 = v0 ? s[e] * c2 : -INFINITY, x1 = v1 ? s[2 + e] * c2 : -INFINITY;
            const float m_new = fmaxf(m_run[e], fmaxf(x0, x1));
            if (m_new > -INFINITY) {
                l_run[e] = l_run[e] * ex2_approx(m_run[e] - m_new) + ex2_approx(x0 - m_new) + ex2_approx(x1 - m_new);
                m_run[e] = m_new;
            }
        }
        __syncwarp();                                     // this stage is refilled by the next iteration
    }
    cp_async_wait<0>();
#pragma unroll
    for (int e = 0; e < 2; ++e) {
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {               // merge the eight lanes that share the column
            const float m_o = __shfl_xor_sync(0xFFFFFFFFu, m_run[e], o);
            const float l_o = __shfl_xor_sync(0xFFFFFFFFu, l_run[e], o);
            const float m_new = fmaxf(m_run[e], m_o);
            if (m_new > -INFINITY)
                l_run[e] = l_run[e] * ex2_approx(m_run[e] - m_new) + l_o * ex2_approx(m_o - m_new);
            m_run[e] = m_new;
        }
    }
    }
    if (MODE == 1) {                                   // this range's statistics; the gradient launch combines them
#pragma unroll
        for (int e = 0; e < 2; ++e)
            if (gid == 0 && 2 * tig + e < G)
                a.part_ml[((size_t)range * a.total_rows + qrow) * a.n_h + g * G + 2 * tig + e] = make_float2(m_run[e], l_run[e]);
        return;
    }
    if (a.lse_in) {                                    // the forward pass saved the statistics: no first sweep
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            m_run[e] = a.lse_in[qrow * a.n_h + g * G + min(2 * tig + e, G - 1)] * kLog2e;
            l_run[e] = 1.f;
        }
    } else if (MODE == 2) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int h = g * G + min(2 * tig + e, G - 1);    // (columns >= G are padding: any finite value will do)
            for (int r = 0; r < a.n_ranges; ++r) {
                const float2 ml = a.part_ml[((size_t)r * a.total_rows + qrow) * a.n_h + h];
                const float m_new = fmaxf(m_run[e], ml.x);
                if (m_new > -INFINITY)
                    l_run[e] = l_run[e] * ex2_approx(m_run[e] - m_new) + ml.y * ex2_approx(ml.x - m_new);
                m_run[e] = m_new;
            }
        }
    }
    float lse2[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        lse2[e] = m_run[e] + log2f(l_run[e]);
        if (writes_row && gid == 0 && 2 * tig + e < G) a.lse2[qrow * a.n_h + g * G + 2 * tig + e] = lse2[e];
    }
    if (MODE == 2 && j_lo >= ke) return;               // (an item of range 0 that only had the row's values to write)

    // ---- sweep 2: gradients ---------------------------------------------------------------------------
    float dq[KS][4];
#pragma unroll
    for (int mt = 0; mt < KS; ++mt) dq[mt][0] = dq[mt][1] = dq[mt][2] = dq[mt][3] = 0.f;
    fetch(j_lo, 0);
    load_v(pos_fetched);
    for (int j0 = j_lo, stage = 0; j0 < ke; j0 += 16, stage ^= 1) {
        fetch(j0 + 16, stage ^ 1);
        cp_async_wait<1>();
        __syncwarp();
        const uint32_t k_s32 = st_s32 + stage * STAGE;
        float s[4], dp[4], p[4], ds[4];
        tile_times(k_s32, qb, s);
        {
            float dp2[4] = {0.f, 0.f, 0.f, 0.f};
            dp[0] = dp[1] = dp[2] = dp[3] = 0.f;
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                mma_bf16_16816(dp, vb[c].x, vb[NC + c].x, vb[c].y, vb[NC + c].y, dobd[c].x, dobd[c].y);
                mma_bf16_16816(dp2, vb[c].z, vb[NC + c].z, vb[c].w, vb[NC + c].w, dobd[c].z, dobd[c].w);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) dp[i] += dp2[i];
        }
        if (j0 + 16 < ke) load_v(pos_fetched);            // the next tile's V' rows, under the rest of this tile's work
        const bool v0 = j0 + gid < ke, v1 = j0 + gid + 8 < ke;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            p[e] = v0 ? ex2_approx(s[e] * c2 - lse2[e]) : 0.f;
            p[2 + e] = v1 ? ex2_approx(s[2 + e] * c2 - lse2[e]) : 0.f;
            ds[e] = p[e] * (dp[e] - delta[e]);
            ds[2 + e] = p[2 + e] * (dp[2 + e] - delta[e]);
        }
        if (a.pbar) {
            // the target of the indexer's loss (Eq. 14) falls out of this sweep: sum the group's heads per
            // key (rows gid, gid + 8), one fp32 atomic per key and KV head
            float r0 = 0.f, r1 = 0.f;
#pragma unroll
            for (int e = 0; e < 2; ++e)
                if (2 * tig + e < G) { r0 += p[e]; r1 += p[2 + e]; }
            r0 += __shfl_xor_sync(0xFFFFFFFFu, r0, 1); r0 += __shfl_xor_sync(0xFFFFFFFFu, r0, 2);
            r1 += __shfl_xor_sync(0xFFFFFFFFu, r1, 1); r1 += __shfl_xor_sync(0xFFFFFFFFu, r1, 2);
            if (tig == 0) {
                float* const prow = a.pbar + irow * a.k_max;
                const float inv_heads = 1.0f / (float)a.n_h;
                if (v0) atomicAdd(prow + j0 + gid, r0 * inv_heads);
                if (v1) atomicAdd(prow + j0 + gid + 8, r1 * inv_heads);
            }
        }
        const uint32_t ds_lo = pack_bf16(ds[0], ds[1]), ds_hi = pack_bf16(ds[2], ds[3]);
        // dQ^T[d, head] += K^T[d, key] dS^T[key, head]
        {
            const uint32_t b0 = movmatrix_t(ds_lo), b1 = movmatrix_t(ds_hi);
            const int mi = lane >> 3;
            const uint32_t addr = k_s32 + ((lane & 7) + (mi >> 1) * 8) * ROW + (mi & 1) * 16;
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                uint32_t a0, a1, a2, a3;
                ldmatrix_x4_trans(a0, a1, a2, a3, addr + mt * 32);
                mma_bf16_16816(dq[mt], a0, a1, a2, a3, b0, b1);
            }
        }
        __syncwarp();                                     // this stage is refilled by the next iteration
    }
    cp_async_wait<0>();

    // ---- dQ: rows of the fragment are d, columns the heads 2 tig, 2 tig + 1 ---------------------------
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int hl = 2 * tig + e;
        if (hl < G) {
            if (MODE == 2) {                           // this range's part: eight lanes fill one 32-byte sector
                float* const dst = a.dq32 + (qrow * a.n_h + (g * G + hl)) * DH;
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) {
                    atomicAdd(dst + mt * 16 + gid, dq[mt][e] * a.scale);
                    atomicAdd(dst + mt * 16 + gid + 8, dq[mt][2 + e] * a.scale);
                }
            } else {
                __nv_bfloat16* const dst = a.dQ + (qrow * a.n_h + (g * G + hl)) * DH;
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) {
                    dst[mt * 16 + gid] = __float2bfloat16(dq[mt][e] * a.scale);
                    dst[mt * 16 + gid + 8] = __float2bfloat16(dq[mt][2 + e] * a.scale);
                }
            }
        }
    }
}

// dQ rows of the range from the fp32 sums
__global__ void __launch_bounds__(256) gsa_bwd_dq_finish_kernel(const float* __restrict__ dq32,
                                                                __nv_bfloat16* __restrict__ dQ, RowRange rr,
                                                                int32_t Lq, int64_t row_elems) {
    const int lr = blockIdx.x;
    const int64_t qrow = (int64_t)(rr.b0 + lr / rr.R) * Lq + rr.q_begin + lr % rr.R;
    for (int64_t i = threadIdx.x * 4; i < row_elems; i += blockDim.x * 4) {
        const float4 v = *reinterpret_cast<const float4*>(dq32 + qrow * row_elems + i);
        __align__(8) __nv_bfloat16 o[4] = {__float2bfloat16(v.x), __float2bfloat16(v.y), __float2bfloat16(v.z),
                                           __float2bfloat16(v.w)};
        *reinterpret_cast<uint2*>(dQ + qrow * row_elems + i) = *reinterpret_cast<const uint2*>(o);
    }
}

template <int DH, int G, int MODE>
cudaError_t launch_bwd_mode(const BwdArgs& a, cudaStream_t st) {
    constexpr int ROW = (DH + 8) * 2;
    constexpr int WARP_SMEM = 2 * 16 * ROW;
    const int smem = kBwdWarps * WARP_SMEM;
    auto kern = gsa_sparse_attn_bwd_kernel<DH, G, MODE>;
    // (set on every call: the attribute belongs to the current device)
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    const int64_t items = (int64_t)a.rr.rows() * a.n_kv * (MODE == 0 ? 1 : a.n_ranges);
    const int64_t ctas = (items + kBwdWarps - 1) / kBwdWarps;
    kern<<<(unsigned)ctas, kBwdWarps * 32, smem, st>>>(a);
    ++g_launches;
    return cudaGetLastError();
}

template <int DH, int G>
cudaError_t launch_bwd_t(const BwdArgs& a, cudaStream_t st) {
    {
        const int64_t warps = (int64_t)a.rr.rows() * a.n_h;
        gsa_bwd_prep_kernel<DH><<<(unsigned)((warps + 7) / 8), 256, 0, st>>>(a.g1, a.out, a.dout, a.dOs, a.dg1, a.delta,
                                                                            a.rr, a.Lq, a.n_h);
        ++g_launches;
        cudaError_t e0 = cudaGetLastError();
        if (e0 != cudaSuccess) return e0;
    }
    if (a.n_ranges <= 1) return launch_bwd_mode<DH, G, 0>(a, st);
    gsa_bwd_range_cuts_kernel<<<(unsigned)((a.rr.rows() + 7) / 8), 256, 0, st>>>(a.idx, a.kt, const_cast<int32_t*>(a.cuts), a.rr,
                                                                                  a.il, a.Lq, a.k_max, a.n_ranges, a.range_keys);
    ++g_launches;
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaMemsetAsync(a.dq32, 0, (size_t)a.total_rows * a.n_h * DH * 4, st);
    if (e == cudaSuccess && !a.lse_in) e = launch_bwd_mode<DH, G, 1>(a, st);
    if (e == cudaSuccess) e = launch_bwd_mode<DH, G, 2>(a, st);
    if (e != cudaSuccess) return e;
    gsa_bwd_dq_finish_kernel<<<a.rr.rows(), 256, 0, st>>>(a.dq32, a.dQ, a.rr, a.Lq, (int64_t)a.n_h * DH);
    ++g_launches;
    return cudaGetLastError();
}

// key ranges of the query-major half: the forward pass's range size; one range when the keys fit one
struct BwdRanges { int range_keys, n_ranges; };
BwdRanges plan_bwd_ranges(const gsa_params_t& p) {
    BwdRanges r;
    r.range_keys = attn_range_keys();
    r.n_ranges = (p.Lk + r.range_keys - 1) / r.range_keys;
    if (r.n_ranges > 48) {
        r.range_keys = ((p.Lk + 47) / 48 + 1023) / 1024 * 1024;
        r.n_ranges = (p.Lk + r.range_keys - 1) / r.range_keys;
    }
    return r;
}

}  // namespace

size_t attn_bwd_range_bytes(const gsa_params_t& p) {
    const BwdRanges br = plan_bwd_ranges(p);
    if (br.n_ranges <= 1) return 0;
    const size_t rows = (size_t)p.B * p.Lq;
    return ((size_t)br.n_ranges * rows * p.n_h * 8 + 255) / 256 * 256 + (rows * p.n_h * p.d_h * 4 + 255) / 256 * 256 +
           (rows * (br.n_ranges + 1) * 4 + 255) / 256 * 256;
}

bool attn_bwd_supported(const gsa_params_t& p) {
    const int G = p.n_h / p.n_kv;
    return (p.d_h == 128 || p.d_h == 64) && (G == 1 || G == 2 || G == 4 || G == 8);
}

cudaError_t launch_sparse_attn_bwd(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* Q,
                                   const __nv_bfloat16* K, const __nv_bfloat16* Vg, const __nv_bfloat16* g1,
                                   const __nv_bfloat16* out, const __nv_bfloat16* dout, const int32_t* idx,
                                   const int32_t* kt, IdxLayout il, __nv_bfloat16* dQ, __nv_bfloat16* dg1,
                                   __nv_bfloat16* dOs, float* lse2, float* delta, float* pbar, const float* lse_in,
                                   void* range_ws, cudaStream_t st) {
    if (rr.rows() <= 0) return cudaSuccess;
    BwdArgs a;
    const BwdRanges br = plan_bwd_ranges(p);
    a.range_keys = br.range_keys; a.n_ranges = br.n_ranges; a.total_rows = (int64_t)p.B * p.Lq;
    a.lse_in = lse_in;
    a.part_ml = (float2*)range_ws;
    a.dq32 = (float*)((char*)range_ws + ((size_t)br.n_ranges * a.total_rows * p.n_h * 8 + 255) / 256 * 256);
    a.cuts = (const int32_t*)((char*)a.dq32 + ((size_t)a.total_rows * p.n_h * p.d_h * 4 + 255) / 256 * 256);
    a.Q = Q; a.K = K; a.Vg = Vg; a.g1 = g1; a.out = out; a.dout = dout; a.idx = idx; a.kt = kt; a.dev_status = t_dev_status;
    a.dQ = dQ; a.dg1 = dg1; a.dOs = dOs; a.lse2 = lse2; a.delta = delta; a.pbar = pbar; a.rr = rr; a.il = il;
    a.Lq = p.Lq; a.Lk = p.Lk; a.n_h = p.n_h; a.n_kv = p.n_kv; a.k_max = p.k_max;
    a.scale = p.sm_scale > 0.f ? p.sm_scale : 1.0f / sqrtf((float)p.d_h);
    const int G = p.n_h / p.n_kv;
#define GSA_BWD_CASE(DH_, G_) if (p.d_h == DH_ && G == G_) return launch_bwd_t<DH_, G_>(a, st)
    GSA_BWD_CASE(128, 1); GSA_BWD_CASE(128, 2); GSA_BWD_CASE(128, 4); GSA_BWD_CASE(128, 8);
    GSA_BWD_CASE(64, 1); GSA_BWD_CASE(64, 2); GSA_BWD_CASE(64, 4); GSA_BWD_CASE(64, 8);
#undef GSA_BWD_CASE
    return cudaErrorInvalidValue;
}

}  // namespace gsa
