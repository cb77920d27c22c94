// The indexer's sparse-phase loss (Sec. 5.1, Eq. 14) and its backward:
//     loss_t = KL( pbar[t, S_t]  ||  softmax_j I[t, s_j] ),    I from Eq. 7 (or Eq. 3 with act = 1).
//
// Two kernels, both one warp per work item with the selected keys as the M of bf16 mma.sync tiles that
// 16-byte asynchronous copies gather into a private, double-buffered shared-memory stage:
//
//  * gsa_attn_probs_mean_kernel, one warp per (query row, KV head): the target pbar.  Eq. 11 gives one
//    attention distribution per head; the indexer score has no head index, so the target is their mean over
//    the heads.  A first sweep over S_t takes the softmax statistics of S^T = K Q^T, a second one adds
//    2^(c S^T - lse) / n_h, summed over the group's heads, into pbar (one fp32 atomic per key and KV head).
//
//  * gsa_indexer_kl_kernel, one warp per query row.  X^T[key, head] = k^I . q^I^T + b on the tensor cores,
//    f = sigmoid (or ReLU), I_j = sum_i w_i f_ij.  Sweep 1: log-sum-exp of I over S_t and the three sums the
//    loss needs.  Sweep 2: dI_j = softmax(I)_j * sum(pbar) - pbar_j,  dX_ij = dI_j w_i f'_ij, then
//        dw_i = sum_j dI_j f_ij          db_i += sum_j dX_ij          dq^I^T[c, i] += k^I^T[c, key] dX[key, i]
//        dk^I[key, c] += dX[key, i] q^I[i, c]   (m16n8k8: the indexer heads are K)
//    dk^I is a sum over every query that selected the key: d^I fp32 additions per selected pair, done with
//    red.global.add.v2.f32 into an fp32 array that a streaming pass rounds to bf16 (32 times fewer than the
//    attention's dK would need, which is why that one inverts the index sets instead).
#include "gsa_common.cuh"

namespace gsa {

namespace {

constexpr int kLossWarps = 4;
constexpr float kLog2eL = 1.4426950408889634f;

__device__ __forceinline__ uint32_t movmatrix_tl(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ float ex2_approx_l(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// D(16x8, fp32) = A(16x8, bf16, row) * B(8x8, bf16, col)
__device__ __forceinline__ void mma_bf16_1688_l(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%7,%8,%9,%10};\n"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a0), "r"(a1), "r"(b0), "f"(0.f), "f"(0.f), "f"(0.f), "f"(0.f));
}
__device__ __forceinline__ void red_add_v2_l(float* addr, float x, float y) {
    asm volatile("red.global.add.v2.f32 [%0], {%1, %2};" ::"l"(addr), "f"(x), "f"(y) : "memory");
}

// ---- the target: mean over the heads of the attention distribution on S_t -----------------------------
struct ProbsArgs {
    const __nv_bfloat16* Q;
    const __nv_bfloat16* K;
    const int32_t* idx;
    const int32_t* kt;
    float* pbar;                  // [B, R, k_max], zeroed by the caller of the kernel
    RowRange rr;
    IdxLayout il;
    int32_t Lq, Lk, n_h, n_kv, k_max;
    float scale;
    int32_t* dev_status;          // where an out-of-range index or budget is reported (may be null)
};

template <int DH, int G>
__global__ void __launch_bounds__(kLossWarps * 32) gsa_attn_probs_mean_kernel(const ProbsArgs a) {
    constexpr int ROW = (DH + 8) * 2;
    constexpr int KTILE = 16 * ROW, QTILE = 8 * ROW;
    constexpr int WARP_SMEM = 2 * KTILE;               // two stages; the Q tile borrows stage 1 first
    static_assert(QTILE <= KTILE, "the Q tile must fit one stage");
    constexpr int KS = DH / 16;
    constexpr int EPL = DH / 32;
    constexpr int CPR = DH / 8;
    extern __shared__ __align__(16) unsigned char loss_smem[];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gid = lane >> 2, tig = lane & 3;
    const int64_t item = (int64_t)blockIdx.x * kLossWarps + warp;
    if (item >= (int64_t)a.rr.rows() * a.n_kv) return;   // (no block-wide barrier below)
    const int lr = a.rr.rows() - 1 - (int)(item / a.n_kv);    // long rows first
    const int g = (int)(item % a.n_kv);
    const int b = a.rr.b0 + lr / a.rr.R, t = a.rr.q_begin + lr % a.rr.R;
    const int64_t qrow = (int64_t)b * a.Lq + t;
    const int64_t irow = a.il.row(b, t);
    const int ke = checked_budget(a.kt[irow], a.k_max, a.dev_status);
    const int32_t* __restrict__ S = a.idx + irow * a.k_max;
    float* __restrict__ prow = a.pbar + irow * a.k_max;

    unsigned char* const ws = loss_smem + warp * WARP_SMEM;
    const uint32_t st_s32 = (uint32_t)__cvta_generic_to_shared(ws);
    const uint32_t q_s32 = st_s32 + KTILE;
#pragma unroll
    for (int hl = 0; hl < 8; ++hl) {
        __nv_bfloat16* qd = reinterpret_cast<__nv_bfloat16*>(ws + KTILE + hl * ROW) + lane * EPL;
#pragma unroll
        for (int e = 0; e < EPL; ++e)
            qd[e] = hl < G ? a.Q[(qrow * a.n_h + (g * G + hl)) * DH + lane * EPL + e] : __float2bfloat16(0.f);
    }
    __syncwarp();
    uint32_t qb[2 * KS];
#pragma unroll
    for (int k2 = 0; k2 < KS / 2; ++k2)
        ldmatrix_x4(qb[4 * k2], qb[4 * k2 + 1], qb[4 * k2 + 2], qb[4 * k2 + 3],
                    q_s32 + (lane & 7) * ROW + (lane >> 3) * 16 + k2 * 64);
    __syncwarp();                                      // stage 1 is free for tiles from here on

    const float c2 = a.scale * kLog2eL;
    const size_t kv_row = (size_t)a.n_kv * DH;
    const __nv_bfloat16* const kbase = a.K + ((size_t)b * a.Lk * a.n_kv + g) * DH;
    auto fetch = [&](int j, int stage) {
        if (j < ke) {
            const int32_t pos16 = checked_pos(S[min(j + (lane & 15), ke - 1)], a.Lk, a.dev_status);
#pragma unroll
            for (int i = 0; i < 16 * CPR / 32; ++i) {
                const int chunk = i * 32 + lane;
                const int r = chunk / CPR, c = chunk % CPR;
                const int32_t p = __shfl_sync(0xFFFFFFFFu, pos16, r);
                cp_async16(st_s32 + stage * KTILE + r * ROW + c * 16, kbase + (size_t)p * kv_row + c * 8);
            }
        }
        cp_async_commit();
    };
    auto scores = [&](int stage, float (&acc)[4]) {
        acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
        const uint32_t addr = st_s32 + stage * KTILE + (lane & 15) * ROW + (lane >> 4) * 16;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4(a0, a1, a2, a3, addr + ks * 32);
            mma_bf16_16816(acc, a0, a1, a2, a3, qb[2 * ks], qb[2 * ks + 1]);
        }
    };

    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    fetch(0, 0);
    for (int j0 = 0, stage = 0; j0 < ke; j0 += 16, stage ^= 1) {
        fetch(j0 + 16, stage ^ 1);
        cp_async_wait<1>();
        __syncwarp();
        float s[4];
        scores(stage, s);
        const bool v0 = j0 + gid < ke, v1 = j0 + gid + 8 < ke;
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const float x0 = v0 ? s[e] * c2 : -INFINITY, x1 = v1 ? s[2 + e] * c2 : -INFINITY;
            const float m_new = fmaxf(m_run[e], fmaxf(x0, x1));
            if (m_new > -INFINITY) {
                l_run[e] = l_run[e] * ex2_approx_l(m_run[e] - m_new) + ex2_approx_l(x0 - m_new) + ex2_approx_l(x1 - m_new);
                m_run[e] = m_new;
            }
        }
        __syncwarp();
    }
    cp_async_wait<0>();
    float lse2[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
            const float m_o = __shfl_xor_sync(0xFFFFFFFFu, m_run[e], o);
            const float l_o = __shfl_xor_sync(0xFFFFFFFFu, l_run[e], o);
            const float m_new = fmaxf(m_run[e], m_o);
            if (m_new > -INFINITY)
                l_run[e] = l_run[e] * ex2_approx_l(m_run[e] - m_new) + l_o * ex2_approx_l(m_o - m_new);
            m_run[e] = m_new;
        }
        lse2[e] = m_run[e] + log2f(l_run[e]);
    }
    __syncwarp();

    const float inv_heads = 1.0f / (float)a.n_h;
    fetch(0, 0);
    for (int j0 = 0, stage = 0; j0 < ke; j0 += 16, stage ^= 1) {
        fetch(j0 + 16, stage ^ 1);
        cp_async_wait<1>();
        __syncwarp();
        float s[4];
        scores(stage, s);
        // the group's heads are columns 0 .. G-1: sum them per key (rows gid, gid + 8)
        float r0 = 0.f, r1 = 0.f;
#pragma unroll
        for (int e = 0; e < 2; ++e)
            if (2 * tig + e < G) {
                r0 += ex2_approx_l(s[e] * c2 - lse2[e]);
                r1 += ex2_approx_l(s[2 + e] * c2 - lse2[e]);
            }
        r0 += __shfl_xor_sync(0xFFFFFFFFu, r0, 1); r0 += __shfl_xor_sync(0xFFFFFFFFu, r0, 2);
        r1 += __shfl_xor_sync(0xFFFFFFFFu, r1, 1); r1 += __shfl_xor_sync(0xFFFFFFFFu, r1, 2);
        if (tig == 0) {
            if (j0 + gid < ke) atomicAdd(prow + j0 + gid, r0 * inv_heads);
            if (j0 + gid + 8 < ke) atomicAdd(prow + j0 + gid + 8, r1 * inv_heads);
        }
        __syncwarp();
    }
    cp_async_wait<0>();
}

// ---- the loss and its backward ------------------------------------------------------------------------
struct KlArgs {
    const __nv_bfloat16* qI;
    const __nv_bfloat16* kI;
    const float* w;
    const float* bI;              // may be null
    const int32_t* idx;
    const int32_t* kt;
    const float* pbar;
    float* loss;                  // [B, R]
    __nv_bfloat16* dqI;           // [B, Lq, HI, dI]
    float* dw;                    // [B, Lq, HI]
    float* dkI32;                 // [B, Lk, dI] fp32, zeroed by the caller of the kernel
    float* dbI;                   // [HI] fp32, zeroed by the caller of the kernel; may be null
    RowRange rr;
    IdxLayout il;
    int32_t Lq, Lk, k_max, act;
    int32_t* dev_status;          // where an out-of-range index or budget is reported (may be null)
};

template <int DI, int HI>
__global__ void __launch_bounds__(kLossWarps * 32) gsa_indexer_kl_kernel(const KlArgs a) {
    constexpr int ROW = (DI + 8) * 2;                  // bytes of a padded tile row (odd multiple of 16)
    constexpr int KTILE = 16 * ROW, QTILE = 8 * ROW;
    constexpr int WARP_SMEM = 2 * KTILE + QTILE;       // two k^I stages and the row's q^I tile
    constexpr int KS = DI / 16;
    constexpr int CPR = DI / 8;
    extern __shared__ __align__(16) unsigned char loss_smem[];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gid = lane >> 2, tig = lane & 3;
    const int64_t item = (int64_t)blockIdx.x * kLossWarps + warp;
    if (item >= a.rr.rows()) return;                   // (no block-wide barrier below)
    const int lr = a.rr.rows() - 1 - (int)item;        // long rows first
    const int b = a.rr.b0 + lr / a.rr.R, t = a.rr.q_begin + lr % a.rr.R;
    const int64_t qrow = (int64_t)b * a.Lq + t;
    const int64_t irow = a.il.row(b, t);
    const int ke = checked_budget(a.kt[irow], a.k_max, a.dev_status);
    const int32_t* __restrict__ S = a.idx + irow * a.k_max;
    const float* __restrict__ prow = a.pbar + irow * a.k_max;

    unsigned char* const ws = loss_smem + warp * WARP_SMEM;
    const uint32_t st_s32 = (uint32_t)__cvta_generic_to_shared(ws);
    const uint32_t q_s32 = st_s32 + 2 * KTILE;
    // q^I of the row as a tile: rows = indexer heads (rows >= HI are zero)
    for (int i = lane; i < 8 * DI; i += 32) {
        const int h = i / DI, c = i % DI;
        reinterpret_cast<__nv_bfloat16*>(ws + 2 * KTILE + h * ROW)[c] =
            h < HI ? a.qI[(qrow * HI + h) * DI + c] : __float2bfloat16(0.f);
    }
    __syncwarp();
    uint32_t qb[2 * KS];                               // B operand of X^T = k^I q^I^T: (k = c, n = head)
#pragma unroll
    for (int k2 = 0; k2 < KS / 2; ++k2)
        ldmatrix_x4(qb[4 * k2], qb[4 * k2 + 1], qb[4 * k2 + 2], qb[4 * k2 + 3],
                    q_s32 + (lane & 7) * ROW + (lane >> 3) * 16 + k2 * 64);
    // this lane's two heads (columns 2 tig, 2 tig + 1)
    float wv[2], bv[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int h = 2 * tig + e;
        wv[e] = h < HI ? a.w[qrow * HI + h] : 0.f;
        bv[e] = (a.bI && h < HI) ? a.bI[h] : 0.f;
    }

    const __nv_bfloat16* const kbase = a.kI + (size_t)b * a.Lk * DI;
    auto fetch = [&](int j, int stage) {
        if (j < ke) {
            const int32_t pos16 = checked_pos(S[min(j + (lane & 15), ke - 1)], a.Lk, a.dev_status);
#pragma unroll
            for (int i = 0; i < 16 * CPR / 32; ++i) {
                const int chunk = i * 32 + lane;
                const int r = chunk / CPR, c = chunk % CPR;
                const int32_t p = __shfl_sync(0xFFFFFFFFu, pos16, r);
                cp_async16(st_s32 + stage * KTILE + r * ROW + c * 16, kbase + (size_t)p * DI + c * 8);
            }
        }
        cp_async_commit();
    };
    // f(x) and f'(x) of the tile's (key, head) entries, and the keys' scores I (rows gid, gid + 8)
    auto tile_scores = [&](int stage, float (&f)[4], float (&fp)[4], float& I0, float& I1) {
        float x[4] = {0.f, 0.f, 0.f, 0.f};
        const uint32_t addr = st_s32 + stage * KTILE + (lane & 15) * ROW + (lane >> 4) * 16;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4(a0, a1, a2, a3, addr + ks * 32);
            mma_bf16_16816(x, a0, a1, a2, a3, qb[2 * ks], qb[2 * ks + 1]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float v = x[i] + bv[i & 1];
            if (a.act == 1) {
                f[i] = fmaxf(v, 0.f);
                fp[i] = v > 0.f ? 1.f : 0.f;
            } else {
                f[i] = 1.0f / (1.0f + __expf(-v));
                fp[i] = f[i] * (1.0f - f[i]);
            }
        }
        I0 = wv[0] * f[0] + wv[1] * f[1];
        I1 = wv[0] * f[2] + wv[1] * f[3];
        I0 += __shfl_xor_sync(0xFFFFFFFFu, I0, 1); I0 += __shfl_xor_sync(0xFFFFFFFFu, I0, 2);
        I1 += __shfl_xor_sync(0xFFFFFFFFu, I1, 1); I1 += __shfl_xor_sync(0xFFFFFFFFu, I1, 2);
    };

    // ---- sweep 1: log-sum-exp of the scores, sum pbar, sum pbar I, sum pbar log pbar ------------------
    float m_run = -INFINITY, l_run = 0.f, s_p = 0.f, s_pi = 0.f, s_plp = 0.f;
    fetch(0, 0);
    for (int j0 = 0, stage = 0; j0 < ke; j0 += 16, stage ^= 1) {
        fetch(j0 + 16, stage ^ 1);
        const bool v0 = j0 + gid < ke, v1 = j0 + gid + 8 < ke;
        const float p0 = v0 ? prow[j0 + gid] : 0.f, p1 = v1 ? prow[j0 + gid + 8] : 0.f;
        cp_async_wait<1>();
        __syncwarp();
        float f[4], fp[4], I0, I1;
        tile_scores(stage, f, fp, I0, I1);
        const float x0 = v0 ? I0 * kLog2eL : -INFINITY, x1 = v1 ? I1 * kLog2eL : -INFINITY;
        const float m_new = fmaxf(m_run, fmaxf(x0, x1));
        if (m_new > -INFINITY) {
            l_run = l_run * ex2_approx_l(m_run - m_new) + ex2_approx_l(x0 - m_new) + ex2_approx_l(x1 - m_new);
            m_run = m_new;
        }
        s_p += p0 + p1;
        s_pi += p0 * I0 + p1 * I1;
        s_plp += (p0 > 0.f ? p0 * __logf(p0) : 0.f) + (p1 > 0.f ? p1 * __logf(p1) : 0.f);
        __syncwarp();
    }
    cp_async_wait<0>();
    // the four lanes of a key hold the same values: merge across the keys only (lane bits 2..4)
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
        const float m_o = __shfl_xor_sync(0xFFFFFFFFu, m_run, o);
        const float l_o = __shfl_xor_sync(0xFFFFFFFFu, l_run, o);
        const float m_new = fmaxf(m_run, m_o);
        if (m_new > -INFINITY) l_run = l_run * ex2_approx_l(m_run - m_new) + l_o * ex2_approx_l(m_o - m_new);
        m_run = m_new;
        s_p += __shfl_xor_sync(0xFFFFFFFFu, s_p, o);
        s_pi += __shfl_xor_sync(0xFFFFFFFFu, s_pi, o);
        s_plp += __shfl_xor_sync(0xFFFFFFFFu, s_plp, o);
    }
    const float lse2 = m_run + log2f(l_run);           // log2 of sum_j exp(I_j)
    if (lane == 0) a.loss[irow] = ke > 0 ? s_plp - s_pi + (lse2 / kLog2eL) * s_p : 0.f;
    __syncwarp();

    // ---- sweep 2: derivatives ----------------------------------------------------------------------------
    float dq[KS][4];                                   // dq^I^T: rows = c, columns = heads 2 tig, 2 tig + 1
#pragma unroll
    for (int mt = 0; mt < KS; ++mt) dq[mt][0] = dq[mt][1] = dq[mt][2] = dq[mt][3] = 0.f;
    float dw_acc[2] = {0.f, 0.f}, db_acc[2] = {0.f, 0.f};
    fetch(0, 0);
    for (int j0 = 0, stage = 0; j0 < ke; j0 += 16, stage ^= 1) {
        const int32_t pos16 = checked_pos(S[min(j0 + (lane & 15), ke - 1)], a.Lk, a.dev_status);
        fetch(j0 + 16, stage ^ 1);
        const bool v0 = j0 + gid < ke, v1 = j0 + gid + 8 < ke;
        const float p0 = v0 ? prow[j0 + gid] : 0.f, p1 = v1 ? prow[j0 + gid + 8] : 0.f;
        cp_async_wait<1>();
        __syncwarp();
        float f[4], fp[4], I0, I1;
        tile_scores(stage, f, fp, I0, I1);
        const float dI0 = v0 ? ex2_approx_l(I0 * kLog2eL - lse2) * s_p - p0 : 0.f;
        const float dI1 = v1 ? ex2_approx_l(I1 * kLog2eL - lse2) * s_p - p1 : 0.f;
        float dx[4];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            dw_acc[e] += dI0 * f[e] + dI1 * f[2 + e];
            dx[e] = dI0 * wv[e] * fp[e];
            dx[2 + e] = dI1 * wv[e] * fp[2 + e];
            db_acc[e] += dx[e] + dx[2 + e];
        }
        const uint32_t dx_lo = pack_bf16(dx[0], dx[1]), dx_hi = pack_bf16(dx[2], dx[3]);
        // dq^I^T[c, head] += k^I^T[c, key] dX[key, head]
        {
            const uint32_t b0 = movmatrix_tl(dx_lo), b1 = movmatrix_tl(dx_hi);
            const int mi = lane >> 3;
            const uint32_t addr = st_s32 + stage * KTILE + ((lane & 7) + (mi >> 1) * 8) * ROW + (mi & 1) * 16;
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                uint32_t a0, a1, a2, a3;
                ldmatrix_x4_trans(a0, a1, a2, a3, addr + mt * 32);
                mma_bf16_16816(dq[mt], a0, a1, a2, a3, b0, b1);
            }
        }
        // dk^I[key, c] += dX[key, head] q^I[head, c]
        {
            const int32_t key0 = __shfl_sync(0xFFFFFFFFu, pos16, gid), key1 = __shfl_sync(0xFFFFFFFFu, pos16, gid + 8);
            float* const dk0 = a.dkI32 + ((size_t)b * a.Lk + key0) * DI + 2 * tig;
            float* const dk1 = a.dkI32 + ((size_t)b * a.Lk + key1) * DI + 2 * tig;
            const uint32_t boff = q_s32 + (lane & 7) * ROW + (lane >> 3) * 16;
#pragma unroll
            for (int n4 = 0; n4 < DI / 32; ++n4) {
                uint32_t bq[4];
                ldmatrix_x4_trans(bq[0], bq[1], bq[2], bq[3], boff + n4 * 64);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float ck[4];
                    mma_bf16_1688_l(ck, dx_lo, dx_hi, bq[i]);
                    const int col = (n4 * 4 + i) * 8;
                    if (v0) red_add_v2_l(dk0 + col, ck[0], ck[1]);
                    if (v1) red_add_v2_l(dk1 + col, ck[2], ck[3]);
                }
            }
        }
        __syncwarp();
    }
    cp_async_wait<0>();

    // ---- per-row results ------------------------------------------------------------------------------------
#pragma unroll
    for (int e = 0; e < 2; ++e) {
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
            dw_acc[e] += __shfl_xor_sync(0xFFFFFFFFu, dw_acc[e], o);
            db_acc[e] += __shfl_xor_sync(0xFFFFFFFFu, db_acc[e], o);
        }
        const int h = 2 * tig + e;
        if (h < HI) {
            if (gid == 0) {
                a.dw[qrow * HI + h] = dw_acc[e];
                if (a.dbI) atomicAdd(a.dbI + h, db_acc[e]);
            }
            __nv_bfloat16* const dst = a.dqI + (qrow * HI + h) * DI;
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                dst[mt * 16 + gid] = __float2bfloat16(dq[mt][e]);
                dst[mt * 16 + gid + 8] = __float2bfloat16(dq[mt][2 + e]);
            }
        }
    }
}

__global__ void __launch_bounds__(256) gsa_f32_to_bf16_kernel(const float* __restrict__ src,
                                                              __nv_bfloat16* __restrict__ dst, int64_t n) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x * 4;
    for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4; i < n; i += stride) {
        const float4 v = *reinterpret_cast<const float4*>(src + i);
        __align__(8) __nv_bfloat16 o[4] = {__float2bfloat16(v.x), __float2bfloat16(v.y), __float2bfloat16(v.z),
                                           __float2bfloat16(v.w)};
        *reinterpret_cast<uint2*>(dst + i) = *reinterpret_cast<const uint2*>(o);
    }
}

template <int DH, int G>
cudaError_t launch_probs_t(const ProbsArgs& a, cudaStream_t st) {
    constexpr int smem = kLossWarps * 2 * 16 * (DH + 8) * 2;
    auto kern = gsa_attn_probs_mean_kernel<DH, G>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    const int64_t items = (int64_t)a.rr.rows() * a.n_kv;
    kern<<<(unsigned)((items + kLossWarps - 1) / kLossWarps), kLossWarps * 32, smem, st>>>(a);
    ++g_launches;
    return cudaGetLastError();
}

template <int DI, int HI>
cudaError_t launch_kl_t(const KlArgs& a, cudaStream_t st) {
    constexpr int smem = kLossWarps * (2 * 16 + 8) * (DI + 8) * 2;
    auto kern = gsa_indexer_kl_kernel<DI, HI>;
    const int64_t items = a.rr.rows();
    kern<<<(unsigned)((items + kLossWarps - 1) / kLossWarps), kLossWarps * 32, smem, st>>>(a);
    ++g_launches;
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attn_probs_mean(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* Q,
                                   const __nv_bfloat16* K, const int32_t* idx, const int32_t* kt, IdxLayout il,
                                   float* pbar, cudaStream_t st) {
    if (rr.rows() <= 0) return cudaSuccess;
    cudaError_t e = cudaMemsetAsync(pbar, 0, (size_t)rr.rows() * p.k_max * 4, st);
    if (e != cudaSuccess) return e;
    ProbsArgs a;
    a.Q = Q; a.K = K; a.idx = idx; a.kt = kt; a.dev_status = t_dev_status; a.pbar = pbar; a.rr = rr; a.il = il;
    a.Lq = p.Lq; a.Lk = p.Lk; a.n_h = p.n_h; a.n_kv = p.n_kv; a.k_max = p.k_max;
    a.scale = p.sm_scale > 0.f ? p.sm_scale : 1.0f / sqrtf((float)p.d_h);
    const int G = p.n_h / p.n_kv;
#define GSA_PROBS_CASE(DH_, G_) if (p.d_h == DH_ && G == G_) return launch_probs_t<DH_, G_>(a, st)
    GSA_PROBS_CASE(128, 1); GSA_PROBS_CASE(128, 2); GSA_PROBS_CASE(128, 4); GSA_PROBS_CASE(128, 8);
    GSA_PROBS_CASE(64, 1); GSA_PROBS_CASE(64, 2); GSA_PROBS_CASE(64, 4); GSA_PROBS_CASE(64, 8);
#undef GSA_PROBS_CASE
    return cudaErrorInvalidValue;
}

cudaError_t launch_indexer_kl(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* qI,
                              const __nv_bfloat16* kI, const float* w, const float* bI, const int32_t* idx,
                              const int32_t* kt, IdxLayout il, const float* pbar, float* loss,
                              __nv_bfloat16* dqI, __nv_bfloat16* dkI, float* dw, float* dbI, float* dkI32,
                              cudaStream_t st) {
    const int64_t n_k = (int64_t)p.B * p.Lk * p.dI;
    cudaError_t e = cudaMemsetAsync(dkI32, 0, (size_t)n_k * 4, st);
    if (e == cudaSuccess && dbI) e = cudaMemsetAsync(dbI, 0, (size_t)p.HI * 4, st);
    if (e != cudaSuccess) return e;
    if (rr.rows() > 0) {
        KlArgs a;
        a.qI = qI; a.kI = kI; a.w = w; a.bI = bI; a.idx = idx; a.kt = kt; a.dev_status = t_dev_status; a.pbar = pbar; a.loss = loss;
        a.dqI = dqI; a.dw = dw; a.dkI32 = dkI32; a.dbI = dbI; a.rr = rr; a.il = il;
        a.Lq = p.Lq; a.Lk = p.Lk; a.k_max = p.k_max; a.act = p.act;
        e = cudaErrorInvalidValue;
#define GSA_KL_CASE(DI_, HI_) if (p.dI == DI_ && p.HI == HI_) e = launch_kl_t<DI_, HI_>(a, st)
        GSA_KL_CASE(64, 8); GSA_KL_CASE(64, 4); GSA_KL_CASE(64, 2); GSA_KL_CASE(64, 1);
        GSA_KL_CASE(32, 8); GSA_KL_CASE(32, 4); GSA_KL_CASE(32, 2); GSA_KL_CASE(32, 1);
#undef GSA_KL_CASE
        if (e != cudaSuccess) return e;
    }
    const int64_t want = (n_k / 4 + 255) / 256;
    gsa_f32_to_bf16_kernel<<<(int)(want < sm_count() * 16 ? (want > 0 ? want : 1) : sm_count() * 16), 256, 0, st>>>(dkI32, dkI, n_k);
    ++g_launches;
    return cudaGetLastError();
}

}  // namespace gsa
