// Gated lightning indexer (Eq. 7) for calls with very few query rows per sequence (decode: one new
// token against a long cache).  A tile of 32 queries x H^I heads would be almost empty there, so
// the work is laid out the other way round: a warp streams the shared indexer keys k^I of one
// sequence 16 at a time straight from HBM into the A fragments of a bf16 MMA (keys are M, the
// contraction index d^I is used in the order the 32-byte loads deliver it) and multiplies them with
// the H^I <= 8 indexer queries of one token (N = heads):
//     S^T[key, head] = k^I[key, :] . q^I[head, :]
//     I[t, key]      = sum_head w[head] * sigmoid(S^T[key, head] + b[head])     (sum across the 4 lanes
//                                                                               that hold a key's heads)
// The kernel is bound by reading k^I once per query row: d^I * 2 bytes per (row, key).
#include "gsa_common.cuh"

namespace gsa {

namespace {

constexpr int kRowsWarps = 8;              // warps per CTA
constexpr int kTilesPerStep = 4;           // 16-key tiles a warp has in flight

struct RowsIdxArgs {
    const __nv_bfloat16* qI;
    const __nv_bfloat16* kI;
    const float* w;
    const float* bI;
    float* scores;
    int64_t row_stride;
    RowRange rr;
    int32_t Lq, Lk;
    int32_t keys_per_cta;
    int32_t act;
};

__device__ __forceinline__ void ldg32(const void* p, uint4& lo, uint4& hi) {
    asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(lo.x), "=r"(lo.y), "=r"(lo.z), "=r"(lo.w), "=r"(hi.x), "=r"(hi.y), "=r"(hi.z), "=r"(hi.w)
                 : "l"(p));
}

template <int DI, int HI>
__global__ void __launch_bounds__(kRowsWarps * 32) gsa_indexer_rows_kernel(const RowsIdxArgs a) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gid = lane >> 2, tig = lane & 3;
    const int lr = blockIdx.y;
    const int b = a.rr.b0 + lr / a.rr.R;
    const int t = a.rr.q_begin + lr % a.rr.R;
    const int n = a.Lk - a.Lq + t + 1;                 // visible keys
    const int key_lo = blockIdx.x * a.keys_per_cta;
    const int key_hi = min(n, key_lo + a.keys_per_cta);
    if (key_lo >= key_hi) return;

    // Lane tig owns the tig-th quarter of every key row (DI/4 consecutive elements); the B operand
    // q^I[head = gid] is read with the same split, so both sides agree on which d a k-index means.
    constexpr int LANE_ELEMS = DI / 4;                 // bf16 per lane and key: 16 (DI 64) or 8 (DI 32)
    uint32_t qb[LANE_ELEMS / 2];
    {
        const __nv_bfloat16* qp = a.qI + (((size_t)b * a.Lq + t) * HI + (gid < HI ? gid : 0)) * DI + tig * LANE_ELEMS;
#pragma unroll
        for (int i = 0; i < LANE_ELEMS / 2; ++i)
            qb[i] = gid < HI ? *reinterpret_cast<const uint32_t*>(qp + 2 * i) : 0u;
    }
    // heads 2*tig, 2*tig+1 are this lane's columns of S^T
    float wv[2], bv[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int h = 2 * tig + e;
        wv[e] = h < HI ? a.w[((size_t)b * a.Lq + t) * HI + h] : 0.f;
        bv[e] = (a.bI && h < HI) ? a.bI[h] * (a.act == 1 ? 1.0f : -1.4426950408889634f) : 0.f;
    }
    const unsigned char* kbase = reinterpret_cast<const unsigned char*>(a.kI) + (size_t)b * a.Lk * DI * 2 +
                                 tig * (LANE_ELEMS * 2);
    float* __restrict__ out_row = a.scores + (int64_t)lr * a.row_stride;

    for (int k0 = key_lo + warp * 16 * kTilesPerStep; k0 < key_hi; k0 += kRowsWarps * 16 * kTilesPerStep) {
        uint32_t ka[kTilesPerStep][2][LANE_ELEMS / 2];          // [tile][key gid / gid+8][packed pairs]
#pragma unroll
        for (int u = 0; u < kTilesPerStep; ++u)
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                // rows past the end of the cache are clamped to the last one; their scores are not stored
                const int key = min(k0 + u * 16 + hf * 8 + gid, a.Lk - 1);
                const unsigned char* kp = kbase + (size_t)key * (DI * 2);
                if constexpr (LANE_ELEMS == 16) {
                    uint4 lo, hi;
                    ldg32(kp, lo, hi);
                    ka[u][hf][0] = lo.x; ka[u][hf][1] = lo.y; ka[u][hf][2] = lo.z; ka[u][hf][3] = lo.w;
                    ka[u][hf][4] = hi.x; ka[u][hf][5] = hi.y; ka[u][hf][6] = hi.z; ka[u][hf][7] = hi.w;
                } else {
                    const uint4 v = __ldg(reinterpret_cast<const uint4*>(kp));
                    ka[u][hf][0] = v.x; ka[u][hf][1] = v.y; ka[u][hf][2] = v.z; ka[u][hf][3] = v.w;
                }
            }
#pragma unroll
        for (int u = 0; u < kTilesPerStep; ++u) {
            float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < LANE_ELEMS / 4; ++ks)          // one k-step uses 4 of the lane's elements
                mma_bf16_16816(s, ka[u][0][2 * ks], ka[u][1][2 * ks], ka[u][0][2 * ks + 1], ka[u][1][2 * ks + 1],
                               qb[2 * ks], qb[2 * ks + 1]);
            // s[0], s[1]: key gid, heads 2tig, 2tig+1;  s[2], s[3]: key gid + 8
            float acc[2];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                float v = 0.f;
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    if (a.act == 1) {                                     // Eq. 3: ReLU
                        v = fmaf(wv[e], fmaxf(s[hf * 2 + e] + bv[e], 0.f), v);
                    } else {
                        float ex, rc;
                        const float arg = fminf(fmaf(s[hf * 2 + e], -1.4426950408889634f, bv[e]), 80.f);
                        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(ex) : "f"(arg));
                        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rc) : "f"(1.0f + ex));
                        v = fmaf(wv[e], rc, v);
                    }
                }
                v += __shfl_xor_sync(0xFFFFFFFFu, v, 1);
                v += __shfl_xor_sync(0xFFFFFFFFu, v, 2);
                acc[hf] = v;
            }
            const int key = k0 + u * 16 + (tig & 1) * 8 + gid;
            if (tig < 2 && key < key_hi) out_row[key] = acc[tig & 1];
        }
    }
}

template <int DI, int HI>
cudaError_t launch_rows_t(const gsa_params_t& p, RowRange rr, const RowsIdxArgs& a0, cudaStream_t st) {
    RowsIdxArgs a = a0;
    const int n_max = p.Lk - p.Lq + rr.q_begin + rr.R;
    // enough CTAs to fill the GPU about four times over, each with a run of keys long enough to stream
    const int64_t want_ctas = (int64_t)sm_count() * 4;
    int64_t per = ((int64_t)n_max * rr.rows() + want_ctas - 1) / want_ctas;
    const int step = kRowsWarps * 16 * kTilesPerStep;
    per = (per + step - 1) / step * step;
    if (per < step) per = step;
    a.keys_per_cta = (int32_t)per;
    dim3 grid((unsigned)((n_max + per - 1) / per), (unsigned)rr.rows());
    gsa_indexer_rows_kernel<DI, HI><<<grid, kRowsWarps * 32, 0, st>>>(a);
    ++g_launches;
    return cudaGetLastError();
}

}  // namespace

bool indexer_rows_preferred(const gsa_params_t& p, RowRange rr) {
    (void)p;
    return rr.R <= 4 && rr.rows() <= 65535;
}

cudaError_t launch_indexer_rows(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* qI,
                                const __nv_bfloat16* kI, const float* w, const float* bI, float* scores,
                                int64_t row_stride, cudaStream_t st) {
    if (rr.rows() <= 0) return cudaSuccess;
    RowsIdxArgs a;
    a.qI = qI; a.kI = kI; a.w = w; a.bI = bI; a.scores = scores; a.row_stride = row_stride;
    a.rr = rr; a.Lq = p.Lq; a.Lk = p.Lk; a.keys_per_cta = 0; a.act = p.act;
#define GSA_ROWS_CASE(DI_, HI_) if (p.dI == DI_ && p.HI == HI_) return launch_rows_t<DI_, HI_>(p, rr, a, st)
    GSA_ROWS_CASE(64, 8); GSA_ROWS_CASE(64, 4); GSA_ROWS_CASE(64, 2); GSA_ROWS_CASE(64, 1);
    GSA_ROWS_CASE(32, 8); GSA_ROWS_CASE(32, 4); GSA_ROWS_CASE(32, 2); GSA_ROWS_CASE(32, 1);
#undef GSA_ROWS_CASE
    return cudaErrorInvalidValue;
}

}  // namespace gsa
