// Gated lightning indexer (Eq. 7) on the CUDA cores: bring-up / cross-check path and the
// path for shapes the tensor-core kernel does not take.  One thread per key position keeps
// its k^I row in registers; the CTA walks a tile of queries whose q^I rows and head weights
// sit in shared memory (broadcast reads), so score rows are written with consecutive
// threads on consecutive s.
#include "gsa_common.cuh"

namespace gsa {

namespace {

constexpr int kKeysPerCta = 128;
constexpr int kQueriesPerCta = 16;

struct SimpleIdxArgs {
    const __nv_bfloat16* qI;
    const __nv_bfloat16* kI;
    const float* w;
    const float* bI;
    float* scores;
    int64_t row_stride;
    RowRange rr;
    int32_t Lq, Lk, HI, act;
};

template <int DI>
__global__ void __launch_bounds__(kKeysPerCta) gsa_indexer_simple_kernel(const SimpleIdxArgs a) {
    __shared__ float sq[kQueriesPerCta * 8 * DI];
    __shared__ float sw[kQueriesPerCta * 8];
    __shared__ float sb[8];

    const int tiles_per_batch = (a.rr.R + kQueriesPerCta - 1) / kQueriesPerCta;
    const int bl = blockIdx.y / tiles_per_batch;                       // local batch index
    const int tr0 = (blockIdx.y % tiles_per_batch) * kQueriesPerCta;   // first row of the tile
    const int nq = min(kQueriesPerCta, a.rr.R - tr0);
    const int b = a.rr.b0 + bl;
    const int t0 = a.rr.q_begin + tr0;
    const int off = a.Lk - a.Lq;
    const int s = blockIdx.x * kKeysPerCta + threadIdx.x;
    if (blockIdx.x * kKeysPerCta > off + t0 + nq - 1) return;          // tile entirely above the diagonal

    const int HI = a.HI;
    for (int i = threadIdx.x; i < nq * HI * DI; i += kKeysPerCta)
        sq[i] = __bfloat162float(a.qI[((size_t)b * a.Lq + t0) * HI * DI + i]);
    for (int i = threadIdx.x; i < nq * HI; i += kKeysPerCta) sw[i] = a.w[((size_t)b * a.Lq + t0) * HI + i];
    if (threadIdx.x < 8) sb[threadIdx.x] = (a.bI && threadIdx.x < HI) ? a.bI[threadIdx.x] : 0.f;

    float k[DI];
    if (s < a.Lk) {
        const uint4* kp = reinterpret_cast<const uint4*>(a.kI + ((size_t)b * a.Lk + s) * DI);
#pragma unroll
        for (int c = 0; c < DI / 8; ++c) {
            const uint4 v = __ldg(kp + c);
            const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 f = __bfloat1622float2(v2[e]);
                k[c * 8 + 2 * e] = f.x;
                k[c * 8 + 2 * e + 1] = f.y;
            }
        }
    }
    __syncthreads();

    for (int qi = 0; qi < nq; ++qi) {
        const int t = t0 + qi;
        if (s > off + t) continue;                                     // not visible (also s >= Lk)
        float acc = 0.f;
        for (int j = 0; j < HI; ++j) {
            const float* q = sq + (qi * HI + j) * DI;
            float x = sb[j];
#pragma unroll
            for (int c = 0; c < DI; ++c) x = fmaf(q[c], k[c], x);
            acc = fmaf(sw[qi * HI + j], a.act == 1 ? fmaxf(x, 0.f) : fast_sigmoid(x), acc);
        }
        a.scores[((int64_t)bl * a.rr.R + tr0 + qi) * a.row_stride + s] = acc;
    }
}

}  // namespace

cudaError_t launch_indexer_simple(const gsa_params_t& p, RowRange rr, const __nv_bfloat16* qI,
                                  const __nv_bfloat16* kI, const float* w, const float* bI,
                                  float* scores, int64_t row_stride, cudaStream_t st) {
    if (rr.rows() <= 0) return cudaSuccess;
    SimpleIdxArgs a;
    a.qI = qI; a.kI = kI; a.w = w; a.bI = bI; a.scores = scores; a.row_stride = row_stride;
    a.rr = rr; a.Lq = p.Lq; a.Lk = p.Lk; a.HI = p.HI; a.act = p.act;
    const int n_max = p.Lk - p.Lq + rr.q_begin + rr.R;                 // visible keys of the last row
    dim3 grid((n_max + kKeysPerCta - 1) / kKeysPerCta,
              rr.nb * ((rr.R + kQueriesPerCta - 1) / kQueriesPerCta));
    if (p.dI == 64) gsa_indexer_simple_kernel<64><<<grid, kKeysPerCta, 0, st>>>(a);
    else if (p.dI == 32) gsa_indexer_simple_kernel<32><<<grid, kKeysPerCta, 0, st>>>(a);
    else return cudaErrorInvalidValue;
    ++g_launches;
    return cudaGetLastError();
}

}  // namespace gsa
