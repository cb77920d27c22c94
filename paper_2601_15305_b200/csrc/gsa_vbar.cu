// Running mean of the score variance: the normaliser V-bar of the adaptive budget (Eq. 8) is an
// exponential moving average of the score variance across the batch.  The paper gives neither the
// momentum nor the start value, so both are the caller's:
//     mean_var = mean over the batch's query rows of Var(I[t, :])
//     v_bar    = momentum * v_bar + (1 - momentum) * mean_var
// One CTA, fp64 partial sums added in a fixed order: the result does not depend on scheduling.
#include "gsa_common.cuh"

namespace gsa {

namespace {

constexpr int kVbarThreads = 1024;

__global__ void __launch_bounds__(kVbarThreads) gsa_vbar_update_kernel(const float* __restrict__ var, int64_t n,
                                                                       float momentum, float* v_bar,
                                                                       float* mean_var) {
    __shared__ double part[kVbarThreads / 32];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    double s = 0.0;
    for (int64_t i = tid; i < n; i += kVbarThreads) s += (double)__ldg(var + i);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    if (lane == 0) part[wid] = s;
    __syncthreads();
    if (tid == 0) {
        double tot = 0.0;
        for (int i = 0; i < kVbarThreads / 32; ++i) tot += part[i];
        const double m = n > 0 ? tot / (double)n : 0.0;
        if (mean_var) *mean_var = (float)m;
        *v_bar = (float)((double)momentum * (double)*v_bar + (1.0 - (double)momentum) * m);
    }
}

}  // namespace

cudaError_t launch_vbar_update(const float* var, int64_t n, float momentum, float* v_bar, float* mean_var,
                               cudaStream_t st) {
    gsa_vbar_update_kernel<<<1, kVbarThreads, 0, st>>>(var, n, momentum, v_bar, mean_var);
    ++g_launches;
    return cudaGetLastError();
}

}  // namespace gsa
