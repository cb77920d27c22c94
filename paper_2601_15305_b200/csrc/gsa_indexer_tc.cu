// placeholder until the tcgen05 kernel lands
#include "gsa_common.cuh"
namespace gsa {
bool indexer_tc_supported(const gsa_params_t&) { return false; }
cudaError_t launch_indexer_tc(const gsa_params_t&, RowRange, const __nv_bfloat16*, const __nv_bfloat16*,
                              const float*, const float*, float*, int64_t, int32_t*, cudaStream_t) {
    return cudaErrorNotSupported;
}
}  // namespace gsa
