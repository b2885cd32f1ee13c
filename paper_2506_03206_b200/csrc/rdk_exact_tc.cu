// Tensor-core contraction for the bf16 layout of the affinity matrix (placeholder until the
// tcgen05 kernel lands).
#include "rdk_common.cuh"

namespace rdk {

int launch_exact_tc(const __nv_bfloat16*, long long, const __nv_bfloat16*, long long, float*, int, int, int,
                    int32_t*, cudaStream_t) {
    set_error("rdk_redistribute_exact: the bf16 tensor-core layout is not available in this build");
    return RDK_ERR_UNSUPPORTED;
}

}  // namespace rdk
