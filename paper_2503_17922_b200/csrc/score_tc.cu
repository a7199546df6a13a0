// Tensor-core (tcgen05) score kernels — placeholder until the kernels land.
#include "wkv_internal.cuh"

namespace wkv {

bool score_tc_supported(const KShape &, int) { return false; }

int launch_score_tc(const KShape &, const void *, const void *, float *, float *, void *, const Workspace &,
                    cudaStream_t)
{
    set_error_detail("tensor-core score kernels are not built");
    return WKV_ERR_UNSUPPORTED;
}

}  // namespace wkv
