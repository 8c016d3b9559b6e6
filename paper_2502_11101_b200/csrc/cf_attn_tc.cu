// Placeholder translation unit for the tensor-core attention kernel.
#include "cf_common.cuh"

namespace cf {

bool attn_tc_supported(const cf_geom*, const cf_batch*) { return false; }

int launch_attn_tc(const cf_geom*, const cf_batch*, const PlanView&, const void*, const void*,
                   const void*, float, const AttnWorkspace&, cudaStream_t) {
    return CF_ERR_UNSUPPORTED;
}

}  // namespace cf
