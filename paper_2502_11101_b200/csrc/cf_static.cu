// An attention entry point for callers that cannot allocate device memory: its scratch space is
// a fixed array that lives in the library image instead of a caller-provided workspace.
#include <cmath>
#include <mutex>

#include "cf_common.cuh"

namespace cf {


// The scratch itself.  Every GPU that loads this library holds these bytes until the process
// exits.  In host code `g_static_scratch` is only a handle: the device address comes from
// cudaGetSymbolAddress (static_scratch_address below).
static __device__ __align__(256) unsigned char g_static_scratch[CF_STATIC_WORKSPACE_BYTES];

static std::mutex g_static_mutex;
static void* g_static_address[kMaxDevices] = {};

// Device address of the scratch array on the current device; looked up once per device.
static int static_scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CF_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_address[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return CF_ERR_CUDA;
        g_static_address[dev] = ptr;
    }
    *out = g_static_address[dev];
    return CF_OK;
}

}  // namespace cf

using namespace cf;

extern "C" int cf_query_prefill_attn_static(const cf_geom* geom, const cf_batch* batch, const void* plan,
                                            const void* q, const void* k_cache, const void* v_cache,
                                            float softmax_scale, void* out, float* lse,
                                            float* doc_scores, float* score_accum, void* stream) {
    if (!batch || !plan) return CF_ERR_INVALID_ARG;
    int rc = validate(geom, batch);
    if (rc != CF_OK) return rc;
    if (attn_workspace_layout(geom, batch, choose_splits(geom, batch, 1), 1, false, nullptr, nullptr) >
        (size_t)CF_STATIC_WORKSPACE_BYTES)
        return CF_ERR_WORKSPACE;            // this batch needs more scratch than the library carries
    void* scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc != CF_OK) return rc;
    const LayerSpan span = {1, 0, 0, 0};
    return run_attn_layers(geom, batch, plan, span, q, k_cache, v_cache, nullptr, nullptr, 0, softmax_scale, out, lse,
                           doc_scores, score_accum, scratch, (size_t)CF_STATIC_WORKSPACE_BYTES,
                           static_cast<cudaStream_t>(stream));
}
