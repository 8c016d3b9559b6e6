// Decoding over the final caches (Algorithm 2, Phase 3: Y <- LLM(C_final); the "Decoding" loop of
// Algorithm 1): every generated token appends its key/value rows to each request's packed final cache
// and attends all rows of it.  The caches come out of cf_assemble_final_cache already re-positioned, so
// nothing is rotated here: each request's used rows are declared as one document whose destination
// equals its source (delta 0) and the attention kernels of the query-time path do the rest -- with one
// query row per head the pass is a stream over the cache, bound by HBM bandwidth.
#include <climits>

#include "cf_common.cuh"

namespace cf {

namespace {

// Integer description of the decoding batch, kept in front of the plan inside the caller's buffer:
// two documents per request (the used rows of its slot, the unused tail), only the first is kept.
struct DecodeArrays {
    int* req_doc_begin;   // [B + 1]
    int* doc_offsets;     // [2 B + 1]
    int* doc_src_start;   // [2 B]
    int* order;           // [2 B]
    int* kept_count;      // [B]
    size_t bytes;         // of the block, a multiple of 256
};

DecodeArrays decode_arrays(void* base, int n_requests) {
    DecodeArrays a;
    int* p = static_cast<int*>(base);
    const size_t nb = (size_t)n_requests;
    a.req_doc_begin = p;
    a.doc_offsets = a.req_doc_begin + nb + 1;
    a.doc_src_start = a.doc_offsets + 2 * nb + 1;
    a.order = a.doc_src_start + 2 * nb;
    a.kept_count = a.order + 2 * nb;
    a.bytes = ((8 * nb + 2) * sizeof(int) + 255) / 256 * 256;
    return a;
}

// The geometry and batch the query-time kernels see for a decoding step.  The positional range is
// widened so that a cache of any length fits one window: positions only enter through the delta,
// which is 0 here.
void decode_views(const cf_geom* geom, int n_requests, int cache_rows, const DecodeArrays& a, cf_geom* g, cf_batch* b) {
    *g = *geom;
    g->pos_range = INT_MAX / 2;
    b->n_requests = n_requests;
    b->n_docs_total = 2 * n_requests;
    b->q_len = 1;
    b->prefix_len = 0;
    b->tail_reserve = 1;
    b->n_reuse = 1;
    b->tiles_hint = cache_rows / kTile + 2;
    b->reserved = 0;
    b->total_tokens = (int64_t)n_requests * cache_rows;
    b->token_stride = (int64_t)geom->n_kv_heads * geom->head_dim;
    b->req_doc_begin = a.req_doc_begin;
    b->doc_offsets = a.doc_offsets;
    b->doc_src_start = a.doc_src_start;
}

int check_decode(const cf_geom* geom, int n_requests, int cache_rows) {
    int rc = validate(geom, nullptr);
    if (rc != CF_OK) return rc;
    if (n_requests <= 0 || n_requests > (1 << 20) || cache_rows <= 0) return CF_ERR_INVALID_ARG;
    if ((long long)n_requests * cache_rows > 0x7fffffffLL - kTile) return CF_ERR_INVALID_ARG;
    return CF_OK;
}

__global__ void decode_setup_kernel(DecodeArrays a, int n_requests, int cache_rows, int pos_range,
                                    const int* __restrict__ rows, int extra_rows, int* status) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b > n_requests) return;
    if (b == n_requests) {
        a.req_doc_begin[b] = 2 * b;
        a.doc_offsets[2 * b] = b * cache_rows;
        return;
    }
    long long used = (long long)rows[b] + extra_rows;
    if (used < 1 || used > cache_rows) {                // the slot cannot hold (or has) that many rows
        atomicCAS(status, 0, CF_ERR_RANGE);
        used = used < 1 ? 1 : cache_rows;
    }
    a.req_doc_begin[b] = 2 * b;
    a.doc_offsets[2 * b] = b * cache_rows;
    a.doc_offsets[2 * b + 1] = b * cache_rows + (int)used;
    // cached where the allocation will put it: the window ends at the query (pos_range - tail_reserve)
    a.doc_src_start[2 * b] = pos_range - 1 - (int)used;
    a.doc_src_start[2 * b + 1] = 0;
    a.order[2 * b] = 0;
    a.order[2 * b + 1] = 1;
    a.kept_count[b] = 1;
}

// One block per (request, layer): the new token's key and value rows go behind the rows in use.
template <typename T>
__global__ void decode_append_kernel(int cache_rows, int row_elems, long long layer_stride, long long new_layer_stride,
                                     const int* __restrict__ rows, int step, const T* __restrict__ k_new,
                                     const T* __restrict__ v_new, T* __restrict__ k_final, T* __restrict__ v_final,
                                     int* status) {
    const int b = blockIdx.x, layer = blockIdx.y;
    const long long row = (long long)rows[b] + step;
    if (row < 0 || row >= cache_rows) {
        if (threadIdx.x == 0 && status) atomicCAS(status, 0, CF_ERR_RANGE);
        return;
    }
    constexpr int E = 16 / sizeof(T);
    const size_t dst = (size_t)layer * layer_stride + ((size_t)b * cache_rows + (size_t)row) * row_elems;
    const size_t src = (size_t)layer * new_layer_stride + (size_t)b * row_elems;
    for (int i = threadIdx.x * E; i < row_elems; i += blockDim.x * E) {
        *reinterpret_cast<uint4*>(k_final + dst + i) = *reinterpret_cast<const uint4*>(k_new + src + i);
        *reinterpret_cast<uint4*>(v_final + dst + i) = *reinterpret_cast<const uint4*>(v_new + src + i);
    }
}

}  // namespace

}  // namespace cf

using namespace cf;

extern "C" {

size_t cf_decode_plan_bytes(const cf_geom* geom, int32_t n_requests, int32_t cache_rows) {
    if (check_decode(geom, n_requests, cache_rows) != CF_OK) return 0;
    const DecodeArrays a = decode_arrays(nullptr, n_requests);
    cf_geom g;
    cf_batch b;
    decode_views(geom, n_requests, cache_rows, a, &g, &b);
    cf_plan_layout L;
    // the layout depends on sizes only; the (null-based) array pointers are not dereferenced on the host
    b.req_doc_begin = b.doc_offsets = b.doc_src_start = reinterpret_cast<const int32_t*>(geom);
    if (cf_plan_layout_of(&g, &b, &L) != CF_OK) return 0;
    return a.bytes + L.total_bytes;
}

int cf_decode_plan(const cf_geom* geom, int32_t n_requests, int32_t cache_rows, const int32_t* rows,
                   int32_t extra_rows, void* decode_plan, size_t decode_plan_bytes, void* stream) {
    int rc = check_decode(geom, n_requests, cache_rows);
    if (rc != CF_OK) return rc;
    if (!rows || !decode_plan) return CF_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(decode_plan) % 256 != 0) return CF_ERR_WORKSPACE;
    const size_t need = cf_decode_plan_bytes(geom, n_requests, cache_rows);
    if (need == 0 || decode_plan_bytes < need) return CF_ERR_WORKSPACE;
    const DecodeArrays a = decode_arrays(decode_plan, n_requests);
    cf_geom g;
    cf_batch b;
    decode_views(geom, n_requests, cache_rows, a, &g, &b);
    void* plan = static_cast<char*>(decode_plan) + a.bytes;
    const PlanView pv = make_plan_view(&g, &b, plan);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    rc = launch_clear_status(pv, s);
    if (rc != CF_OK) return rc;
    decode_setup_kernel<<<(n_requests + 1 + 255) / 256, 256, 0, s>>>(a, n_requests, cache_rows, g.pos_range, rows,
                                                                   extra_rows, pv.status);
    if (cudaGetLastError() != cudaSuccess) return CF_ERR_CUDA;
    return launch_plan(make_geom_view(&g), make_batch_view(&b), pv, 0, a.order, a.kept_count, -1, nullptr, 0, nullptr,
                       CF_ALLOC_ALIGN, s);
}

int cf_decode_status(const cf_geom* geom, int32_t n_requests, int32_t cache_rows, const void* decode_plan, void* stream) {
    int rc = check_decode(geom, n_requests, cache_rows);
    if (rc != CF_OK) return rc;
    if (!decode_plan) return CF_ERR_INVALID_ARG;
    const DecodeArrays a = decode_arrays(const_cast<void*>(decode_plan), n_requests);
    cf_geom g;
    cf_batch b;
    decode_views(geom, n_requests, cache_rows, a, &g, &b);
    return cf_plan_status(&g, &b, static_cast<const char*>(decode_plan) + a.bytes, stream);
}

size_t cf_decode_workspace_bytes(const cf_geom* geom, int32_t n_requests, int32_t cache_rows, int32_t n_layers) {
    if (check_decode(geom, n_requests, cache_rows) != CF_OK) return 0;
    const DecodeArrays a = decode_arrays(nullptr, n_requests);
    cf_geom g;
    cf_batch b;
    decode_views(geom, n_requests, cache_rows, a, &g, &b);
    b.req_doc_begin = b.doc_offsets = b.doc_src_start = reinterpret_cast<const int32_t*>(geom);
    return cf_attn_workspace_bytes_layers(&g, &b, n_layers);
}

int cf_decode_attn(const cf_geom* geom, int32_t n_requests, int32_t cache_rows, const void* decode_plan,
                   int32_t n_layers, const void* q, int64_t q_layer_stride, const void* k_final,
                   const void* v_final, int64_t kv_layer_stride, float softmax_scale, void* out,
                   int64_t out_layer_stride, float* lse, void* workspace, size_t workspace_bytes, void* stream) {
    int rc = check_decode(geom, n_requests, cache_rows);
    if (rc != CF_OK) return rc;
    if (!decode_plan || q_layer_stride < 0 || kv_layer_stride < 0 || out_layer_stride < 0) return CF_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(decode_plan) % 256 != 0) return CF_ERR_WORKSPACE;
    const DecodeArrays a = decode_arrays(const_cast<void*>(decode_plan), n_requests);
    cf_geom g;
    cf_batch b;
    decode_views(geom, n_requests, cache_rows, a, &g, &b);
    const LayerSpan span = {n_layers, q_layer_stride, kv_layer_stride, out_layer_stride};
    return run_attn_layers(&g, &b, static_cast<const char*>(decode_plan) + a.bytes, span, q, k_final, v_final, nullptr,
                           nullptr, 0, softmax_scale, out, lse, nullptr, nullptr, workspace, workspace_bytes,
                           static_cast<cudaStream_t>(stream), nullptr, nullptr, 0, 0, -1, 0,
                           /*keys_in_place=*/true);           // the final caches are used where they lie
}

int cf_decode_append(const cf_geom* geom, int32_t n_requests, int32_t cache_rows, int32_t n_layers,
                     void* k_final, void* v_final, int64_t kv_layer_stride, const int32_t* rows, int32_t step,
                     const void* k_new, const void* v_new, int64_t new_layer_stride, int32_t* status, void* stream) {
    int rc = check_decode(geom, n_requests, cache_rows);
    if (rc != CF_OK) return rc;
    if (!k_final || !v_final || !rows || !k_new || !v_new || n_layers <= 0 || n_layers > 65535 || step < 0)
        return CF_ERR_INVALID_ARG;
    const int row_elems = geom->n_kv_heads * geom->head_dim;
    const int esize = geom->dtype == CF_BF16 ? 2 : 4;
    const void* ptrs[4] = {k_final, v_final, k_new, v_new};
    for (const void* p : ptrs)
        if (reinterpret_cast<uintptr_t>(p) % 16) return CF_ERR_INVALID_ARG;
    if ((kv_layer_stride * esize) % 16 || (new_layer_stride * esize) % 16) return CF_ERR_INVALID_ARG;
    if (n_layers > 1 && (kv_layer_stride < (int64_t)n_requests * cache_rows * row_elems ||
                         new_layer_stride < (int64_t)n_requests * row_elems))
        return CF_ERR_INVALID_ARG;
    const dim3 grid((unsigned)n_requests, (unsigned)n_layers);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (geom->dtype == CF_BF16)
        decode_append_kernel<__nv_bfloat16><<<grid, 128, 0, s>>>(
            cache_rows, row_elems, kv_layer_stride, new_layer_stride, rows, step, static_cast<const __nv_bfloat16*>(k_new),
            static_cast<const __nv_bfloat16*>(v_new), static_cast<__nv_bfloat16*>(k_final),
            static_cast<__nv_bfloat16*>(v_final), status);
    else
        decode_append_kernel<float><<<grid, 128, 0, s>>>(cache_rows, row_elems, kv_layer_stride, new_layer_stride, rows, step,
                                                         static_cast<const float*>(k_new), static_cast<const float*>(v_new),
                                                         static_cast<float*>(k_final), static_cast<float*>(v_final), status);
    return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

}  // extern "C"
