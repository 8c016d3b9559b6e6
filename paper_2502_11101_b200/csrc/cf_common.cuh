// Shared declarations of the CUDA side: views of the caller's buffers, small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cachefocus.h"
#include "cachefocus_debug.h"

namespace cf {

constexpr int kTile = CF_TILE_TOKENS;
constexpr int kMaxDocs = CF_MAX_DOCS_PER_REQUEST;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct GeomView {
    int n_q_heads, n_kv_heads, head_dim, dtype, rope_layout, pos_range;
    double rope_theta;
};

struct BatchView {
    int n_requests, n_docs_total, q_len, prefix_len, tail_reserve, n_reuse;
    long long total_tokens, token_stride;
    const int* req_doc_begin;
    const int* doc_offsets;
    const int* doc_src_start;
};

// Typed pointers into a plan buffer (see cf_plan_layout).
struct PlanView {
    int* status;
    int* kept;
    int* kept_count;
    int* dst_start;
    int* group;
    int* n_reuse;
    int* query_start;
    int* n_tiles;
    int* tile_begin;
    int* doc_tile_begin;
    int* doc_tile_count;
    int* tile_doc;
    int* tile_row0;
    int* tile_len;
    float2* trig;
    int max_tiles;
};

// First tile slot of request b: an upper bound of the tiles all earlier requests can own
// (a document of len tokens owns ceil(len/kTile) <= 1 + len/kTile tiles).
__host__ __device__ inline int tile_base(int doc_begin, int row_begin) {
    return doc_begin + row_begin / kTile;
}

GeomView make_geom_view(const cf_geom* g);
BatchView make_batch_view(const cf_batch* b);
PlanView make_plan_view(const cf_geom* g, const cf_batch* b, void* plan);
int validate(const cf_geom* g, const cf_batch* b);
int sm_count();
// Index of the current device for per-device caches (attributes such as the dynamic shared memory
// limit of a kernel and the SM count belong to a device, not to the process); -1 if unknown.
constexpr int kMaxDevices = 64;
int current_device();
// One flag per device: true once the calling site has configured its kernel on that device.
struct PerDeviceOnce {
    bool done[kMaxDevices] = {};
};
// Sets the dynamic shared memory limit of `kernel` once per device; CF_OK or CF_ERR_CUDA.
template <typename K>
int configure_smem_once(PerDeviceOnce& once, K kernel, int bytes) {
    const int dev = current_device();
    if (dev >= 0 && once.done[dev]) return CF_OK;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess)
        return CF_ERR_CUDA;
    if (dev >= 0) once.done[dev] = true;
    return CF_OK;
}
int choose_splits(const cf_geom* g, const cf_batch* b, int n_layers);
int choose_row_group(const cf_geom* g, const cf_batch* b);
int tiles_per_request_bound(const cf_batch* b);

// Partial results of the attention kernels, one slice per split, merged by the combine kernel.
// All logits are in base-2 units: t = (q.k) * softmax_scale * log2(e).
// A call covers n_layers layers; (layer, request) pairs are numbered lb = layer * B + request.
struct AttnWorkspace {
    float* part_o;     // [L*B][n_splits][Hq*Lq][D] sum_t 2^(t - m) v_t, not normalised (unset if m = -inf);
                       //                           fp32, or bf16 in the same index order when part_bf16 is set
    float* part_m;     // [L*B][n_splits][Hq*Lq]    reference maximum m (-inf if the part is empty)
    float* part_l;     // [L*B][n_splits][Hq*Lq]    sum_t 2^(t - m)
    float* tile_lse2;  // [L][max_tiles][Hq*Lq]     log2 of sum over the tile's tokens of 2^t
    float* row_lse2;   // [L*B][Hq*Lq]              log2 of the full softmax denominator
    int n_splits;
    int part_bf16;     // the tensor-core kernel stores its partial O rows as bf16
    int n_layers;
    int max_tiles;     // tile slots per layer in tile_lse2
    int rg_rows;       // query rows per CTA of the tensor-core kernel: 256 (two row tiles) or 128
    // Key blocks besides the documents (the query-self block, a shared prefix cache) of a call that has some.
    // self_mode 1 (CUDA-core path): the query-self block is one more part, (self_m, self_l, self_o) like
    // (part_m, part_l, part_o) in fp32.  self_mode 2 (tensor-core path): the blocks are further key tiles of
    // the last parts, and part_ld holds every part's sum over the documents' keys alone.  self_mode 0: none.
    float* self_o;     // [L*B][Hq*Lq][D]
    float* self_m;     // [L*B][Hq*Lq]
    float* self_l;     // [L*B][Hq*Lq]
    float* part_ld;    // [L*B][n_splits][Hq*Lq]    like part_l, the documents' keys only (self_mode 2)
    int self_mode;
    int keys_in_place; // every document's destination equals its source (decoding over final caches): no rotation
};
// part_layers > 0: the partial results (and the further key blocks' buffers) are sized for that many layers only, the
// per-tile and per-row log-sum-exps for n_layers (calls that fill one layer slot at a time and score the slots later).
size_t attn_workspace_layout(const cf_geom* g, const cf_batch* b, int n_splits, int n_layers, bool with_self,
                             AttnWorkspace* ws, void* base, int part_layers = 0);

// Where the layers of a call sit (element strides between consecutive layers).
struct LayerSpan {
    int n_layers;
    long long q_stride, kv_stride, out_stride;
};

// ---- launchers (each returns a CF_* code) -------------------------------------------------
int launch_plan(const GeomView& gv, const BatchView& bv, const PlanView& pv, int mode,
                const int* order, const int* kept_count, int query_start, const float* score_accum,
                int keep, const int* keep_per_request, int strategy, cudaStream_t stream);
int launch_merge_attn(const cf_geom* g, long long n_rows, int q_len, const void* out_a, const float* lse_a,
                      const void* out_b, const float* lse_b, void* out, float* lse, cudaStream_t stream);
int launch_clear_status(const PlanView& pv, cudaStream_t stream);
int launch_wait_probe(const PlanView& pv, long long limit_cycles, cudaStream_t stream);
int launch_reposition(const cf_geom* g, const cf_batch* b, const PlanView& pv, int n_layers,
                      long long layer_stride, const void* k_in, void* k_out, cudaStream_t stream);
int launch_assemble(const cf_geom* g, const cf_batch* b, const PlanView& pv, int n_layers, long long layer_stride,
                    long long self_stride, int out_rows, const void* k_in, const void* v_in, const void* k_self,
                    const void* v_self, void* k_out, void* v_out, int* final_rows, cudaStream_t stream);
int launch_attn_simt(const cf_geom* g, const cf_batch* b, const PlanView& pv, const LayerSpan& span,
                     const void* q, const void* k, const void* v, float scale_log2,
                     const AttnWorkspace& ws, cudaStream_t stream);
int launch_attn_tc(const cf_geom* g, const cf_batch* b, const PlanView& pv, const LayerSpan& span,
                   const void* q, const void* k, const void* v, const void* k_self, const void* v_self,
                   long long self_stride, const void* k_prefix, const void* v_prefix, long long prefix_stride,
                   int prefix_len, float scale_log2, const AttnWorkspace& ws, cudaStream_t stream);
bool attn_tc_supported(const cf_geom* g, const cf_batch* b);
int launch_combine(const cf_geom* g, const cf_batch* b, const PlanView& pv, const LayerSpan& span,
                   const AttnWorkspace& ws, void* out, float* lse, float* doc_scores,
                   float* score_accum, cudaStream_t stream);
int launch_self_block(const cf_geom* g, const cf_batch* b, const LayerSpan& span, long long self_stride,
                      const void* q, const void* k_self, const void* v_self, const void* k_prefix, const void* v_prefix,
                      long long prefix_stride, int prefix_len, float scale_log2, const AttnWorkspace& ws,
                      cudaStream_t stream);
// Shared body of the attention entry points (k_self = v_self = null: cached documents only).
int run_attn_layers(const cf_geom* geom, const cf_batch* batch, const void* plan, const LayerSpan& span,
                    const void* q, const void* k_cache, const void* v_cache, const void* k_self,
                    const void* v_self, long long self_stride, float softmax_scale,
                    void* out, float* lse, float* doc_scores, float* score_accum, void* workspace,
                    size_t workspace_bytes, cudaStream_t stream, const void* k_prefix = nullptr,
                    const void* v_prefix = nullptr, long long prefix_stride = 0, int prefix_len = 0, int slot = -1,
                    int n_slots = 0, bool keys_in_place = false);
// Document scores of the layers held in a workspace: doc_scores[l] = s^l (optional), S += s^l in layer order.
int launch_scores(const cf_geom* g, const cf_batch* b, const PlanView& pv, const AttnWorkspace& ws, float* doc_scores,
                  float* score_accum, cudaStream_t stream);

// Arguments of the cache-construction attention kernels (cf_document_prefill_attn).
struct DocAttnArgs {
    int n_docs, n_layers, max_doc_len, prefix_len, n_q_heads, n_kv_heads;
    long long total_tokens, token_stride, q_layer_stride, kv_layer_stride, prefix_layer_stride, out_layer_stride;
    const int* doc_offsets;
    float scale_log2;
};
int launch_docattn_simt(const cf_geom* g, const DocAttnArgs& a, const void* q, const void* k, const void* v,
                        const void* kp, const void* vp, void* out, float* lse, cudaStream_t stream);
bool docattn_tc_supported(const cf_geom* g, const cf_doc_batch* docs);
int launch_docattn_tc(const cf_geom* g, const DocAttnArgs& a, const void* q, const void* k, const void* v,
                      const void* kp, const void* vp, void* out, float* lse, int* status, cudaStream_t stream);
int attn_path();

// ---- device helpers -----------------------------------------------------------------------
__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_float(float x);
template <> __device__ __forceinline__ float from_float<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float x) {
    return __float2bfloat16_rn(x);
}

// Eq. 2 on one slice (a, b) with (c, s) = cos, sin of the delta angle; fp32, fused multiply-adds.
__device__ __forceinline__ void rotate_pair(float a, float b, float c, float s, float& ya, float& yb) {
    ya = fmaf(a, c, -(b * s));
    yb = fmaf(a, s, b * c);
}

}  // namespace cf
