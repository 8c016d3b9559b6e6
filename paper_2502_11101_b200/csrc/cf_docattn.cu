// Attention of the offline cache construction, C_d <- LLM(C_prefix, d) (Sec. 2.2): the tokens of every
// document attend the shared prefix cache and the document's own earlier tokens under the causal mask of
// Eq. 1; documents do not see each other, so the batch is block-diagonal over a packed store.
// This file holds the portable CUDA-core kernel (any storage type, head_dim 64 or 128) and the entry
// point; the tensor-core kernel for bf16 / head_dim 128 is in cf_docattn_tc.cu.
//
// Rows of a (document, kv head) are numbered token-major, r = token * G + g (G = query heads per kv
// head), so that a block of consecutive rows needs the keys up to its last token only.
#include <cmath>

#include "cf_common.cuh"

namespace cf {

namespace {

constexpr int kDocThreads = 256;
constexpr int kDocRows = 64;      // query rows per CTA
constexpr int kDocSub = 32;       // keys per inner step

template <int D>
constexpr size_t doc_smem_bytes() {
    return sizeof(float) * (size_t)(kDocRows * (D + 1) + kDocSub * (D + 1) + kDocSub * D + kDocRows * (kDocSub + 1));
}

template <typename T, int D>
__global__ void __launch_bounds__(kDocThreads)
docattn_simt_kernel(DocAttnArgs a, const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                    const T* __restrict__ k_prefix, const T* __restrict__ v_prefix, T* __restrict__ out,
                    float* __restrict__ lse) {
    extern __shared__ float smem[];
    float (*Qs)[D + 1] = reinterpret_cast<float (*)[D + 1]>(smem);
    float (*Ks)[D + 1] = reinterpret_cast<float (*)[D + 1]>(smem + kDocRows * (D + 1));
    float (*Vs)[D] = reinterpret_cast<float (*)[D]>(smem + (kDocRows + kDocSub) * (D + 1));
    float (*Ps)[kDocSub + 1] =
        reinterpret_cast<float (*)[kDocSub + 1]>(smem + (kDocRows + kDocSub) * (D + 1) + kDocSub * D);

    const int tid = threadIdx.x;
    const int group = a.n_q_heads / a.n_kv_heads;
    const int layer = blockIdx.z / a.n_docs, doc = blockIdx.z - layer * a.n_docs;
    const int kvh = blockIdx.y;
    const int row_first = a.doc_offsets[doc];
    const int len = a.doc_offsets[doc + 1] - row_first;
    const int rows = len * group;
    const int r0 = blockIdx.x * kDocRows;
    if (r0 >= rows) return;
    const int n_rows = min(kDocRows, rows - r0);
    q += (size_t)layer * a.q_layer_stride;
    out += (size_t)layer * a.out_layer_stride;
    k += (size_t)layer * a.kv_layer_stride;
    v += (size_t)layer * a.kv_layer_stride;
    k_prefix += (size_t)layer * a.prefix_layer_stride;
    v_prefix += (size_t)layer * a.prefix_layer_stride;

    for (int idx = tid; idx < kDocRows * D; idx += kDocThreads) {
        const int rr = idx / D, d = idx - rr * D;
        float val = 0.f;
        if (rr < n_rows) {
            const int row = r0 + rr;
            const int j = row / group, g = row - j * group;
            val = to_float(q[((size_t)(row_first + j) * a.n_q_heads + kvh * group + g) * D + d]);
        }
        Qs[rr][d] = val;
    }

    const int r = tid >> 2, q4 = tid & 3;
    const int my_token = (r0 + min(r, n_rows - 1)) / group;            // rows beyond the end follow the last valid row
    const int last_token = (r0 + n_rows - 1) / group;                  // the block needs document keys 0..last_token
    const int n_keys = a.prefix_len + last_token + 1;
    float m = -INFINITY, l = 0.f;
    float acc[D / 4];
#pragma unroll
    for (int i = 0; i < D / 4; ++i) acc[i] = 0.f;

    for (int sub = 0; sub < n_keys; sub += kDocSub) {
        __syncthreads();
        for (int idx = tid; idx < kDocSub * D; idx += kDocThreads) {
            const int t = idx / D, d = idx - t * D;
            const int key = sub + t;                                   // index in [prefix ; document]
            float kv = 0.f, vv = 0.f;
            if (key < a.prefix_len) {
                kv = to_float(k_prefix[((size_t)key * a.n_kv_heads + kvh) * D + d]);
                vv = to_float(v_prefix[((size_t)key * a.n_kv_heads + kvh) * D + d]);
            } else if (key < n_keys) {
                const size_t off = (size_t)(row_first + key - a.prefix_len) * a.token_stride + (size_t)kvh * D + d;
                kv = to_float(k[off]);
                vv = to_float(v[off]);
            }
            Ks[t][d] = kv;
            Vs[t][d] = vv;
        }
        __syncthreads();
        float sc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) sc[i] = 0.f;
        for (int d = 0; d < D; ++d) {
            const float qv = Qs[r][d];
#pragma unroll
            for (int i = 0; i < 8; ++i) sc[i] = fmaf(qv, Ks[q4 * 8 + i][d], sc[i]);
        }
        // causal mask: the prefix and document tokens 0..my_token are visible
        const int visible = a.prefix_len + my_token + 1;
        float sub_max = -INFINITY;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            sc[i] = (sub + q4 * 8 + i < visible) ? sc[i] * a.scale_log2 : -INFINITY;
            sub_max = fmaxf(sub_max, sc[i]);
        }
        sub_max = fmaxf(sub_max, __shfl_xor_sync(0xffffffffu, sub_max, 1));
        sub_max = fmaxf(sub_max, __shfl_xor_sync(0xffffffffu, sub_max, 2));
        const float m_new = fmaxf(m, sub_max);                         // finite from the first step on: key 0 is visible
        const float alpha = exp2f(m - m_new);
        float sub_sum = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float pr = exp2f(sc[i] - m_new);
            Ps[r][q4 * 8 + i] = pr;
            sub_sum += pr;
        }
        sub_sum += __shfl_xor_sync(0xffffffffu, sub_sum, 1);
        sub_sum += __shfl_xor_sync(0xffffffffu, sub_sum, 2);
        l = fmaf(l, alpha, sub_sum);
        m = m_new;
#pragma unroll
        for (int i = 0; i < D / 4; ++i) acc[i] *= alpha;
        __syncwarp();
        for (int t = 0; t < kDocSub; ++t) {
            const float pr = Ps[r][t];
#pragma unroll
            for (int i = 0; i < D / 4; ++i) acc[i] = fmaf(pr, Vs[t][4 * i + q4], acc[i]);
        }
    }
    if (r < n_rows) {
        const int row = r0 + r;
        const int j = row / group, g = row - j * group;
        const int h = kvh * group + g;
        const float inv = 1.f / l;
        T* dst = out + ((size_t)(row_first + j) * a.n_q_heads + h) * D;
#pragma unroll
        for (int i = 0; i < D / 4; ++i) dst[4 * i + q4] = from_float<T>(acc[i] * inv);
        if (q4 == 0 && lse)
            lse[((size_t)layer * a.n_q_heads + h) * a.total_tokens + row_first + j] = (m + log2f(l)) * kLn2;
    }
}

template <typename T, int D>
int launch_docattn_simt_typed(const DocAttnArgs& a, const void* q, const void* k, const void* v, const void* kp,
                              const void* vp, void* out, float* lse, cudaStream_t stream) {
    const int group = a.n_q_heads / a.n_kv_heads;
    const long long chunks = ((long long)a.max_doc_len * group + kDocRows - 1) / kDocRows;
    if (chunks > 0x7fffffffLL || a.n_kv_heads > 65535 || (long long)a.n_docs * a.n_layers > 65535) return CF_ERR_INVALID_ARG;
    static PerDeviceOnce configured;
    if (configure_smem_once(configured, docattn_simt_kernel<T, D>, (int)doc_smem_bytes<D>()) != CF_OK) return CF_ERR_CUDA;
    dim3 grid((unsigned)chunks, (unsigned)a.n_kv_heads, (unsigned)(a.n_docs * a.n_layers));
    docattn_simt_kernel<T, D><<<grid, kDocThreads, doc_smem_bytes<D>(), stream>>>(
        a, static_cast<const T*>(q), static_cast<const T*>(k), static_cast<const T*>(v), static_cast<const T*>(kp),
        static_cast<const T*>(vp), static_cast<T*>(out), lse);
    return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

}  // namespace

int launch_docattn_simt(const cf_geom* g, const DocAttnArgs& a, const void* q, const void* k, const void* v,
                        const void* kp, const void* vp, void* out, float* lse, cudaStream_t stream) {
    if (g->dtype == CF_BF16)
        return g->head_dim == 128 ? launch_docattn_simt_typed<__nv_bfloat16, 128>(a, q, k, v, kp, vp, out, lse, stream)
                                  : launch_docattn_simt_typed<__nv_bfloat16, 64>(a, q, k, v, kp, vp, out, lse, stream);
    return g->head_dim == 128 ? launch_docattn_simt_typed<float, 128>(a, q, k, v, kp, vp, out, lse, stream)
                              : launch_docattn_simt_typed<float, 64>(a, q, k, v, kp, vp, out, lse, stream);
}

}  // namespace cf

using namespace cf;

extern "C" int cf_document_prefill_attn(const cf_geom* geom, const cf_doc_batch* docs, int32_t n_layers,
                                        const void* q, int64_t q_layer_stride, const void* k, const void* v,
                                        int64_t kv_layer_stride, const void* k_prefix, const void* v_prefix,
                                        int64_t prefix_layer_stride, float softmax_scale, void* out,
                                        int64_t out_layer_stride, float* lse, int32_t* status, void* stream) {
    int rc = validate(geom, nullptr);
    if (rc != CF_OK) return rc;
    if (!docs || docs->n_docs < 0 || docs->total_tokens < 0 || docs->max_doc_len < 0 || docs->prefix_len < 0 ||
        n_layers <= 0 || !(softmax_scale >= 0.0f) || !std::isfinite(softmax_scale))
        return CF_ERR_INVALID_ARG;
    if (docs->n_docs == 0 || docs->total_tokens == 0 || docs->max_doc_len == 0) return CF_OK;
    if (!docs->doc_offsets || !q || !k || !v || !out || (docs->prefix_len > 0 && (!k_prefix || !v_prefix)))
        return CF_ERR_INVALID_ARG;
    const int esize = geom->dtype == CF_BF16 ? 2 : 4;
    const int64_t row = (int64_t)geom->n_kv_heads * geom->head_dim;
    if (docs->token_stride < row || (docs->token_stride * esize) % 16 || docs->total_tokens > 0x7fffffffLL - kTile)
        return CF_ERR_INVALID_ARG;
    const void* ptrs[4] = {q, k, v, out};
    for (const void* p : ptrs)
        if (reinterpret_cast<uintptr_t>(p) % 16) return CF_ERR_INVALID_ARG;
    if (docs->prefix_len > 0 && (reinterpret_cast<uintptr_t>(k_prefix) % 16 || reinterpret_cast<uintptr_t>(v_prefix) % 16))
        return CF_ERR_INVALID_ARG;
    if (n_layers > 1) {
        const int64_t q_rows = docs->total_tokens * geom->n_q_heads * geom->head_dim;
        if (q_layer_stride < q_rows || out_layer_stride < q_rows ||
            kv_layer_stride < docs->total_tokens * docs->token_stride ||
            (docs->prefix_len > 0 && prefix_layer_stride < docs->prefix_len * row) || (q_layer_stride * esize) % 16 ||
            (out_layer_stride * esize) % 16 || (kv_layer_stride * esize) % 16 || (prefix_layer_stride * esize) % 16)
            return CF_ERR_INVALID_ARG;
    }
    DocAttnArgs a;
    a.n_docs = docs->n_docs;
    a.n_layers = n_layers;
    a.max_doc_len = docs->max_doc_len;
    a.prefix_len = docs->prefix_len;
    a.n_q_heads = geom->n_q_heads;
    a.n_kv_heads = geom->n_kv_heads;
    a.total_tokens = docs->total_tokens;
    a.token_stride = docs->token_stride;
    a.q_layer_stride = q_layer_stride;
    a.kv_layer_stride = kv_layer_stride;
    a.prefix_layer_stride = prefix_layer_stride;
    a.out_layer_stride = out_layer_stride;
    a.doc_offsets = docs->doc_offsets;
    a.scale_log2 = (softmax_scale == 0.0f ? 1.0f / std::sqrt((float)geom->head_dim) : softmax_scale) * kLog2e;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (attn_path() == 0 && docattn_tc_supported(geom, docs))
        return launch_docattn_tc(geom, a, q, k, v, k_prefix, v_prefix, out, lse, status, s);
    return launch_docattn_simt(geom, a, q, k, v, k_prefix, v_prefix, out, lse, s);
}
