// The causal block of the query tokens over their own keys and values (footnote to Eq. 1;
// Algorithm 2, "layer_l" beyond the cached documents): row j of the query sees query tokens 0..j.
// It is a few MFLOP per layer, so it runs on the CUDA cores: one warp per query row, lanes over the
// keys for the logits and over the head dimension for the weighted values.  The result is left in
// the workspace as one more part of the split-KV decomposition (reference maximum, sum,
// unnormalised row), which the merge kernel folds into the output after the documents' parts.
#include "cf_common.cuh"

namespace cf {

namespace {

constexpr int kSelfThreads = 256;
constexpr int kSelfRows = 32;          // query rows per block: four per warp
constexpr int kSelfMaxLq = 128;

// Bytes of the padded key rows in shared memory, rounded up so that the value rows behind them can be
// written with 16-byte stores.
template <typename T, int D>
__host__ __device__ constexpr size_t self_keys_bytes(int lq) {
    return ((size_t)lq * (D + 2) * sizeof(T) + 15) / 16 * 16;
}

template <typename T, int D>
__global__ void __launch_bounds__(kSelfThreads)
self_block_kernel(AttnWorkspace ws, LayerSpan span, long long self_stride, int n_requests, int n_q_heads,
                  int n_kv_heads, int lq, float scale_log2, const T* __restrict__ q,
                  const T* __restrict__ k_self, const T* __restrict__ v_self) {
    extern __shared__ __align__(16) unsigned char self_smem[];
    constexpr int kPitch = D + 2;                                   // odd number of 32-bit words per key row: no bank conflicts
    T* Ks = reinterpret_cast<T*>(self_smem);                        // [lq][kPitch]
    T* Vs = reinterpret_cast<T*>(self_smem + self_keys_bytes<T, D>(lq));   // [lq][D], 16-byte aligned
    float* Qs = reinterpret_cast<float*>(Vs + (size_t)lq * D);      // [warps][D]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int group = n_q_heads / n_kv_heads;
    const int rows = group * lq;                                    // rows that share this kv head
    const int kvh = blockIdx.y;
    const int lb = blockIdx.z;                                      // layer * B + request
    const int layer = lb / n_requests, b = lb - layer * n_requests;
    const int rows_total = n_q_heads * lq;
    q += (size_t)layer * span.q_stride;
    k_self += (size_t)layer * self_stride + (size_t)b * lq * n_kv_heads * D;
    v_self += (size_t)layer * self_stride + (size_t)b * lq * n_kv_heads * D;

    // 16-byte loads; the padded key rows are only 4-byte aligned, so they are stored word by word
    constexpr int kVec = 16 / (int)sizeof(T), kWords = 4;           // elements and 32-bit words per vector
    for (int idx = tid; idx < lq * (D / kVec); idx += kSelfThreads) {
        const int t = idx / (D / kVec), c = idx - t * (D / kVec);
        const size_t src = ((size_t)t * n_kv_heads + kvh) * D + c * kVec;
        const uint4 kq = *reinterpret_cast<const uint4*>(k_self + src);
        const uint4 vq = *reinterpret_cast<const uint4*>(v_self + src);
        uint32_t* kd = reinterpret_cast<uint32_t*>(Ks + (size_t)t * kPitch + c * kVec);
        kd[0] = kq.x; kd[1] = kq.y; kd[kWords - 2] = kq.z; kd[kWords - 1] = kq.w;
        *reinterpret_cast<uint4*>(Vs + (size_t)t * D + c * kVec) = vq;
    }
    __syncthreads();

    float* qrow = Qs + warp * D;
    for (int rr = warp; rr < kSelfRows; rr += kSelfThreads / 32) {
        const int row = blockIdx.x * kSelfRows + rr;                // row among those of this kv head
        if (row >= rows) break;
        const int g = row / lq, j = row - g * lq;
        const int h = kvh * group + g;
        __syncwarp();
        for (int d = lane; d < D; d += 32) qrow[d] = to_float(q[(((size_t)b * lq + j) * n_q_heads + h) * D + d]);
        __syncwarp();
        // logits of keys lane, lane + 32, ... (at most four per lane)
        float s[kSelfMaxLq / 32];
        float m = -INFINITY;
#pragma unroll
        for (int c = 0; c < kSelfMaxLq / 32; ++c) {
            const int t = lane + 32 * c;
            s[c] = -INFINITY;
            if (t <= j) {
                float acc0 = 0.f, acc1 = 0.f;
                const T* kr = Ks + (size_t)t * kPitch;
#pragma unroll 8
                for (int d = 0; d < D; d += 2) {
                    acc0 = fmaf(qrow[d], to_float(kr[d]), acc0);
                    acc1 = fmaf(qrow[d + 1], to_float(kr[d + 1]), acc1);
                }
                s[c] = (acc0 + acc1) * scale_log2;
            }
            m = fmaxf(m, s[c]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        float l = 0.f;
#pragma unroll
        for (int c = 0; c < kSelfMaxLq / 32; ++c) {
            s[c] = s[c] > -INFINITY ? exp2f(s[c] - m) : 0.f;        // key 0 is always visible, so m is finite
            l += s[c];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
        // weighted values: D / 32 dimensions per lane, keys in order
        constexpr int V = D / 32;
        float o_acc[V];
#pragma unroll
        for (int i = 0; i < V; ++i) o_acc[i] = 0.f;
#pragma unroll
        for (int c = 0; c < kSelfMaxLq / 32; ++c) {
            if (32 * c > j) break;
            const int n = min(32, j + 1 - 32 * c);
            for (int u = 0; u < n; ++u) {
                const float p = __shfl_sync(0xffffffffu, s[c], u);
                const T* vr = Vs + (size_t)(32 * c + u) * D + lane * V;
#pragma unroll
                for (int i = 0; i < V; ++i) o_acc[i] = fmaf(p, to_float(vr[i]), o_acc[i]);
            }
        }
        const size_t slot = (size_t)lb * rows_total + (size_t)kvh * rows + row;
#pragma unroll
        for (int i = 0; i < V; ++i) ws.self_o[slot * D + lane * V + i] = o_acc[i];
        if (lane == 0) {
            ws.self_m[slot] = m;
            ws.self_l[slot] = l;
        }
    }
}

template <typename T, int D>
int launch_self_typed(const cf_geom* g, const cf_batch* b, const LayerSpan& span, long long self_stride,
                      const void* q, const void* k_self, const void* v_self, float scale_log2,
                      const AttnWorkspace& ws, cudaStream_t stream) {
    const int rows = (g->n_q_heads / g->n_kv_heads) * b->q_len;
    const size_t smem = self_keys_bytes<T, D>(b->q_len) + (size_t)b->q_len * D * sizeof(T) +
                        (size_t)(kSelfThreads / 32) * D * sizeof(float);
    static PerDeviceOnce configured;
    if (configure_smem_once(configured, self_block_kernel<T, D>,
                            (int)(self_keys_bytes<T, D>(kSelfMaxLq) + (size_t)kSelfMaxLq * D * sizeof(T) +
                                  (kSelfThreads / 32) * D * sizeof(float))) != CF_OK)
        return CF_ERR_CUDA;
    dim3 grid((unsigned)((rows + kSelfRows - 1) / kSelfRows), (unsigned)g->n_kv_heads,
              (unsigned)(b->n_requests * span.n_layers));
    self_block_kernel<T, D><<<grid, kSelfThreads, smem, stream>>>(
        ws, span, self_stride, b->n_requests, g->n_q_heads, g->n_kv_heads, b->q_len, scale_log2,
        static_cast<const T*>(q), static_cast<const T*>(k_self), static_cast<const T*>(v_self));
    return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

}  // namespace

int launch_self_block(const cf_geom* g, const cf_batch* b, const LayerSpan& span, long long self_stride,
                      const void* q, const void* k_self, const void* v_self, float scale_log2,
                      const AttnWorkspace& ws, cudaStream_t stream) {
    if (b->q_len > kSelfMaxLq) return CF_ERR_UNSUPPORTED;
    if ((long long)b->n_requests * span.n_layers > 65535 || g->n_kv_heads > 65535) return CF_ERR_INVALID_ARG;
    if (g->dtype == CF_BF16)
        return g->head_dim == 128
                   ? launch_self_typed<__nv_bfloat16, 128>(g, b, span, self_stride, q, k_self, v_self, scale_log2, ws, stream)
                   : launch_self_typed<__nv_bfloat16, 64>(g, b, span, self_stride, q, k_self, v_self, scale_log2, ws, stream);
    return g->head_dim == 128
               ? launch_self_typed<float, 128>(g, b, span, self_stride, q, k_self, v_self, scale_log2, ws, stream)
               : launch_self_typed<float, 64>(g, b, span, self_stride, q, k_self, v_self, scale_log2, ws, stream);
}

}  // namespace cf
