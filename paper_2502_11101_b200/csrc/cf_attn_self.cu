// The key blocks besides the documents on the CUDA-core path: a shared prefix cache (Sec. 2.2: every query row sees
// all of it) and the causal block of the query tokens over their own keys and values (footnote to Eq. 1;
// Algorithm 2, "layer_l" beyond the cached documents: row j of the query sees query tokens 0..j).
// They are a few MFLOP per layer, so they run on the CUDA cores: one warp per query row, lanes over the
// keys for the logits and over the head dimension for the weighted values, the keys in chunks of 128 with a
// running maximum and sum.  The result is left in the workspace as one more part of the split-KV decomposition
// (reference maximum, sum, unnormalised row), which the merge kernel folds into the output after the documents' parts.
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

// Where the keys of the block come from: first the rows of a shared prefix cache (every query row sees them), then
// the query tokens' own rows (row j sees tokens 0..j).  Either may be absent.
struct ExtraKeys {
    const void* k_prefix;
    const void* v_prefix;
    long long prefix_stride;      // elements between layers of the prefix tensors
    int prefix_len;
    const void* k_self;
    const void* v_self;
    long long self_stride;
};

template <typename T, int D>
__global__ void __launch_bounds__(kSelfThreads)
self_block_kernel(AttnWorkspace ws, LayerSpan span, ExtraKeys ek, int n_requests, int n_q_heads, int n_kv_heads, int lq,
                  float scale_log2, const T* __restrict__ q) {
    extern __shared__ __align__(16) unsigned char self_smem[];
    constexpr int kPitch = D + 2;                                   // odd number of 32-bit words per key row: no bank conflicts
    T* Ks = reinterpret_cast<T*>(self_smem);                        // [kSelfMaxLq][kPitch]
    T* Vs = reinterpret_cast<T*>(self_smem + self_keys_bytes<T, D>(kSelfMaxLq));   // [kSelfMaxLq][D], 16-byte aligned
    float* Qs = reinterpret_cast<float*>(Vs + (size_t)kSelfMaxLq * D);             // [warps][D]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int group = n_q_heads / n_kv_heads;
    const int rows = group * lq;                                    // rows that share this kv head
    const int kvh = blockIdx.y;
    const int lb = blockIdx.z;                                      // layer * B + request
    const int layer = lb / n_requests, b = lb - layer * n_requests;
    const int rows_total = n_q_heads * lq;
    q += (size_t)layer * span.q_stride;
    const bool with_self = ek.k_self != nullptr;
    const int n_prefix_chunks = (ek.prefix_len + kSelfMaxLq - 1) / kSelfMaxLq;
    const int n_chunks = n_prefix_chunks + (with_self ? 1 : 0);

    // this warp's rows (four of the block's 32) keep a running maximum, sum and unnormalised output across the chunks
    constexpr int kRowsPerWarp = kSelfRows / (kSelfThreads / 32);
    constexpr int V = D / 32;
    float m_run[kRowsPerWarp], l_run[kRowsPerWarp], o_acc[kRowsPerWarp][V];
#pragma unroll
    for (int x = 0; x < kRowsPerWarp; ++x) {
        m_run[x] = -INFINITY;
        l_run[x] = 0.f;
#pragma unroll
        for (int i = 0; i < V; ++i) o_acc[x][i] = 0.f;
    }

    for (int c = 0; c < n_chunks; ++c) {
        const bool self_chunk = c == n_prefix_chunks;
        const int first = self_chunk ? 0 : c * kSelfMaxLq;          // first key row of the chunk in its tensor
        const int n_keys = self_chunk ? lq : min(kSelfMaxLq, ek.prefix_len - first);
        const T* k_src = self_chunk ? static_cast<const T*>(ek.k_self) + (size_t)layer * ek.self_stride + (size_t)b * lq * n_kv_heads * D
                                    : static_cast<const T*>(ek.k_prefix) + (size_t)layer * ek.prefix_stride + (size_t)first * n_kv_heads * D;
        const T* v_src = self_chunk ? static_cast<const T*>(ek.v_self) + (size_t)layer * ek.self_stride + (size_t)b * lq * n_kv_heads * D
                                    : static_cast<const T*>(ek.v_prefix) + (size_t)layer * ek.prefix_stride + (size_t)first * n_kv_heads * D;
        __syncthreads();                                            // the previous chunk has been consumed
        // 16-byte loads; the padded key rows are only 4-byte aligned, so they are stored word by word
        constexpr int kVec = 16 / (int)sizeof(T), kWords = 4;       // elements and 32-bit words per vector
        for (int idx = tid; idx < n_keys * (D / kVec); idx += kSelfThreads) {
            const int t = idx / (D / kVec), cc = idx - t * (D / kVec);
            const size_t src = ((size_t)t * n_kv_heads + kvh) * D + cc * kVec;
            const uint4 kq = *reinterpret_cast<const uint4*>(k_src + src);
            const uint4 vq = *reinterpret_cast<const uint4*>(v_src + src);
            uint32_t* kd = reinterpret_cast<uint32_t*>(Ks + (size_t)t * kPitch + cc * kVec);
            kd[0] = kq.x; kd[1] = kq.y; kd[kWords - 2] = kq.z; kd[kWords - 1] = kq.w;
            *reinterpret_cast<uint4*>(Vs + (size_t)t * D + cc * kVec) = vq;
        }
        __syncthreads();

        float* qrow = Qs + warp * D;
#pragma unroll
        for (int x = 0; x < kRowsPerWarp; ++x) {
            const int row = blockIdx.x * kSelfRows + warp + x * (kSelfThreads / 32);   // row among those of this kv head
            if (row >= rows) break;
            const int g = row / lq, j = row - g * lq;
            const int h = kvh * group + g;
            const int last = self_chunk ? j : n_keys - 1;           // last visible key of the chunk (causal mask of the self block)
            __syncwarp();
            for (int d = lane; d < D; d += 32) qrow[d] = to_float(q[(((size_t)b * lq + j) * n_q_heads + h) * D + d]);
            __syncwarp();
            // logits of keys lane, lane + 32, ... (at most four per lane)
            float sc[kSelfMaxLq / 32];
            float cmax = -INFINITY;
#pragma unroll
            for (int u = 0; u < kSelfMaxLq / 32; ++u) {
                const int t = lane + 32 * u;
                sc[u] = -INFINITY;
                if (t <= last) {
                    float acc0 = 0.f, acc1 = 0.f;
                    const T* kr = Ks + (size_t)t * kPitch;
#pragma unroll 8
                    for (int d = 0; d < D; d += 2) {
                        acc0 = fmaf(qrow[d], to_float(kr[d]), acc0);
                        acc1 = fmaf(qrow[d + 1], to_float(kr[d + 1]), acc1);
                    }
                    sc[u] = (acc0 + acc1) * scale_log2;
                }
                cmax = fmaxf(cmax, sc[u]);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, o));
            const float m_new = fmaxf(m_run[x], cmax);              // key 0 of a chunk is always visible: finite
            const float alpha = exp2f(m_run[x] - m_new);            // first chunk: 0
            float lsum = 0.f;
#pragma unroll
            for (int u = 0; u < kSelfMaxLq / 32; ++u) {
                sc[u] = sc[u] > -INFINITY ? exp2f(sc[u] - m_new) : 0.f;
                lsum += sc[u];
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
            l_run[x] = fmaf(l_run[x], alpha, lsum);
            m_run[x] = m_new;
            // weighted values: D / 32 dimensions per lane, keys in order
#pragma unroll
            for (int i = 0; i < V; ++i) o_acc[x][i] *= alpha;
#pragma unroll
            for (int u = 0; u < kSelfMaxLq / 32; ++u) {
                if (32 * u > last) break;
                const int n = min(32, last + 1 - 32 * u);
                for (int k = 0; k < n; ++k) {
                    const float p = __shfl_sync(0xffffffffu, sc[u], k);
                    const T* vr = Vs + (size_t)(32 * u + k) * D + lane * V;
#pragma unroll
                    for (int i = 0; i < V; ++i) o_acc[x][i] = fmaf(p, to_float(vr[i]), o_acc[x][i]);
                }
            }
        }
    }
#pragma unroll
    for (int x = 0; x < kRowsPerWarp; ++x) {
        const int row = blockIdx.x * kSelfRows + warp + x * (kSelfThreads / 32);
        if (row >= rows) break;
        const size_t slot = (size_t)lb * rows_total + (size_t)kvh * rows + row;
#pragma unroll
        for (int i = 0; i < V; ++i) ws.self_o[slot * D + lane * V + i] = o_acc[x][i];
        if (lane == 0) {
            ws.self_m[slot] = m_run[x];
            ws.self_l[slot] = l_run[x];
        }
    }
}

template <typename T, int D>
int launch_self_typed(const cf_geom* g, const cf_batch* b, const LayerSpan& span, const ExtraKeys& ek, const void* q,
                      float scale_log2, const AttnWorkspace& ws, cudaStream_t stream) {
    const int rows = (g->n_q_heads / g->n_kv_heads) * b->q_len;
    const size_t smem = self_keys_bytes<T, D>(kSelfMaxLq) + (size_t)kSelfMaxLq * D * sizeof(T) +
                        (size_t)(kSelfThreads / 32) * D * sizeof(float);
    static PerDeviceOnce configured;
    if (configure_smem_once(configured, self_block_kernel<T, D>, (int)smem) != CF_OK) return CF_ERR_CUDA;
    dim3 grid((unsigned)((rows + kSelfRows - 1) / kSelfRows), (unsigned)g->n_kv_heads,
              (unsigned)(b->n_requests * span.n_layers));
    self_block_kernel<T, D><<<grid, kSelfThreads, smem, stream>>>(ws, span, ek, b->n_requests, g->n_q_heads, g->n_kv_heads,
                                                                 b->q_len, scale_log2, static_cast<const T*>(q));
    return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

}  // namespace

int launch_self_block(const cf_geom* g, const cf_batch* b, const LayerSpan& span, long long self_stride,
                      const void* q, const void* k_self, const void* v_self, const void* k_prefix, const void* v_prefix,
                      long long prefix_stride, int prefix_len, float scale_log2, const AttnWorkspace& ws,
                      cudaStream_t stream) {
    if (k_self && b->q_len > kSelfMaxLq) return CF_ERR_UNSUPPORTED;
    if (!k_self && prefix_len <= 0) return CF_ERR_INVALID_ARG;
    if ((long long)b->n_requests * span.n_layers > 65535 || g->n_kv_heads > 65535) return CF_ERR_INVALID_ARG;
    const ExtraKeys ek = {k_prefix, v_prefix, prefix_stride, prefix_len > 0 ? prefix_len : 0, k_self, v_self, self_stride};
    if (g->dtype == CF_BF16)
        return g->head_dim == 128 ? launch_self_typed<__nv_bfloat16, 128>(g, b, span, ek, q, scale_log2, ws, stream)
                                  : launch_self_typed<__nv_bfloat16, 64>(g, b, span, ek, q, scale_log2, ws, stream);
    return g->head_dim == 128 ? launch_self_typed<float, 128>(g, b, span, ek, q, scale_log2, ws, stream)
                              : launch_self_typed<float, 64>(g, b, span, ek, q, scale_log2, ws, stream);
}

}  // namespace cf
