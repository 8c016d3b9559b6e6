// Portable CUDA-core version of the fused re-position + query-prefill attention (Eq. 5 fused
// into Eq. 1), and the kernels that merge split partials and reduce document scores.  This
// kernel serves the geometries the tensor-core kernel does not cover (fp32 storage, head_dim
// 64) and is the second implementation the tensor-core kernel is checked against.
#include <algorithm>
#include <type_traits>

#include "cf_common.cuh"

namespace cf {

constexpr int kSimtThreads = 256;
constexpr int kSimtRows = 64;     // query rows per CTA
constexpr int kSimtSub = 32;      // key rows per inner step

template <int D>
constexpr size_t simt_smem_bytes() {
    return sizeof(float) * (size_t)(kSimtRows * (D + 1) + kSimtSub * (D + 1) + kSimtSub * D +
                                    kSimtRows * (kSimtSub + 1));
}

template <typename T, int D, int LAYOUT>
__global__ void __launch_bounds__(kSimtThreads)
attn_simt_kernel(BatchView bv, PlanView pv, AttnWorkspace ws, LayerSpan span, int n_q_heads, int n_kv_heads,
                 float scale_log2, const T* __restrict__ q, const T* __restrict__ k_cache,
                 const T* __restrict__ v_cache) {
    extern __shared__ float smem[];
    float (*Qs)[D + 1] = reinterpret_cast<float (*)[D + 1]>(smem);
    float (*Ks)[D + 1] = reinterpret_cast<float (*)[D + 1]>(smem + kSimtRows * (D + 1));
    float (*Vs)[D] = reinterpret_cast<float (*)[D]>(smem + (kSimtRows + kSimtSub) * (D + 1));
    float (*Ps)[kSimtSub + 1] =
        reinterpret_cast<float (*)[kSimtSub + 1]>(smem + (kSimtRows + kSimtSub) * (D + 1) + kSimtSub * D);

    const int tid = threadIdx.x;
    const int group = n_q_heads / n_kv_heads;
    const int lq = bv.q_len;
    const int rows = group * lq;                                   // query rows sharing one kv head
    const int row_chunks = (rows + kSimtRows - 1) / kSimtRows;
    const int lb = blockIdx.z;                                     // layer * B + request
    const int layer = lb / bv.n_requests;
    const int b = lb - layer * bv.n_requests;
    q += (size_t)layer * span.q_stride;
    k_cache += (size_t)layer * span.kv_stride;
    v_cache += (size_t)layer * span.kv_stride;
    const int kvh = blockIdx.y / row_chunks;
    const int r0 = (blockIdx.y - kvh * row_chunks) * kSimtRows;
    const int n_rows = min(kSimtRows, rows - r0);
    const int split = blockIdx.x;
    const int rows_total = n_q_heads * lq;

    for (int idx = tid; idx < kSimtRows * D; idx += kSimtThreads) {
        const int rr = idx / D, d = idx - rr * D;
        float val = 0.f;
        if (rr < n_rows) {
            const int row = r0 + rr;
            const int g = row / lq, j = row - g * lq;
            const int h = kvh * group + g;
            val = to_float(q[(((size_t)b * lq + j) * n_q_heads + h) * D + d]);
        }
        Qs[rr][d] = val;
    }

    const int doc0 = bv.req_doc_begin[b];
    const int base = tile_base(doc0, bv.doc_offsets[doc0]);
    const int n_tiles = pv.n_tiles[b];
    const int t_begin = (int)((long long)n_tiles * split / ws.n_splits);
    const int t_end = (int)((long long)n_tiles * (split + 1) / ws.n_splits);

    const int r = tid >> 2, q4 = tid & 3;
    float m = -INFINITY, l = 0.f;
    float acc[D / 4];
#pragma unroll
    for (int k = 0; k < D / 4; ++k) acc[k] = 0.f;
    const size_t row_global = (size_t)kvh * rows + r0 + r;

    for (int ti = t_begin; ti < t_end; ++ti) {
        const int doc = pv.tile_doc[base + ti];
        const long long row0 = pv.tile_row0[base + ti];
        const int len = pv.tile_len[base + ti];
        const float2* trig = pv.trig + (size_t)doc * (D / 2);
        float l_tile = 0.f;
        for (int sub = 0; sub < len; sub += kSimtSub) {
            const int n = min(kSimtSub, len - sub);
            __syncthreads();
            // keys: rotate each slice by the document's delta (Eq. 5), round to the storage type
            for (int idx = tid; idx < kSimtSub * (D / 2); idx += kSimtThreads) {
                const int t = idx / (D / 2), p = idx - t * (D / 2);
                const int ia = LAYOUT == CF_ROPE_HALF ? p : 2 * p;
                const int ib = LAYOUT == CF_ROPE_HALF ? p + D / 2 : 2 * p + 1;
                float ya = 0.f, yb = 0.f;
                if (t < n) {
                    const T* src = k_cache + (row0 + sub + t) * bv.token_stride + (size_t)kvh * D;
                    const float2 cs = trig[p];
                    rotate_pair(to_float(src[ia]), to_float(src[ib]), cs.x, cs.y, ya, yb);
                    ya = to_float(from_float<T>(ya));
                    yb = to_float(from_float<T>(yb));
                }
                Ks[t][ia] = ya;
                Ks[t][ib] = yb;
            }
            for (int idx = tid; idx < kSimtSub * D; idx += kSimtThreads) {
                const int t = idx / D, d = idx - t * D;
                Vs[t][d] = t < n ? to_float(v_cache[(row0 + sub + t) * bv.token_stride + (size_t)kvh * D + d]) : 0.f;
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
            float sub_max = -INFINITY;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                sc[i] = (q4 * 8 + i < n) ? sc[i] * scale_log2 : -INFINITY;
                sub_max = fmaxf(sub_max, sc[i]);
            }
            sub_max = fmaxf(sub_max, __shfl_xor_sync(0xffffffffu, sub_max, 1));
            sub_max = fmaxf(sub_max, __shfl_xor_sync(0xffffffffu, sub_max, 2));
            const float m_new = fmaxf(m, sub_max);
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
            l_tile = fmaf(l_tile, alpha, sub_sum);
            m = m_new;
#pragma unroll
            for (int k = 0; k < D / 4; ++k) acc[k] *= alpha;
            __syncwarp();
            for (int t = 0; t < kSimtSub; ++t) {
                const float pr = Ps[r][t];
#pragma unroll
                for (int k = 0; k < D / 4; ++k) acc[k] = fmaf(pr, Vs[t][4 * k + q4], acc[k]);
            }
        }
        if (q4 == 0 && r < n_rows)
            ws.tile_lse2[((size_t)layer * ws.max_tiles + base + ti) * rows_total + row_global] = m + log2f(l_tile);
    }
    if (r < n_rows) {
        const size_t slot = ((size_t)lb * ws.n_splits + split) * rows_total + row_global;
        if (q4 == 0) {
            ws.part_m[slot] = m;
            ws.part_l[slot] = l;
        }
#pragma unroll
        for (int k = 0; k < D / 4; ++k) ws.part_o[slot * D + 4 * k + q4] = acc[k];
    }
}

// D/32 consecutive elements of a partial O row (fp32 or bf16) as floats.
template <int V>
__device__ __forceinline__ void load_part(const float* p, float (&x)[V]) {
    if (V == 4) {
        const float4 t = *reinterpret_cast<const float4*>(p);
        x[0] = t.x; x[1] = t.y; x[V - 2] = t.z; x[V - 1] = t.w;
    } else {
        const float2 t = *reinterpret_cast<const float2*>(p);
        x[0] = t.x; x[1] = t.y;
    }
}
template <int V>
__device__ __forceinline__ void load_part(const __nv_bfloat16* p, float (&x)[V]) {
    if (V == 4) {
        const uint2 t = *reinterpret_cast<const uint2*>(p);
        x[0] = __uint_as_float(t.x << 16); x[1] = __uint_as_float(t.x & 0xffff0000u);
        x[V - 2] = __uint_as_float(t.y << 16); x[V - 1] = __uint_as_float(t.y & 0xffff0000u);
    } else {
        const uint32_t t = *reinterpret_cast<const uint32_t*>(p);
        x[0] = __uint_as_float(t << 16); x[1] = __uint_as_float(t & 0xffff0000u);
    }
}
template <int V>
__device__ __forceinline__ void store_row(float* p, const float (&x)[V]) {
#pragma unroll
    for (int i = 0; i < V; ++i) p[i] = x[i];
}
template <int V>
__device__ __forceinline__ void store_row(__nv_bfloat16* p, const float (&x)[V]) {
#pragma unroll
    for (int i = 0; i < V; i += 2)
        *reinterpret_cast<__nv_bfloat162*>(p + i) = __floats2bfloat162_rn(x[i], x[i + 1]);
}

constexpr int kCombineRows = 4;       // query rows (warps) per block of the merge kernel
constexpr int kCombineDepth = 8;      // parts whose loads are in flight together

// Merge the parts of one query row (one warp per row, D/32 output dimensions per lane):
// out = sum_p w_p O_p / sum_p w_p l_p with w_p = 2^(m_p - max m), and the row's log-sum-exp.
// Parts are visited in index order and the warp reductions have a fixed shape, so the result does
// not depend on scheduling.
template <typename T, int D, typename P>
__global__ void __launch_bounds__(32 * kCombineRows)
combine_kernel(AttnWorkspace ws, int n_requests, long long n_rows_all, long long out_layer_stride, int n_q_heads,
               int lq, T* __restrict__ out, float* __restrict__ lse) {
    constexpr int V = D / 32;
    static_assert(CF_MAX_SPLITS <= 64, "two parts per lane");
    const int lane = threadIdx.x & 31;
    const long long row_all = (long long)blockIdx.x * kCombineRows + (threadIdx.x >> 5);
    if (row_all >= n_rows_all) return;
    const int rows_total = n_q_heads * lq;
    const int lb = (int)(row_all / rows_total), rg = (int)(row_all - (long long)lb * rows_total);   // lb = layer * B + request
    const int layer = lb / n_requests, b = lb - layer * n_requests;
    const int h = rg / lq, j = rg - h * lq;
    const int n_parts = ws.n_splits;
    const size_t slot0 = (size_t)lb * n_parts * rows_total + rg;      // part p sits at slot0 + p * rows_total

    float m[2], l[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int p = lane + 32 * k;
        m[k] = p < n_parts ? ws.part_m[slot0 + (size_t)p * rows_total] : -INFINITY;
        l[k] = m[k] > -INFINITY ? ws.part_l[slot0 + (size_t)p * rows_total] : 0.f;
    }
    float m_max = fmaxf(m[0], m[1]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m_max = fmaxf(m_max, __shfl_xor_sync(0xffffffffu, m_max, o));
    float w[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) w[k] = m[k] > -INFINITY ? exp2f(m[k] - m_max) : 0.f;
    float l_sum = fmaf(l[1], w[1], l[0] * w[0]);                      // fixed-shape tree: deterministic
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l_sum += __shfl_xor_sync(0xffffffffu, l_sum, o);

    float acc[V];
#pragma unroll
    for (int i = 0; i < V; ++i) acc[i] = 0.f;
    const P* po = reinterpret_cast<const P*>(ws.part_o) + slot0 * D + lane * V;
    const size_t stride = (size_t)rows_total * D;
    for (int p0 = 0; p0 < n_parts; p0 += kCombineDepth) {             // independent loads in flight
        float wp[kCombineDepth], x[kCombineDepth][V];
#pragma unroll
        for (int u = 0; u < kCombineDepth; ++u) {
            const int p = p0 + u;
            wp[u] = __shfl_sync(0xffffffffu, (p & 32) ? w[1] : w[0], p & 31);
            if (p >= n_parts) wp[u] = 0.f;
            if (wp[u] > 0.f) load_part<V>(po + (size_t)p * stride, x[u]);
        }
#pragma unroll
        for (int u = 0; u < kCombineDepth; ++u)
            if (wp[u] > 0.f) {
#pragma unroll
                for (int i = 0; i < V; ++i) acc[i] = fmaf(x[u][i], wp[u], acc[i]);
            }
    }
    // the documents' share of the row: what the document scores are measured against
    float docs_l = l_sum;
    if (ws.self_mode == 2) {
        // further key blocks were tiles of some parts: every part reports its sum over the documents alone
        float ld[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int p = lane + 32 * k;
            ld[k] = (p < n_parts && m[k] > -INFINITY) ? ws.part_ld[slot0 + (size_t)p * rows_total] : 0.f;
        }
        docs_l = fmaf(ld[1], w[1], ld[0] * w[0]);                       // same tree as l_sum, no subtraction
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) docs_l += __shfl_xor_sync(0xffffffffu, docs_l, o);
    }
    const float docs_lse2 = docs_l > 0.f ? m_max + log2f(docs_l) : -INFINITY;
    float m_all = m_max, l_all = l_sum;
    if (ws.self_mode == 1) {                                           // the query-self block joins as one more part
        const size_t srow = (size_t)lb * rows_total + rg;
        const float ms = ws.self_m[srow], ls = ws.self_l[srow];
        float xs[V];
        load_part<V>(ws.self_o + srow * D + lane * V, xs);
        m_all = fmaxf(m_max, ms);
        const float wd = l_sum > 0.f ? exp2f(m_max - m_all) : 0.f, wsf = exp2f(ms - m_all);
#pragma unroll
        for (int i = 0; i < V; ++i) acc[i] = fmaf(xs[i], wsf, acc[i] * wd);
        l_all = fmaf(ls, wsf, l_sum * wd);
    }
    const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
#pragma unroll
    for (int i = 0; i < V; ++i) acc[i] *= inv;
    store_row<V>(out + (size_t)layer * out_layer_stride + (((size_t)b * lq + j) * n_q_heads + h) * D + lane * V, acc);
    if (lane == 0) {
        ws.row_lse2[(size_t)lb * rows_total + rg] = docs_lse2;
        if (lse) lse[(size_t)lb * rows_total + rg] = (l_all > 0.f ? m_all + log2f(l_all) : -INFINITY) * kLn2;
    }
}

constexpr int kScoreThreads = 1024;

// Document scores (footnote of Sec. 2.4; Algorithm 2: S <- S + s^l): one block per document sums
// 2^(tile_lse - row_lse) over the document's tiles and all query rows of every layer of the call,
// each layer in a fixed order, then adds the layers' scores to S in layer order.  Up to eight
// layers are reduced side by side by groups of threads.
__global__ void __launch_bounds__(kScoreThreads)
score_kernel(BatchView bv, PlanView pv, AttnWorkspace ws, int rows_total, float* __restrict__ doc_scores,
             float* __restrict__ score_accum) {
    __shared__ float s_red[kScoreThreads / 32];
    __shared__ float s_layer[CF_MAX_LAYERS_PER_CALL];
    const int doc = blockIdx.x;
    const int n_layers = ws.n_layers;
    const int count = pv.doc_tile_count[doc];
    if (count == 0) {
        if (doc_scores)
            for (int l = threadIdx.x; l < n_layers; l += kScoreThreads) doc_scores[(size_t)l * bv.n_docs_total + doc] = 0.f;
        return;
    }
    int lo = 0, hi = bv.n_requests;                 // request that owns the document
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (bv.req_doc_begin[mid] <= doc) lo = mid; else hi = mid;
    }
    int groups = 1;                                 // power of two, at most min(n_layers, 8)
    while (groups * 2 <= n_layers && groups < 8) groups *= 2;
    const int gs = kScoreThreads / groups;          // threads per group, a multiple of 128
    const int g = threadIdx.x / gs, t = threadIdx.x - g * gs;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int warps_per_group = gs >> 5;
    const int rounds = (n_layers + groups - 1) / groups;
    const size_t tile0 = (size_t)pv.doc_tile_begin[doc];
    const int n = count * rows_total;
    for (int rd = 0; rd < rounds; ++rd) {
        const int layer = rd * groups + g;
        float sum = 0.f;
        if (layer < n_layers) {
            const float* __restrict__ row_lse2 = ws.row_lse2 + ((size_t)layer * bv.n_requests + lo) * rows_total;
            const float* __restrict__ tile_lse2 = ws.tile_lse2 + ((size_t)layer * ws.max_tiles + tile0) * rows_total;
#pragma unroll 4
            for (int idx = t; idx < n; idx += gs) sum += exp2f(tile_lse2[idx] - row_lse2[idx % rows_total]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) s_red[warp] = sum;
        __syncthreads();
        if (t == 0 && layer < n_layers) {
            float total = 0.f;
            for (int k = 0; k < warps_per_group; ++k) total += s_red[g * warps_per_group + k];
            s_layer[layer] = total / (float)rows_total;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        float acc = score_accum ? score_accum[doc] : 0.f;
        for (int l = 0; l < n_layers; ++l) {
            if (doc_scores) doc_scores[(size_t)l * bv.n_docs_total + doc] = s_layer[l];
            acc += s_layer[l];
        }
        if (score_accum) score_accum[doc] = acc;
    }
}

// Softmax attention over the union of two disjoint key sets from the results over each set:
// one warp per (block, query token, head); weights 2^(lse - max) so nothing overflows.
template <typename T, int D>
__global__ void __launch_bounds__(256)
merge_attn_kernel(long long n_rows, int n_q_heads, int lq, const T* out_a, const float* lse_a,
                  const T* out_b, const float* lse_b, T* out, float* lse) {   // out may alias out_a or out_b, lse likewise
    constexpr int V = D / 32;
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);     // index into out: (block, token, head)
    if (row >= n_rows) return;
    const long long blk = row / ((long long)lq * n_q_heads);
    const int rem = (int)(row - blk * lq * n_q_heads);
    const int j = rem / n_q_heads, h = rem - j * n_q_heads;
    const long long li = (blk * n_q_heads + h) * lq + j;                      // index into lse: (block, head, token)
    const float la = lse_a[li], lb = lse_b[li];
    const float m = fmaxf(la, lb);
    const float wa = la > -INFINITY ? expf(la - m) : 0.f, wb = lb > -INFINITY ? expf(lb - m) : 0.f;
    const float inv = wa + wb > 0.f ? 1.f / (wa + wb) : 0.f;
#pragma unroll
    for (int i = 0; i < V; ++i) {
        const long long e = row * D + lane * V + i;
        out[e] = from_float<T>((to_float(out_a[e]) * wa + to_float(out_b[e]) * wb) * inv);
    }
    if (lane == 0 && lse) lse[li] = wa + wb > 0.f ? m + logf(wa + wb) : -INFINITY;
}

int launch_merge_attn(const cf_geom* g, long long n_rows, int q_len, const void* out_a, const float* lse_a,
                      const void* out_b, const float* lse_b, void* out, float* lse, cudaStream_t stream) {
    const long long blocks = (n_rows + 7) / 8;
    if (blocks <= 0 || blocks > 0x7fffffffLL) return CF_ERR_INVALID_ARG;
    auto run = [&](auto kernel, auto* typed) {
        using T = std::remove_pointer_t<decltype(typed)>;
        kernel<<<(unsigned)blocks, 256, 0, stream>>>(n_rows, g->n_q_heads, q_len, static_cast<const T*>(out_a), lse_a,
                                                    static_cast<const T*>(out_b), lse_b, static_cast<T*>(out), lse);
    };
    if (g->dtype == CF_BF16) {
        if (g->head_dim == 128) run(merge_attn_kernel<__nv_bfloat16, 128>, (__nv_bfloat16*)nullptr);
        else run(merge_attn_kernel<__nv_bfloat16, 64>, (__nv_bfloat16*)nullptr);
    } else {
        if (g->head_dim == 128) run(merge_attn_kernel<float, 128>, (float*)nullptr);
        else run(merge_attn_kernel<float, 64>, (float*)nullptr);
    }
    return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

template <typename T, int D>
static int launch_simt_typed(const cf_geom* g, const cf_batch* b, const PlanView& pv, const LayerSpan& span,
                             const void* q, const void* k, const void* v, float scale_log2,
                             const AttnWorkspace& ws, cudaStream_t stream) {
    const int rows = (g->n_q_heads / g->n_kv_heads) * b->q_len;
    const int row_chunks = (rows + kSimtRows - 1) / kSimtRows;
    if ((long long)g->n_kv_heads * row_chunks > 65535 || (long long)b->n_requests * span.n_layers > 65535)
        return CF_ERR_INVALID_ARG;
    dim3 grid((unsigned)ws.n_splits, (unsigned)(g->n_kv_heads * row_chunks), (unsigned)(b->n_requests * span.n_layers));
    BatchView bv = make_batch_view(b);
    const size_t smem = simt_smem_bytes<D>();
    static PerDeviceOnce configured[2];              // per (T, D) instantiation and slice layout
    auto run = [&](auto kernel, int which) {
        if (configure_smem_once(configured[which], kernel, (int)smem) != CF_OK) return CF_ERR_CUDA;
        kernel<<<grid, kSimtThreads, smem, stream>>>(bv, pv, ws, span, g->n_q_heads, g->n_kv_heads, scale_log2,
                                                     static_cast<const T*>(q), static_cast<const T*>(k),
                                                     static_cast<const T*>(v));
        return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
    };
    if (g->rope_layout == CF_ROPE_HALF) return run(attn_simt_kernel<T, D, CF_ROPE_HALF>, 0);
    return run(attn_simt_kernel<T, D, CF_ROPE_INTERLEAVED>, 1);
}

int launch_attn_simt(const cf_geom* g, const cf_batch* b, const PlanView& pv, const LayerSpan& span,
                     const void* q, const void* k, const void* v, float scale_log2,
                     const AttnWorkspace& ws, cudaStream_t stream) {
    if (g->dtype == CF_BF16) {
        if (g->head_dim == 128) return launch_simt_typed<__nv_bfloat16, 128>(g, b, pv, span, q, k, v, scale_log2, ws, stream);
        return launch_simt_typed<__nv_bfloat16, 64>(g, b, pv, span, q, k, v, scale_log2, ws, stream);
    }
    if (g->head_dim == 128) return launch_simt_typed<float, 128>(g, b, pv, span, q, k, v, scale_log2, ws, stream);
    return launch_simt_typed<float, 64>(g, b, pv, span, q, k, v, scale_log2, ws, stream);
}

template <typename T, int D>
static int launch_combine_typed(const cf_geom* g, const cf_batch* b, const LayerSpan& span, const AttnWorkspace& ws,
                                void* out, float* lse, cudaStream_t stream) {
    const long long rows_all = (long long)span.n_layers * b->n_requests * g->n_q_heads * b->q_len;
    const long long blocks = (rows_all + kCombineRows - 1) / kCombineRows;
    if (blocks > 0x7fffffffLL || ws.n_splits > CF_MAX_SPLITS) return CF_ERR_INVALID_ARG;
    if (ws.part_bf16)
        combine_kernel<T, D, __nv_bfloat16><<<(unsigned)blocks, 32 * kCombineRows, 0, stream>>>(
            ws, b->n_requests, rows_all, span.out_stride, g->n_q_heads, b->q_len, static_cast<T*>(out), lse);
    else
        combine_kernel<T, D, float><<<(unsigned)blocks, 32 * kCombineRows, 0, stream>>>(
            ws, b->n_requests, rows_all, span.out_stride, g->n_q_heads, b->q_len, static_cast<T*>(out), lse);
    return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

int launch_combine(const cf_geom* g, const cf_batch* b, const PlanView& pv, const LayerSpan& span,
                   const AttnWorkspace& ws, void* out, float* lse, float* doc_scores, float* score_accum,
                   cudaStream_t stream) {
    int rc;
    if (g->dtype == CF_BF16)
        rc = g->head_dim == 128 ? launch_combine_typed<__nv_bfloat16, 128>(g, b, span, ws, out, lse, stream)
                                : launch_combine_typed<__nv_bfloat16, 64>(g, b, span, ws, out, lse, stream);
    else
        rc = g->head_dim == 128 ? launch_combine_typed<float, 128>(g, b, span, ws, out, lse, stream)
                                : launch_combine_typed<float, 64>(g, b, span, ws, out, lse, stream);
    if (rc != CF_OK) return rc;
    return launch_scores(g, b, pv, ws, doc_scores, score_accum, stream);
}

int launch_scores(const cf_geom* g, const cf_batch* b, const PlanView& pv, const AttnWorkspace& ws, float* doc_scores,
                  float* score_accum, cudaStream_t stream) {
    if (b->n_docs_total > 0 && (doc_scores || score_accum)) {
        score_kernel<<<(unsigned)b->n_docs_total, kScoreThreads, 0, stream>>>(make_batch_view(b), pv, ws,
                                                                   g->n_q_heads * b->q_len, doc_scores,
                                                                   score_accum);
        if (cudaGetLastError() != cudaSuccess) return CF_ERR_CUDA;
    }
    return CF_OK;
}

}  // namespace cf
