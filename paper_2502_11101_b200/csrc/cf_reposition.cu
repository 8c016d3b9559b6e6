// Cache Re-Positioning as a standalone streaming kernel (Eq. 5; Algorithm 2, Phase 2):
// every key row of every kept document is rotated by the document's delta and written back.
// The work is one read and one write of the key store, so the kernel is laid out for HBM:
// 16-byte vectors, each thread owning both halves of a slice group so a row is read once,
// several independent vectors in flight per thread.
#include <algorithm>

#include "cf_common.cuh"

namespace cf {

constexpr int kRepoThreads = 256;
constexpr int kRepoUnroll = 4;

template <typename T> struct Vec16;
template <> struct Vec16<__nv_bfloat16> { static constexpr int kElems = 8; };
template <> struct Vec16<float> { static constexpr int kElems = 4; };

template <typename T>
__device__ __forceinline__ void unpack(const uint4& v, float (&f)[Vec16<T>::kElems]);
template <>
__device__ __forceinline__ void unpack<__nv_bfloat16>(const uint4& v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
template <>
__device__ __forceinline__ void unpack<float>(const uint4& v, float (&f)[4]) {
    f[0] = __uint_as_float(v.x);
    f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z);
    f[3] = __uint_as_float(v.w);
}

template <typename T>
__device__ __forceinline__ uint4 pack(const float (&f)[Vec16<T>::kElems]);
template <>
__device__ __forceinline__ uint4 pack<__nv_bfloat16>(const float (&f)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t*>(&h);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}
template <>
__device__ __forceinline__ uint4 pack<float>(const float (&f)[4]) {
    return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]),
                      __float_as_uint(f[3]));
}

// One work item = one 16-byte vector of the first half of a (row, head) and its partner in the
// second half (HALF layout), or one self-contained vector (INTERLEAVED layout).
template <typename T, int D, int LAYOUT>
__global__ void __launch_bounds__(kRepoThreads)
reposition_kernel(BatchView bv, PlanView pv, int n_kv_heads, long long layer_stride,
                  const T* k_in, T* k_out) {
    constexpr int E = Vec16<T>::kElems;
    constexpr int kVecPerHead = D / E;                                    // 16-byte vectors per (row, head)
    constexpr int kItemsPerHead = LAYOUT == CF_ROPE_HALF ? kVecPerHead / 2 : kVecPerHead;
    constexpr int kPartner = LAYOUT == CF_ROPE_HALF ? (D / 2) : 0;       // element distance to the partner

    const int b = blockIdx.z;
    const int layer = blockIdx.y;
    const int base = pv.tile_begin[b];                              // = tile_base of the request, one load instead of two
    const int n_tiles = pv.n_tiles[b];
    const T* src = k_in + (long long)layer * layer_stride;
    T* dst = k_out + (long long)layer * layer_stride;
    const int items_per_row = n_kv_heads * kItemsPerHead;

    for (int ti = blockIdx.x; ti < n_tiles; ti += gridDim.x) {
        const int doc = pv.tile_doc[base + ti];
        const long long row0 = pv.tile_row0[base + ti];
        const int len = pv.tile_len[base + ti];
        const float2* trig = pv.trig + (size_t)doc * (D / 2);
        const int n_items = len * items_per_row;
        for (int it0 = threadIdx.x; it0 < n_items; it0 += kRepoThreads * kRepoUnroll) {
            uint4 va[kRepoUnroll], vb[kRepoUnroll];
            long long off[kRepoUnroll];
            int slice0[kRepoUnroll];
#pragma unroll
            for (int u = 0; u < kRepoUnroll; ++u) {
                const int it = it0 + u * kRepoThreads;
                if (it < n_items) {
                    const int row = it / items_per_row;
                    const int rem = it - row * items_per_row;
                    const int head = rem / kItemsPerHead;
                    const int vec = rem - head * kItemsPerHead;
                    off[u] = (row0 + row) * bv.token_stride + head * D + vec * E;
                    slice0[u] = LAYOUT == CF_ROPE_HALF ? vec * E : vec * (E / 2);
                    va[u] = *reinterpret_cast<const uint4*>(src + off[u]);
                    if (LAYOUT == CF_ROPE_HALF) vb[u] = *reinterpret_cast<const uint4*>(src + off[u] + kPartner);
                }
            }
#pragma unroll
            for (int u = 0; u < kRepoUnroll; ++u) {
                const int it = it0 + u * kRepoThreads;
                if (it < n_items) {
                    float a[E], ya[E];
                    unpack<T>(va[u], a);
                    if (LAYOUT == CF_ROPE_HALF) {
                        float c[E], yc[E];
                        unpack<T>(vb[u], c);
#pragma unroll
                        for (int e = 0; e < E; ++e) {
                            const float2 cs = __ldg(trig + slice0[u] + e);
                            rotate_pair(a[e], c[e], cs.x, cs.y, ya[e], yc[e]);
                        }
                        *reinterpret_cast<uint4*>(dst + off[u]) = pack<T>(ya);
                        *reinterpret_cast<uint4*>(dst + off[u] + kPartner) = pack<T>(yc);
                    } else {
#pragma unroll
                        for (int e = 0; e < E; e += 2) {
                            const float2 cs = __ldg(trig + slice0[u] + e / 2);
                            rotate_pair(a[e], a[e + 1], cs.x, cs.y, ya[e], ya[e + 1]);
                        }
                        *reinterpret_cast<uint4*>(dst + off[u]) = pack<T>(ya);
                    }
                }
            }
        }
    }
}

// Algorithm 2, Phase 2, assembled: per layer and request, the re-positioned keys and the values of
// the surviving documents, packed in rank order, followed by the query tokens' own keys and values.
// The blocks of a (layer, request) stride over the key tiles of the plan's list (tiles are listed
// in rank order, so a tile's first output row is the sum of the lengths of the tiles before it);
// index n_tiles stands for the query rows, appended last.  Everything is moved in 16-byte vectors.
template <typename T, int D, int LAYOUT>
__global__ void __launch_bounds__(kRepoThreads)
assemble_kernel(BatchView bv, PlanView pv, int n_kv_heads, long long layer_stride, long long self_stride,
                int out_rows, const T* __restrict__ k_in, const T* __restrict__ v_in,
                const T* __restrict__ k_self, const T* __restrict__ v_self, T* __restrict__ k_out,
                T* __restrict__ v_out, int* __restrict__ final_rows) {
    constexpr int E = Vec16<T>::kElems;
    constexpr int kVecPerHead = D / E;
    __shared__ int s_red[kRepoThreads / 32];
    const int b = blockIdx.z, layer = blockIdx.y;
    const int base = pv.tile_begin[b];                              // = tile_base of the request, one load instead of two
    const int n_tiles = pv.n_tiles[b];
    const int row_vecs = n_kv_heads * kVecPerHead;                  // 16-byte vectors of one dense output row
    const long long out_base = (((long long)layer * bv.n_requests + b) * out_rows) * (long long)n_kv_heads * D;
    constexpr int kItemsPerHead = LAYOUT == CF_ROPE_HALF ? kVecPerHead / 2 : kVecPerHead;
    constexpr int kPartner = LAYOUT == CF_ROPE_HALF ? (D / 2) : 0;
    const int items_per_row = n_kv_heads * kItemsPerHead;
    // blocks stride over the tiles, so a grid smaller than the tile count still covers every tile
    for (int ti = blockIdx.x; ti <= n_tiles; ti += gridDim.x) {
        // rows of the tiles before this one (ti == n_tiles: of all tiles)
        int before = 0;
        for (int t = threadIdx.x; t < ti; t += kRepoThreads) before += pv.tile_len[base + t];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
        __syncthreads();                                            // the previous round's readers are done
        if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = before;
        __syncthreads();
        before = 0;
#pragma unroll
        for (int w = 0; w < kRepoThreads / 32; ++w) before += s_red[w];

        if (ti == n_tiles) {                                        // the query tokens' own keys and values
            const int lq = bv.q_len;
            if (before + lq > out_rows) {
                if (threadIdx.x == 0) atomicCAS(pv.status, 0, CF_ERR_WORKSPACE);
                continue;
            }
            if (layer == 0 && threadIdx.x == 0) final_rows[b] = before + lq;
            const long long src0 = (long long)layer * self_stride + (long long)b * lq * n_kv_heads * D;
            for (int idx = threadIdx.x; idx < lq * row_vecs; idx += kRepoThreads) {
                const long long off = (long long)idx * E;
                const long long dst = out_base + (long long)before * n_kv_heads * D + off;
                *reinterpret_cast<uint4*>(k_out + dst) = *reinterpret_cast<const uint4*>(k_self + src0 + off);
                *reinterpret_cast<uint4*>(v_out + dst) = *reinterpret_cast<const uint4*>(v_self + src0 + off);
            }
            continue;
        }
        const int len = pv.tile_len[base + ti];
        if (before + len > out_rows) continue;                      // reported by the block of the query rows
        const long long row0 = pv.tile_row0[base + ti];
        const float2* trig = pv.trig + (size_t)pv.tile_doc[base + ti] * (D / 2);
        const T* ksrc = k_in + (long long)layer * layer_stride;
        const T* vsrc = v_in + (long long)layer * layer_stride;
        for (int it = threadIdx.x; it < len * items_per_row; it += kRepoThreads) {
            const int row = it / items_per_row;
            const int rem = it - row * items_per_row;
            const int head = rem / kItemsPerHead;
            const int vec = rem - head * kItemsPerHead;
            const long long src = (row0 + row) * bv.token_stride + head * D + vec * E;
            const long long dst = out_base + ((long long)(before + row) * n_kv_heads + head) * D + vec * E;
            const int slice0 = LAYOUT == CF_ROPE_HALF ? vec * E : vec * (E / 2);
            float a[E], ya[E];
            unpack<T>(*reinterpret_cast<const uint4*>(ksrc + src), a);
            *reinterpret_cast<uint4*>(v_out + dst) = *reinterpret_cast<const uint4*>(vsrc + src);
            if (LAYOUT == CF_ROPE_HALF) {
                float c[E], yc[E];
                unpack<T>(*reinterpret_cast<const uint4*>(ksrc + src + kPartner), c);
                *reinterpret_cast<uint4*>(v_out + dst + kPartner) = *reinterpret_cast<const uint4*>(vsrc + src + kPartner);
#pragma unroll
                for (int e = 0; e < E; ++e) {
                    const float2 cs = __ldg(trig + slice0 + e);
                    rotate_pair(a[e], c[e], cs.x, cs.y, ya[e], yc[e]);
                }
                *reinterpret_cast<uint4*>(k_out + dst) = pack<T>(ya);
                *reinterpret_cast<uint4*>(k_out + dst + kPartner) = pack<T>(yc);
            } else {
#pragma unroll
                for (int e = 0; e < E; e += 2) {
                    const float2 cs = __ldg(trig + slice0 + e / 2);
                    rotate_pair(a[e], a[e + 1], cs.x, cs.y, ya[e], ya[e + 1]);
                }
                *reinterpret_cast<uint4*>(k_out + dst) = pack<T>(ya);
            }
        }
    }
}

template <typename T, int D>
static int launch_assemble_typed(const cf_geom* g, const cf_batch* b, const PlanView& pv, int n_layers,
                                 long long layer_stride, long long self_stride, int out_rows, const void* k_in,
                                 const void* v_in, const void* k_self, const void* v_self, void* k_out, void* v_out,
                                 int* final_rows, cudaStream_t stream) {
    const int tiles = std::min(tiles_per_request_bound(b), 1 << 16);
    if (n_layers > 65535 || b->n_requests > 65535) return CF_ERR_INVALID_ARG;
    dim3 grid((unsigned)tiles + 1, (unsigned)n_layers, (unsigned)b->n_requests);
    BatchView bv = make_batch_view(b);
    auto args = [&](auto kernel) {
        kernel<<<grid, kRepoThreads, 0, stream>>>(bv, pv, g->n_kv_heads, layer_stride, self_stride, out_rows,
                                                  static_cast<const T*>(k_in), static_cast<const T*>(v_in),
                                                  static_cast<const T*>(k_self), static_cast<const T*>(v_self),
                                                  static_cast<T*>(k_out), static_cast<T*>(v_out), final_rows);
    };
    if (g->rope_layout == CF_ROPE_HALF) args(assemble_kernel<T, D, CF_ROPE_HALF>);
    else args(assemble_kernel<T, D, CF_ROPE_INTERLEAVED>);
    return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

int launch_assemble(const cf_geom* g, const cf_batch* b, const PlanView& pv, int n_layers, long long layer_stride,
                    long long self_stride, int out_rows, const void* k_in, const void* v_in, const void* k_self,
                    const void* v_self, void* k_out, void* v_out, int* final_rows, cudaStream_t stream) {
    if (g->dtype == CF_BF16) {
        if (g->head_dim == 128)
            return launch_assemble_typed<__nv_bfloat16, 128>(g, b, pv, n_layers, layer_stride, self_stride, out_rows, k_in, v_in, k_self, v_self, k_out, v_out, final_rows, stream);
        return launch_assemble_typed<__nv_bfloat16, 64>(g, b, pv, n_layers, layer_stride, self_stride, out_rows, k_in, v_in, k_self, v_self, k_out, v_out, final_rows, stream);
    }
    if (g->head_dim == 128)
        return launch_assemble_typed<float, 128>(g, b, pv, n_layers, layer_stride, self_stride, out_rows, k_in, v_in, k_self, v_self, k_out, v_out, final_rows, stream);
    return launch_assemble_typed<float, 64>(g, b, pv, n_layers, layer_stride, self_stride, out_rows, k_in, v_in, k_self, v_self, k_out, v_out, final_rows, stream);
}

template <typename T, int D>
static int launch_typed(const cf_geom* g, const cf_batch* b, const PlanView& pv, int n_layers,
                        long long layer_stride, const void* k_in, void* k_out, cudaStream_t stream) {
    const int tiles = tiles_per_request_bound(b);
    dim3 grid((unsigned)std::min(tiles, 1 << 16), (unsigned)n_layers, (unsigned)b->n_requests);
    if (n_layers > 65535 || b->n_requests > 65535) return CF_ERR_INVALID_ARG;
    BatchView bv = make_batch_view(b);
    if (g->rope_layout == CF_ROPE_HALF)
        reposition_kernel<T, D, CF_ROPE_HALF><<<grid, kRepoThreads, 0, stream>>>(
            bv, pv, g->n_kv_heads, layer_stride, static_cast<const T*>(k_in), static_cast<T*>(k_out));
    else
        reposition_kernel<T, D, CF_ROPE_INTERLEAVED><<<grid, kRepoThreads, 0, stream>>>(
            bv, pv, g->n_kv_heads, layer_stride, static_cast<const T*>(k_in), static_cast<T*>(k_out));
    return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

int launch_reposition(const cf_geom* g, const cf_batch* b, const PlanView& pv, int n_layers,
                      long long layer_stride, const void* k_in, void* k_out, cudaStream_t stream) {
    if (g->dtype == CF_BF16) {
        if (g->head_dim == 128) return launch_typed<__nv_bfloat16, 128>(g, b, pv, n_layers, layer_stride, k_in, k_out, stream);
        return launch_typed<__nv_bfloat16, 64>(g, b, pv, n_layers, layer_stride, k_in, k_out, stream);
    }
    if (g->head_dim == 128) return launch_typed<float, 128>(g, b, pv, n_layers, layer_stride, k_in, k_out, stream);
    return launch_typed<float, 64>(g, b, pv, n_layers, layer_stride, k_in, k_out, stream);
}

}  // namespace cf
