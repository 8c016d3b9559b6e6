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
    const int doc0 = bv.req_doc_begin[b];
    const int base = tile_base(doc0, bv.doc_offsets[doc0]);
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
