// Tensor-core kernel of the cache-construction attention, C_d <- LLM(C_prefix, d) (Sec. 2.2), for bf16
// storage and head_dim 128: block-diagonal causal attention over a packed store.
//
// One CTA owns 128 query rows of a (layer, document, kv head); rows are numbered token-major
// (r = token * G + g), so the CTA needs the prefix cache and the document's keys up to its last token
// only.  Keys are walked in tiles of up to 128: first the prefix tiles (every key visible), then the
// document's own tiles, where row r sees the keys up to its own token (causal mask of Eq. 1).
//   warps 0-3  softmax, one query row per thread (= TMEM lane); running maximum and sum per row
//   warp 4     one lane issues the TMA loads and the tcgen05.mma instructions
// S = Q K^T and O += P V accumulate in tensor memory (128 + 128 columns); P goes back through tensor
// memory as bf16 over the S columns already consumed.  There is one K and one V buffer: the next key
// tile is fetched as soon as QK^T has read the current one, the next value tile as soon as PV has.  A CTA
// holds 96 KB of shared memory and 256 tensor-memory columns, so two CTAs share an SM and overlap each
// other's waits.  The result is complete per row (a document is short: no split over CTAs, no merge).
// Every mbarrier wait is bounded; on expiry the CTA reports CF_ERR_TIMEOUT in the status word.
#include "cf_tc_util.cuh"

namespace cf {

namespace {

using namespace tc;

constexpr int kDocTcThreads = 160;
constexpr int kDocTcSmem = 3 * kTileBytes + 1024 + 128;      // Q, K, V tiles; alignment slack; barriers

struct DocMaps {
    CUtensorMap k[4], v[4];        // the documents' keys and values, one map per box height
    CUtensorMap kp[4], vp[4];      // the prefix cache
};

struct DocBars {
    unsigned long long k_full, v_full, s_full, p_ready, o_done;
    unsigned int tmem_base;
    volatile int abort_flag;
};

struct KeyTile {
    int row0, len, doc_first;      // doc_first: document token of the tile's first key, -1 for a prefix tile
};

__device__ __forceinline__ KeyTile key_tile(int i, int n_prefix_tiles, int prefix_len, int row_first, int n_doc_keys) {
    KeyTile t;
    if (i < n_prefix_tiles) {
        t.row0 = i * kTile;
        t.len = min(kTile, prefix_len - t.row0);
        t.doc_first = -1;
    } else {
        const int d0 = (i - n_prefix_tiles) * kTile;
        t.row0 = row_first + d0;
        t.len = min(kTile, n_doc_keys - d0);
        t.doc_first = d0;
    }
    return t;
}

__global__ void __launch_bounds__(kDocTcThreads, 2)
docattn_tc_kernel(const __grid_constant__ DocMaps maps, DocAttnArgs a, const __nv_bfloat16* __restrict__ q,
                  __nv_bfloat16* __restrict__ out, float* __restrict__ lse, int* status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t q_base = smem_u32(smem), k_base = q_base + kTileBytes, v_base = k_base + kTileBytes;
    DocBars* bars = reinterpret_cast<DocBars*>(smem + 3 * kTileBytes);
    volatile int* abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int group = a.n_q_heads / a.n_kv_heads;
    const int layer = blockIdx.z / a.n_docs, doc = blockIdx.z - layer * a.n_docs;
    const int kvh = blockIdx.y;
    const int row_first = a.doc_offsets[doc];
    const int len = a.doc_offsets[doc + 1] - row_first;
    const int rows = len * group;
    const int r0 = blockIdx.x * kTile;
    if (r0 >= rows) return;
    const int rows_here = min(kTile, rows - r0);
    const int n_doc_keys = (r0 + rows_here - 1) / group + 1;         // document tokens 0 .. the last row's token
    const int n_prefix_tiles = (a.prefix_len + kTile - 1) / kTile;
    const int n_tiles = n_prefix_tiles + (n_doc_keys + kTile - 1) / kTile;
    q += (size_t)layer * a.q_layer_stride;
    out += (size_t)layer * a.out_layer_stride;

    // Keys or values of key tile i into their buffer (issued by the one thread of warp 4 that also issues the MMAs).
    auto load = [&](int i, bool values) {
        const KeyTile t = key_tile(i, n_prefix_tiles, a.prefix_len, row_first, n_doc_keys);
        const int boxes = (t.len + kBoxRows - 1) / kBoxRows;
        const CUtensorMap* map = t.doc_first < 0 ? (values ? &maps.vp[boxes - 1] : &maps.kp[boxes - 1])
                                                 : (values ? &maps.v[boxes - 1] : &maps.k[boxes - 1]);
        const uint32_t bar = smem_u32(values ? &bars->v_full : &bars->k_full);
        const uint32_t dst = values ? v_base : k_base;
        mbar_expect_tx(bar, boxes * 2 * kBoxBytes);
        tma_load_4d(dst, map, 0, kvh, t.row0, layer, bar);
        tma_load_4d(dst + kHalfBytes, map, 64, kvh, t.row0, layer, bar);
    };
    // query rows of this CTA: every load is issued before the first is used (one round trip to memory, not thirteen)
    constexpr int kQLoads = (kTile * 16 + kDocTcThreads - 1) / kDocTcThreads;
    uint4 qv[kQLoads];
#pragma unroll
    for (int i = 0; i < kQLoads; ++i) {
        const int idx = tid + i * kDocTcThreads;
        const int chunk = idx & 15, r = idx >> 4;
        qv[i] = make_uint4(0u, 0u, 0u, 0u);
        if (r < rows_here) {
            const int row = r0 + r;
            const int j = row / group, g = row - j * group;
            qv[i] = __ldg(reinterpret_cast<const uint4*>(q + ((size_t)(row_first + j) * a.n_q_heads + kvh * group + g) * kD + chunk * 8));
        }
    }
    if (warp == 4) {
        if (lane == 0) {
            mbar_init(smem_u32(&bars->k_full), 1);
            mbar_init(smem_u32(&bars->v_full), 1);
            mbar_init(smem_u32(&bars->s_full), 1);
            mbar_init(smem_u32(&bars->p_ready), 128);
            mbar_init(smem_u32(&bars->o_done), 1);
            bars->abort_flag = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            load(0, false);                                         // the first key and value tile travel during the set-up
            load(0, true);
        }
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(smem_u32(&bars->tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // query rows into swizzled shared memory (zero rows beyond the valid ones)
#pragma unroll
    for (int i = 0; i < kQLoads; ++i) {
        const int idx = tid + i * kDocTcThreads;
        const int chunk = idx & 15, r = idx >> 4;
        if (idx < kTile * 16) *reinterpret_cast<uint4*>(smem + (chunk >> 3) * kHalfBytes + swz(r, chunk & 7)) = qv[i];
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;

    if (warp == 4) {
        if (lane == 0) {
            // ---------------------------------------------------------- TMA loads and MMA issue
            auto issue_s = [&](int i) -> bool {
                const int n_keys = (key_tile(i, n_prefix_tiles, a.prefix_len, row_first, n_doc_keys).len + 15) & ~15;
                if (!mbar_wait(smem_u32(&bars->k_full), i & 1, abort_flag)) return false;
                tc_fence_after();
                const uint64_t a0 = smem_desc(q_base, 16, 1024), b0 = smem_desc(k_base, 16, 1024);
                const uint32_t idesc = instr_desc(n_keys, false);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint64_t off = (uint64_t)(((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4);
                    umma(tmem, a0 + off, b0 + off, idesc, kk > 0);
                }
                umma_commit(smem_u32(&bars->s_full));
                return true;
            };
            bool ok = issue_s(0);
            for (int i = 0; i < n_tiles && ok; ++i) {
                const bool more = i + 1 < n_tiles;
                if (more) {                                           // QK^T(i) has read the key buffer
                    ok = mbar_wait(smem_u32(&bars->s_full), i & 1, abort_flag);
                    if (!ok) break;
                    load(i + 1, false);
                }
                const int n_keys = (key_tile(i, n_prefix_tiles, a.prefix_len, row_first, n_doc_keys).len + 15) & ~15;
                ok = mbar_wait(smem_u32(&bars->v_full), i & 1, abort_flag) &&
                     mbar_wait(smem_u32(&bars->p_ready), i & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint64_t b0 = smem_desc(v_base, kHalfBytes, 1024);
                const uint32_t idesc_o = instr_desc(kD, true);
                for (int kk = 0; kk < (n_keys >> 4); ++kk)            // 16 keys = 8 packed P columns per instruction
                    umma_ts(tmem + 128, tmem + kk * 8, b0 + (uint64_t)(kk * 128), idesc_o, (i > 0 || kk > 0) ? 1u : 0u);
                umma_commit(smem_u32(&bars->o_done));
                if (more) {
                    ok = issue_s(i + 1);                              // behind PV(i) in the pipe: may overwrite P(i)
                    if (!ok) break;
                    ok = mbar_wait(smem_u32(&bars->o_done), i & 1, abort_flag);   // PV(i) has read the value buffer
                    if (!ok) break;
                    load(i + 1, true);
                }
            }
        }
    } else {
        // -------------------------------------------------------------- softmax, one row per thread
        const int r = tid;                                              // 0..127 = TMEM lane
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        const uint32_t s_addr = tmem + lane_addr, o_addr = tmem + lane_addr + 128;
        const bool row_valid = r < rows_here;
        const int row = r0 + min(r, rows_here - 1);                     // rows beyond the end follow the last valid one
        const int token = row / group;
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        for (int i = 0; i < n_tiles; ++i) {
            const KeyTile t = key_tile(i, n_prefix_tiles, a.prefix_len, row_first, n_doc_keys);
            // visible keys of this tile: all of a prefix tile; document tokens up to the row's own
            const int vis = t.doc_first < 0 ? t.len : max(0, min(t.len, token - t.doc_first + 1));
            const int n_chunks = (t.len + 31) >> 5;
            ok = mbar_wait(smem_u32(&bars->s_full), i & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            uint32_t sv[32];
            float tile_max = -INFINITY;
            for (int c = 0; c < n_chunks; ++c) {
                tmem_ld32(s_addr + c * 32, sv);
                tile_max = fmaxf(tile_max, chunk_max<true>(sv, vis - c * 32));
            }
            // The reference maximum of a row only moves when a tile exceeds it by more than 2^8: any reference within
            // the exponent range is exact enough, since P (bf16) and the sums (fp32) keep their relative precision,
            // and the rescale of O below becomes rare after the first tile.
            const float t_max = tile_max * a.scale_log2;
            const float m_new = t_max > m_run + 8.0f ? t_max : m_run;   // finite from the first tile on
            const float alpha = fast_exp2(m_run - m_new);               // first tile: 0
            if (i > 0) {
                ok = mbar_wait(smem_u32(&bars->o_done), (i - 1) & 1, abort_flag);   // PV(i-1) is complete
                if (!ok) break;
                tc_fence_after();
                if (__any_sync(0xffffffffu, alpha != 1.f)) {
                    for (int cc = 0; cc < 8; ++cc) {
                        uint32_t o[16];
                        tmem_ld16(o_addr + cc * 16, o);
#pragma unroll
                        for (int x = 0; x < 16; ++x) o[x] = __float_as_uint(__uint_as_float(o[x]) * alpha);
                        tmem_st16(o_addr + cc * 16, o);
                    }
                }
            }
            float tile_sum = 0.f;
            for (int c = 0; c < n_chunks; ++c) {
                tmem_ld32(s_addr + c * 32, sv);
                tile_sum += chunk_exp<true>(sv, vis - c * 32, a.scale_log2, -m_new);
                tmem_st16_async(s_addr + c * 16, sv);                   // over S columns already in registers
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            tc_fence_before();
            mbar_arrive(smem_u32(&bars->p_ready));
            l_run = fmaf(l_run, alpha, tile_sum);
            m_run = m_new;
        }
        if (ok) ok = mbar_wait(smem_u32(&bars->o_done), (n_tiles - 1) & 1, abort_flag);
        if (ok) {
            tc_fence_after();
            const float inv = 1.f / l_run;
            // rows leave through shared memory (the query tile: every QK^T has completed) for 256-byte stores
            unsigned char* stage = smem;
            auto stage_chunk = [&](const uint32_t (&o)[32], int c) {       // 32 dims of the row: four 16-byte pieces
#pragma unroll
                for (int x = 0; x < 4; ++x) {
                    const int chunk = c * 4 + x;
                    *reinterpret_cast<uint4*>(stage + r * 256 + ((chunk ^ (r & 15)) << 4)) =
                        make_uint4(pack_bf16(__uint_as_float(o[8 * x]) * inv, __uint_as_float(o[8 * x + 1]) * inv),
                                   pack_bf16(__uint_as_float(o[8 * x + 2]) * inv, __uint_as_float(o[8 * x + 3]) * inv),
                                   pack_bf16(__uint_as_float(o[8 * x + 4]) * inv, __uint_as_float(o[8 * x + 5]) * inv),
                                   pack_bf16(__uint_as_float(o[8 * x + 6]) * inv, __uint_as_float(o[8 * x + 7]) * inv));
                }
            };
            uint32_t oa[32], ob[32];                                        // the load of the next piece travels under the packing of this one
            tmem_ld32_async(o_addr, oa);
            tmem_ld_wait(oa);
            tmem_ld32_async(o_addr + 32, ob);
            stage_chunk(oa, 0);
            tmem_ld_wait(ob);
            tmem_ld32_async(o_addr + 64, oa);
            stage_chunk(ob, 1);
            tmem_ld_wait(oa);
            tmem_ld32_async(o_addr + 96, ob);
            stage_chunk(oa, 2);
            tmem_ld_wait(ob);
            stage_chunk(ob, 3);
            __syncwarp();
            const int warp_row0 = warp * 32;
#pragma unroll
            for (int x = 0; x < 16; ++x) {                              // two rows per step, 16 lanes each
                const int rr = warp_row0 + 2 * x + (lane >> 4), chunk = lane & 15;
                if (rr < rows_here) {
                    const int rw = r0 + rr;
                    const int j = rw / group, g = rw - j * group;
                    const uint4 val = *reinterpret_cast<const uint4*>(stage + rr * 256 + ((chunk ^ (rr & 15)) << 4));
                    *reinterpret_cast<uint4*>(out + ((size_t)(row_first + j) * a.n_q_heads + kvh * group + g) * kD + chunk * 8) = val;
                }
            }
            if (row_valid && lse) {
                const int g = row - token * group;
                lse[((size_t)layer * a.n_q_heads + kvh * group + g) * a.total_tokens + row_first + token] =
                    (m_run + log2f(l_run)) * kLn2;
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (bars->abort_flag) {
        // a wait expired: let the (at most two) loads in flight land before the shared memory is given back
        if (warp == 4 && lane == 0) {
            const long long t0 = clock64();
            while (clock64() - t0 < kWaitLimitCycles / 64) {}
        }
        if (tid == 0 && status) atomicCAS(status, 0, CF_ERR_TIMEOUT);
        __syncthreads();
    }
    if (warp == 4) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem) : "memory");
    }
}

}  // namespace

bool docattn_tc_supported(const cf_geom* g, const cf_doc_batch* docs) {
    return g->dtype == CF_BF16 && g->head_dim == 128 && docs->total_tokens > 0;
}

int launch_docattn_tc(const cf_geom* g, const DocAttnArgs& a, const void* q, const void* k, const void* v,
                      const void* kp, const void* vp, void* out, float* lse, int* status, cudaStream_t stream) {
    const int group = a.n_q_heads / a.n_kv_heads;
    const long long row_tiles = ((long long)a.max_doc_len * group + kTile - 1) / kTile;
    if (row_tiles > 0x7fffffffLL || a.n_kv_heads > 65535 || (long long)a.n_docs * a.n_layers > 65535) return CF_ERR_INVALID_ARG;
    DocMaps maps;
    const unsigned long long row_bytes = (unsigned long long)a.token_stride * 2;
    const unsigned long long layer_bytes = a.n_layers > 1 ? (unsigned long long)a.kv_layer_stride * 2
                                                          : (unsigned long long)a.total_tokens * row_bytes;
    const unsigned long long prow = (unsigned long long)a.n_kv_heads * kD * 2;
    const unsigned long long player = a.n_layers > 1 ? (unsigned long long)a.prefix_layer_stride * 2
                                                     : (unsigned long long)a.prefix_len * prow;
    for (int i = 0; i < 4; ++i) {
        int rc = make_rows_map(&maps.k[i], k, a.n_kv_heads, (unsigned long long)a.total_tokens, row_bytes, a.n_layers,
                               layer_bytes, (i + 1) * kBoxRows);
        if (rc != CF_OK) return rc;
        rc = make_rows_map(&maps.v[i], v, a.n_kv_heads, (unsigned long long)a.total_tokens, row_bytes, a.n_layers,
                           layer_bytes, (i + 1) * kBoxRows);
        if (rc != CF_OK) return rc;
        if (a.prefix_len > 0) {
            rc = make_rows_map(&maps.kp[i], kp, a.n_kv_heads, (unsigned long long)a.prefix_len, prow, a.n_layers, player,
                               (i + 1) * kBoxRows);
            if (rc != CF_OK) return rc;
            rc = make_rows_map(&maps.vp[i], vp, a.n_kv_heads, (unsigned long long)a.prefix_len, prow, a.n_layers, player,
                               (i + 1) * kBoxRows);
            if (rc != CF_OK) return rc;
        } else {
            maps.kp[i] = maps.k[i];
            maps.vp[i] = maps.v[i];
        }
    }
    static PerDeviceOnce configured;
    if (configure_smem_once(configured, docattn_tc_kernel, kDocTcSmem) != CF_OK) return CF_ERR_CUDA;
    dim3 grid((unsigned)row_tiles, (unsigned)a.n_kv_heads, (unsigned)(a.n_docs * a.n_layers));
    docattn_tc_kernel<<<grid, kDocTcThreads, kDocTcSmem, stream>>>(maps, a, static_cast<const __nv_bfloat16*>(q),
                                                                  static_cast<__nv_bfloat16*>(out), lse, status);
    return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

}  // namespace cf
