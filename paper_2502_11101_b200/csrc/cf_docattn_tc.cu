// Tensor-core kernel of the cache-construction attention, C_d <- LLM(C_prefix, d) (Sec. 2.2), for bf16
// storage and head_dim 128: block-diagonal causal attention over a packed store.
//
// A work item is 128 query rows of a (layer, document, kv head); rows are numbered token-major
// (r = token * G + g), so an item needs the prefix cache and the document's keys up to its last token
// only.  Keys are walked in tiles of up to 128: first the prefix tiles (every key visible), then the
// document's own tiles, where row r sees the keys up to its own token (causal mask of Eq. 1).
//   warps 0-3  softmax, one query row per thread (= TMEM lane); running maximum and sum per row
//   warp 4     one lane issues the TMA loads and the tcgen05.mma instructions
// S = Q K^T and O += P V accumulate in tensor memory (128 + 128 columns); P goes back through tensor
// memory as bf16 over the S columns already consumed.  There is one K and one V buffer: the next key
// tile is fetched as soon as QK^T has read the current one, the next value tile as soon as PV has.  A CTA
// holds 96 KB of shared memory and 256 tensor-memory columns, so two CTAs share an SM and overlap each
// other's waits.  The result is complete per row (a document is short: no split over CTAs, no merge).
// CTAs are persistent: CTA c takes items c, c + grid, c + 2 grid, ...  An item holds whole tokens
// ((128 / G) * G rows), so its query rows are one box of the query tensor: they and the item's first key
// tile are requested as soon as the last QK^T of the current item has read the query tile, and the next
// item's first QK^T runs under the epilogue of the current one.  Rows leave through the value buffer, by
// bulk copy when the item is a whole box of the output, row by row for the ragged last item of a
// document; the next item's first value tile may only overwrite the buffer once they are out.  Barriers
// live for the whole kernel; their parities follow running counts of key tiles and items.
// Every mbarrier wait is bounded; on expiry the CTA reports CF_ERR_TIMEOUT in the status word.
#include <algorithm>

#include "cf_tc_util.cuh"

namespace cf {

namespace {

using namespace tc;

constexpr int kDocTcThreads = 160;
constexpr int kDocTcSmem = 3 * kTileBytes + 1024 + 128;      // Q, K, V tiles; alignment slack; barriers

struct DocMaps {
    CUtensorMap k[4], v[4];        // the documents' keys and values, one map per box height
    CUtensorMap kp[4], vp[4];      // the prefix cache
    CUtensorMap qm, om;            // the queries and the output: boxes of 64 dims x G heads x (128 / G) tokens
};

struct DocBars {
    unsigned long long k_full, v_full, s_full, p_ready, o_done;    // one phase per key tile
    unsigned long long q_full, staged, stage_free;                 // one phase per item
    unsigned int tmem_base;
    volatile int abort_flag;
};

// A key tile: up to 128 keys, first those of the prefix cache (rows p_row0 .. of the prefix tensors, visible to every
// row), then those of the document (store rows d_row0 .., document tokens doc_first ..).  When the prefix length is a
// multiple of the copy boxes' 32 rows the two parts share tiles (`joined`: the keys of an item are the sequence
// [prefix; document tokens] cut every 128); otherwise the prefix has tiles of its own.
struct KeyTile {
    int p_row0, p_len, d_row0, d_len, doc_first, len;
};

__device__ __forceinline__ KeyTile key_tile(int i, bool joined, int n_prefix_tiles, int prefix_len, int row_first, int n_doc_keys) {
    KeyTile t;
    if (joined) {
        const int k0 = i * kTile;
        t.p_row0 = k0;
        t.p_len = max(0, min(kTile, prefix_len - k0));
        t.doc_first = max(0, k0 - prefix_len);
        t.d_len = max(0, min(kTile - t.p_len, n_doc_keys - t.doc_first));
    } else if (i < n_prefix_tiles) {
        t.p_row0 = i * kTile;
        t.p_len = min(kTile, prefix_len - t.p_row0);
        t.doc_first = 0;
        t.d_len = 0;
    } else {
        t.p_row0 = 0;
        t.p_len = 0;
        t.doc_first = (i - n_prefix_tiles) * kTile;
        t.d_len = min(kTile, n_doc_keys - t.doc_first);
    }
    t.d_row0 = row_first + t.doc_first;
    t.len = t.p_len + t.d_len;
    return t;
}

// A work item: index w = row tile + row_tiles * (kv head + n_kv_heads * (layer * n_docs + document)).
struct DocItem {
    int w, layer, kvh, row_first, r0, rows_here, n_doc_keys, n_tiles;
    bool valid;
};

// Shape of the item space.  An item holds whole tokens: rows_per_tile = (128 / G) * G rows, so that its query rows are one
// box of the query tensor (G heads x 128 / G tokens) and arrive by bulk copy.
struct DocGrid {
    int row_tiles, total, group, n_prefix_tiles, rows_per_tile, joined, prefix_len;
};

__device__ __forceinline__ DocItem doc_item(const DocAttnArgs& a, const DocGrid& dg, int w) {
    const int row_tiles = dg.row_tiles, total = dg.total, group = dg.group, n_prefix_tiles = dg.n_prefix_tiles;
    DocItem it;
    it.w = w;
    it.valid = false;
    if (w >= total) return it;
    const int x = w % row_tiles, yz = w / row_tiles;
    it.kvh = yz % a.n_kv_heads;
    const int z = yz / a.n_kv_heads;
    it.layer = z / a.n_docs;
    const int doc = z - it.layer * a.n_docs;
    it.row_first = __ldg(a.doc_offsets + doc);
    const int rows = (__ldg(a.doc_offsets + doc + 1) - it.row_first) * group;
    it.r0 = x * dg.rows_per_tile;
    if (it.r0 >= rows) return it;
    it.rows_here = min(dg.rows_per_tile, rows - it.r0);
    it.n_doc_keys = (it.r0 + it.rows_here - 1) / group + 1;       // document tokens 0 .. the last row's token
    it.n_tiles = dg.joined ? (dg.prefix_len + it.n_doc_keys + kTile - 1) / kTile
                           : n_prefix_tiles + (it.n_doc_keys + kTile - 1) / kTile;
    it.valid = true;
    return it;
}
// The CTA's next item with rows in it, from index w on (steps of the grid size); invalid when there is none.
__device__ __forceinline__ DocItem next_item(const DocAttnArgs& a, const DocGrid& dg, int w) {
    DocItem it = doc_item(a, dg, w);
    while (!it.valid && it.w < dg.total) it = doc_item(a, dg, it.w + (int)gridDim.x);
    return it;
}

__global__ void __launch_bounds__(kDocTcThreads, 2)
docattn_tc_kernel(const __grid_constant__ DocMaps maps, DocAttnArgs a, DocGrid dg,
                  __nv_bfloat16* __restrict__ out_all, float* __restrict__ lse, int* status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t q_base = smem_u32(smem), k_base = q_base + kTileBytes, v_base = k_base + kTileBytes;
    DocBars* bars = reinterpret_cast<DocBars*>(smem + 3 * kTileBytes);
    volatile int* abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int group = dg.group, n_prefix_tiles = dg.n_prefix_tiles;
    const bool joined = dg.joined != 0;
    DocItem cur = next_item(a, dg, (int)blockIdx.x);
    if (!cur.valid) return;                                         // uniform over the CTA

    // Keys or values of key tile i of an item into their buffer (issued by the one thread of warp 4 that also issues the MMAs).
    auto load = [&](const DocItem& it, int i, bool values) {
        const KeyTile t = key_tile(i, joined, n_prefix_tiles, a.prefix_len, it.row_first, it.n_doc_keys);
        const int p_boxes = (t.p_len + kBoxRows - 1) / kBoxRows, d_boxes = (t.d_len + kBoxRows - 1) / kBoxRows;
        const uint32_t bar = smem_u32(values ? &bars->v_full : &bars->k_full);
        const uint32_t dst = values ? v_base : k_base;
        mbar_expect_tx(bar, (p_boxes + d_boxes) * 2 * kBoxBytes);
        if (p_boxes > 0) {
            const CUtensorMap* map = values ? &maps.vp[p_boxes - 1] : &maps.kp[p_boxes - 1];
            tma_load_4d(dst, map, 0, it.kvh, t.p_row0, it.layer, bar);
            tma_load_4d(dst + kHalfBytes, map, 64, it.kvh, t.p_row0, it.layer, bar);
        }
        if (d_boxes > 0) {                                          // behind the prefix rows (a whole number of boxes)
            const CUtensorMap* map = values ? &maps.v[d_boxes - 1] : &maps.k[d_boxes - 1];
            const uint32_t d_dst = dst + t.p_len * 128;
            tma_load_4d(d_dst, map, 0, it.kvh, t.d_row0, it.layer, bar);
            tma_load_4d(d_dst + kHalfBytes, map, 64, it.kvh, t.d_row0, it.layer, bar);
        }
    };
    // Query rows of an item (whole tokens, G heads each) into the query tile, one copy per 64-dim half.
    auto load_q = [&](const DocItem& it) {
        const uint32_t bar = smem_u32(&bars->q_full);
        mbar_expect_tx(bar, dg.rows_per_tile * 256);
        tma_load_4d(q_base, &maps.qm, 0, it.kvh * group, it.row_first + it.r0 / group, it.layer, bar);
        tma_load_4d(q_base + kHalfBytes, &maps.qm, 64, it.kvh * group, it.row_first + it.r0 / group, it.layer, bar);
    };
    // rows of the query tile behind the box are never written: zero them once (their results are not stored)
    for (int idx = tid; idx < (kTile - dg.rows_per_tile) * 16; idx += kDocTcThreads) {
        const int chunk = idx & 15, r = dg.rows_per_tile + (idx >> 4);
        *reinterpret_cast<uint4*>(smem + (chunk >> 3) * kHalfBytes + swz(r, chunk & 7)) = make_uint4(0u, 0u, 0u, 0u);
    }
    fence_proxy_async();
    if (warp == 4) {
        if (lane == 0) {
            mbar_init(smem_u32(&bars->k_full), 1);
            mbar_init(smem_u32(&bars->v_full), 1);
            mbar_init(smem_u32(&bars->s_full), 1);
            mbar_init(smem_u32(&bars->p_ready), 128);
            mbar_init(smem_u32(&bars->o_done), 1);
            mbar_init(smem_u32(&bars->q_full), 1);
            mbar_init(smem_u32(&bars->staged), 128);
            mbar_init(smem_u32(&bars->stage_free), 128);
            bars->abort_flag = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            load_q(cur);                                            // the first tiles travel during the set-up
            load(cur, 0, false);
            load(cur, 0, true);
        }
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(smem_u32(&bars->tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();                                                // barriers are initialised, tensor memory is allocated
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;

    if (warp == 4) {
        if (lane == 0) {
            // ---------------------------------------------------------- TMA loads and MMA issue
            const uint64_t a0 = smem_desc(q_base, 16, 1024), bk = smem_desc(k_base, 16, 1024);
            const uint64_t bv = smem_desc(v_base, kHalfBytes, 1024);
            const uint32_t idesc_o = instr_desc(kD, true);
            int g = 0, n = 0;                                       // key tiles and items before the current one
            auto issue_s = [&](const DocItem& it, int i, int gi) -> bool {
                const int n_keys = (key_tile(i, joined, n_prefix_tiles, a.prefix_len, it.row_first, it.n_doc_keys).len + 15) & ~15;
                if (!mbar_wait(smem_u32(&bars->k_full), gi & 1, abort_flag)) return false;
                tc_fence_after();
                const uint32_t idesc = instr_desc(n_keys, false);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint64_t off = (uint64_t)(((kk >> 2) * kHalfBytes + (kk & 3) * 32) >> 4);
                    umma(tmem, a0 + off, bk + off, idesc, kk > 0);
                }
                umma_commit(smem_u32(&bars->s_full));
                return true;
            };
            bool ok = mbar_wait(smem_u32(&bars->q_full), 0, abort_flag);
            if (ok) ok = issue_s(cur, 0, 0);
            while (ok) {
                const DocItem nxt = next_item(a, dg, cur.w + (int)gridDim.x);
                for (int i = 0; i < cur.n_tiles && ok; ++i) {
                    const bool last = i + 1 == cur.n_tiles;
                    // QK^T(i) has completed: the key buffer is free, and after the item's last one the query tile too
                    ok = mbar_wait(smem_u32(&bars->s_full), (g + i) & 1, abort_flag);
                    if (!ok) break;
                    if (!last) {
                        load(cur, i + 1, false);
                    } else if (nxt.valid) {
                        load_q(nxt);
                        load(nxt, 0, false);
                    }
                    const int n_keys = (key_tile(i, joined, n_prefix_tiles, a.prefix_len, cur.row_first, cur.n_doc_keys).len + 15) & ~15;
                    ok = mbar_wait(smem_u32(&bars->v_full), (g + i) & 1, abort_flag) &&
                         mbar_wait(smem_u32(&bars->p_ready), (g + i) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    for (int kk = 0; kk < (n_keys >> 4); ++kk)        // 16 keys = 8 packed P columns per instruction
                        umma_ts(tmem + 128, tmem + kk * 8, bv + (uint64_t)(kk * 128), idesc_o, (i > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(smem_u32(&bars->o_done));
                    // the next QK^T sits behind PV(i) in the pipe, so it may overwrite P(i); the next item's first one
                    // also needs its query rows in shared memory
                    if (!last) {
                        ok = issue_s(cur, i + 1, g + i + 1);
                    } else if (nxt.valid) {
                        ok = mbar_wait(smem_u32(&bars->q_full), (n + 1) & 1, abort_flag);
                        if (ok) ok = issue_s(nxt, 0, g + i + 1);
                    }
                    if (!ok) break;
                    ok = mbar_wait(smem_u32(&bars->o_done), (g + i) & 1, abort_flag);   // PV(i) has read the value buffer
                    if (!ok) break;
                    if (!last) {
                        load(cur, i + 1, true);
                    } else if (nxt.valid) {                         // the rows of this item leave through the value buffer
                        ok = mbar_wait(smem_u32(&bars->stage_free), n & 1, abort_flag);
                        if (ok) load(nxt, 0, true);
                    }
                }
                if (!nxt.valid) break;
                g += cur.n_tiles;
                ++n;
                cur = nxt;
            }
        }
    } else {
        // -------------------------------------------------------------- softmax, one row per thread
        const int r = tid;                                              // 0..127 = TMEM lane
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        const uint32_t s_addr = tmem + lane_addr, o_addr = tmem + lane_addr + 128;
        int g = 0, n = 0;                                               // key tiles and items before the current one
        bool ok = true;
        while (ok) {
            const DocItem nxt = next_item(a, dg, cur.w + (int)gridDim.x);
            const bool row_valid = r < cur.rows_here;
            const int row = cur.r0 + min(r, cur.rows_here - 1);         // rows beyond the end follow the last valid one
            const int token = row / group;
            float m_run = -INFINITY, l_run = 0.f;
            for (int i = 0; i < cur.n_tiles; ++i) {
                const KeyTile t = key_tile(i, joined, n_prefix_tiles, a.prefix_len, cur.row_first, cur.n_doc_keys);
                // visible keys of this tile: all of its prefix keys; document tokens up to the row's own
                const int vis = t.p_len + max(0, min(t.d_len, token - t.doc_first + 1));
                const int n_chunks = (t.len + 31) >> 5;
                ok = mbar_wait(smem_u32(&bars->s_full), (g + i) & 1, abort_flag);
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
                    ok = mbar_wait(smem_u32(&bars->o_done), (g + i - 1) & 1, abort_flag);   // PV(i-1) is complete
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
                    tmem_st16_async(s_addr + c * 16, sv);               // over S columns already in registers
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                tc_fence_before();
                mbar_arrive(smem_u32(&bars->p_ready));
                l_run = fmaf(l_run, alpha, tile_sum);
                m_run = m_new;
            }
            if (!ok) break;
            ok = mbar_wait(smem_u32(&bars->o_done), (g + cur.n_tiles - 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            {
                const float inv = 1.f / l_run;
                // Rows leave through shared memory (the value buffer: every PV has completed), laid out like the query
                // tile (two 64-dim halves, 128-byte swizzle): an item of whole tokens is one box of the output tensor and
                // goes out by bulk copy; the ragged last item of a document goes out row by row.
                unsigned char* stage = smem + 2 * kTileBytes;
                auto stage_chunk = [&](const uint32_t (&o)[32], int c) {   // 32 dims of the row: four 16-byte pieces
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const int chunk = c * 4 + x;
                        *reinterpret_cast<uint4*>(stage + (chunk >> 3) * kHalfBytes + swz(r, chunk & 7)) =
                            make_uint4(pack_bf16(__uint_as_float(o[8 * x]) * inv, __uint_as_float(o[8 * x + 1]) * inv),
                                       pack_bf16(__uint_as_float(o[8 * x + 2]) * inv, __uint_as_float(o[8 * x + 3]) * inv),
                                       pack_bf16(__uint_as_float(o[8 * x + 4]) * inv, __uint_as_float(o[8 * x + 5]) * inv),
                                       pack_bf16(__uint_as_float(o[8 * x + 6]) * inv, __uint_as_float(o[8 * x + 7]) * inv));
                    }
                };
                uint32_t oa[32], ob[32];                                // the load of the next piece travels under the packing of this one
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
                if (row_valid && lse) {
                    const int gq = row - token * group;
                    lse[((size_t)cur.layer * a.n_q_heads + cur.kvh * group + gq) * a.total_tokens + cur.row_first + token] =
                        (m_run + log2f(l_run)) * kLn2;
                }
                fence_proxy_async();
                tc_fence_before();
                mbar_arrive(smem_u32(&bars->staged));
                ok = mbar_wait(smem_u32(&bars->staged), n & 1, abort_flag);   // every row of the item is staged
                if (!ok) break;
                if (cur.rows_here == dg.rows_per_tile) {
                    if (tid == 0) {
                        const int token0 = cur.row_first + cur.r0 / group;
                        tma_store_4d(&maps.om, smem_u32(stage), 0, cur.kvh * group, token0, cur.layer);
                        tma_store_4d(&maps.om, smem_u32(stage) + kHalfBytes, 64, cur.kvh * group, token0, cur.layer);
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the copies have read the staging rows
                    }
                } else {
                    __nv_bfloat16* out = out_all + (size_t)cur.layer * a.out_layer_stride;
                    const int warp_row0 = warp * 32;
#pragma unroll 4
                    for (int x = 0; x < 16; ++x) {                      // two rows per step, 16 lanes each
                        const int rr = warp_row0 + 2 * x + (lane >> 4), chunk = lane & 15;
                        if (rr < cur.rows_here) {
                            const int rw = cur.r0 + rr;
                            const int j = rw / group, gq = rw - j * group;
                            const uint4 val = *reinterpret_cast<const uint4*>(stage + (chunk >> 3) * kHalfBytes + swz(rr, chunk & 7));
                            *reinterpret_cast<uint4*>(out + ((size_t)(cur.row_first + j) * a.n_q_heads + cur.kvh * group + gq) * kD + chunk * 8) = val;
                        }
                    }
                }
                // once every thread is here the value buffer may be overwritten by the next item's first value tile
                mbar_arrive(smem_u32(&bars->stage_free));
            }
            if (!nxt.valid) break;
            g += cur.n_tiles;
            ++n;
            cur = nxt;
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
    return g->dtype == CF_BF16 && g->head_dim == 128 && docs->total_tokens > 0 &&
           g->n_q_heads / g->n_kv_heads <= kTile;                   // an item holds at least one whole token
}

int launch_docattn_tc(const cf_geom* g, const DocAttnArgs& a, const void* q, const void* k, const void* v,
                      const void* kp, const void* vp, void* out, float* lse, int* status, cudaStream_t stream) {
    const int group = a.n_q_heads / a.n_kv_heads;
    if (group > kTile) return CF_ERR_UNSUPPORTED;
    const int rows_per_tile = (kTile / group) * group;              // whole tokens
    const long long row_tiles = ((long long)a.max_doc_len * group + rows_per_tile - 1) / rows_per_tile;
    const long long total = row_tiles * a.n_kv_heads * (long long)a.n_docs * a.n_layers;   // work items, empty ones included
    if (row_tiles <= 0 || total > 0x7fffffffLL - 65536) return CF_ERR_INVALID_ARG;
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
    {   // queries [layers][tokens][q heads][128] as (64 dims, q heads, tokens, layers); the two halves are fetched one by one
        EncodeTiledFn fn = encode_fn();
        if (!fn) return CF_ERR_CUDA;
        const unsigned long long qrow = (unsigned long long)a.n_q_heads * kD * 2;
        const unsigned long long qlayer = a.n_layers > 1 ? (unsigned long long)a.q_layer_stride * 2
                                                          : (unsigned long long)a.total_tokens * qrow;
        const cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)a.n_q_heads, (cuuint64_t)a.total_tokens, (cuuint64_t)a.n_layers};
        const cuuint64_t strides[3] = {(cuuint64_t)kD * 2, (cuuint64_t)qrow, (cuuint64_t)qlayer};
        const cuuint32_t box[4] = {64, (cuuint32_t)group, (cuuint32_t)(kTile / group), 1};
        const cuuint32_t elem[4] = {1, 1, 1, 1};
        if (fn(&maps.qm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(q), dims, strides, box, elem,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return CF_ERR_CUDA;
        // the output has the layout of the queries; its layers may lie further apart
        const cuuint64_t ostrides[3] = {(cuuint64_t)kD * 2, (cuuint64_t)qrow,
                                        a.n_layers > 1 ? (cuuint64_t)a.out_layer_stride * 2 : (cuuint64_t)a.total_tokens * qrow};
        if (fn(&maps.om, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, out, dims, ostrides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return CF_ERR_CUDA;
    }
    static PerDeviceOnce configured;
    if (configure_smem_once(configured, docattn_tc_kernel, kDocTcSmem) != CF_OK) return CF_ERR_CUDA;
    const int ctas = sm_count() > 0 ? 2 * sm_count() : 296;         // persistent: two CTAs per SM
    const unsigned grid = (unsigned)std::min<long long>(total, ctas);
    const DocGrid dg = {(int)row_tiles, (int)total, group, (a.prefix_len + kTile - 1) / kTile, rows_per_tile,
                        a.prefix_len % kBoxRows == 0 ? 1 : 0, a.prefix_len};
    docattn_tc_kernel<<<grid, kDocTcThreads, kDocTcSmem, stream>>>(maps, a, dg, static_cast<__nv_bfloat16*>(out), lse, status);
    return cudaGetLastError() == cudaSuccess ? CF_OK : CF_ERR_CUDA;
}

}  // namespace cf
