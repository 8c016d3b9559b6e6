"""CPU oracle for the CacheFocus query-time path (arXiv 2502.11101).

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, double-precision restatement of what
the method computes, written from the paper so that the CUDA library can be checked
against it.  Nothing in the product path may import it; it imports nothing from the
product either.  Only the tests, the smoke check and the benchmark's CPU-baseline leg
call it.

What it follows, step by step:

* rotary rotation of each two-dimensional slice of a key (Eq. 2) and re-positioning of a
  cached key from position i to position j by the rotation R_j R_i^T = R_(j-i) (Eq. 5);
* Adaptive Re-Positioning: the number of parallel position windows N_reuse (Eq. 6) and
  the assignment of sequential positions inside each window (Sec. 2.3.1), anchored next
  to the query (Sec. 2.5, Fig. 4 caption);
* scaled dot-product attention of the query tokens over the concatenated, re-positioned
  document caches (Eq. 1), with the attention mass each document receives accumulated
  "document-wise" (footnote of Sec. 2.4);
* Layer-Adaptive Cache Pruning: scores accumulate over layers, every pruning layer keeps
  the best documents and the survivors are re-allocated ("align" / "sort", Sec. 2.5)
  (Algorithm 2, Phases 1 and 2); the linear pruning schedule of App. C;
* the attention of the offline cache construction (Sec. 2.2): every document attends the shared
  prefix cache and itself, causally, independently of the other documents;
* decoding over the final cache (Algorithm 2, Phase 3): each new token's key/value row is appended and
  its query row attends the whole cache.

Pins (tests/test_oracle_*.py): closed forms of the rotation group, the identity of
Eq. 5, an independent complex-number statement of rotary encoding, the printed examples
of Sec. 3.3 (k=20, N_reuse=k/5) and App. C (L=28, n=4, k=40, k_finish=5), allocation
invariants checked by brute force, brute-force attention with Python loops, the
N_reuse=1 special case against a library attention routine, the closed form for Q=0; for the
cache-construction attention a library causal attention over [prefix; document], Python loops, the
Q=0 closed form, causality and the composition of the pinned prefix and self blocks; for the decoding
steps the rows of a library causal attention over [cache; new tokens], the Q=0 closed form and the
agreement of a step with the pinned query_prefill_attn over the cache it has grown.

Parity unpinned (conventions the paper leaves open, no figure or code to compare with):
which two coordinates form a slice (both common layouts are implemented), round-robin
versus contiguous splitting of ranks into windows, and the exact placement picture of
Fig. 4 beyond "next to the query, in order".
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

ROPE_HALF = 0          # slice p pairs coordinates (p, p + D/2)
ROPE_INTERLEAVED = 1   # slice p pairs coordinates (2p, 2p + 1)

ALLOC_NONE = 0         # survivors keep their positions (gaps stay)
ALLOC_ALIGN = 1        # Dynamic Positional Allocation: re-pack, previous order kept
ALLOC_SORT = 2         # Attention-Guided Allocation: re-pack by accumulated score


class RangeError(ValueError):
    """The kept documents do not fit the positional range."""


# --------------------------------------------------------------------------- rotation
def rope_inv_freq(theta: float, head_dim: int) -> np.ndarray:
    """Angle per position of slice p: theta^(-2p/D), p = 0..D/2-1 (the standard rotary
    frequencies; Eq. 2 only names the angle r_i = i * this)."""
    p = np.arange(head_dim // 2, dtype=np.float64)
    return np.power(np.float64(theta), -2.0 * p / head_dim)


def rope_rotate(x: np.ndarray, delta, theta: float, layout: int = ROPE_HALF) -> np.ndarray:
    """Rotate every two-dimensional slice of `x[..., D]` by `delta` positions (Eq. 2):
    (a, b) -> (a cos r - b sin r, a sin r + b cos r), r = delta * inv_freq[p].
    `delta` is a scalar or an array matching x.shape[:-1]."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    ang = np.asarray(delta, dtype=np.float64)[..., None] * rope_inv_freq(theta, d)
    c, s = np.cos(ang), np.sin(ang)
    y = np.empty_like(x)
    if layout == ROPE_HALF:
        a, b = x[..., : d // 2], x[..., d // 2:]
        y[..., : d // 2] = a * c - b * s
        y[..., d // 2:] = a * s + b * c
    elif layout == ROPE_INTERLEAVED:
        a, b = x[..., 0::2], x[..., 1::2]
        y[..., 0::2] = a * c - b * s
        y[..., 1::2] = a * s + b * c
    else:
        raise ValueError("unknown rope layout")
    return y


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Values of `x` rounded to the nearest bfloat16 (8 significand bits, ties to even), returned
    as float64: the storage format of a 16-bit cache, written out from its definition."""
    bits = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    bits = (bits + 0x7FFF + ((bits >> 16) & 1)) & 0xFFFF0000
    return bits.astype(np.uint32).view(np.float32).astype(np.float64)


# ------------------------------------------------------------------------- allocation
def n_reuse_eq6(n_kept: int, capacity: int, cache_len: int) -> int:
    """Eq. 6: ceil(k / (L / l_C)).  L / l_C, the number of caches that fit without
    reuse, is taken as a whole number of caches (floor)."""
    per_group = capacity // cache_len
    if per_group <= 0:
        raise RangeError("a document is longer than the usable positional range")
    return -(-n_kept // per_group)


def allocate_positions(doc_len: Sequence[int], order: Sequence[int], pos_range: int,
                       prefix_len: int = 0, tail_reserve: int = 0, n_reuse: int = 0,
                       query_start: int = -1) -> Tuple[np.ndarray, np.ndarray, int, int]:
    """Destination positions for the kept documents (Sec. 2.3.1, Sec. 2.5).

    `order[r]` is the document at rank r; rank 0 is placed closest to the query.  The
    kept documents are dealt round-robin into N_reuse groups (parallel windows); inside
    a group documents take sequential positions, packed backwards from the query start
    so that every window ends where the query begins.  `n_reuse=0` selects Eq. 6 with
    l_C = the longest kept document; `query_start<0` puts the query at the end of the
    usable range, query_start = pos_range - tail_reserve, the one anchor for which every
    later re-allocation of a pruned set is guaranteed to fit (a window then holds at most
    floor(capacity / l_C) documents of at most l_C tokens).  Only position differences
    enter the attention (text after Eq. 2), so the anchor itself does not change results.

    Returns (dst_start[n_docs] with -1 for documents not kept, group[n_docs] likewise,
    n_reuse, query_start)."""
    doc_len = np.asarray(doc_len, dtype=np.int64)
    n_docs = doc_len.shape[0]
    order = [int(i) for i in order]
    n_kept = len(order)
    if len(set(order)) != n_kept or any(i < 0 or i >= n_docs for i in order):
        raise ValueError("order must list distinct document ids")
    dst_start = np.full(n_docs, -1, dtype=np.int64)
    group = np.full(n_docs, -1, dtype=np.int64)
    capacity = pos_range - prefix_len - tail_reserve
    if n_kept == 0:
        qs = pos_range - tail_reserve if query_start < 0 else query_start
        return dst_start, group, max(1, n_reuse), qs
    cache_len = int(max(doc_len[i] for i in order))
    if cache_len <= 0 or any(doc_len[i] <= 0 for i in order):
        raise ValueError("documents must have at least one token")
    if n_reuse <= 0:
        n_reuse = n_reuse_eq6(n_kept, capacity, cache_len)
    group_total = [0] * n_reuse
    for r, i in enumerate(order):
        group_total[r % n_reuse] += int(doc_len[i])
    if query_start < 0:
        query_start = pos_range - tail_reserve
    if query_start + tail_reserve > pos_range or max(group_total) > query_start - prefix_len:
        raise RangeError("kept documents do not fit the positional range")
    cursor = [query_start] * n_reuse
    for r, i in enumerate(order):
        g = r % n_reuse
        cursor[g] -= int(doc_len[i])
        dst_start[i] = cursor[g]
        group[i] = g
    return dst_start, group, n_reuse, query_start


# ----------------------------------------------------------------------- re-positioning
def reposition_keys(k_store: np.ndarray, doc_offsets: Sequence[int], doc_src_start: Sequence[int],
                    dst_start: Sequence[int], kept: Sequence[int], theta: float,
                    layout: int = ROPE_HALF) -> np.ndarray:
    """Eq. 5 applied to a packed key store `k_store[T, Hkv, D]`: token t of kept document
    i was encoded at src_start[i] + t and is re-encoded at dst_start[i] + t, i.e. rotated
    by delta_i = dst_start[i] - src_start[i].  Values are unchanged; rows of documents not
    in `kept` are returned as they are.  Output is float64."""
    out = np.array(k_store, dtype=np.float64, copy=True)
    for i in kept:
        lo, hi = int(doc_offsets[i]), int(doc_offsets[i + 1])
        delta = float(int(dst_start[i]) - int(doc_src_start[i]))
        out[lo:hi] = rope_rotate(out[lo:hi], np.full(out[lo:hi].shape[:-1], delta), theta, layout)
    return out


# --------------------------------------------------------------------------- attention
def query_prefill_attn(q: np.ndarray, k_rot: np.ndarray, v_store: np.ndarray,
                       doc_offsets: Sequence[int], kept: Sequence[int], n_docs: int,
                       scale: Optional[float] = None, doc_base: int = 0
                       ) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """Eq. 1 for the query rows over the kept documents' caches, plus document scores.

    q[Lq, Hq, D]; k_rot, v_store[T, Hkv, D] (keys already re-positioned); query head h
    reads key/value head h // (Hq // Hkv).  `kept` holds ids local to the request,
    `doc_offsets[doc_base + i]` is the first store row of local document i.
    Returns out[Lq, Hq, D], lse[Hq, Lq] (natural log of the softmax denominator),
    mass[Hq, Lq, n_docs] (softmax probability falling on each document's tokens) and
    doc_scores[n_docs] = mean of mass over heads and query rows (0 for documents not kept).
    The softmax runs over exactly the tokens of the kept documents."""
    q = np.asarray(q, dtype=np.float64)
    lq, hq, d = q.shape
    hkv = k_rot.shape[1]
    g = hq // hkv
    if scale is None or scale == 0.0:
        scale = 1.0 / math.sqrt(d)
    rows: List[np.ndarray] = []
    seg: List[Tuple[int, int, int]] = []
    pos = 0
    for i in kept:
        lo, hi = int(doc_offsets[doc_base + i]), int(doc_offsets[doc_base + i + 1])
        rows.append(np.arange(lo, hi))
        seg.append((int(i), pos, pos + hi - lo))
        pos += hi - lo
    out = np.zeros((lq, hq, d))
    lse = np.full((hq, lq), -np.inf)
    mass = np.zeros((hq, lq, n_docs))
    if pos == 0:
        return out, lse, mass, np.zeros(n_docs)
    sel = np.concatenate(rows)
    k_sel = np.asarray(k_rot, dtype=np.float64)[sel]
    v_sel = np.asarray(v_store, dtype=np.float64)[sel]
    for h in range(hq):
        kvh = h // g
        s = (q[:, h, :] @ k_sel[:, kvh, :].T) * scale
        m = s.max(axis=1, keepdims=True)
        e = np.exp(s - m)
        denom = e.sum(axis=1, keepdims=True)
        p = e / denom
        out[:, h, :] = p @ v_sel[:, kvh, :]
        lse[h] = (m + np.log(denom))[:, 0]
        for i, a, b in seg:
            mass[h, :, i] = p[:, a:b].sum(axis=1)
    doc_scores = mass.sum(axis=(0, 1)) / float(hq * lq)
    return out, lse, mass, doc_scores


# ----------------------------------------------------------------------------- pruning
def query_self_block(q: np.ndarray, k_self: np.ndarray, v_self: np.ndarray,
                     scale: Optional[float] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 1 for the query tokens over their own keys and values, with the causal mask the footnote
    to Eq. 1 refers to: query row j sees the query tokens 0..j.

    q[Lq, Hq, D]; k_self, v_self[Lq, Hkv, D] (keys encoded at the query's positions).
    Returns out[Lq, Hq, D] and lse[Hq, Lq] of this block alone."""
    q = np.asarray(q, dtype=np.float64)
    k_self = np.asarray(k_self, dtype=np.float64)
    v_self = np.asarray(v_self, dtype=np.float64)
    lq, hq, d = q.shape
    g = hq // k_self.shape[1]
    if scale is None or scale == 0.0:
        scale = 1.0 / math.sqrt(d)
    out = np.zeros((lq, hq, d))
    lse = np.zeros((hq, lq))
    for h in range(hq):
        kvh = h // g
        for j in range(lq):
            s = (k_self[:j + 1, kvh, :] @ q[j, h, :]) * scale
            m = s.max()
            e = np.exp(s - m)
            out[j, h, :] = (e / e.sum()) @ v_self[:j + 1, kvh, :]
            lse[h, j] = m + math.log(e.sum())
    return out, lse


def merge_softmax_blocks(out_a: np.ndarray, lse_a: np.ndarray, out_b: np.ndarray, lse_b: np.ndarray
                         ) -> Tuple[np.ndarray, np.ndarray]:
    """Softmax attention over the union of two disjoint key sets from the results over each:
    the outputs are averaged with weights exp(lse) (out[Lq, Hq, D], lse[Hq, Lq])."""
    lse = np.logaddexp(lse_a, lse_b)
    wa = np.exp(lse_a - lse).T[:, :, None]
    wb = np.exp(lse_b - lse).T[:, :, None]
    return wa * out_a + wb * out_b, lse


def document_prefill_attn(q_doc: np.ndarray, k_doc: np.ndarray, v_doc: np.ndarray,
                           k_prefix: Optional[np.ndarray] = None, v_prefix: Optional[np.ndarray] = None,
                           scale: Optional[float] = None) -> Tuple[np.ndarray, np.ndarray]:
    """The attention inside the offline cache construction C_d <- LLM(C_prefix, d) of Sec. 2.2 (the two
    unnumbered equations there; O(l_c^2 k) in the complexity paragraph of Sec. 3.3), one layer, one
    document: token t of the document attends the shared prefix cache and the document's own tokens
    0..t under the causal mask of Eq. 1; other documents are invisible (documents are cached in
    parallel, independently of each other and of any query).

    q_doc[len, Hq, D]; k_doc, v_doc[len, Hkv, D]; k_prefix, v_prefix[P, Hkv, D] or None (P = 0).
    Queries and keys are taken as already rotary-encoded (prefix at 0..P-1, the document right behind
    it).  Returns out[len, Hq, D] and lse[Hq, len]."""
    q_doc = np.asarray(q_doc, dtype=np.float64)
    k_doc = np.asarray(k_doc, dtype=np.float64)
    v_doc = np.asarray(v_doc, dtype=np.float64)
    n, hq, d = q_doc.shape
    hkv = k_doc.shape[1]
    g = hq // hkv
    if k_prefix is None or len(k_prefix) == 0:
        k_prefix = np.zeros((0, hkv, d))
        v_prefix = np.zeros((0, hkv, d))
    k_all = np.concatenate([np.asarray(k_prefix, dtype=np.float64), k_doc])
    v_all = np.concatenate([np.asarray(v_prefix, dtype=np.float64), v_doc])
    p_len = k_all.shape[0] - n
    if scale is None or scale == 0.0:
        scale = 1.0 / math.sqrt(d)
    out = np.zeros((n, hq, d))
    lse = np.zeros((hq, n))
    for h in range(hq):
        kvh = h // g
        for t in range(n):
            vis = p_len + t + 1                               # the prefix, then document tokens 0..t
            s = (k_all[:vis, kvh, :] @ q_doc[t, h, :]) * scale
            m = s.max()
            e = np.exp(s - m)
            out[t, h, :] = (e / e.sum()) @ v_all[:vis, kvh, :]
            lse[h, t] = m + math.log(e.sum())
    return out, lse


def assemble_final_cache(k_rot: np.ndarray, v_store: np.ndarray, doc_offsets: Sequence[int],
                         order: Sequence[int], k_self: np.ndarray, v_self: np.ndarray, doc_base: int = 0
                         ) -> Tuple[np.ndarray, np.ndarray]:
    """Algorithm 2, Phase 2 for one layer of one request: the re-positioned keys and the values of the
    surviving documents in rank order, then the query tokens' own keys and values (C_Q, unchanged).
    k_rot, v_store[T, Hkv, D]; k_self, v_self[Lq, Hkv, D].  Returns (K_final, V_final)."""
    ks, vs = [], []
    for i in order:
        lo, hi = int(doc_offsets[doc_base + i]), int(doc_offsets[doc_base + i + 1])
        ks.append(np.asarray(k_rot, dtype=np.float64)[lo:hi])
        vs.append(np.asarray(v_store, dtype=np.float64)[lo:hi])
    ks.append(np.asarray(k_self, dtype=np.float64))
    vs.append(np.asarray(v_self, dtype=np.float64))
    return np.concatenate(ks), np.concatenate(vs)


def decode_steps(k_final: np.ndarray, v_final: np.ndarray, q_new: np.ndarray, k_new: np.ndarray,
                 v_new: np.ndarray, scale: Optional[float] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Decoding over a final cache (Algorithm 2, Phase 3: Y <- LLM(C_final); the "Decoding" loop of
    Algorithm 1), one layer, one request, attention only: step t appends the new token's key and value
    to the cache (K <- concat(K_past, K_current) in the text under Eq. 1) and the token's single query
    row per head attends every row of the cache, its own included (Eq. 1).

    k_final, v_final[n, Hkv, D] (keys already at their final positions); q_new[a, Hq, D];
    k_new, v_new[a, Hkv, D] with the keys rotary-encoded at the tokens' own positions.
    Returns out[a, Hq, D] and lse[a, Hq]."""
    k_cache = np.asarray(k_final, dtype=np.float64)
    v_cache = np.asarray(v_final, dtype=np.float64)
    q_new = np.asarray(q_new, dtype=np.float64)
    a, hq, d = q_new.shape
    g = hq // k_cache.shape[1]
    if scale is None or scale == 0.0:
        scale = 1.0 / math.sqrt(d)
    out = np.zeros((a, hq, d))
    lse = np.zeros((a, hq))
    for t in range(a):
        k_cache = np.concatenate([k_cache, np.asarray(k_new[t], dtype=np.float64)[None]])
        v_cache = np.concatenate([v_cache, np.asarray(v_new[t], dtype=np.float64)[None]])
        for h in range(hq):
            s = (k_cache[:, h // g, :] @ q_new[t, h, :]) * scale
            m = s.max()
            e = np.exp(s - m)
            out[t, h, :] = (e / e.sum()) @ v_cache[:, h // g, :]
            lse[t, h] = m + math.log(e.sum())
    return out, lse


def prune_topk(score_accum: Sequence[float], order: Sequence[int], keep: int, strategy: int
               ) -> List[int]:
    """Algorithm 2, pruning step: among the documents in `order` keep the `keep` with the
    largest accumulated score (ties: lower id wins) and return their new order.
    "align" and "none" leave survivors in their previous relative order; "sort" orders
    them by accumulated score, best first (rank 0 sits next to the query)."""
    order = [int(i) for i in order]
    keep = min(keep, len(order))
    ranked = sorted(order, key=lambda i: (-float(score_accum[i]), i))
    survivors = set(ranked[:keep])
    if strategy == ALLOC_SORT:
        return ranked[:keep]
    return [i for i in order if i in survivors]


def prune_schedule_linear(n_layers: int, every: int, k: int, k_finish: int) -> List[Tuple[int, int]]:
    """App. C: pruning after every `every`-th layer (1-based), removing
    k_prune = (k - k_finish) / (L / n) documents each time; a remainder of the division
    is removed at the last pruning layer so exactly k_finish remain."""
    n_prunes = n_layers // every
    if n_prunes == 0:
        return []
    k_prune = (k - k_finish) // n_prunes
    out = []
    kept = k
    for j in range(1, n_prunes + 1):
        kept = k_finish if j == n_prunes else kept - k_prune
        out.append((j * every, kept))
    return out


# --------------------------------------------------------------------------- the stack
def run_stack(q_layers: np.ndarray, k_store: np.ndarray, v_store: np.ndarray,
              doc_len: Sequence[int], doc_offsets: Sequence[int], doc_src_start: Sequence[int],
              theta: float, pos_range: int, schedule: Sequence[Tuple[int, int]], strategy: int,
              tail_reserve: int, prefix_len: int = 0, n_reuse: int = 0,
              order0: Optional[Sequence[int]] = None, layout: int = ROPE_HALF,
              scale: Optional[float] = None, doc_base: int = 0, final_reposition: bool = True,
              key_round=None) -> Dict[str, object]:
    """Algorithm 2 for one request.  `q_layers[L, Lq, Hq, D]` holds each layer's query
    states (the projections and feed-forward blocks that would produce them are outside
    this path); `k_store`, `v_store[L, T, Hkv, D]`; `doc_len`, `doc_src_start` are the
    request's own documents, `doc_offsets[doc_base + i]` their first store rows.

    Per layer l = 1..L: re-position the kept caches, attend, S += s^l; after a layer
    named in `schedule` keep the top documents and re-allocate them (same query start).
    Phase 2 re-positions the final survivors in every layer.

    `key_round`, if given, is applied to the re-positioned keys before a layer attends them: the
    re-positioned cache of Eq. 5 is again a cache and may be held in the cache's storage type (a
    rounding function such as round_to_bf16); by default the keys stay exact."""
    n_layers = q_layers.shape[0]
    n_docs = len(doc_len)
    order = list(range(n_docs)) if order0 is None else [int(i) for i in order0]
    sched = {int(l): int(keep) for l, keep in schedule}
    local_off = [int(doc_offsets[doc_base + i]) for i in range(n_docs + 1)]
    dst, group, n_reuse_used, qs = allocate_positions(doc_len, order, pos_range, prefix_len,
                                                      tail_reserve, n_reuse, -1)
    accum = np.zeros(n_docs)
    layers = []
    for l in range(1, n_layers + 1):
        k_rot = reposition_keys(k_store[l - 1], local_off, doc_src_start, dst, order, theta, layout)
        if key_round is not None:
            k_rot = key_round(k_rot)
        out, lse, mass, scores = query_prefill_attn(q_layers[l - 1], k_rot, v_store[l - 1],
                                                    local_off, order, n_docs, scale)
        accum = accum + scores
        rec = {"out": out, "lse": lse, "doc_scores": scores, "score_accum": accum.copy(),
               "order_in": list(order), "dst_start": dst.copy(), "n_reuse": n_reuse_used}
        if l in sched:
            order = prune_topk(accum, order, sched[l], strategy)
            if strategy == ALLOC_NONE:
                kept = set(order)
                dst = np.array([dst[i] if i in kept else -1 for i in range(n_docs)], dtype=np.int64)
                group = np.array([group[i] if i in kept else -1 for i in range(n_docs)], dtype=np.int64)
            else:
                dst, group, n_reuse_used, _ = allocate_positions(doc_len, order, pos_range, prefix_len,
                                                                 tail_reserve, n_reuse, qs)
            rec["order_out"] = list(order)
        layers.append(rec)
    result: Dict[str, object] = {"layers": layers, "order": list(order), "dst_start": dst,
                                 "group": group, "query_start": qs, "score_accum": accum,
                                 "n_reuse": n_reuse_used}
    if final_reposition:
        result["k_final"] = [reposition_keys(k_store[l], local_off, doc_src_start, dst, order, theta, layout)
                             for l in range(n_layers)]
    return result
