"""Pins for the oracle's attention, document scores and the layer loop (Eq. 1, Algorithm 2)."""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import ALLOC_ALIGN, ALLOC_NONE, ALLOC_SORT


def _rng(seed):
    return np.random.default_rng(seed)


def _case(seed, lens, hq=4, hkv=2, d=16, lq=3):
    rng = _rng(seed)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(int)
    q = rng.standard_normal((lq, hq, d))
    k = rng.standard_normal((off[-1], hkv, d))
    v = rng.standard_normal((off[-1], hkv, d))
    return q, k, v, off


def test_brute_force_loops():
    lens = [3, 5, 2, 4]
    q, k, v, off = _case(0, lens)
    kept = [2, 0, 3]
    out, lse, mass, scores = oracle.query_prefill_attn(q, k, v, off, kept, len(lens))
    lq, hq, d = q.shape
    g = hq // k.shape[1]
    for h in range(hq):
        for j in range(lq):
            logits, owner, vals = [], [], []
            for i in kept:
                for t in range(off[i], off[i + 1]):
                    acc = 0.0
                    for c in range(d):
                        acc += q[j, h, c] * k[t, h // g, c]
                    logits.append(acc / math.sqrt(d))
                    owner.append(i)
                    vals.append(v[t, h // g])
            denom = sum(math.exp(x) for x in logits)
            probs = [math.exp(x) / denom for x in logits]
            expect = sum(p * val for p, val in zip(probs, vals))
            assert np.allclose(out[j, h], expect, atol=1e-12)
            assert math.isclose(lse[h, j], math.log(denom), abs_tol=1e-12)
            for i in range(len(lens)):
                m = sum(p for p, o in zip(probs, owner) if o == i)
                assert math.isclose(mass[h, j, i], m, abs_tol=1e-12)
    assert scores[1] == 0.0
    assert np.allclose(scores, mass.mean(axis=(0, 1)))


def test_masses_and_scores_sum_to_one():
    lens = [7, 1, 12, 5, 9]
    q, k, v, off = _case(1, lens, hq=6, hkv=2, d=32, lq=5)
    out, lse, mass, scores = oracle.query_prefill_attn(q, k, v, off, [4, 1, 0, 2], len(lens))
    assert np.allclose(mass.sum(axis=2), 1.0, atol=1e-13)
    assert math.isclose(scores.sum(), 1.0, abs_tol=1e-13)
    assert scores[3] == 0.0
    # a single kept document takes all the mass
    _, _, _, single = oracle.query_prefill_attn(q, k, v, off, [2], len(lens))
    assert math.isclose(single[2], 1.0, abs_tol=1e-14) and single.sum() == single[2]


def test_zero_query_closed_form():
    # Q = 0 gives uniform attention: score_i = len_i / T, output = mean of the kept values
    lens = [4, 10, 6]
    q, k, v, off = _case(2, lens)
    q[:] = 0.0
    out, lse, mass, scores = oracle.query_prefill_attn(q, k, v, off, [0, 1, 2], 3)
    assert np.allclose(scores, np.array(lens) / 20.0, atol=1e-14)
    assert np.allclose(lse, math.log(20.0), atol=1e-14)
    g = q.shape[1] // k.shape[1]
    for h in range(q.shape[1]):
        assert np.allclose(out[:, h], v[:, h // g].mean(axis=0), atol=1e-13)


def test_duplicate_documents_score_equally_and_order_is_irrelevant():
    lens = [6, 6, 3]
    q, k, v, off = _case(3, lens)
    k[off[1]:off[2]] = k[off[0]:off[1]]
    v[off[1]:off[2]] = v[off[0]:off[1]]
    o1, l1, m1, s1 = oracle.query_prefill_attn(q, k, v, off, [0, 1, 2], 3)
    o2, l2, m2, s2 = oracle.query_prefill_attn(q, k, v, off, [2, 1, 0], 3)
    assert math.isclose(s1[0], s1[1], rel_tol=1e-13)
    assert np.allclose(o1, o2, atol=1e-13) and np.allclose(s1, s2, atol=1e-14) and np.allclose(l1, l2)


def test_gqa_equals_mha_on_repeated_heads():
    lens = [5, 8]
    q, k, v, off = _case(4, lens, hq=6, hkv=2, d=16, lq=4)
    o_gqa, lse_gqa, _, s_gqa = oracle.query_prefill_attn(q, k, v, off, [0, 1], 2)
    k_rep, v_rep = np.repeat(k, 3, axis=1), np.repeat(v, 3, axis=1)      # head h reads kv head h // 3
    o_mha, lse_mha, _, s_mha = oracle.query_prefill_attn(q, k_rep, v_rep, off, [0, 1], 2)
    assert np.allclose(o_gqa, o_mha, atol=1e-14) and np.allclose(s_gqa, s_mha, atol=1e-15)


def _textbook_rope(x, pos, theta):
    d = x.shape[-1]
    freq = theta ** (-2.0 * np.arange(d // 2) / d)
    z = (x[..., : d // 2] + 1j * x[..., d // 2:]) * np.exp(1j * pos[..., None] * freq)
    return np.concatenate([z.real, z.imag], axis=-1)


@pytest.mark.parametrize("theta", [1e4, 1e6])
def test_single_window_equals_library_attention(theta):
    """With N_reuse = 1 and no prefix the path is ordinary rotary attention of the query
    tokens over one contiguous sequence: raw keys encoded directly at their final positions,
    fed to a library attention routine."""
    rng = _rng(5)
    lens = [9, 14, 6, 11]
    hq, hkv, d, lq = 4, 2, 32, 5
    off = np.concatenate([[0], np.cumsum(lens)]).astype(int)
    total = off[-1]
    raw_k = rng.standard_normal((total, hkv, d))
    v = rng.standard_normal((total, hkv, d))
    raw_q = rng.standard_normal((lq, hq, d))
    src = [0, 0, 0, 0]
    cached = np.empty_like(raw_k)
    for i, n in enumerate(lens):
        pos = (src[i] + np.arange(n, dtype=np.float64))[:, None] * np.ones((1, hkv))
        cached[off[i]:off[i + 1]] = _textbook_rope(raw_k[off[i]:off[i + 1]], pos, theta)
    order = [1, 3, 0, 2]
    dst, group, n_reuse, qs = oracle.allocate_positions(lens, order, 4096, tail_reserve=lq, n_reuse=1,
                                                        query_start=total)
    assert n_reuse == 1 and qs == total
    q_enc = _textbook_rope(raw_q, (qs + np.arange(lq, dtype=np.float64))[:, None] * np.ones((1, hq)), theta)
    k_rot = oracle.reposition_keys(cached, off, src, dst, order, theta)
    out, lse, mass, scores = oracle.query_prefill_attn(q_enc, k_rot, v, off, order, len(lens))
    # textbook: the sequence is the documents laid out by final position
    seq_k = np.empty_like(raw_k)
    seq_v = np.empty_like(v)
    for i, n in enumerate(lens):
        pos = (dst[i] + np.arange(n, dtype=np.float64))[:, None] * np.ones((1, hkv))
        seq_k[dst[i]:dst[i] + n] = _textbook_rope(raw_k[off[i]:off[i + 1]], pos, theta)
        seq_v[dst[i]:dst[i] + n] = v[off[i]:off[i + 1]]
    tq = torch.from_numpy(q_enc).permute(1, 0, 2)[None]                       # [1, Hq, Lq, D]
    tk = torch.from_numpy(np.repeat(seq_k, hq // hkv, axis=1)).permute(1, 0, 2)[None]
    tv = torch.from_numpy(np.repeat(seq_v, hq // hkv, axis=1)).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)[0].permute(1, 0, 2).numpy()
    assert np.allclose(out, ref, atol=1e-11)


def test_shift_invariance_of_positions():
    # shifting every destination position and the query positions by a constant changes nothing
    rng = _rng(6)
    lens = [7, 5, 9]
    hq, hkv, d, lq, theta = 2, 1, 32, 4, 1e4
    off = np.concatenate([[0], np.cumsum(lens)]).astype(int)
    cached = rng.standard_normal((off[-1], hkv, d))
    v = rng.standard_normal((off[-1], hkv, d))
    raw_q = rng.standard_normal((lq, hq, d))
    src = [0, 0, 0]
    results = []
    for shift in (0, 100, 1234):
        dst = np.array([20, 5, 27]) + shift
        qs = 40 + shift
        q_enc = oracle.rope_rotate(raw_q, (qs + np.arange(lq, dtype=np.float64))[:, None] * np.ones((1, hq)), theta)
        k_rot = oracle.reposition_keys(cached, off, src, dst, [0, 1, 2], theta)
        results.append(oracle.query_prefill_attn(q_enc, k_rot, v, off, [0, 1, 2], 3))
    for r in results[1:]:
        assert np.allclose(r[0], results[0][0], atol=1e-9)
        assert np.allclose(r[3], results[0][3], atol=1e-10)


def _stack_case(seed, n_docs=6, n_layers=4, hq=4, hkv=2, d=16, lq=3):
    rng = _rng(seed)
    lens = rng.integers(3, 9, size=n_docs)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(int)
    q = rng.standard_normal((n_layers, lq, hq, d))
    k = rng.standard_normal((n_layers, off[-1], hkv, d))
    v = rng.standard_normal((n_layers, off[-1], hkv, d))
    return lens, off, q, k, v


@pytest.mark.parametrize("strategy", [ALLOC_NONE, ALLOC_ALIGN, ALLOC_SORT])
def test_stack_follows_algorithm2(strategy):
    lens, off, q, k, v = _stack_case(7)
    n_docs, n_layers = len(lens), q.shape[0]
    sched = [(2, 4), (3, 2)]
    res = oracle.run_stack(q, k, v, lens, off, [0] * n_docs, 1e4, 64, sched, strategy, tail_reserve=3)
    # replay by hand, layer by layer
    order = list(range(n_docs))
    dst, group, n_reuse, qs = oracle.allocate_positions(lens, order, 64, 0, 3)
    accum = np.zeros(n_docs)
    for l in range(1, n_layers + 1):
        rec = res["layers"][l - 1]
        assert rec["order_in"] == order
        k_rot = oracle.reposition_keys(k[l - 1], off, [0] * n_docs, dst, order, 1e4)
        out, lse, mass, s = oracle.query_prefill_attn(q[l - 1], k_rot, v[l - 1], off, order, n_docs)
        accum += s                                            # S <- S + s^l, never reset
        assert np.allclose(rec["out"], out) and np.allclose(rec["score_accum"], accum)
        for i in range(n_docs):
            if i not in order:
                assert rec["doc_scores"][i] == 0.0            # pruned documents are not attended
        if l in dict(sched):
            order = oracle.prune_topk(accum, order, dict(sched)[l], strategy)
            if strategy == ALLOC_NONE:
                dst = np.array([dst[i] if i in order else -1 for i in range(n_docs)])
            else:
                dst, group, n_reuse, _ = oracle.allocate_positions(lens, order, 64, 0, 3, 0, qs)
    assert res["order"] == order and len(order) == 2
    assert np.array_equal(res["dst_start"], dst)
    # Phase 2: survivors re-positioned in every layer, everything else untouched
    for l in range(n_layers):
        expect = oracle.reposition_keys(k[l], off, [0] * n_docs, dst, order, 1e4)
        assert np.array_equal(res["k_final"][l], expect)
    if strategy == ALLOC_NONE:
        first = res["layers"][0]["dst_start"]
        assert all(res["dst_start"][i] == first[i] for i in order)       # positions never moved
    else:
        ends = sorted(int(res["dst_start"][i]) + int(lens[i]) for i in order)
        assert ends[-1] == res["query_start"]                            # re-packed next to the query
    if strategy == ALLOC_SORT:
        final = [res["score_accum"][i] for i in order]
        # order was fixed at the last pruning layer (layer 3) from the scores of that time
        at_prune = res["layers"][2]["score_accum"]
        assert [at_prune[i] for i in order] == sorted([at_prune[i] for i in order], reverse=True)
        assert len(final) == 2


def test_self_block_and_merge_equal_textbook_causal_attention():
    """Documents in one window (N_reuse = 1) followed by the query: attention of the query rows over
    the re-positioned caches, merged with the causal query-self block, is ordinary causal attention
    over the whole sequence with every key encoded directly at its final position (library routine)."""
    import torch
    rng = np.random.default_rng(5)
    hq, hkv, d, lq, theta = 4, 2, 16, 6, 1e4
    doc_len = [5, 9, 3]
    offsets = np.concatenate([[0], np.cumsum(doc_len)])
    total = int(offsets[-1])
    raw_k = rng.standard_normal((total, hkv, d))
    v_docs = rng.standard_normal((total, hkv, d))
    raw_q = rng.standard_normal((lq, hq, d))
    raw_kq = rng.standard_normal((lq, hkv, d))
    v_q = rng.standard_normal((lq, hkv, d))
    src = [0, 0, 0]
    def at(x, first):                                              # encode token t of x at position first + t
        return oracle.rope_rotate(x, (first + np.arange(x.shape[0]))[:, None] * np.ones((1, x.shape[1])), theta)
    k_store = np.concatenate([at(raw_k[offsets[i]:offsets[i + 1]], src[i]) for i in range(3)])
    order = [2, 0, 1]
    dst, _, n_reuse, qs = oracle.allocate_positions(doc_len, order, 64, n_reuse=1, query_start=40)
    assert n_reuse == 1
    k_rot = oracle.reposition_keys(k_store, offsets, src, dst, order, theta)
    q = at(raw_q, qs)
    k_self = at(raw_kq, qs)
    o_docs, lse_docs, _, _ = oracle.query_prefill_attn(q, k_rot, v_docs, offsets, order, 3)
    o_self, lse_self = oracle.query_self_block(q, k_self, v_q)
    o_full, lse_full = oracle.merge_softmax_blocks(o_docs, lse_docs, o_self, lse_self)
    # the same thing as one sequence: documents sorted by position, then the query tokens
    by_pos = sorted(range(3), key=lambda i: dst[i])
    keys = np.concatenate([at(raw_k[offsets[i]:offsets[i + 1]], dst[i]) for i in by_pos] + [k_self])
    vals = np.concatenate([v_docs[offsets[i]:offsets[i + 1]] for i in by_pos] + [v_q])
    n = keys.shape[0]
    q_all = np.zeros((n, hq, d))
    q_all[n - lq:] = q
    g = hq // hkv
    qt = torch.from_numpy(q_all).permute(1, 0, 2)                      # [Hq, n, D]
    kt = torch.from_numpy(keys).permute(1, 0, 2).repeat_interleave(g, dim=0)
    vt = torch.from_numpy(vals).permute(1, 0, 2).repeat_interleave(g, dim=0)
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True).permute(1, 0, 2).numpy()
    assert np.allclose(o_full, ref[n - lq:], atol=1e-12)
    # the merged denominator is the denominator over the union
    s = np.einsum("jhd,thd->hjt", q, np.repeat(keys, g, axis=1)) / np.sqrt(d)
    mask = np.arange(n)[None, :] <= (n - lq + np.arange(lq))[:, None]
    lse_ref = np.log(np.where(mask[None], np.exp(s), 0.0).sum(axis=2))
    assert np.allclose(lse_full, lse_ref, atol=1e-12)


def test_merge_of_two_halves_is_attention_over_the_whole():
    rng = np.random.default_rng(6)
    lq, hq, d, t = 3, 2, 8, 10
    q = rng.standard_normal((lq, hq, d))
    k = rng.standard_normal((t, hq, d))
    v = rng.standard_normal((t, hq, d))
    whole = oracle.query_prefill_attn(q, k, v, [0, t], [0], 1)
    a = oracle.query_prefill_attn(q, k[:4], v[:4], [0, 4], [0], 1)
    b = oracle.query_prefill_attn(q, k[4:], v[4:], [0, 6], [0], 1)
    out, lse = oracle.merge_softmax_blocks(a[0], a[1], b[0], b[1])
    assert np.allclose(out, whole[0], atol=1e-13) and np.allclose(lse, whole[1], atol=1e-13)


def test_assembled_final_cache_holds_the_pieces_in_order():
    rng = np.random.default_rng(7)
    hkv, d, lq = 2, 8, 3
    doc_len = [4, 2, 5]
    offsets = np.concatenate([[0], np.cumsum(doc_len)])
    k_rot = rng.standard_normal((11, hkv, d))
    v = rng.standard_normal((11, hkv, d))
    k_self = rng.standard_normal((lq, hkv, d))
    v_self = rng.standard_normal((lq, hkv, d))
    order = [2, 0]                                                   # document 1 was pruned
    kf, vf = oracle.assemble_final_cache(k_rot, v, offsets, order, k_self, v_self)
    assert kf.shape == (5 + 4 + lq, hkv, d)
    assert np.array_equal(kf[:5], k_rot[6:11]) and np.array_equal(kf[5:9], k_rot[0:4]) and np.array_equal(kf[9:], k_self)
    assert np.array_equal(vf[:5], v[6:11]) and np.array_equal(vf[5:9], v[0:4]) and np.array_equal(vf[9:], v_self)
    # a later token attending the assembled cache = the survivors' caches and the query block, merged
    q_new = rng.standard_normal((1, 4, d))
    whole = oracle.query_prefill_attn(q_new, kf, vf, [0, kf.shape[0]], [0], 1)
    docs = oracle.query_prefill_attn(q_new, k_rot, v, offsets, order, 3)
    tail = oracle.query_prefill_attn(q_new, k_self, v_self, [0, lq], [0], 1)
    out, lse = oracle.merge_softmax_blocks(docs[0], docs[1], tail[0], tail[1])
    assert np.allclose(out, whole[0], atol=1e-13) and np.allclose(lse, whole[1], atol=1e-13)
