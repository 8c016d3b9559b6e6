"""Pins for the oracle's cache-construction attention (Sec. 2.2: C_d <- LLM(C_prefix, d))."""
import math

import numpy as np
import pytest
import torch

import oracle


def _case(seed, n, p_len, hq=4, hkv=2, d=16):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((n, hq, d)), rng.standard_normal((n, hkv, d)), rng.standard_normal((n, hkv, d)),
            rng.standard_normal((p_len, hkv, d)), rng.standard_normal((p_len, hkv, d)))


@pytest.mark.parametrize("n,p_len,hq,hkv", [(7, 3, 4, 2), (12, 0, 2, 2), (1, 5, 6, 2), (9, 9, 3, 1)])
def test_equals_library_causal_attention_over_prefix_and_document(n, p_len, hq, hkv):
    """One causal softmax attention over the sequence [prefix ; document] by a library routine; the rows of
    the document are what the oracle returns (the prefix rows' own queries are irrelevant to them)."""
    d = 16
    q, k, v, kp, vp = _case(n + p_len, n, p_len, hq, hkv, d)
    out, lse = oracle.document_prefill_attn(q, k, v, kp, vp)
    g = hq // hkv
    q_all = np.concatenate([np.zeros((p_len, hq, d)), q])
    k_all = np.repeat(np.concatenate([kp, k]), g, axis=1)
    v_all = np.repeat(np.concatenate([vp, v]), g, axis=1)
    t = lambda x: torch.from_numpy(x).permute(1, 0, 2)[None]               # [1, heads, seq, d]
    ref = torch.nn.functional.scaled_dot_product_attention(t(q_all), t(k_all), t(v_all), is_causal=True)
    ref = ref[0].permute(1, 0, 2).numpy()[p_len:]
    assert np.allclose(out, ref, atol=1e-12)


def test_brute_force_loops():
    n, p_len, hq, hkv, d = 5, 2, 4, 2, 8
    q, k, v, kp, vp = _case(1, n, p_len, hq, hkv, d)
    out, lse = oracle.document_prefill_attn(q, k, v, kp, vp, scale=0.3)
    for h in range(hq):
        kv = h // 2
        for t in range(n):
            keys = [kp[i, kv] for i in range(p_len)] + [k[i, kv] for i in range(t + 1)]
            vals = [vp[i, kv] for i in range(p_len)] + [v[i, kv] for i in range(t + 1)]
            logits = [0.3 * sum(q[t, h, c] * key[c] for c in range(d)) for key in keys]
            denom = sum(math.exp(x) for x in logits)
            expect = sum(math.exp(x) / denom * val for x, val in zip(logits, vals))
            assert np.allclose(out[t, h], expect, atol=1e-12)
            assert math.isclose(lse[h, t], math.log(denom), abs_tol=1e-12)


def test_zero_query_closed_form():
    # uniform weights: token t averages the prefix values and the document's values 0..t
    n, p_len = 6, 4
    q, k, v, kp, vp = _case(2, n, p_len)
    q[:] = 0.0
    out, lse = oracle.document_prefill_attn(q, k, v, kp, vp)
    for t in range(n):
        for h in range(4):
            expect = (vp[:, h // 2].sum(axis=0) + v[:t + 1, h // 2].sum(axis=0)) / (p_len + t + 1)
            assert np.allclose(out[t, h], expect, atol=1e-13)
        assert np.allclose(lse[:, t], math.log(p_len + t + 1), atol=1e-13)


def test_first_token_without_prefix_returns_its_own_value():
    q, k, v, _, _ = _case(3, 4, 0)
    out, lse = oracle.document_prefill_attn(q, k, v)
    for h in range(4):
        assert np.allclose(out[0, h], v[0, h // 2], atol=1e-14)
        assert math.isclose(lse[h, 0], float(q[0, h] @ k[0, h // 2]) / math.sqrt(16), abs_tol=1e-13)


def test_later_tokens_and_other_documents_are_invisible():
    n, p_len = 8, 3
    q, k, v, kp, vp = _case(4, n, p_len)
    out, lse = oracle.document_prefill_attn(q, k, v, kp, vp)
    k2, v2 = k.copy(), v.copy()
    k2[5:] += 3.0                                               # tokens 5.. change: rows 0..4 must not
    v2[5:] -= 2.0
    out2, lse2 = oracle.document_prefill_attn(q, k2, v2, kp, vp)
    assert np.array_equal(out[:5], out2[:5]) and np.array_equal(lse[:, :5], lse2[:, :5])
    assert not np.allclose(out[5:], out2[5:])
    # a document's result is the same whether or not it is cut out of a longer packed array
    out3, _ = oracle.document_prefill_attn(q[:4], k[:4], v[:4], kp, vp)
    assert np.allclose(out3, out[:4], atol=1e-14)


def test_is_the_merge_of_the_prefix_block_and_the_causal_self_block():
    """The same result composed from two functions pinned elsewhere: attention over the prefix alone
    (query_prefill_attn with the prefix as its one document) and the causal block of the tokens over
    themselves (query_self_block), joined by merge_softmax_blocks."""
    n, p_len = 9, 5
    q, k, v, kp, vp = _case(5, n, p_len, hq=6, hkv=2, d=32)
    out, lse = oracle.document_prefill_attn(q, k, v, kp, vp)
    o_p, lse_p, _, _ = oracle.query_prefill_attn(q, kp, vp, [0, p_len], [0], 1)
    o_s, lse_s = oracle.query_self_block(q, k, v)
    o_m, lse_m = oracle.merge_softmax_blocks(o_p, lse_p, o_s, lse_s)
    assert np.allclose(out, o_m, atol=1e-12) and np.allclose(lse, lse_m, atol=1e-12)
