"""Pins for the oracle's decoding steps over a final cache (Algorithm 2, Phase 3; Algorithm 1, decoding loop)."""
import numpy as np
import pytest
import torch

import oracle


def _case(seed, n, a, hq, hkv, d):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((n, hkv, d)), rng.standard_normal((n, hkv, d)), rng.standard_normal((a, hq, d)),
            rng.standard_normal((a, hkv, d)), rng.standard_normal((a, hkv, d)))


@pytest.mark.parametrize("n,a,hq,hkv", [(9, 4, 4, 2), (1, 3, 2, 2), (17, 1, 6, 1), (0, 5, 3, 3)])
def test_steps_are_rows_of_a_library_causal_attention(n, a, hq, hkv):
    """Causal attention of a library routine over the sequence [cache rows ; new tokens]: the rows of the new
    tokens are the decoding steps (token t sees the cache and the new tokens 0..t)."""
    d = 16
    kf, vf, q, kn, vn = _case(3 * n + a, n, a, hq, hkv, d)
    out, lse = oracle.decode_steps(kf, vf, q, kn, vn)
    g = hq // hkv
    q_all = np.concatenate([np.zeros((n, hq, d)), q])
    k_all = np.repeat(np.concatenate([kf, kn]), g, axis=1)
    v_all = np.repeat(np.concatenate([vf, vn]), g, axis=1)
    t = lambda x: torch.from_numpy(x).permute(1, 0, 2)[None]               # [1, heads, seq, d]
    ref = torch.nn.functional.scaled_dot_product_attention(t(q_all), t(k_all), t(v_all), is_causal=True)
    assert np.allclose(out, ref[0].permute(1, 0, 2).numpy()[n:], atol=1e-12)


def test_zero_query_gives_the_mean_of_the_values_seen_so_far():
    kf, vf, q, kn, vn = _case(5, 6, 3, 4, 2, 8)
    out, lse = oracle.decode_steps(kf, vf, np.zeros_like(q), kn, vn, scale=0.7)
    for t in range(3):
        seen = np.concatenate([vf, vn[:t + 1]])
        for h in range(4):
            assert np.allclose(out[t, h], seen[:, h // 2].mean(axis=0), atol=1e-13)
            assert abs(lse[t, h] - np.log(6 + t + 1)) < 1e-13


def test_a_step_equals_the_pinned_query_attention_over_the_grown_cache():
    """Step t against query_prefill_attn (itself pinned by loops, closed forms and a library routine) given
    the cache with the first t + 1 new rows appended as one document."""
    kf, vf, q, kn, vn = _case(11, 10, 4, 6, 2, 16)
    out, lse = oracle.decode_steps(kf, vf, q, kn, vn, scale=0.21)
    for t in range(4):
        k_all, v_all = np.concatenate([kf, kn[:t + 1]]), np.concatenate([vf, vn[:t + 1]])
        o_ref, lse_ref, _, _ = oracle.query_prefill_attn(q[t:t + 1], k_all, v_all, [0, len(k_all)], [0], 1, scale=0.21)
        assert np.allclose(out[t], o_ref[0], atol=1e-12) and np.allclose(lse[t], lse_ref[:, 0], atol=1e-12)


def test_the_newest_token_is_attended_and_later_ones_are_not():
    kf, vf, q, kn, vn = _case(2, 4, 3, 2, 2, 8)
    base, _ = oracle.decode_steps(kf, vf, q, kn, vn)
    vn2 = vn.copy()
    vn2[2] += 100.0                                        # only the last step may notice
    moved, _ = oracle.decode_steps(kf, vf, q, kn, vn2)
    assert np.array_equal(base[:2], moved[:2]) and not np.allclose(base[2], moved[2])
    vn3 = vn.copy()
    vn3[0] += 100.0                                        # every step sees the first new token
    moved, _ = oracle.decode_steps(kf, vf, q, kn, vn3)
    assert all(not np.allclose(base[t], moved[t]) for t in range(3))
