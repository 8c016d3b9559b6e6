"""The seeded input generator: reproducible, shaped like the named configurations."""
import numpy as np
import torch

from paper_2502_11101_b200 import workloads as W


def test_metadata_shapes_and_ranges():
    for cid, cfg in W.CONFIGS.items():
        meta = W.make_meta(cfg, seed=0)
        assert meta.n_docs_total == cfg.n_docs * cfg.batch
        assert meta.doc_len.min() >= cfg.doc_len_lo and meta.doc_len.max() <= cfg.doc_len_hi
        assert meta.doc_offsets[0] == 0 and np.array_equal(np.diff(meta.doc_offsets), meta.doc_len)
        assert all(len(p) == cfg.n_planted for p in meta.planted)
        for b in range(cfg.batch):
            scales = meta.key_scale[b * cfg.n_docs:(b + 1) * cfg.n_docs]
            rest = np.sort(np.delete(scales, meta.planted[b]))
            assert np.all(np.diff(rest) > 0)                     # a strict ladder, no two alike
            assert rest.max() < W.PLANTED_SCALE
    assert W.CONFIGS[3].kept_at_layer(4) == 50 and W.CONFIGS[3].kept_at_layer(5) == 25
    assert W.CONFIGS[3].kept_at_layer(28) == 6


def test_values_are_reproducible_and_chunk_independent():
    cfg = W.scaled_config(W.CONFIGS[3], n_layers=2, n_docs=5)
    meta = W.make_meta(cfg, seed=3)
    k1, v1 = W.make_kv(meta)
    k2 = torch.empty_like(k1[1])
    v2 = torch.empty_like(v1[1])
    W.fill_kv_layer(meta, 1, k2, v2, chunk_tokens=37)            # different chunking, same values
    assert torch.equal(k1[1], k2) and torch.equal(v1[1], v2)
    assert not torch.equal(k1[0], k1[1])
    q = W.make_q(meta)
    assert q.shape == (2, 1, cfg.q_len, cfg.n_q_heads, cfg.head_dim) and q.dtype == torch.bfloat16
    assert torch.equal(q[1], W.make_q(meta, layers=range(1, 2))[0])
    other = W.make_meta(cfg, seed=4)
    assert not torch.equal(W.make_q(other), q)


def test_values_look_standard_normal_and_keys_carry_the_scale():
    x = W.hashed_normal(0, W.TENSOR_V, 0, 200000)
    assert abs(float(x.mean())) < 0.01 and abs(float(x.std()) - 1.0) < 0.01
    assert float(x.abs().max()) <= 3.47
    cfg = W.CONFIGS[1]
    meta = W.make_meta(cfg, seed=0)
    k, v = W.make_kv(meta)
    for i in range(meta.n_docs_total):
        rows = k[0, meta.doc_offsets[i]:meta.doc_offsets[i + 1]].double()
        assert abs(float(rows.std()) / meta.key_scale[i] - 1.0) < 0.05
