"""Full-size runs in the launch configurations bench.py times (Session.run_stack with one attention call
per run of layers between two pruning layers, and with one call per layer), checked on sampled
outputs the oracle computes one by one and on properties that hold at any size.

Nothing the oracle consumes comes from the CUDA path: layer 1 attends every document in retrieval
order, so its allocation and outputs are fixed by the inputs alone."""
import types

import numpy as np
import pytest
import torch

import oracle
from paper_2502_11101_b200 import workloads as W
from paper_2502_11101_b200.session import Session

pytestmark = pytest.mark.gpu


def _run_full(cfg, samples, batch_layers):
    meta = W.make_meta(cfg, 0)
    dev = "cuda:0"
    q = W.make_q(meta, dev)
    k, v = W.make_kv(meta, dev)
    sess = Session(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.torch_dtype, cfg.pos_range, cfg.rope_theta,
                   cfg.q_len, meta.doc_len, meta.req_doc_begin, meta.doc_src_start, tail_reserve=cfg.q_len, device=dev)
    # integer state after Init: bit-exact against the oracle's allocation, every request
    sess.init()
    plan0 = sess.read_plan()
    for b in range(cfg.batch):
        lo, hi = int(meta.req_doc_begin[b]), int(meta.req_doc_begin[b + 1])
        dst, grp, n_reuse, qs = oracle.allocate_positions(meta.doc_len[lo:hi], range(hi - lo), cfg.pos_range, 0, cfg.q_len)
        assert np.array_equal(plan0["dst_start"][lo:hi], dst) and np.array_equal(plan0["group"][lo:hi], grp)
        assert int(plan0["n_reuse"][b]) == n_reuse and int(plan0["query_start"][b]) == qs
    out = torch.empty_like(q)
    lse = torch.empty((cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.q_len), device=dev)
    scores = torch.empty((cfg.n_layers, meta.n_docs_total), device=dev)
    sess.run_stack(q, k, v, cfg.schedule, oracle.ALLOC_ALIGN, out, lse, None, scores, batch_layers=batch_layers)
    torch.cuda.synchronize()
    assert sess.status() == 0
    # ---- sampled outputs of layer 1 (all documents kept, retrieval order)
    g = cfg.group_size
    for b, h in samples:
        lo, hi = int(meta.req_doc_begin[b]), int(meta.req_doc_begin[b + 1])
        n = hi - lo
        r0, r1 = int(meta.doc_offsets[lo]), int(meta.doc_offsets[hi])
        kvh = h // g
        k_req = k[0, r0:r1, kvh:kvh + 1].double().cpu().numpy()
        v_req = v[0, r0:r1, kvh:kvh + 1].double().cpu().numpy()
        off = meta.doc_offsets[lo:hi + 1] - r0
        dst, _, _, _ = oracle.allocate_positions(meta.doc_len[lo:hi], range(n), cfg.pos_range, 0, cfg.q_len)
        k_rot = oracle.reposition_keys(k_req, off, meta.doc_src_start[lo:hi], dst, range(n), cfg.rope_theta)
        q_h = q[0, b, :, h:h + 1].double().cpu().numpy()
        o_ref, lse_ref, mass, _ = oracle.query_prefill_attn(q_h, k_rot, v_req, off, range(n), n)
        o_got = out[0, b, :, h].float().cpu().numpy()
        assert np.all(np.abs(o_got - o_ref[:, 0]) <= 1e-2 + 2e-2 * np.abs(o_ref[:, 0])), (b, h)
        assert np.all(np.abs(lse[0, b, h].cpu().numpy() - lse_ref[0]) <= 1e-2), (b, h)
    # ---- properties that hold at any size
    sc = scores.cpu().numpy()
    for layer in range(1, cfg.n_layers + 1):
        for b in range(cfg.batch):
            lo, hi = int(meta.req_doc_begin[b]), int(meta.req_doc_begin[b + 1])
            s = sc[layer - 1, lo:hi]
            assert abs(float(s.sum()) - 1.0) < 2e-3, (layer, b)                 # masses of a request sum to 1
            assert int((s > 0).sum()) == cfg.kept_at_layer(layer), (layer, b)   # pruned documents score exactly 0
    plan = sess.read_plan()
    final_keep = cfg.schedule[-1][1]
    for b in range(cfg.batch):
        lo, hi = int(meta.req_doc_begin[b]), int(meta.req_doc_begin[b + 1])
        order = plan["order"][b]
        assert len(order) == final_keep and len(set(order)) == final_keep
        assert set(meta.planted[b]) <= set(order), "planted documents must survive every pruning layer"
        qs = int(plan["query_start"][b])
        spans = {}
        for i in order:                                                          # allocation invariants
            d0 = int(plan["dst_start"][lo + i])
            assert 0 <= d0 and d0 + int(meta.doc_len[lo + i]) <= qs
            spans.setdefault(int(plan["group"][lo + i]), []).append((d0, d0 + int(meta.doc_len[lo + i])))
        for win in spans.values():
            win.sort()
            assert win[-1][1] == qs and all(a[1] == c[0] for a, c in zip(win, win[1:]))
        pruned = np.setdiff1d(np.arange(hi - lo), order)
        assert np.all(plan["dst_start"][lo + pruned] == -1)
    return plan0


@pytest.mark.parametrize("batch_layers", [True, False])
def test_config4_full_size_sampled(batch_layers):
    _run_full(W.CONFIGS[4], samples=[(0, 0), (1, 13), (3, 27)], batch_layers=batch_layers)


@pytest.mark.parametrize("batch_layers", [True, False])
def test_config5_four_layers_full_batch_sampled(batch_layers):
    # the full 32-layer store is 90 GB; four layers keep the launch configuration (8 requests x 120
    # documents x 32 heads, six parallel windows) and hold 11 GB; the batched variant runs layers 1-2
    # in one call
    schedule = ((2, 60), (3, 30)) if batch_layers else ((1, 60), (2, 30), (3, 15))
    cfg = W.scaled_config(W.CONFIGS[5], n_layers=4, schedule=schedule)
    plan0 = _run_full(cfg, samples=[(0, 0), (5, 17), (7, 31)], batch_layers=batch_layers)
    assert all(int(x) == 6 for x in plan0["n_reuse"])


def _run_against_whole_oracle(cfg, sample_heads, min_margin=5e-4):
    """The stack issued call by call (one attention call per layer) with the plan read back after
    every pruning step, against oracle.run_stack request by request: kept set, order, positions and
    windows bit-exact after every cut; every layer's document scores and log-sum-exp of the sampled
    heads, and their outputs, within tolerance."""
    from tests import harness
    dev = "cuda:0"
    one = types.SimpleNamespace(cfg=W.scaled_config(cfg, batch=1))      # cut_margins reads the configuration only
    # the first seed whose decisive score gaps (every cut, every request) are clear of the score error
    for seed in range(6):
        meta = W.make_meta(cfg, seed)
        q = W.make_q(meta, dev)
        k, v = W.make_kv(meta, dev)
        # the oracle's inputs: the same seeded tensors, widened exactly (bf16 -> fp32) and upcast per layer inside
        q_h, k_h, v_h = q.float().cpu().numpy(), k.float().cpu().numpy(), v.float().cpu().numpy()
        ref = []
        for b in range(cfg.batch):
            lo, hi = int(meta.req_doc_begin[b]), int(meta.req_doc_begin[b + 1])
            ref.append(oracle.run_stack(q_h[:, b], k_h, v_h, meta.doc_len[lo:hi], meta.doc_offsets, meta.doc_src_start[lo:hi],
                                        cfg.rope_theta, cfg.pos_range, cfg.schedule, oracle.ALLOC_ALIGN,
                                        tail_reserve=cfg.q_len, doc_base=lo, final_reposition=False))
            if harness.cut_margins(one, ref[-1:], oracle.ALLOC_ALIGN) < min_margin:
                break                                       # this seed is rejected: no need for its other requests
        else:
            break
        del q, k, v
    assert len(ref) == cfg.batch and harness.cut_margins(meta, ref, oracle.ALLOC_ALIGN) >= min_margin, \
        "no seed with clear margins"
    sess = Session(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.torch_dtype, cfg.pos_range, cfg.rope_theta,
                   cfg.q_len, meta.doc_len, meta.req_doc_begin, meta.doc_src_start, tail_reserve=cfg.q_len, device=dev)
    sess.set_live_docs(cfg.n_docs)
    sess.init()
    sched = dict(cfg.schedule)
    out = torch.empty_like(q[0])
    lse = torch.empty((cfg.batch, cfg.n_q_heads, cfg.q_len), device=dev)
    for layer in range(1, cfg.n_layers + 1):
        sess.attend(q[layer - 1], k[layer - 1], v[layer - 1], out, lse)
        s_got = sess.doc_scores.cpu().numpy()
        o_got, l_got = out.float().cpu().numpy(), lse.cpu().numpy()
        for b in range(cfg.batch):
            lo, hi = int(meta.req_doc_begin[b]), int(meta.req_doc_begin[b + 1])
            rec = ref[b]["layers"][layer - 1]
            n_kept = len(rec["order_in"])
            s_err = np.abs(s_got[lo:hi] - rec["doc_scores"])
            assert np.all(s_err <= 1e-2 / n_kept + 2e-2 * np.abs(rec["doc_scores"])), (layer, b)
            assert set(np.nonzero(s_got[lo:hi])[0]) == set(rec["order_in"]), (layer, b)
            for h in sample_heads:
                assert np.all(np.abs(o_got[b, :, h] - rec["out"][:, h]) <= 1e-2 + 2e-2 * np.abs(rec["out"][:, h])), (layer, b, h)
                assert np.all(np.abs(l_got[b, h] - rec["lse"][h]) <= 1e-2), (layer, b, h)
        if layer in sched:
            sess.prune(sched[layer], oracle.ALLOC_ALIGN)
            plan = sess.read_plan()
            for b in range(cfg.batch):
                lo, hi = int(meta.req_doc_begin[b]), int(meta.req_doc_begin[b + 1])
                rec = ref[b]["layers"][layer - 1]
                assert plan["order"][b] == rec["order_out"], (layer, b)
                if layer < cfg.n_layers:
                    nxt = ref[b]["layers"][layer]
                    assert np.array_equal(plan["dst_start"][lo:hi], nxt["dst_start"]), (layer, b)
                    assert int(plan["n_reuse"][b]) == nxt["n_reuse"], (layer, b)
    assert sess.status() == 0
    plan = sess.read_plan()
    for b in range(cfg.batch):
        lo, hi = int(meta.req_doc_begin[b]), int(meta.req_doc_begin[b + 1])
        assert plan["order"][b] == ref[b]["order"]
        assert np.array_equal(plan["dst_start"][lo:hi], ref[b]["dst_start"])
        assert np.array_equal(plan["group"][lo:hi], ref[b]["group"])
        assert np.all(np.abs(sess.score_accum.cpu().numpy()[lo:hi] - ref[b]["score_accum"])
                      <= 1e-2 + 2e-2 * np.abs(ref[b]["score_accum"]))


def test_config4_full_size_every_cut_against_the_oracle():
    _run_against_whole_oracle(W.CONFIGS[4], sample_heads=(0, 13, 27))


def test_config5_four_layers_every_cut_against_the_oracle():
    cfg = W.scaled_config(W.CONFIGS[5], n_layers=4, schedule=((1, 60), (2, 30), (3, 15)))
    _run_against_whole_oracle(cfg, sample_heads=(0, 17, 31))


def test_config5_sixteen_layers_full_batch_sampled():
    # half of the 32-layer stack: 45 GB of keys and values resident, the schedule's first two cuts at
    # their own layers (4 and 12); the 32-layer store (90.6 GB plus the final keys) is not run
    cfg = W.scaled_config(W.CONFIGS[5], n_layers=16, schedule=((4, 60), (12, 30)))
    plan0 = _run_full(cfg, samples=[(0, 0), (3, 9), (7, 31)], batch_layers=True)
    assert all(int(x) == 6 for x in plan0["n_reuse"])
