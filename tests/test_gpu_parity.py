"""Parity of the CUDA library (through the C ABI) with the CPU oracle on seeded workloads.

Tolerances: integer results (positions, windows, kept sets and their order) bit-exact; rotated
keys within 1 bf16 ulp (4 fp32 ulp for fp32 storage) of the fp64 value; attention outputs within
1e-2 + 2e-2*|ref|; document scores within 1e-2/n_kept + 2e-2*|ref|."""
import numpy as np
import pytest
import torch

import oracle
from paper_2502_11101_b200 import workloads as W
from tests import harness

pytestmark = pytest.mark.gpu

STRATEGIES = [oracle.ALLOC_NONE, oracle.ALLOC_ALIGN, oracle.ALLOC_SORT]


@pytest.fixture(scope="module", autouse=True)
def _library():
    assert torch.cuda.is_available()
    from paper_2502_11101_b200 import build
    build.build()
    import paper_2502_11101_b200 as cf
    cf.load_library()


def _pick_seed(cfg, strategy, min_margin=2e-3, tries=6):
    """First seed whose oracle run has no decisive score gap inside the tolerance."""
    for seed in range(tries):
        meta = W.make_meta(cfg, seed)
        ref = harness.oracle_stack(meta, W.make_q(meta), *W.make_kv(meta), strategy, final_reposition=False)
        if harness.cut_margins(meta, ref, strategy) >= min_margin:
            return seed
    raise AssertionError("no seed with a safe margin")


@pytest.mark.parametrize("strategy", STRATEGIES)
def test_config1_tiny_fp32(strategy):
    cfg = W.CONFIGS[1]
    rep = harness.run_and_compare(cfg, _pick_seed(cfg, strategy), strategy)
    assert rep["out_max_abs"] < 1e-4 and rep["score_max_rel"] < 1e-4      # fp32 path is much tighter


@pytest.mark.parametrize("strategy", [oracle.ALLOC_ALIGN, oracle.ALLOC_SORT])
def test_config2_llama_layer(strategy):
    cfg = W.CONFIGS[2]
    harness.run_and_compare(cfg, _pick_seed(cfg, strategy), strategy)


@pytest.mark.parametrize("strategy", STRATEGIES)
def test_config3_qwen_stack(strategy):
    cfg = W.CONFIGS[3]
    harness.run_and_compare(cfg, _pick_seed(cfg, strategy, min_margin=1e-3), strategy, min_margin=1e-3)


def test_config4_reduced_batch_of_requests():
    cfg = W.scaled_config(W.CONFIGS[4], n_layers=5, batch=2, schedule=((1, 50), (3, 25), (4, 12)))
    harness.run_and_compare(cfg, _pick_seed(cfg, oracle.ALLOC_ALIGN, 1e-3), oracle.ALLOC_ALIGN, min_margin=1e-3)


def test_config5_reduced_parallel_windows():
    cfg = W.scaled_config(W.CONFIGS[5], n_layers=3, batch=2, schedule=((1, 60), (2, 30)))
    meta = W.make_meta(cfg, 0)
    dst, grp, n_reuse, qs = oracle.allocate_positions(meta.doc_len[:120], range(120), 4096, 0, 64)
    assert n_reuse == 6                                   # six parallel windows inside the 4096 range
    harness.run_and_compare(cfg, _pick_seed(cfg, oracle.ALLOC_ALIGN, 1e-3), oracle.ALLOC_ALIGN, min_margin=1e-3)


@pytest.mark.parametrize("dtype,head_dim", [("bf16", 128), ("bf16", 64), ("f32", 128), ("f32", 64)])
def test_ragged_document_lengths(dtype, head_dim):
    lens = [1, 63, 64, 65, 127, 128, 129, 200, 300, 17, 256, 31]
    cfg = W.WorkloadConfig("ragged", 2, 8, 2, head_dim, dtype, 1e4, 4096, len(lens), 1, 300, 5, 1, 2,
                           ((1, 7),))
    harness.run_and_compare(cfg, 1, oracle.ALLOC_ALIGN, doc_len_override=lens, min_margin=1e-3)


def test_forced_window_counts():
    cfg = W.scaled_config(W.CONFIGS[2], n_docs=12, n_planted=2, schedule=((1, 6),))
    for n_reuse in (1, 3, 12):                            # sequential, k/4, fully parallel (Sec. 3.3)
        harness.run_and_compare(cfg, 0, oracle.ALLOC_ALIGN, n_reuse=n_reuse, min_margin=1e-3)


def test_window_count_policies_of_the_reuse_study():
    """The policies of Sec. 3.3 on k = 20 documents (the case its text works through): N_reuse = k, 1, k/5
    (four windows of five documents, each position used four times) and a fixed 5, besides Eq. 6."""
    cfg = W.scaled_config(W.CONFIGS[2], n_docs=20, n_planted=4, schedule=((1, 10),))
    for n_reuse in (20, 1, 20 // 5, 5, 0):
        report = harness.run_and_compare(cfg, 0, oracle.ALLOC_ALIGN, n_reuse=n_reuse, min_margin=1e-3)
        assert report["margin"] >= 1e-3


def test_keep_larger_than_live_set_and_no_pruning():
    cfg = W.scaled_config(W.CONFIGS[3], n_layers=3, n_docs=9, n_planted=2, schedule=((1, 20), (2, 9)))
    harness.run_and_compare(cfg, 0, oracle.ALLOC_SORT, min_margin=1e-3)


def test_results_are_bitwise_reproducible():
    cfg = W.scaled_config(W.CONFIGS[3], n_layers=2, n_docs=20, schedule=((1, 10),))
    meta = W.make_meta(cfg, 0)
    q = W.make_q(meta)
    k, v = W.make_kv(meta)
    a = harness.gpu_stack(meta, q, k, v, oracle.ALLOC_ALIGN)
    b = harness.gpu_stack(meta, q, k, v, oracle.ALLOC_ALIGN)
    for key in ("out", "lse", "scores", "accum", "k_final"):
        assert np.array_equal(a[key], b[key]), key


@pytest.mark.parametrize("heads,q_len,lens", [
    ((4, 4), 16, [128]),                                   # one full tile, one row tile
    ((4, 4), 16, [40, 128, 7]),                            # ragged tiles
    ((12, 2), 48, [130, 160, 192, 128, 150]),              # two row tiles (288 rows), two-tile documents
    ((28, 4), 64, [128, 192, 161, 140, 177, 133]),         # 448 rows: two row groups per kv head
    ((20, 2), 60, [130, 160, 128]),                        # 600 rows: five row tiles, one per CTA
])
def test_tensor_core_kernel_matches_cuda_core_kernel(heads, q_len, lens):
    """Same inputs through both attention kernels of the library."""
    import paper_2502_11101_b200 as cf
    from paper_2502_11101_b200.session import Session
    cfg = W.WorkloadConfig("tc-vs-simt", 1, heads[0], heads[1], 128, "bf16", 1e6, 32768, len(lens), 1, 400, q_len,
                           1, 1, ())
    meta = W.make_meta(cfg, 3, doc_len_override=lens)
    q, (k, v) = W.make_q(meta).cuda(), [t.cuda() for t in W.make_kv(meta)]
    results = []
    try:
        for path in (1, 0):
            cf.cf_set_attn_path(path)
            sess = Session(cfg.n_q_heads, cfg.n_kv_heads, 128, torch.bfloat16, cfg.pos_range, cfg.rope_theta, q_len,
                           meta.doc_len, meta.req_doc_begin, meta.doc_src_start, tail_reserve=q_len)
            sess.init()
            out = torch.full_like(q[0], float("nan"))
            lse = torch.full((1, cfg.n_q_heads, q_len), float("nan"), device="cuda")
            sess.attend(q[0], k[0], v[0], out, lse)
            torch.cuda.synchronize()
            assert sess.status() == 0
            results.append((out.float().cpu(), lse.cpu(), sess.doc_scores.cpu()))
    finally:
        cf.cf_set_attn_path(0)
    (o_a, l_a, s_a), (o_b, l_b, s_b) = results
    assert torch.all((o_a - o_b).abs() <= 1e-2 + 2e-2 * o_a.abs()), float((o_a - o_b).abs().max())
    assert torch.all((l_a - l_b).abs() <= 1e-3), float((l_a - l_b).abs().max())
    assert torch.all((s_a - s_b).abs() <= 1e-3 * s_a.abs() + 1e-6)


@pytest.mark.parametrize("which", ["config3", "config4-reduced", "ragged-f32-d64", "ragged-bf16-d64"])
def test_layer_batched_calls_match_oracle(which):
    """Layers between two pruning layers in one library call (cf_query_prefill_attn_layers)."""
    if which == "config3":                                 # segments of 4, 8, 8 and 8 layers
        cfg = W.CONFIGS[3]
    elif which == "config4-reduced":                       # two requests x segments of 2, 2 and 1 layers
        cfg = W.scaled_config(W.CONFIGS[4], n_layers=5, batch=2, schedule=((2, 50), (4, 25)))
    else:                                                  # CUDA-core kernel, ragged tiles, segments of 3 and 2
        lens = [1, 63, 64, 65, 127, 128, 129, 200, 300, 17, 256, 31]
        dtype = "f32" if "f32" in which else "bf16"
        cfg = W.WorkloadConfig("ragged", 5, 8, 2, 64, dtype, 1e4, 4096, len(lens), 1, 300, 5, 1, 2, ((3, 7),))
        harness.run_and_compare(cfg, 1, oracle.ALLOC_ALIGN, doc_len_override=lens, min_margin=1e-3, batch_layers=True)
        return
    harness.run_and_compare(cfg, _pick_seed(cfg, oracle.ALLOC_ALIGN, 1e-3), oracle.ALLOC_ALIGN, min_margin=1e-3,
                            batch_layers=True)


def test_layer_batched_call_is_reproducible_and_agrees_with_single_layer_calls():
    import paper_2502_11101_b200 as cf
    from paper_2502_11101_b200.session import Session
    cfg = W.scaled_config(W.CONFIGS[3], n_layers=3, n_docs=20, schedule=())
    meta = W.make_meta(cfg, 0)
    q = W.make_q(meta).cuda()
    k, v = [t.cuda() for t in W.make_kv(meta)]
    # the store with a gap between layers: the layer stride is an argument of its own
    pad = 24
    k_wide = torch.zeros((3, meta.total_tokens + pad, cfg.n_kv_heads, 128), dtype=torch.bfloat16, device="cuda")
    v_wide = torch.zeros_like(k_wide)
    k_wide[:, :meta.total_tokens] = k
    v_wide[:, :meta.total_tokens] = v
    runs = []
    for mode in ("layers", "layers", "layers-strided", "single"):
        sess = Session(cfg.n_q_heads, cfg.n_kv_heads, 128, torch.bfloat16, cfg.pos_range, cfg.rope_theta, cfg.q_len,
                       meta.doc_len, meta.req_doc_begin, meta.doc_src_start, tail_reserve=cfg.q_len)
        sess.init()
        out = torch.full_like(q, float("nan"))
        lse = torch.full((3, 1, cfg.n_q_heads, cfg.q_len), float("nan"), device="cuda")
        scores = torch.full((3, meta.n_docs_total), float("nan"), device="cuda")
        if mode == "layers":
            sess.attend_layers(q, k, v, out, lse, scores)
        elif mode == "layers-strided":
            sess.attend_layers(q, k_wide[:, :meta.total_tokens], v_wide[:, :meta.total_tokens], out, lse, scores)
        else:
            for i in range(3):
                sess.attend(q[i], k[i], v[i], out[i], lse[i])
                scores[i].copy_(sess.doc_scores)
        torch.cuda.synchronize()
        assert sess.status() == 0
        runs.append([t.float().cpu() for t in (out, lse, scores, sess.score_accum)])
    for a, b in zip(runs[0], runs[1]):
        assert torch.equal(a, b)                                        # run to run
    for a, b in zip(runs[0], runs[2]):
        assert torch.equal(a, b)                                        # a layer stride changes nothing
    o_a, l_a, s_a, acc_a = runs[0]
    o_b, l_b, s_b, acc_b = runs[3]
    assert torch.all((o_a - o_b).abs() <= 1e-2 + 2e-2 * o_b.abs())
    assert torch.all((l_a - l_b).abs() <= 1e-3)
    assert torch.all((s_a - s_b).abs() <= 1e-3 * s_b.abs() + 1e-6)
    assert torch.allclose(acc_a, s_a.sum(0), rtol=1e-5) and torch.allclose(acc_a, acc_b, rtol=1e-3)


@pytest.mark.parametrize("which", ["config3", "ragged-f32-d64"])
def test_deferred_document_scores_equal_the_per_layer_calls(which):
    """cf_query_prefill_attn_slot + cf_accumulate_scores against cf_query_prefill_attn layer by layer: the same outputs
    bit for bit, the same per-layer scores and S up to the rounding of fp32 sums taken in another order (five layers in
    four slots: two groups, the second partly filled);
    the per-layer calls themselves are compared with the oracle by the stack tests."""
    import paper_2502_11101_b200 as cf
    from paper_2502_11101_b200.session import Session
    if which == "config3":
        cfg = W.scaled_config(W.CONFIGS[3], n_layers=5, n_docs=20, schedule=())
    else:
        cfg = W.WorkloadConfig("ragged", 5, 8, 2, 64, "f32", 1e4, 4096, 7, 5, 70, 5, 1, 2, ())   # CUDA-core kernels
    meta = W.make_meta(cfg, 1)
    q = W.make_q(meta).cuda()
    k, v = [t.cuda() for t in W.make_kv(meta)]
    n_slots, nd = 4, meta.n_docs_total
    runs = []
    for mode in ("single", "slots"):
        sess = Session(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.torch_dtype, cfg.pos_range, cfg.rope_theta,
                       cfg.q_len, meta.doc_len, meta.req_doc_begin, meta.doc_src_start, tail_reserve=cfg.q_len)
        sess.init()
        out = torch.full_like(q, float("nan"))
        lse = torch.full((5, cfg.batch, cfg.n_q_heads, cfg.q_len), float("nan"), device="cuda")
        scores = torch.full((5, nd), float("nan"), device="cuda")
        if mode == "single":
            for i in range(5):
                sess.attend(q[i], k[i], v[i], out[i], lse[i])
                scores[i].copy_(sess.doc_scores)
        else:
            work = torch.empty(cf.cf_attn_workspace_bytes_slots(sess.geom, sess.batch, n_slots), dtype=torch.uint8, device="cuda")
            work.fill_(0xFF)                                             # nothing in it needs zeroing
            for first in (0, 4):
                filled = min(n_slots, 5 - first)
                for i in range(filled):
                    cf.cf_query_prefill_attn_slot(sess.geom, sess.batch, sess.plan, i, n_slots, q[first + i], k[first + i],
                                                  v[first + i], out[first + i], work, lse[first + i])
                cf.cf_accumulate_scores(sess.geom, sess.batch, sess.plan, filled, n_slots, work,
                                        scores[first:first + filled], sess.score_accum)
        torch.cuda.synchronize()
        assert sess.status() == 0
        runs.append([t.float().cpu() for t in (out, lse, scores, sess.score_accum)])
    for i, (a, b) in enumerate(zip(*runs)):
        assert not torch.isnan(a).any() and not torch.isnan(b).any()
        if i < 2:
            assert torch.equal(a, b)                                     # outputs and log-sum-exps: the same kernels
        else:                                                            # a layer's rows are summed by a quarter of the block
            assert torch.allclose(a, b, rtol=1e-5, atol=1e-9)
    with pytest.raises(cf.CacheFocusError):                              # a slot beyond the capacity
        cf.cf_query_prefill_attn_slot(sess.geom, sess.batch, sess.plan, 4, n_slots, q[0], k[0], v[0], out[0], work)
    with pytest.raises(cf.CacheFocusError):                              # more slots to score than there are
        cf.cf_accumulate_scores(sess.geom, sess.batch, sess.plan, 5, n_slots, work, None, sess.score_accum)


@pytest.mark.parametrize("simt", [False, True])
def test_deferred_scores_with_prefix_and_query_self_block(simt):
    """cf_query_prefill_attn_slot_full + cf_accumulate_scores against cf_query_prefill_attn_prefix layer by layer
    (three layers in two slots; a 40-token prefix and the causal block of the query tokens): the same outputs bit for
    bit, scores and S up to fp32 rounding.  Both kernel families."""
    import paper_2502_11101_b200 as cf
    from paper_2502_11101_b200.session import Session
    hq, hkv, d, q_len, prefix, n_layers = 8, 2, 128, 20, 40, 3
    lens = np.array([130, 64, 17, 96, 200], dtype=np.int32)
    n = len(lens)
    gen = torch.Generator().manual_seed(9)
    rnd = lambda *shape: torch.randn(shape, generator=gen).bfloat16().cuda()
    q, k, v = rnd(n_layers, 1, q_len, hq, d), rnd(n_layers, int(lens.sum()), hkv, d), rnd(n_layers, int(lens.sum()), hkv, d)
    kp, vp = rnd(n_layers, prefix, hkv, d), rnd(n_layers, prefix, hkv, d)
    ks, vs = rnd(n_layers, 1, q_len, hkv, d), rnd(n_layers, 1, q_len, hkv, d)
    cf.cf_set_attn_path(1 if simt else 0)
    try:
        runs = []
        for mode in ("calls", "slots"):
            sess = Session(hq, hkv, d, torch.bfloat16, 4096, 1e4, q_len, lens, np.array([0, n], dtype=np.int32),
                           np.full(n, prefix, dtype=np.int32), tail_reserve=q_len, prefix_len=prefix)
            sess.init()
            out = torch.full_like(q, float("nan"))
            lse = torch.full((n_layers, 1, hq, q_len), float("nan"), device="cuda")
            scores = torch.full((n_layers, n), float("nan"), device="cuda")
            if mode == "calls":
                sess.reserve_workspace(1, with_self=True)
                for i in range(n_layers):
                    cf.cf_query_prefill_attn_prefix(sess.geom, sess.batch, sess.plan, q[i:i + 1], k[i:i + 1], v[i:i + 1],
                                                    kp[i:i + 1], vp[i:i + 1], out[i:i + 1], sess.workspace, lse=lse[i:i + 1],
                                                    doc_scores=scores[i:i + 1], score_accum=sess.score_accum,
                                                    k_self=ks[i:i + 1], v_self=vs[i:i + 1])
            else:
                work = torch.empty(cf.cf_attn_workspace_bytes_slots_full(sess.geom, sess.batch, 2), dtype=torch.uint8, device="cuda")
                for first, filled in ((0, 2), (2, 1)):
                    for i in range(filled):
                        l = first + i
                        cf.cf_query_prefill_attn_slot_full(sess.geom, sess.batch, sess.plan, i, 2, q[l], k[l], v[l], out[l], work,
                                                           k_prefix=kp[l], v_prefix=vp[l], k_self=ks[l], v_self=vs[l], lse=lse[l])
                    cf.cf_accumulate_scores(sess.geom, sess.batch, sess.plan, filled, 2, work, scores[first:first + filled],
                                            sess.score_accum)
            torch.cuda.synchronize()
            assert sess.status() == 0
            runs.append([t.float().cpu() for t in (out, lse, scores, sess.score_accum)])
    finally:
        cf.cf_set_attn_path(0)
    for i, (a, b) in enumerate(zip(*runs)):
        assert not torch.isnan(a).any() and not torch.isnan(b).any()
        assert torch.equal(a, b) if i < 2 else torch.allclose(a, b, rtol=1e-5, atol=1e-9)


def test_interleaved_slice_layout():
    import paper_2502_11101_b200 as cf
    from paper_2502_11101_b200.session import Session
    cfg = W.scaled_config(W.CONFIGS[2], n_docs=6, n_planted=1, n_q_heads=4, n_kv_heads=2)
    meta = W.make_meta(cfg, 0)
    q = W.make_q(meta)
    k, v = W.make_kv(meta)
    sess = Session(4, 2, 128, torch.bfloat16, 4096, 1e4, cfg.q_len, meta.doc_len, meta.req_doc_begin,
                   meta.doc_src_start, tail_reserve=cfg.q_len, rope_layout=cf.CF_ROPE_INTERLEAVED)
    qg, kg, vg = q.cuda(), k.cuda(), v.cuda()
    out = torch.empty_like(qg[0])
    sess.init()
    sess.attend(qg[0], kg[0], vg[0], out)
    k_rot = torch.empty_like(kg[0])
    sess.reposition(kg[0], k_rot)
    plan = sess.read_plan()
    order = plan["order"][0]
    kr = oracle.reposition_keys(k[0].double().numpy(), meta.doc_offsets, meta.doc_src_start, plan["dst_start"],
                                order, 1e4, oracle.ROPE_INTERLEAVED)
    o_ref, _, _, s_ref = oracle.query_prefill_attn(q[0, 0].double().numpy(), kr, v[0].double().numpy(),
                                                   meta.doc_offsets, order, cfg.n_docs)
    err = np.abs(k_rot.float().cpu().numpy() - kr) / harness.rotated_key_tolerance(kr, "bf16", interleaved=True)
    assert err.max() <= 1.0
    assert np.all(np.abs(out[0].float().cpu().numpy() - o_ref) <= 1e-2 + 2e-2 * np.abs(o_ref))
    assert np.allclose(sess.doc_scores.cpu().numpy(), s_ref, rtol=2e-2, atol=1e-3)


def test_fused_equals_reposition_then_attend():
    """Rotating on the way in (fused) and re-positioning the store first, then attending with a zero
    delta, are the same computation: outputs agree bit for bit."""
    from paper_2502_11101_b200.session import Session
    cfg = W.scaled_config(W.CONFIGS[3], n_layers=1, n_docs=12, n_planted=2, schedule=())
    meta = W.make_meta(cfg, 2)
    q, (k, v) = W.make_q(meta).cuda(), [t.cuda() for t in W.make_kv(meta)]

    def session(src_start):
        return Session(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.torch_dtype, cfg.pos_range, cfg.rope_theta,
                       cfg.q_len, meta.doc_len, meta.req_doc_begin, src_start, tail_reserve=cfg.q_len)
    fused = session(meta.doc_src_start)
    fused.init()
    out_a = torch.empty_like(q[0])
    fused.attend(q[0], k[0], v[0], out_a)
    k_rot = torch.empty_like(k[0])
    fused.reposition(k[0], k_rot)
    moved = session(fused.read_plan()["dst_start"])       # the store now sits at its destination
    moved.init()
    out_b = torch.empty_like(q[0])
    moved.attend(q[0], k_rot, v[0], out_b)
    assert torch.equal(out_a, out_b)
    assert torch.equal(fused.doc_scores, moved.doc_scores)


def test_argument_errors_are_reported_not_faulted():
    import paper_2502_11101_b200 as cf
    from paper_2502_11101_b200.session import Session
    cfg = W.scaled_config(W.CONFIGS[2], n_docs=4, n_planted=1)
    meta = W.make_meta(cfg, 0)
    sess = Session(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.torch_dtype, cfg.pos_range, cfg.rope_theta,
                   cfg.q_len, meta.doc_len, meta.req_doc_begin, meta.doc_src_start, tail_reserve=cfg.q_len)
    q, (k, v) = W.make_q(meta).cuda(), [t.cuda() for t in W.make_kv(meta)]
    out = torch.empty_like(q[0])
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(cf.CacheFocusError) as e:
        cf.cf_query_prefill_attn(sess.geom, sess.batch, sess.plan, q[0], k[0], v[0], out, small)
    assert e.value.code == cf.CF_ERR_WORKSPACE
    with pytest.raises(cf.CacheFocusError) as e:
        cf.cf_plan_init(sess.geom, sess.batch, small)
    assert e.value.code == cf.CF_ERR_WORKSPACE
    q3, k3, v3 = q[:1].expand(3, *q.shape[1:]), k[:1].expand(3, *k.shape[1:]), v[:1].expand(3, *v.shape[1:])
    out3 = torch.empty((3,) + tuple(out.shape), dtype=out.dtype, device="cuda")
    with pytest.raises(cf.CacheFocusError) as e:             # layers that overlap (stride 0)
        cf.cf_query_prefill_attn_layers(sess.geom, sess.batch, sess.plan, q3, k3, v3, out3, sess.workspace)
    assert e.value.code == cf.CF_ERR_INVALID_ARG
    with pytest.raises(cf.CacheFocusError) as e:
        cf.cf_query_prefill_attn_layers(sess.geom, sess.batch, sess.plan, q3.contiguous(), k3.contiguous(),
                                        v3.contiguous(), out3, small)
    assert e.value.code == cf.CF_ERR_WORKSPACE
    assert cf.cf_attn_workspace_bytes_layers(sess.geom, sess.batch, cf.CF_MAX_LAYERS_PER_CALL + 1) == 0
    bad = cf.make_geom(5, 2, 128, cf.CF_BF16, 4096, 1e4)
    with pytest.raises(cf.CacheFocusError) as e:
        cf.cf_plan_layout_of(bad, sess.batch)
    assert e.value.code == cf.CF_ERR_INVALID_ARG
    # a range too small for the documents is reported through the plan's status word
    tight = Session(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.torch_dtype, 100 + cfg.q_len, cfg.rope_theta,
                    cfg.q_len, meta.doc_len, meta.req_doc_begin, meta.doc_src_start, tail_reserve=cfg.q_len)
    tight.init()
    assert tight.status() == cf.CF_ERR_RANGE


def test_degenerate_batches():
    """A request without documents, a one-token document, keep = 0: results are defined, nothing faults."""
    import paper_2502_11101_b200 as cf
    from paper_2502_11101_b200.session import Session
    lens = np.array([1, 130, 17], dtype=np.int32)                    # request 0: one token; request 1: none; request 2: two docs
    req = np.array([0, 1, 1, 3], dtype=np.int32)
    src = np.zeros(3, dtype=np.int32)
    hq, hkv, d, lq = 4, 2, 128, 5
    sess = Session(hq, hkv, d, torch.bfloat16, 4096, 1e4, lq, lens, req, src, tail_reserve=lq)
    gen = torch.Generator().manual_seed(0)
    total = int(lens.sum())
    q = torch.randn((3, lq, hq, d), generator=gen).bfloat16().cuda()
    k = torch.randn((total, hkv, d), generator=gen).bfloat16().cuda()
    v = torch.randn((total, hkv, d), generator=gen).bfloat16().cuda()
    out = torch.full_like(q, float("nan"))
    lse = torch.full((3, hq, lq), float("nan"), device="cuda")
    for path in (0, 1):
        cf.cf_set_attn_path(path)
        try:
            sess.init()
            sess.attend(q, k, v, out, lse)
            torch.cuda.synchronize()
        finally:
            cf.cf_set_attn_path(0)
        assert sess.status() == 0
        o = out.float().cpu().numpy()
        # one-token document: the softmax has a single term, the output is that value row (to the
        # tolerance of attention outputs: the one weight is a bf16 number near 1, not exactly 1)
        for h in range(hq):
            assert np.allclose(o[0, :, h], v[0, h // 2].float().cpu().numpy(), atol=1e-2, rtol=2e-2)
        assert np.all(o[1] == 0.0) and np.all(np.isneginf(lse[1].cpu().numpy()))   # nothing to attend
        s = sess.doc_scores.cpu().numpy()
        assert abs(s[0] - 1.0) < 1e-4 and abs(s[1] + s[2] - 1.0) < 1e-3
        # oracle for request 2 (no position change matters for the check of masses: compare outputs)
        dst, _, _, _ = oracle.allocate_positions(lens[1:], [0, 1], 4096, 0, lq)
        off = np.array([0, 130, 147])
        kr = oracle.reposition_keys(k[1:].double().cpu().numpy(), off, [0, 0], dst, [0, 1], 1e4)
        o_ref, lse_ref, _, s_ref = oracle.query_prefill_attn(q[2].double().cpu().numpy(), kr, v[1:].double().cpu().numpy(),
                                                             off, [0, 1], 2)
        assert np.all(np.abs(o[2] - o_ref) <= 1e-2 + 2e-2 * np.abs(o_ref))
        assert np.allclose(s[1:], s_ref, rtol=2e-2, atol=1e-3)
    # keep = 0 empties every request; the next layer then attends nothing
    sess.prune(0, oracle.ALLOC_ALIGN)
    sess.attend(q, k, v, out, lse)
    torch.cuda.synchronize()
    assert sess.status() == 0 and sess.read_plan()["order"] == [[], [], []]
    assert np.all(out.float().cpu().numpy() == 0.0) and np.all(sess.doc_scores.cpu().numpy() == 0.0)


def test_store_smaller_than_one_tile():
    """A store of five rows in all: every bulk copy reaches past the end of the store."""
    cfg = W.WorkloadConfig("five-rows", 2, 4, 2, 128, "bf16", 1e4, 4096, 1, 5, 5, 3, 1, 1, ())
    for batch_layers in (False, True):
        harness.run_and_compare(cfg, 0, oracle.ALLOC_ALIGN, min_margin=0.0, batch_layers=batch_layers)


@pytest.mark.parametrize("heads", [(32, 32), (12, 2)])
def test_single_query_row(heads):
    """q_len = 1 (the shape of a decoding step over the kept caches): one row per head."""
    cfg = W.WorkloadConfig("one-row", 2, heads[0], heads[1], 128, "bf16", 1e4, 4096, 8, 100, 200, 1, 2, 2, ((1, 4),))
    for batch_layers in (False, True):
        harness.run_and_compare(cfg, _pick_seed(cfg, oracle.ALLOC_ALIGN, 1e-3), oracle.ALLOC_ALIGN, min_margin=1e-3,
                                batch_layers=batch_layers)


def test_linear_pruning_schedule_of_the_paper():
    """App. C: prune every n = 4 layers by a constant amount down to k_finish = 5 (schedule from the library)."""
    import paper_2502_11101_b200 as cf
    base = W.CONFIGS[3]
    schedule = tuple(cf.cf_schedule_linear(base.n_layers, 4, base.n_docs, 5))
    assert schedule == tuple(oracle.prune_schedule_linear(base.n_layers, 4, base.n_docs, 5)) and len(schedule) == 7
    cfg = W.scaled_config(base, schedule=schedule)
    harness.run_and_compare(cfg, _pick_seed(cfg, oracle.ALLOC_ALIGN, 1e-3), oracle.ALLOC_ALIGN, min_margin=1e-3,
                            batch_layers=True)


@pytest.mark.parametrize("which", ["config3", "config2-mha", "config4-reduced", "ragged-f32-d64", "config1-f32"])
def test_query_self_block_merged_in(which):
    """cf_query_prefill_attn_full: the causal block of the query tokens over themselves joins the softmax."""
    if which == "config3":
        cfg = W.scaled_config(W.CONFIGS[3], n_layers=6, schedule=((2, 25), (4, 12)))
    elif which == "config2-mha":
        cfg = W.CONFIGS[2]
    elif which == "config4-reduced":
        cfg = W.scaled_config(W.CONFIGS[4], n_layers=3, batch=2, schedule=((2, 50),))
    elif which == "config1-f32":
        cfg = W.CONFIGS[1]
    else:
        lens = [1, 63, 64, 65, 127, 128, 129, 200, 300, 17, 256, 31]
        cfg = W.WorkloadConfig("ragged", 3, 8, 2, 64, "f32", 1e4, 4096, len(lens), 1, 300, 5, 1, 2, ((2, 7),))
        for batch_layers in (False, True):
            harness.run_and_compare(cfg, 1, oracle.ALLOC_ALIGN, doc_len_override=lens, min_margin=1e-3,
                                    batch_layers=batch_layers, self_block=True)
        return
    seed = _pick_seed(cfg, oracle.ALLOC_ALIGN, 1e-3)
    for batch_layers in (False, True):
        harness.run_and_compare(cfg, seed, oracle.ALLOC_ALIGN, min_margin=1e-3, batch_layers=batch_layers,
                                self_block=True)


def test_query_self_block_argument_errors():
    import paper_2502_11101_b200 as cf
    from paper_2502_11101_b200.session import Session
    cfg = W.scaled_config(W.CONFIGS[2], n_docs=4, n_planted=1, q_len=130)      # more query tokens than one key tile
    meta = W.make_meta(cfg, 0)
    sess = Session(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.torch_dtype, cfg.pos_range, cfg.rope_theta,
                   cfg.q_len, meta.doc_len, meta.req_doc_begin, meta.doc_src_start, tail_reserve=cfg.q_len)
    q, (k, v), (ks, vs) = W.make_q(meta).cuda(), [t.cuda() for t in W.make_kv(meta)], [t.cuda() for t in W.make_kv_self(meta)]
    out = torch.empty_like(q)
    sess.init()
    for path in (0, 1):
        cf.cf_set_attn_path(path)
        try:
            with pytest.raises(cf.CacheFocusError) as e:
                sess.attend_layers(q, k, v, out, k_self=ks, v_self=vs)
            assert e.value.code == cf.CF_ERR_UNSUPPORTED
        finally:
            cf.cf_set_attn_path(0)
    sess.attend_layers(q, k, v, out)                                            # without the block the batch is fine
    torch.cuda.synchronize()
    assert sess.status() == 0


@pytest.mark.parametrize("dtype,head_dim", [("bf16", 128), ("f32", 64)])
def test_assembled_final_cache(dtype, head_dim):
    """cf_assemble_final_cache: survivors' re-positioned keys and values in rank order, then the query rows."""
    from paper_2502_11101_b200.session import Session
    cfg = W.WorkloadConfig("assemble", 3, 8, 2, head_dim, dtype, 1e4, 4096, 9, 20, 150, 6, 2, 2, ((1, 5), (2, 3)))
    seed = _pick_seed(cfg, oracle.ALLOC_SORT, 1e-3)
    meta = W.make_meta(cfg, seed)
    q = W.make_q(meta)
    k, v = W.make_kv(meta)
    k_self, v_self = W.make_kv_self(meta)
    ref = harness.oracle_stack(meta, q, k, v, oracle.ALLOC_SORT)
    sess = Session(cfg.n_q_heads, cfg.n_kv_heads, head_dim, cfg.torch_dtype, cfg.pos_range, cfg.rope_theta, cfg.q_len,
                   meta.doc_len, meta.req_doc_begin, meta.doc_src_start, tail_reserve=cfg.q_len)
    qg, kg, vg, ksg, vsg = [t.cuda() for t in (q, k, v, k_self, v_self)]
    out = torch.empty_like(qg)
    sess.run_stack(qg, kg, vg, cfg.schedule, oracle.ALLOC_SORT, out)
    out_rows = 3 * 150 + cfg.q_len + 7
    sentinel = 12288.0                                               # exact in bf16
    k_out = torch.full((cfg.n_layers, cfg.batch, out_rows, cfg.n_kv_heads, head_dim), sentinel, dtype=cfg.torch_dtype, device="cuda")
    v_out = torch.full_like(k_out, sentinel)
    final_rows = torch.full((cfg.batch,), -1, dtype=torch.int32, device="cuda")
    sess.assemble(kg, vg, ksg, vsg, k_out, v_out, final_rows)
    torch.cuda.synchronize()
    assert sess.status() == 0
    kf_got, vf_got = k_out.float().cpu().numpy(), v_out.float().cpu().numpy()
    for b in range(cfg.batch):
        lo = int(meta.req_doc_begin[b])
        order = ref[b]["order"]
        assert sess.read_plan()["order"][b] == order
        for l in range(cfg.n_layers):
            kf, vf = oracle.assemble_final_cache(ref[b]["k_final"][l], v[l].double().numpy(), meta.doc_offsets, order,
                                                 k_self[l, b].double().numpy(), v_self[l, b].double().numpy(), doc_base=lo)
            n = kf.shape[0]
            assert int(final_rows[b]) == n
            n_docs_rows = n - cfg.q_len
            err = np.abs(kf_got[l, b, :n_docs_rows] - kf[:n_docs_rows]) / harness.rotated_key_tolerance(kf[:n_docs_rows], dtype)
            assert err.max() <= 1.0
            assert np.array_equal(kf_got[l, b, n_docs_rows:n], kf[n_docs_rows:])          # the query rows are copies
            assert np.array_equal(vf_got[l, b, :n], vf)                                   # values are copies
            assert np.all(kf_got[l, b, n:] == sentinel) and np.all(vf_got[l, b, n:] == sentinel)
    # a buffer that is too small is reported, not overrun
    small_k = torch.full((cfg.n_layers, cfg.batch, 10, cfg.n_kv_heads, head_dim), sentinel, dtype=cfg.torch_dtype, device="cuda")
    small_v = torch.full_like(small_k, sentinel)
    sess.assemble(kg, vg, ksg, vsg, small_k, small_v, final_rows)
    torch.cuda.synchronize()
    import paper_2502_11101_b200 as cf
    assert sess.status() == cf.CF_ERR_WORKSPACE


@pytest.mark.parametrize("group,q_len", [(8, 32), (7, 37), (3, 43), (8, 64), (5, 77)])
def test_row_counts_around_the_row_tile_boundaries(group, q_len):
    """256, 259, 129, 512 and 385 query rows per kv head: full row groups, a three-row remainder, one
    row over a tile, two full groups, an odd number of row tiles."""
    lens = [129, 64, 192, 1, 128]
    cfg = W.WorkloadConfig("row-tiles", 2, 2 * group, 2, 128, "bf16", 1e4, 8192, len(lens), 1, 300, q_len, 1, 1, ())
    for batch_layers, self_block in ((False, False), (True, True)):
        harness.run_and_compare(cfg, 3, oracle.ALLOC_ALIGN, doc_len_override=lens, min_margin=0.0,
                                batch_layers=batch_layers, self_block=self_block)


@pytest.mark.parametrize("case", range(10))
def test_random_shapes(case):
    """Seeded random geometries around the tile boundaries of the tensor-core kernel (row counts next to
    128 and 256, one- to three-tile documents, several requests), without pruning so that no score gap
    can decide a result; random call granularity and query-self block."""
    rng = np.random.default_rng(1000 + case)
    n_kv = int(rng.choice([1, 2, 4]))
    group = int(rng.choice([1, 2, 3, 5, 7, 8]))
    q_len = int(rng.choice([1, 3, 16, 18, 19, 26, 32, 37, 43, 64]))
    n_docs = int(rng.integers(1, 7))
    batch = int(rng.integers(1, 4))
    n_layers = int(rng.integers(1, 4))
    lens = [int(x) for x in rng.choice([1, 31, 32, 33, 95, 96, 97, 127, 128, 129, 191, 192, 193, 257, 300],
                                       size=n_docs * batch)]
    cfg = W.WorkloadConfig(f"random-{case}", n_layers, n_kv * group, n_kv, 128, "bf16", 1e4, 8192, n_docs, 1, 300,
                           q_len, batch, 1, ())
    harness.run_and_compare(cfg, case, oracle.ALLOC_ALIGN, doc_len_override=lens, min_margin=0.0,
                            batch_layers=bool(rng.integers(0, 2)), self_block=bool(rng.integers(0, 2)))


def test_query_self_block_when_a_request_has_no_documents():
    """With nothing cached to attend, the layer's attention is the causal query-self block alone."""
    import paper_2502_11101_b200 as cf
    from paper_2502_11101_b200.session import Session
    lens = np.array([40, 130], dtype=np.int32)                       # request 0: none; request 1: two documents
    req = np.array([0, 0, 2], dtype=np.int32)
    hq, hkv, d, lq = 4, 2, 128, 7
    gen = torch.Generator().manual_seed(1)
    q = torch.randn((1, 2, lq, hq, d), generator=gen).bfloat16().cuda()
    k = torch.randn((1, 170, hkv, d), generator=gen).bfloat16().cuda()
    v = torch.randn((1, 170, hkv, d), generator=gen).bfloat16().cuda()
    ks = torch.randn((1, 2, lq, hkv, d), generator=gen).bfloat16().cuda()
    vs = torch.randn((1, 2, lq, hkv, d), generator=gen).bfloat16().cuda()
    for path in (0, 1):
        cf.cf_set_attn_path(path)
        try:
            sess = Session(hq, hkv, d, torch.bfloat16, 4096, 1e4, lq, lens, req, np.zeros(2, dtype=np.int32), tail_reserve=lq)
            sess.init()
            out = torch.full_like(q, float("nan"))
            lse = torch.full((1, 2, hq, lq), float("nan"), device="cuda")
            scores = torch.full((1, 2), float("nan"), device="cuda")
            sess.attend_layers(q, k, v, out, lse, scores, k_self=ks, v_self=vs)
            torch.cuda.synchronize()
        finally:
            cf.cf_set_attn_path(0)
        assert sess.status() == 0
        o_self, lse_self = oracle.query_self_block(q[0, 0].double().cpu().numpy(), ks[0, 0].double().cpu().numpy(),
                                                   vs[0, 0].double().cpu().numpy())
        got = out[0, 0].float().cpu().numpy()
        assert np.all(np.abs(got - o_self) <= 1e-2 + 2e-2 * np.abs(o_self))
        assert np.all(np.abs(lse[0, 0].cpu().numpy() - lse_self) <= 1e-2)
        # request 1: documents and the block, merged
        dst, _, _, _ = oracle.allocate_positions(lens, [0, 1], 4096, 0, lq)
        kr = oracle.reposition_keys(k[0].double().cpu().numpy(), [0, 40, 170], [0, 0], dst, [0, 1], 1e4)
        o_d, lse_d, _, s_ref = oracle.query_prefill_attn(q[0, 1].double().cpu().numpy(), kr, v[0].double().cpu().numpy(),
                                                         [0, 40, 170], [0, 1], 2)
        o_s, lse_s = oracle.query_self_block(q[0, 1].double().cpu().numpy(), ks[0, 1].double().cpu().numpy(),
                                             vs[0, 1].double().cpu().numpy())
        o_ref, lse_ref = oracle.merge_softmax_blocks(o_d, lse_d, o_s, lse_s)
        got = out[0, 1].float().cpu().numpy()
        assert np.all(np.abs(got - o_ref) <= 1e-2 + 2e-2 * np.abs(o_ref))
        assert np.all(np.abs(lse[0, 1].cpu().numpy() - lse_ref) <= 1e-2)
        assert np.allclose(scores[0].cpu().numpy(), s_ref, rtol=2e-2, atol=1e-3)


def test_pinned_prefix_attended_by_its_own_call_and_merged():
    """A shared prefix cache (Algorithm 2, C_prefix): attended by a call of its own with delta 0, merged
    with the documents' result by cf_merge_attn; it is in no kept list, so it is never pruned and the
    documents' scores are those of the documents alone."""
    import paper_2502_11101_b200 as cf
    from paper_2502_11101_b200.session import Session
    hq, hkv, d, lq, prefix, pos_range, theta = 8, 2, 128, 6, 40, 4096, 1e4
    lens = np.array([130, 64, 17, 96, 200], dtype=np.int32)
    gen = torch.Generator().manual_seed(2)
    q = torch.randn((2, 1, lq, hq, d), generator=gen).bfloat16()
    k = torch.randn((2, int(lens.sum()), hkv, d), generator=gen).bfloat16()
    v = torch.randn((2, int(lens.sum()), hkv, d), generator=gen).bfloat16()
    kp = torch.randn((2, prefix, hkv, d), generator=gen).bfloat16()          # prefix keys, as cached at positions 0..39
    vp = torch.randn((2, prefix, hkv, d), generator=gen).bfloat16()
    docs = Session(hq, hkv, d, torch.bfloat16, pos_range, theta, lq, lens, np.array([0, 5], dtype=np.int32),
                   np.full(5, prefix, dtype=np.int32), tail_reserve=lq, prefix_len=prefix)
    qs = pos_range - lq
    # the prefix as the one "document" of a batch of its own; cached where the allocation will put it => delta 0
    pre = Session(hq, hkv, d, torch.bfloat16, pos_range, theta, lq, np.array([prefix], dtype=np.int32),
                  np.array([0, 1], dtype=np.int32), np.array([qs - prefix], dtype=np.int32), tail_reserve=lq)
    qg, kg, vg, kpg, vpg = [t.cuda() for t in (q, k, v, kp, vp)]
    docs.init()
    pre.init()
    assert int(pre.read_plan()["dst_start"][0]) == qs - prefix
    out_a, out_b = torch.empty_like(qg), torch.empty_like(qg)
    lse_a = torch.empty((2, 1, hq, lq), device="cuda")
    lse_b = torch.empty_like(lse_a)
    scores = torch.empty((2, 5), device="cuda")
    for layer in range(2):
        docs.attend(qg[layer], kg[layer], vg[layer], out_a[layer], lse_a[layer])
        scores[layer].copy_(docs.doc_scores)
        pre.attend(qg[layer], kpg[layer], vpg[layer], out_b[layer], lse_b[layer])
        if layer == 0:
            docs.prune(3, oracle.ALLOC_ALIGN)
    out = torch.empty_like(qg)
    lse = torch.empty_like(lse_a)
    cf.cf_merge_attn(docs.geom, out_a, lse_a, out_b, lse_b, out, lse)
    torch.cuda.synchronize()
    assert docs.status() == 0 and pre.status() == 0
    # oracle: one softmax over the prefix (keys as cached) and the kept documents (keys re-positioned)
    offsets = np.concatenate([[0], np.cumsum(lens)])
    order = list(range(5))
    accum = np.zeros(5)
    for layer in range(2):
        dst, _, _, _ = oracle.allocate_positions(lens, order, pos_range, prefix, lq)
        assert np.all(dst[order] >= prefix)                                  # documents stay clear of the prefix positions
        k_rot = oracle.reposition_keys(k[layer].double().numpy(), offsets, np.full(5, prefix), dst, order, theta)
        k_all = np.concatenate([kp[layer].double().numpy(), k_rot])
        v_all = np.concatenate([vp[layer].double().numpy(), v[layer].double().numpy()])
        off_all = np.concatenate([[0], prefix + offsets])
        o_ref, lse_ref, _, _ = oracle.query_prefill_attn(q[layer, 0].double().numpy(), k_all, v_all, off_all,
                                                         [0] + [1 + i for i in order], 6)
        _, _, _, s_docs = oracle.query_prefill_attn(q[layer, 0].double().numpy(), k_rot, v[layer].double().numpy(),
                                                    offsets, order, 5)
        got = out[layer, 0].float().cpu().numpy()
        assert np.all(np.abs(got - o_ref) <= 1e-2 + 2e-2 * np.abs(o_ref))
        assert np.all(np.abs(lse[layer, 0].cpu().numpy() - lse_ref) <= 1e-2)
        assert np.allclose(scores[layer].cpu().numpy(), s_docs, rtol=2e-2, atol=1e-3)
        accum += s_docs
        if layer == 0:
            order = oracle.prune_topk(accum, order, 3, oracle.ALLOC_ALIGN)
    assert docs.read_plan()["order"][0] == order


def test_decoding_step_over_the_assembled_final_cache():
    """A new token's query row attends a request's final cache straight out of cf_assemble_final_cache:
    each request's packed rows are one "document" cached where the allocation puts it (delta 0), the
    unused tail of its slot a second document that is never kept."""
    from paper_2502_11101_b200.session import Session
    cfg = W.WorkloadConfig("decode", 2, 8, 2, 128, "bf16", 1e4, 4096, 7, 20, 150, 5, 2, 2, ((1, 3),))
    seed = _pick_seed(cfg, oracle.ALLOC_ALIGN, 1e-3)
    meta = W.make_meta(cfg, seed)
    q, (k, v), (k_self, v_self) = W.make_q(meta), W.make_kv(meta), W.make_kv_self(meta)
    ref = harness.oracle_stack(meta, q, k, v, oracle.ALLOC_ALIGN)
    sess = Session(cfg.n_q_heads, cfg.n_kv_heads, 128, cfg.torch_dtype, cfg.pos_range, cfg.rope_theta, cfg.q_len,
                   meta.doc_len, meta.req_doc_begin, meta.doc_src_start, tail_reserve=cfg.q_len)
    qg, kg, vg, ksg, vsg = [t.cuda() for t in (q, k, v, k_self, v_self)]
    sess.run_stack(qg, kg, vg, cfg.schedule, oracle.ALLOC_ALIGN, torch.empty_like(qg))
    out_rows = 3 * 150 + cfg.q_len + 9
    k_out = torch.zeros((cfg.n_layers, cfg.batch, out_rows, cfg.n_kv_heads, 128), dtype=torch.bfloat16, device="cuda")
    v_out = torch.zeros_like(k_out)
    final_rows = torch.zeros(cfg.batch, dtype=torch.int32, device="cuda")
    sess.assemble(kg, vg, ksg, vsg, k_out, v_out, final_rows)
    rows = final_rows.cpu().numpy()
    # the decoding batch: per request (final cache, unused tail), only the first kept
    doc_len = np.stack([rows, out_rows - rows], axis=1).reshape(-1).astype(np.int32)
    qs = cfg.pos_range - 1
    src = np.stack([qs - rows, np.zeros_like(rows)], axis=1).reshape(-1).astype(np.int32)
    dec = Session(cfg.n_q_heads, cfg.n_kv_heads, 128, cfg.torch_dtype, cfg.pos_range, cfg.rope_theta, 1, doc_len,
                  np.arange(cfg.batch + 1, dtype=np.int32) * 2, src, tail_reserve=1, n_reuse=1)
    order = torch.tensor([0, 1] * cfg.batch, dtype=torch.int32, device="cuda")
    kept_count = torch.ones(cfg.batch, dtype=torch.int32, device="cuda")
    dec.set_live_docs(1)
    dec.init(order, kept_count)
    gen = torch.Generator().manual_seed(3)
    q_new = torch.randn((cfg.n_layers, cfg.batch, 1, cfg.n_q_heads, 128), generator=gen).bfloat16().cuda()
    out = torch.empty_like(q_new)
    lse = torch.empty((cfg.n_layers, cfg.batch, cfg.n_q_heads, 1), device="cuda")
    dec.attend_layers(q_new, k_out.view(cfg.n_layers, cfg.batch * out_rows, cfg.n_kv_heads, 128),
                      v_out.view(cfg.n_layers, cfg.batch * out_rows, cfg.n_kv_heads, 128), out, lse)
    torch.cuda.synchronize()
    assert dec.status() == 0 and sess.status() == 0
    assert [len(o) for o in dec.read_plan()["order"]] == [1] * cfg.batch
    for b in range(cfg.batch):
        lo = int(meta.req_doc_begin[b])
        for l in range(cfg.n_layers):
            kf, vf = oracle.assemble_final_cache(ref[b]["k_final"][l], v[l].double().numpy(), meta.doc_offsets,
                                                 ref[b]["order"], k_self[l, b].double().numpy(),
                                                 v_self[l, b].double().numpy(), doc_base=lo)
            assert kf.shape[0] == rows[b]
            o_ref, lse_ref, _, _ = oracle.query_prefill_attn(q_new[l, b].double().cpu().numpy(), kf, vf,
                                                             [0, kf.shape[0]], [0], 1)
            got = out[l, b].float().cpu().numpy()
            assert np.all(np.abs(got - o_ref) <= 1e-2 + 2e-2 * np.abs(o_ref))
            assert np.all(np.abs(lse[l, b].cpu().numpy() - lse_ref) <= 1e-2)


@pytest.mark.parametrize("prefix,q_len,heads,with_self", [
    (40, 6, (8, 2), False),          # one prefix tile, one row tile, both warpgroups on alternate tiles
    (200, 48, (12, 2), True),        # two prefix tiles, 288 rows per kv head, the query-self block behind them
    (130, 64, (8, 2), True),         # 256 rows: two row tiles side by side
    (128, 3, (4, 4), True),          # a full prefix tile, fewer document tiles than parts
])
def test_pinned_prefix_attended_inside_the_call(prefix, q_len, heads, with_self):
    _pinned_prefix_case(prefix, q_len, heads, with_self)


@pytest.mark.parametrize("prefix,q_len,heads,with_self", [
    (40, 6, (8, 2), False),          # a prefix alone: one chunk of keys
    (200, 48, (12, 2), True),        # two chunks of prefix keys, then the causal chunk of the query tokens
    (128, 3, (4, 4), True),          # a full chunk
])
def test_pinned_prefix_on_the_cuda_core_path(prefix, q_len, heads, with_self):
    """The same cases through the CUDA-core kernels: prefix and query-self block are one more part of the merge."""
    import paper_2502_11101_b200 as cf
    cf.cf_set_attn_path(1)
    try:
        _pinned_prefix_case(prefix, q_len, heads, with_self)
    finally:
        cf.cf_set_attn_path(0)


def _pinned_prefix_case(prefix, q_len, heads, with_self):
    """cf_query_prefill_attn_prefix: the shared prefix cache rides along as further key tiles (delta 0, seen by
    every query row), with or without the causal query-self block behind it; one softmax over prefix, kept
    documents and query tokens in the oracle.  Document scores stay those of the documents alone, pruning
    included; two layers in one call as well as one by one."""
    import paper_2502_11101_b200 as cf
    from paper_2502_11101_b200.session import Session
    hq, hkv = heads
    d, pos_range, theta = 128, 4096, 1e4
    lens = np.array([130, 64, 17, 96, 200, 128, 33], dtype=np.int32)
    n = len(lens)
    gen = torch.Generator().manual_seed(5)
    rnd = lambda *shape: torch.randn(shape, generator=gen).bfloat16()
    q, k, v = rnd(2, 1, q_len, hq, d), rnd(2, int(lens.sum()), hkv, d), rnd(2, int(lens.sum()), hkv, d)
    kp, vp = rnd(2, prefix, hkv, d), rnd(2, prefix, hkv, d)
    ks, vs = rnd(2, 1, q_len, hkv, d), rnd(2, 1, q_len, hkv, d)
    sess = Session(hq, hkv, d, torch.bfloat16, pos_range, theta, q_len, lens, np.array([0, n], dtype=np.int32),
                   np.full(n, prefix, dtype=np.int32), tail_reserve=q_len, prefix_len=prefix)
    qg, kg, vg, kpg, vpg, ksg, vsg = [t.cuda() for t in (q, k, v, kp, vp, ks, vs)]
    offsets = np.concatenate([[0], np.cumsum(lens)])

    def reference(order):
        """Per layer: (out, lse) over prefix + documents (+ query tokens), and the documents' scores."""
        res = []
        for layer in range(2):
            dst, _, _, _ = oracle.allocate_positions(lens, order, pos_range, prefix, q_len)
            assert np.all(dst[order] >= prefix)
            k_rot = oracle.reposition_keys(k[layer].double().numpy(), offsets, np.full(n, prefix), dst, order, theta)
            k_all = np.concatenate([kp[layer].double().numpy(), k_rot])
            v_all = np.concatenate([vp[layer].double().numpy(), v[layer].double().numpy()])
            qd = q[layer, 0].double().numpy()
            o_ref, lse_ref, _, _ = oracle.query_prefill_attn(qd, k_all, v_all, np.concatenate([[0], prefix + offsets]),
                                                             [0] + [1 + i for i in order], n + 1)
            if with_self:
                o_self, lse_self = oracle.query_self_block(qd, ks[layer, 0].double().numpy(), vs[layer, 0].double().numpy())
                o_ref, lse_ref = oracle.merge_softmax_blocks(o_ref, lse_ref, o_self, lse_self)
            _, _, _, s_docs = oracle.query_prefill_attn(qd, k_rot, v[layer].double().numpy(), offsets, order, n)
            res.append((o_ref, lse_ref, s_docs))
        return res

    def check(out, lse, scores, ref):
        for layer in range(2):
            o_ref, lse_ref, s_docs = ref[layer]
            got = out[layer, 0].float().cpu().numpy()
            assert np.all(np.abs(got - o_ref) <= 1e-2 + 2e-2 * np.abs(o_ref)), layer
            assert np.all(np.abs(lse[layer, 0].cpu().numpy() - lse_ref) <= 1e-2), layer
            s_got = scores[layer].cpu().numpy()
            assert np.all(np.abs(s_got - s_docs) <= 1e-2 / max(1, int((s_docs > 0).sum())) + 2e-2 * s_docs), layer
            assert abs(float(s_got.sum()) - 1.0) < 1e-3

    out = torch.full_like(qg, float("nan"))
    lse = torch.full((2, 1, hq, q_len), float("nan"), device="cuda")
    scores = torch.full((2, n), float("nan"), device="cuda")
    sess.init()
    sess.reserve_workspace(2, with_self=True)
    self_kv = dict(k_self=ksg, v_self=vsg) if with_self else {}
    # both layers in one call, every document kept
    cf.cf_query_prefill_attn_prefix(sess.geom, sess.batch, sess.plan, qg, kg, vg, kpg, vpg, out, sess.workspace,
                                    lse=lse, doc_scores=scores, score_accum=sess.score_accum, **self_kv)
    torch.cuda.synchronize()
    assert sess.status() == 0
    order = list(range(n))
    ref = reference(order)
    check(out, lse, scores, ref)
    accum = ref[0][2] + ref[1][2]
    assert np.all(np.abs(sess.score_accum.cpu().numpy() - accum) <= 1e-2 + 2e-2 * accum)
    # a pruning step on those sums, then layer by layer over the survivors
    sess.prune(3, oracle.ALLOC_ALIGN)
    order = oracle.prune_topk(accum, order, 3, oracle.ALLOC_ALIGN)
    assert sess.read_plan()["order"][0] == order
    out.fill_(float("nan"))
    for layer in range(2):
        kw = {key: t[layer:layer + 1] for key, t in self_kv.items()}
        cf.cf_query_prefill_attn_prefix(sess.geom, sess.batch, sess.plan, qg[layer:layer + 1], kg[layer:layer + 1],
                                        vg[layer:layer + 1], kpg[layer:layer + 1], vpg[layer:layer + 1],
                                        out[layer:layer + 1], sess.workspace, lse=lse[layer:layer + 1],
                                        doc_scores=scores[layer:layer + 1], **kw)
    torch.cuda.synchronize()
    assert sess.status() == 0
    check(out, lse, scores, reference(order))
    # the same through the library's stack driver: layer 1 over every document, pruning on its scores, layer 2
    out2 = torch.full_like(qg, float("nan"))
    lse2 = torch.full_like(lse, float("nan"))
    scores2 = torch.full_like(scores, float("nan"))
    sess.run_stack(qg, kg, vg, ((1, 3),), oracle.ALLOC_ALIGN, out2, lse2, None, scores2, batch_layers=False,
                   k_prefix=kpg, v_prefix=vpg, **self_kv)
    torch.cuda.synchronize()
    assert sess.status() == 0
    first = reference(list(range(n)))
    order2 = oracle.prune_topk(first[0][2], list(range(n)), 3, oracle.ALLOC_ALIGN)
    assert sess.read_plan()["order"][0] == order2
    check(out2, lse2, scores2, [first[0], reference(order2)[1]])

