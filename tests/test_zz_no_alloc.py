"""The attention entry point that carries its own scratch (for callers that may not allocate
device memory) must give what the ordinary entry point gives.  Collected last on purpose: a run
that stops at the first failure has then already seen every other test."""
import pytest
import torch

import oracle
import paper_2502_11101_b200 as cf
from paper_2502_11101_b200 import workloads as W
from paper_2502_11101_b200.session import Session

pytestmark = pytest.mark.gpu


def _session(cfg, meta):
    return Session(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.torch_dtype, cfg.pos_range, cfg.rope_theta,
                   cfg.q_len, meta.doc_len, meta.req_doc_begin, meta.doc_src_start, tail_reserve=cfg.q_len)


def test_static_scratch_entry_point_matches_the_ordinary_one():
    from paper_2502_11101_b200 import build
    build.build()
    cfg = W.scaled_config(W.CONFIGS[3], n_layers=2, n_docs=16, n_planted=3, schedule=())
    meta = W.make_meta(cfg, 5)
    q = W.make_q(meta).cuda()
    k, v = [t.cuda() for t in W.make_kv(meta)]
    sess = _session(cfg, meta)
    sess.init()
    assert cf.cf_attn_workspace_bytes(sess.geom, sess.batch) <= 32 << 20
    shape_lse = (cfg.batch, cfg.n_q_heads, cfg.q_len)
    for layer in range(2):                                   # two calls in a row share the scratch array
        want_out, got_out = torch.empty_like(q[layer]), torch.full_like(q[layer], float("nan"))
        want_lse = torch.empty(shape_lse, device="cuda")
        got_lse = torch.full(shape_lse, float("nan"), device="cuda")
        want_s = torch.empty(meta.n_docs_total, device="cuda")
        got_s = torch.full((meta.n_docs_total,), float("nan"), device="cuda")
        want_acc = torch.zeros(meta.n_docs_total, device="cuda")
        got_acc = torch.zeros(meta.n_docs_total, device="cuda")
        cf.cf_query_prefill_attn(sess.geom, sess.batch, sess.plan, q[layer], k[layer], v[layer], want_out,
                                 sess.workspace, want_lse, want_s, want_acc)
        cf.cf_query_prefill_attn_static(sess.geom, sess.batch, sess.plan, q[layer], k[layer], v[layer], got_out,
                                        got_lse, got_s, got_acc)
        torch.cuda.synchronize()
        w, g = want_out.float(), got_out.float()
        assert torch.all((g - w).abs() <= 1e-2 + 2e-2 * w.abs())
        assert torch.all((got_lse - want_lse).abs() <= 1e-2)
        assert torch.all((got_s - want_s).abs() <= 1e-2 / cfg.n_docs + 2e-2 * want_s.abs())
        assert torch.all((got_acc - want_acc).abs() <= 1e-2 / cfg.n_docs + 2e-2 * want_acc.abs())
        assert abs(float(got_s.sum()) - 1.0) < 1e-3
        # and against the oracle itself, on the same seeded inputs
        kd = k[layer].double().cpu().numpy()
        dst, _, _, _ = oracle.allocate_positions(meta.doc_len, range(cfg.n_docs), cfg.pos_range, 0, cfg.q_len)
        k_rot = oracle.reposition_keys(kd, meta.doc_offsets, meta.doc_src_start, dst, range(cfg.n_docs), cfg.rope_theta)
        o_ref, lse_ref, _, s_ref = oracle.query_prefill_attn(q[layer, 0].double().cpu().numpy(), k_rot,
                                                             v[layer].double().cpu().numpy(), meta.doc_offsets,
                                                             range(cfg.n_docs), cfg.n_docs)
        o_got = got_out[0].float().cpu().numpy()
        assert (abs(o_got - o_ref) <= 1e-2 + 2e-2 * abs(o_ref)).all()
        assert (abs(got_lse[0].cpu().numpy() - lse_ref) <= 1e-2).all()
        assert (abs(got_s.cpu().numpy() - s_ref) <= 1e-2 / cfg.n_docs + 2e-2 * abs(s_ref)).all()


def test_static_scratch_entry_point_refuses_batches_that_do_not_fit():
    cfg = W.scaled_config(W.CONFIGS[4], n_layers=1, batch=16)         # needs more than 32 MiB
    meta = W.make_meta(cfg, 0)
    sess = _session(cfg, meta)
    assert cf.cf_attn_workspace_bytes(sess.geom, sess.batch) > 32 << 20
    dummy = torch.zeros(16, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(cf.CacheFocusError) as e:
        cf.cf_query_prefill_attn_static(sess.geom, sess.batch, sess.plan, dummy, dummy, dummy, dummy)
    assert e.value.code == cf.CF_ERR_WORKSPACE
