"""Decoding over the final caches (cf_decode_append / cf_decode_plan / cf_decode_attn) against the oracle's
decode_steps: the caches come out of cf_assemble_final_cache, every step appends one token per request and
its query row attends the grown cache."""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_11101_b200 as cf
from paper_2502_11101_b200 import workloads as W
from paper_2502_11101_b200.session import Session
from tests import harness

pytestmark = pytest.mark.gpu


def _final_caches(cfg, seed, slack):
    """Runs the stack and Phase 2 on the GPU; returns the packed final caches, the rows in use, and the
    oracle's final caches per (layer, request)."""
    meta = W.make_meta(cfg, seed)
    q, (k, v), (k_self, v_self) = W.make_q(meta), W.make_kv(meta), W.make_kv_self(meta)
    ref = harness.oracle_stack(meta, q, k, v, oracle.ALLOC_ALIGN)
    assert harness.cut_margins(meta, ref, oracle.ALLOC_ALIGN) >= 1e-3
    sess = Session(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.torch_dtype, cfg.pos_range, cfg.rope_theta, cfg.q_len,
                   meta.doc_len, meta.req_doc_begin, meta.doc_src_start, tail_reserve=cfg.q_len)
    qg, kg, vg, ksg, vsg = [t.cuda() for t in (q, k, v, k_self, v_self)]
    sess.run_stack(qg, kg, vg, cfg.schedule, oracle.ALLOC_ALIGN, torch.empty_like(qg))
    keep = cfg.schedule[-1][1] if cfg.schedule else cfg.n_docs
    cache_rows = keep * cfg.doc_len_hi + cfg.q_len + slack
    k_fin = torch.zeros((cfg.n_layers, cfg.batch, cache_rows, cfg.n_kv_heads, cfg.head_dim), dtype=cfg.torch_dtype, device="cuda")
    v_fin = torch.zeros_like(k_fin)
    rows = torch.zeros(cfg.batch, dtype=torch.int32, device="cuda")
    sess.assemble(kg, vg, ksg, vsg, k_fin, v_fin, rows)
    torch.cuda.synchronize()
    assert sess.status() == 0
    want = {}
    for b in range(cfg.batch):
        lo = int(meta.req_doc_begin[b])
        for l in range(cfg.n_layers):
            want[l, b] = oracle.assemble_final_cache(ref[b]["k_final"][l], v[l].double().numpy(), meta.doc_offsets,
                                                     ref[b]["order"], k_self[l, b].double().numpy(),
                                                     v_self[l, b].double().numpy(), doc_base=lo)
    return sess.geom, k_fin, v_fin, rows, cache_rows, want


@pytest.mark.parametrize("which", ["gqa-bf16-tensor-core", "mha-f32-cuda-core"])
def test_four_decoding_steps_over_the_assembled_caches(which):
    if which == "gqa-bf16-tensor-core":
        cfg = W.WorkloadConfig("decode", 2, 8, 2, 128, "bf16", 1e4, 4096, 7, 20, 150, 5, 2, 2, ((1, 3),))
        steps, layers_per_call = 4, 2                      # both layers of a step in one call
    else:
        cfg = W.WorkloadConfig("decode", 2, 4, 4, 64, "f32", 1e4, 2048, 6, 10, 70, 3, 2, 2, ((1, 3),))
        steps, layers_per_call = 4, 1                      # one call per layer, as a running model issues them
    seed = next(s for s in range(20) if _margin_ok(cfg, s))
    geom, k_fin, v_fin, rows, cache_rows, want = _final_caches(cfg, seed, slack=steps + 3)
    rows_h = rows.cpu().numpy()
    L, B, hq, hkv, d = cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    gen = torch.Generator().manual_seed(7)
    q_new = torch.randn((steps, L, B, hq, d), generator=gen).to(cfg.torch_dtype)
    k_new = torch.randn((steps, L, B, hkv, d), generator=gen).to(cfg.torch_dtype)
    v_new = torch.randn((steps, L, B, hkv, d), generator=gen).to(cfg.torch_dtype)
    plan = torch.zeros(cf.cf_decode_plan_bytes(geom, B, cache_rows), dtype=torch.uint8, device="cuda")
    work = torch.empty(cf.cf_decode_workspace_bytes(geom, B, cache_rows, layers_per_call), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got_out = torch.full((steps, L, B, hq, d), float("nan"), dtype=cfg.torch_dtype, device="cuda")
    got_lse = torch.full((steps, L, B, hq), float("nan"), device="cuda")
    untouched_k = k_fin.clone()
    for t in range(steps):
        cf.cf_decode_append(geom, B, cache_rows, k_fin, v_fin, rows, t, k_new[t].cuda(), v_new[t].cuda(), status)
        cf.cf_decode_plan(geom, B, cache_rows, rows, t + 1, plan)
        qt = q_new[t].cuda()
        for l0 in range(0, L, layers_per_call):
            l1 = l0 + layers_per_call
            cf.cf_decode_attn(geom, B, cache_rows, plan, qt[l0:l1], k_fin[l0:l1], v_fin[l0:l1], got_out[t, l0:l1], work,
                              got_lse[t, l0:l1])
    torch.cuda.synchronize()
    assert cf.cf_decode_status(geom, B, cache_rows, plan) == 0 and int(status.item()) == 0
    for b in range(B):
        n = int(rows_h[b])
        # the appended rows sit right behind the rows in use, bit for bit; nothing else moved
        assert torch.equal(k_fin[:, b, n:n + steps].cpu(), k_new[:, :, b].transpose(0, 1))
        assert torch.equal(v_fin[:, b, n:n + steps].cpu(), v_new[:, :, b].transpose(0, 1))
        assert torch.equal(k_fin[:, b, :n], untouched_k[:, b, :n]) and torch.equal(k_fin[:, b, n + steps:], untouched_k[:, b, n + steps:])
        for l in range(L):
            kf, vf = want[l, b]
            assert kf.shape[0] == n
            o_ref, lse_ref = oracle.decode_steps(kf, vf, q_new[:, l, b].double().numpy(), k_new[:, l, b].double().numpy(),
                                                 v_new[:, l, b].double().numpy())
            got = got_out[:, l, b].float().cpu().numpy()
            assert np.all(np.abs(got - o_ref) <= 1e-2 + 2e-2 * np.abs(o_ref)), (l, b)
            assert np.all(np.abs(got_lse[:, l, b].cpu().numpy() - lse_ref) <= 1e-2), (l, b)


def _margin_ok(cfg, seed):
    meta = W.make_meta(cfg, seed)
    q, (k, v) = W.make_q(meta), W.make_kv(meta)
    ref = harness.oracle_stack(meta, q, k, v, oracle.ALLOC_ALIGN, final_reposition=False)
    return harness.cut_margins(meta, ref, oracle.ALLOC_ALIGN) >= 1e-3


def test_decode_calls_report_a_full_slot():
    geom = cf.make_geom(4, 4, 64, cf.CF_F32, 2048, 1e4)
    B, cache_rows = 2, 40
    plan = torch.zeros(cf.cf_decode_plan_bytes(geom, B, cache_rows), dtype=torch.uint8, device="cuda")
    rows = torch.tensor([10, 40], dtype=torch.int32, device="cuda")          # the second slot is full
    cf.cf_decode_plan(geom, B, cache_rows, rows, 1, plan)
    assert cf.cf_decode_status(geom, B, cache_rows, plan) == cf.CF_ERR_RANGE
    k_fin = torch.zeros((1, B, cache_rows, 4, 64), device="cuda")
    v_fin = torch.zeros_like(k_fin)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    new = torch.ones((1, B, 4, 64), device="cuda")
    cf.cf_decode_append(geom, B, cache_rows, k_fin, v_fin, rows, 0, new, new, status)
    torch.cuda.synchronize()
    assert int(status.item()) == cf.CF_ERR_RANGE
    assert bool(torch.all(k_fin[0, 0, 10] == 1)) and float(k_fin[0, 1].abs().sum()) == 0.0   # the full slot was skipped
    with pytest.raises(cf.CacheFocusError):
        cf.cf_decode_plan(geom, B, cache_rows, rows, 1, plan[: plan.numel() // 2])


@pytest.mark.parametrize("layers_per_call", [1, 2])
def test_bench_sized_caches_one_step(layers_per_call):
    """Caches of the size bench.py times for decoding (28 query / 4 kv heads, four requests with up to 16 000 rows in
    use: every CTA walks tens of full key tiles), ragged fill levels, one appended token; every (layer, request) against
    the oracle."""
    L, B, hq, hkv, d, cache_rows = 2, 4, 28, 4, 128, 16064
    geom = cf.make_geom(hq, hkv, d, cf.CF_BF16, 32768, 1e6)
    used = np.array([16000, 15001, 9000, 127], dtype=np.int32)
    gen = torch.Generator().manual_seed(11)
    k_fin = torch.randn((L, B, cache_rows, hkv, d), generator=gen).bfloat16()
    v_fin = torch.randn((L, B, cache_rows, hkv, d), generator=gen).bfloat16()
    q_new = torch.randn((L, B, hq, d), generator=gen).bfloat16()
    k_new = torch.randn((L, B, hkv, d), generator=gen).bfloat16()
    v_new = torch.randn((L, B, hkv, d), generator=gen).bfloat16()
    kg, vg, rows = k_fin.cuda(), v_fin.cuda(), torch.from_numpy(used).cuda()
    plan = torch.zeros(cf.cf_decode_plan_bytes(geom, B, cache_rows), dtype=torch.uint8, device="cuda")
    work = torch.empty(cf.cf_decode_workspace_bytes(geom, B, cache_rows, layers_per_call), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.full((L, B, hq, d), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((L, B, hq), float("nan"), device="cuda")
    cf.cf_decode_append(geom, B, cache_rows, kg, vg, rows, 0, k_new.cuda(), v_new.cuda(), status)
    cf.cf_decode_plan(geom, B, cache_rows, rows, 1, plan)
    qg = q_new.cuda()
    for l0 in range(0, L, layers_per_call):
        l1 = l0 + layers_per_call
        cf.cf_decode_attn(geom, B, cache_rows, plan, qg[l0:l1], kg[l0:l1], vg[l0:l1], out[l0:l1], work, lse[l0:l1])
    torch.cuda.synchronize()
    assert cf.cf_decode_status(geom, B, cache_rows, plan) == 0 and int(status.item()) == 0
    for l in range(L):
        for b in range(B):
            n = int(used[b])
            o_ref, lse_ref = oracle.decode_steps(k_fin[l, b, :n].double().numpy(), v_fin[l, b, :n].double().numpy(),
                                                 q_new[l, b][None].double().numpy(), k_new[l, b][None].double().numpy(),
                                                 v_new[l, b][None].double().numpy())
            got = out[l, b].float().cpu().numpy()
            assert np.all(np.abs(got - o_ref[0]) <= 1e-2 + 2e-2 * np.abs(o_ref[0])), (l, b)
            assert np.all(np.abs(lse[l, b].cpu().numpy() - lse_ref[0]) <= 1e-2), (l, b)
