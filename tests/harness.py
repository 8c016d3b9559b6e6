"""Runs the CUDA library and the CPU oracle on the same seeded workload and compares them."""
from __future__ import annotations

from typing import Dict, List, Optional

import numpy as np
import torch

import oracle
from paper_2502_11101_b200 import workloads as W

OUT_ATOL, OUT_RTOL = 1e-2, 2e-2          # attention outputs: |g - o| <= atol + rtol |o|
SCORE_RTOL = 2e-2                        # scores: |g - o| <= 1e-2 / n_kept + rtol |o|


def bf16_ulp(x: np.ndarray) -> np.ndarray:
    """Spacing of bf16 numbers at the binade of |x| (8 significand bits)."""
    ax = np.maximum(np.abs(x), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(ax)) - 7)


def f32_ulp(x: np.ndarray) -> np.ndarray:
    ax = np.maximum(np.abs(x), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(ax)) - 23)


def rotated_key_tolerance(want: np.ndarray, dtype: str, interleaved: bool = False) -> np.ndarray:
    """Allowed |gpu - oracle| for re-positioned keys `want` [..., D]: one rounding to the storage type at
    the result (one bf16 spacing; nothing for fp32 storage) plus 4 fp32 spacings at the magnitude of
    the two-dimensional slice the coordinate belongs to.  A rotation keeps the norm of a slice, so a
    nearly cancelled coordinate cannot be more exact than fp32 arithmetic on its slice allows."""
    if interleaved:
        norm = np.repeat(np.sqrt(want[..., 0::2] ** 2 + want[..., 1::2] ** 2), 2, axis=-1)
    else:
        half = want.shape[-1] // 2
        norm = np.sqrt(want[..., :half] ** 2 + want[..., half:] ** 2)
        norm = np.concatenate([norm, norm], axis=-1)
    arith = 4.0 * f32_ulp(norm)
    return arith if dtype == "f32" else bf16_ulp(want) + arith


def oracle_stack(meta: W.WorkloadMeta, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, strategy: int,
                 schedule=None, final_reposition: bool = True, n_reuse: int = 0, scale: Optional[float] = None,
                 key_round=None) -> List[Dict]:
    """`key_round` (e.g. oracle.round_to_bf16): the layers attend re-positioned keys held in the store's type."""
    cfg = meta.cfg
    qd, kd, vd = q.double().cpu().numpy(), k.double().cpu().numpy(), v.double().cpu().numpy()
    res = []
    for b in range(cfg.batch):
        lo, hi = int(meta.req_doc_begin[b]), int(meta.req_doc_begin[b + 1])
        res.append(oracle.run_stack(qd[:, b], kd, vd, meta.doc_len[lo:hi], meta.doc_offsets,
                                    meta.doc_src_start[lo:hi], cfg.rope_theta, cfg.pos_range,
                                    cfg.schedule if schedule is None else schedule, strategy,
                                    tail_reserve=cfg.q_len, n_reuse=n_reuse, doc_base=lo,
                                    final_reposition=final_reposition, scale=scale, key_round=key_round))
    return res


def cut_margins(meta: W.WorkloadMeta, ref: List[Dict], strategy: int, schedule=None) -> float:
    """Smallest relative score gap that decides an integer result: at every cut of the schedule,
    and for "sort" between neighbouring survivors."""
    cfg = meta.cfg
    worst = np.inf
    for b in range(cfg.batch):
        for layer, keep in (cfg.schedule if schedule is None else schedule):
            rec = ref[b]["layers"][layer - 1]
            vals = sorted((rec["score_accum"][i] for i in rec["order_in"]), reverse=True)
            if keep < len(vals):
                worst = min(worst, (vals[keep - 1] - vals[keep]) / vals[keep - 1])
            if strategy == oracle.ALLOC_SORT:
                for a, c in zip(vals[:keep], vals[1:keep]):
                    worst = min(worst, (a - c) / a)
    return float(worst)


def add_self_block(meta: W.WorkloadMeta, ref: List[Dict], q: torch.Tensor, k_self: torch.Tensor,
                   v_self: torch.Tensor, scale: Optional[float] = None) -> None:
    """Replace every layer's output and log-sum-exp of the oracle run by the merge with the causal
    query-self block (document scores are defined on the documents alone and stay)."""
    qd, ks, vs = q.double().cpu().numpy(), k_self.double().cpu().numpy(), v_self.double().cpu().numpy()
    for b in range(meta.cfg.batch):
        for l, rec in enumerate(ref[b]["layers"]):
            o_self, lse_self = oracle.query_self_block(qd[l, b], ks[l, b], vs[l, b], scale)
            rec["out"], rec["lse"] = oracle.merge_softmax_blocks(rec["out"], rec["lse"], o_self, lse_self)


PAD_SENTINEL = 12288.0                   # exact in bf16 and fp32: fills the padding of a padded store


def padded_store(t: torch.Tensor, token_stride: int, device) -> torch.Tensor:
    """`t` [L, T, Hkv, D] on `device` as a view into a store whose rows are `token_stride` elements
    apart; the padding behind every row holds PAD_SENTINEL."""
    n_layers, total, hkv, d = t.shape
    base = torch.full((n_layers, total, token_stride), PAD_SENTINEL, dtype=t.dtype, device=device)
    view = base[:, :, :hkv * d].view(n_layers, total, hkv, d)
    view.copy_(t)
    return view


def padding_of(view: torch.Tensor, token_stride: int) -> torch.Tensor:
    """The padding columns of a store made by padded_store."""
    n_layers, total, hkv, d = view.shape
    base = torch.as_strided(view, (n_layers, total, token_stride), (total * token_stride, token_stride, 1))
    return base[:, :, hkv * d:]


def gpu_stack(meta: W.WorkloadMeta, q, k, v, strategy: int, schedule=None, device="cuda:0", n_reuse: int = 0,
              with_final: bool = True, batch_layers: bool = False, k_self=None, v_self=None,
              driver: str = "library", softmax_scale: float = 0.0, token_stride: Optional[int] = None):
    from paper_2502_11101_b200.session import Session
    cfg = meta.cfg
    sess = Session(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.torch_dtype, cfg.pos_range, cfg.rope_theta,
                   cfg.q_len, meta.doc_len, meta.req_doc_begin, meta.doc_src_start, tail_reserve=cfg.q_len,
                   n_reuse=n_reuse, token_stride=token_stride, device=device)
    qg = q.to(device)
    if token_stride is None:
        kg, vg = k.to(device), v.to(device)
        k_final = kg.clone() if with_final else None
    else:
        kg, vg = padded_store(k, token_stride, device), padded_store(v, token_stride, device)
        k_final = padded_store(k, token_stride, device) if with_final else None
    n_layers = q.shape[0]
    out = torch.full_like(qg, float("nan"))
    lse = torch.full((n_layers, cfg.batch, cfg.n_q_heads, cfg.q_len), float("nan"), device=device)
    scores = torch.full((n_layers, meta.n_docs_total), float("nan"), device=device)
    sched = cfg.schedule if schedule is None else schedule
    sess.run_stack(qg, kg, vg, sched, strategy, out, lse, k_final, scores, batch_layers=batch_layers,
                   k_self=None if k_self is None else k_self.to(device),
                   v_self=None if v_self is None else v_self.to(device), driver=driver, softmax_scale=softmax_scale)
    torch.cuda.synchronize()
    status = sess.status()
    if token_stride is not None:                            # nothing may be written between the rows
        for t in (kg, vg) + ((k_final,) if with_final else ()):
            assert bool(torch.all(padding_of(t, token_stride) == PAD_SENTINEL)), "padding of the store was written"
    return {"out": out.float().cpu().numpy(), "lse": lse.cpu().numpy(), "scores": scores.cpu().numpy(),
            "accum": sess.score_accum.cpu().numpy(), "plan": sess.read_plan(), "status": status,
            "k_final": None if k_final is None else k_final.float().cpu().numpy(), "session": sess}


def compare(meta: W.WorkloadMeta, ref: List[Dict], got: Dict, k_store: torch.Tensor) -> Dict[str, float]:
    """Element-by-element comparison; raises AssertionError with the offending quantity."""
    cfg = meta.cfg
    n_layers = len(ref[0]["layers"])
    assert got["status"] == 0, f"device status {got['status']}"
    report = {"out_max_abs": 0.0, "score_max_rel": 0.0, "lse_max_abs": 0.0, "key_max_ulp": 0.0}
    for b in range(cfg.batch):
        lo, hi = int(meta.req_doc_begin[b]), int(meta.req_doc_begin[b + 1])
        r = ref[b]
        # integer results: bit-exact
        assert got["plan"]["order"][b] == r["order"], f"request {b}: kept set/order differs"
        assert np.array_equal(got["plan"]["dst_start"][lo:hi], r["dst_start"]), f"request {b}: dst_start differs"
        assert np.array_equal(got["plan"]["group"][lo:hi], r["group"]), f"request {b}: window index differs"
        assert int(got["plan"]["query_start"][b]) == r["query_start"]
        assert int(got["plan"]["n_reuse"][b]) == r["n_reuse"]
        for l in range(n_layers):
            rec = r["layers"][l]
            o_ref = rec["out"]
            o_got = got["out"][l, b]
            err = np.abs(o_got - o_ref)
            assert np.all(err <= OUT_ATOL + OUT_RTOL * np.abs(o_ref)), \
                f"request {b} layer {l + 1}: output error {err.max():.3e}"
            report["out_max_abs"] = max(report["out_max_abs"], float(err.max()))
            lse_err = np.abs(got["lse"][l, b] - rec["lse"])
            assert np.all(lse_err <= 1e-2), f"request {b} layer {l + 1}: lse error {lse_err.max():.3e}"
            report["lse_max_abs"] = max(report["lse_max_abs"], float(lse_err.max()))
            s_ref = rec["doc_scores"]
            s_got = got["scores"][l, lo:hi]
            n_kept = len(rec["order_in"])
            s_err = np.abs(s_got - s_ref)
            assert np.all(s_err <= 1e-2 / n_kept + SCORE_RTOL * np.abs(s_ref)), \
                f"request {b} layer {l + 1}: score error {s_err.max():.3e}"
            kept = np.array(rec["order_in"])
            report["score_max_rel"] = max(report["score_max_rel"], float((s_err[kept] / s_ref[kept]).max()))
            pruned = np.setdiff1d(np.arange(hi - lo), kept)
            assert np.all(s_got[pruned] == 0.0), "pruned documents must score exactly 0"
            assert abs(float(s_got.sum()) - 1.0) < 1e-3, "document scores of a request must sum to 1"
        acc_err = np.abs(got["accum"][lo:hi] - r["score_accum"])
        assert np.all(acc_err <= 1e-2 + SCORE_RTOL * np.abs(r["score_accum"]))
    if got["k_final"] is not None:
        k_in = k_store.float().cpu().numpy()
        half = cfg.head_dim // 2
        for b in range(cfg.batch):
            lo = int(meta.req_doc_begin[b])
            survivors = set(ref[b]["order"])
            for l in range(n_layers):
                kf_ref = ref[b]["k_final"][l]
                for i in range(int(meta.req_doc_begin[b + 1]) - lo):
                    a, c = int(meta.doc_offsets[lo + i]), int(meta.doc_offsets[lo + i + 1])
                    if i in survivors:
                        want = kf_ref[a:c]
                        # one rounding to the storage type at the result, plus fp32 arithmetic at the
                        # magnitude of the slice (a slice keeps its norm under rotation)
                        tol = rotated_key_tolerance(want, cfg.dtype)
                        err = np.abs(got["k_final"][l, a:c] - want) / tol
                        assert err.max() <= 1.0, f"rotated key off by {err.max():.3f} tol (layer {l + 1}, doc {i})"
                        report["key_max_ulp"] = max(report["key_max_ulp"], float(err.max()))
                    else:
                        assert np.array_equal(got["k_final"][l, a:c], k_in[l, a:c]), "pruned rows must stay untouched"
    return report


def run_and_compare(cfg: W.WorkloadConfig, seed: int, strategy: int, device="cuda:0", n_reuse: int = 0,
                    min_margin: float = 2e-3, doc_len_override=None, batch_layers: bool = False,
                    self_block: bool = False, driver: str = "library", softmax_scale: float = 0.0,
                    token_stride: Optional[int] = None, key_round=None) -> Dict[str, float]:
    meta = W.make_meta(cfg, seed, doc_len_override)
    q = W.make_q(meta)
    k, v = W.make_kv(meta)
    scale = softmax_scale if softmax_scale else None
    ref = oracle_stack(meta, q, k, v, strategy, n_reuse=n_reuse, scale=scale, key_round=key_round)
    margin = cut_margins(meta, ref, strategy)
    assert margin >= min_margin, f"workload rejected: decisive score gap {margin:.2e} below {min_margin:.0e}"
    k_self = v_self = None
    if self_block:
        k_self, v_self = W.make_kv_self(meta)
        add_self_block(meta, ref, q, k_self, v_self, scale)
    got = gpu_stack(meta, q, k, v, strategy, device=device, n_reuse=n_reuse, batch_layers=batch_layers,
                    k_self=k_self, v_self=v_self, driver=driver, softmax_scale=softmax_scale,
                    token_stride=token_stride)
    report = compare(meta, ref, got, k)
    report["margin"] = margin
    return report
