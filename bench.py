#!/usr/bin/env python
"""Benchmark of the CacheFocus query-time path on B200.

One "step" is one pass of the whole hot path for one batch of synthetic requests: positional
allocation, then per layer the fused re-position + query-prefill attention with document scores
and score accumulation, pruning + re-allocation at the scheduled layers, and the final
re-positioning of the surviving caches in every layer (Algorithm 2, Phases 1 and 2).

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--workload 3]

Prints one JSON line (rank 0).  `value` = cached KV tokens (one token position of one layer of a
kept document) processed per second with inputs resident in HBM; `e2e` = the same with the
query and the cache store starting in pinned host memory every step.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2502_11101_b200 import workloads as W  # noqa: E402

METRIC = "cached KV tokens/s through reposition+query-prefill attn"
# DRAM bytes (read + write) of one attention-kernel launch, averaged over the launches of a step, from the
# ncu capture summarised under profiles/; quoted only while the kernel's sources still hash to `kernel_sha`.
NCU_TRAFFIC = {("configs[2]", "layer-batched", "tcgen05"):
               {"bytes_per_launch": 25.65e6, "kernel_sha": "5e8cbfebacd3ff26", "summary": "profiles/attn_tc_kernel_workload3.md"}}
UNIT = "tokens/s"
STRATEGY_ALIGN = 1


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"hbm_gbs": float(p["hbm_gbs"]), "tflops": float(p["bf16_tflops"]),
                "tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "tflops": 1590.0, "tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.samples = []
        self.proc = None
        self.thread = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            parts = [s.strip() for s in line.split(",")]
            if len(parts) >= 7:
                try:
                    self.samples.append((time.time(), float(parts[0]), float(parts[1]), parts[3:7]))
                except ValueError:
                    pass

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        inside = [s for s in self.samples if t0 <= s[0] <= t1 + 0.15] or self.samples[-3:]
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for s in inside for i in range(4) if s[3][i].lower().startswith("active")})
        return {"sm_mhz": float(np.median([s[1] for s in inside])), "sm_max_mhz": inside[0][2],
                "reasons": reasons, "samples": len(inside)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def token_layers(cfg, meta, kept_lists):
    """Cached tokens visited per layer given the kept sets in force at each layer."""
    per_layer = []
    for layer in range(1, cfg.n_layers + 1):
        total = 0
        for b in range(cfg.batch):
            base = int(meta.req_doc_begin[b])
            total += int(sum(int(meta.doc_len[base + i]) for i in kept_lists[layer - 1][b]))
        per_layer.append(total)
    return per_layer


class GpuWorkload:
    """A ring of resident input sets (distinct seeds) so that consecutive steps never find their
    inputs in L2, plus the session and output buffers of the library."""

    def __init__(self, cfg, seed, device, ring, batch_layers=True, self_block=False, n_reuse=0, prefix=0):
        from paper_2502_11101_b200.session import Session
        self.cfg, self.device = cfg, device
        self.batch_layers = batch_layers
        self.self_kernel = False            # set by main(): the query-self block runs as a kernel of its own
        self.meta = W.make_meta(cfg, seed)
        m = self.meta
        self.sess = Session(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.torch_dtype, cfg.pos_range,
                            cfg.rope_theta, cfg.q_len, m.doc_len, m.req_doc_begin, m.doc_src_start,
                            tail_reserve=cfg.q_len, n_reuse=n_reuse, prefix_len=prefix, device=device)
        self.prefix_kv = None
        if prefix:                                   # a shared prefix cache attended by every layer (random contents)
            shape = (cfg.n_layers, prefix, cfg.n_kv_heads, cfg.head_dim)
            self.prefix_kv = (torch.empty(shape, dtype=cfg.torch_dtype, device=device).normal_(),
                              torch.empty(shape, dtype=cfg.torch_dtype, device=device).normal_())
        self.slots = []
        self.self_kv = []
        for r in range(ring):
            # same documents (lengths, relevance), fresh tensor contents per slot
            mr = W.make_meta(cfg, seed + 1000 * r, doc_len_override=m.doc_len) if r else m
            mr.key_scale[:] = m.key_scale
            q = W.make_q(mr, device)
            k, v = W.make_kv(mr, device)
            self.slots.append((q, k, v))
            self.self_kv.append(W.make_kv_self(mr, device) if self_block else (None, None))
        q0 = self.slots[0][0]
        self.out = torch.empty_like(q0)
        self.lse = torch.empty((cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.q_len), device=device)
        self.k_final = torch.empty_like(self.slots[0][1])

    def step(self, slot):
        q, k, v = self.slots[slot % len(self.slots)]
        k_self, v_self = self.self_kv[slot % len(self.slots)]
        self.sess.run_stack(q, k, v, self.cfg.schedule, STRATEGY_ALIGN, self.out, self.lse, self.k_final,
                            batch_layers=self.batch_layers, k_self=k_self, v_self=v_self,
                            k_prefix=None if self.prefix_kv is None else self.prefix_kv[0],
                            v_prefix=None if self.prefix_kv is None else self.prefix_kv[1])

    def calls(self):
        """(first, last) layer ranges of the attention calls of one step."""
        from paper_2502_11101_b200 import binding as B
        n = self.cfg.n_layers
        if not self.batch_layers:
            return [(i, i + 1) for i in range(n)]
        cuts = sorted(l for l, _ in self.cfg.schedule if l < n) + [n]
        out, first = [], 0
        for last in cuts:
            for lo in range(first, last, B.CF_MAX_LAYERS_PER_CALL):
                out.append((lo, min(last, lo + B.CF_MAX_LAYERS_PER_CALL)))
            first = last
        return out

    def kept_per_layer(self, slot=0):
        """One instrumented step: the kept sets seen by every layer."""
        q, k, v = self.slots[slot]
        cfg, sess = self.cfg, self.sess
        sched = dict(cfg.schedule)
        sess.set_live_docs(cfg.n_docs)
        sess.init()
        kept = []
        current = sess.read_plan()["order"]
        for layer in range(1, cfg.n_layers + 1):
            kept.append(current)
            sess.attend(q[layer - 1], k[layer - 1], v[layer - 1], self.out[layer - 1], self.lse[layer - 1])
            if layer in sched:
                sess.prune(sched[layer], STRATEGY_ALIGN)
                current = sess.read_plan()["order"]
        return kept, current

    def launches_per_step(self):
        cfg = self.cfg
        # clear status + plan init + per attention call (attention, merge, scores; the query-self block if asked
        # for) + prune/plan kernels + final re-positioning
        # (on the tensor-core path the block is a key tile of the attention kernel, not a launch)
        per_call = 4 if self.self_kernel else 3
        prunes = sum(1 for l, _ in cfg.schedule if l <= cfg.n_layers)
        if not self.batch_layers:
            # one call per layer: the stack driver leaves the layers' scores in up to eight workspace
            # slots and adds them to S with one launch before each pruning layer, when the slots are full and at the end
            cuts, slots, groups, filled = {l for l, _ in cfg.schedule}, min(8, cfg.n_layers), 0, 0
            for layer in range(1, cfg.n_layers + 1):
                filled += 1
                if layer in cuts or filled == slots or layer == cfg.n_layers:
                    groups, filled = groups + 1, 0
            return 2 + (per_call - 1) * cfg.n_layers + groups + prunes + 1
        return 2 + per_call * len(self.calls()) + prunes + 1


def time_steps(fn, steps, warmup, world):
    import torch.distributed as dist
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    start.record()
    for i in range(steps):
        fn(warmup + i)
    stop.record()
    torch.cuda.synchronize()
    t1 = time.time()
    if world > 1:
        dist.barrier()
    return start.elapsed_time(stop), t0, t1


def reposition_roofline(device, peaks, layers=8, iters=5):
    """Standalone cf_reposition_keys (Algorithm 2, Phase 2) over a store shaped like the largest
    configuration (32 kv heads, 8 requests x 120 documents of 160-200 tokens): every key row of
    `layers` layers is rotated in place.  Bytes = one read and one write of the key store."""
    from paper_2502_11101_b200.session import Session
    cfg = W.scaled_config(W.CONFIGS[5], n_layers=layers)
    meta = W.make_meta(cfg, 0)
    sess = Session(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.torch_dtype, cfg.pos_range, cfg.rope_theta,
                   cfg.q_len, meta.doc_len, meta.req_doc_begin, meta.doc_src_start, tail_reserve=cfg.q_len,
                   device=device)
    k = torch.empty((layers, meta.total_tokens, cfg.n_kv_heads, cfg.head_dim), dtype=torch.bfloat16, device=device)
    v_scratch = torch.empty_like(k[0])
    for layer in range(layers):
        W.fill_kv_layer(meta, layer, k[layer], v_scratch)
    del v_scratch
    sess.set_live_docs(cfg.n_docs)
    sess.init()
    for _ in range(3):
        sess.reposition(k, k, layers, k.stride(0))
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(iters):
        sess.reposition(k, k, layers, k.stride(0))
    stop.record()
    torch.cuda.synchronize()
    ms = start.elapsed_time(stop) / iters
    nbytes = 2 * k.numel() * k.element_size()
    gbs = nbytes / ms / 1e6
    assert sess.status() == 0
    return {"kernel": "cf_reposition_keys", "workload": f"configs[4]-shaped key store, {layers} of 32 layers, in place",
            "bound": "hbm", "bytes_per_launch": nbytes, "ms_per_launch": ms, "achieved": gbs, "peak": peaks["hbm_gbs"],
            "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "frac_of_8tbs_nominal": gbs / 8000.0,
            "peak_source": peaks["source"]}


def assemble_roofline(device, peaks, layers=2, iters=5):
    """cf_assemble_final_cache (Phase 2 with the final caches packed per request) over a store shaped
    like the largest configuration, every document kept: K and V are read once and written once."""
    from paper_2502_11101_b200.session import Session
    cfg = W.scaled_config(W.CONFIGS[5], n_layers=layers)
    meta = W.make_meta(cfg, 0)
    sess = Session(cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.torch_dtype, cfg.pos_range, cfg.rope_theta,
                   cfg.q_len, meta.doc_len, meta.req_doc_begin, meta.doc_src_start, tail_reserve=cfg.q_len,
                   device=device)
    k, v = W.make_kv(meta, device)
    k_self, v_self = W.make_kv_self(meta, device)
    out_rows = int(max(meta.doc_offsets[meta.req_doc_begin[b + 1]] - meta.doc_offsets[meta.req_doc_begin[b]]
                       for b in range(cfg.batch))) + cfg.q_len
    k_out = torch.empty((layers, cfg.batch, out_rows, cfg.n_kv_heads, cfg.head_dim), dtype=torch.bfloat16, device=device)
    v_out = torch.empty_like(k_out)
    final_rows = torch.zeros(cfg.batch, dtype=torch.int32, device=device)
    sess.set_live_docs(cfg.n_docs)
    sess.init()
    for _ in range(2):
        sess.assemble(k, v, k_self, v_self, k_out, v_out, final_rows)
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(iters):
        sess.assemble(k, v, k_self, v_self, k_out, v_out, final_rows)
    stop.record()
    torch.cuda.synchronize()
    ms = start.elapsed_time(stop) / iters
    assert sess.status() == 0
    moved = int(final_rows.sum().item()) * layers * cfg.n_kv_heads * cfg.head_dim * 2      # rows x row bytes
    nbytes = 4 * moved                                                                    # K and V, read and written
    gbs = nbytes / ms / 1e6
    return {"kernel": "cf_assemble_final_cache", "workload": f"configs[4]-shaped store, {layers} of 32 layers, every document kept",
            "bound": "hbm", "bytes_per_launch": nbytes, "ms_per_launch": ms, "achieved": gbs, "peak": peaks["hbm_gbs"],
            "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "peak_source": peaks["source"]}


def decode_roofline(cf, device, peaks, label, n_q_heads, n_kv_heads, requests, rows_used, layers, layers_per_call, iters=10):
    """One decoding step's attention over final caches of `rows_used` rows per request (cf_decode_attn; Algorithm 2,
    Phase 3): one query row per head streams the cache once.  Bytes = the keys and values attended."""
    geom = cf.make_geom(n_q_heads, n_kv_heads, 128, torch.bfloat16, 1 << 20, 1e4)
    cache_rows = rows_used + 64
    k_fin = torch.empty((layers, requests, cache_rows, n_kv_heads, 128), dtype=torch.bfloat16, device=device).normal_()
    v_fin = torch.empty_like(k_fin).normal_()
    q = torch.empty((layers, requests, n_q_heads, 128), dtype=torch.bfloat16, device=device).normal_()
    out = torch.empty_like(q)
    rows = torch.full((requests,), rows_used - 1, dtype=torch.int32, device=device)
    plan = torch.zeros(cf.cf_decode_plan_bytes(geom, requests, cache_rows), dtype=torch.uint8, device=device)
    work = torch.empty(cf.cf_decode_workspace_bytes(geom, requests, cache_rows, layers_per_call), dtype=torch.uint8, device=device)
    cf.cf_decode_plan(geom, requests, cache_rows, rows, 1, plan)

    def step():
        for l0 in range(0, layers, layers_per_call):
            l1 = l0 + layers_per_call
            cf.cf_decode_attn(geom, requests, cache_rows, plan, q[l0:l1], k_fin[l0:l1], v_fin[l0:l1], out[l0:l1], work)

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.graph(graph, stream=side):
        step()
    graph.replay()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(iters):
        graph.replay()
    stop.record()
    torch.cuda.synchronize()
    ms = start.elapsed_time(stop) / iters
    assert cf.cf_decode_status(geom, requests, cache_rows, plan) == 0
    nbytes = 2 * layers * requests * rows_used * n_kv_heads * 128 * 2
    gbs = nbytes / ms / 1e6
    return {"kernel": "cf_decode_attn", "workload": label, "q_heads": n_q_heads, "kv_heads": n_kv_heads,
            "requests": requests, "rows_per_request": rows_used, "layers_resident": layers,
            "layers_per_call": layers_per_call, "bound": "hbm", "bytes_per_step": nbytes, "ms_per_step": ms,
            "us_per_layer": 1e3 * ms / layers, "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": gbs / peaks["hbm_gbs"], "peak_source": peaks["source"]}


def docattn_roofline(cf, device, peaks, n_q_heads=12, n_kv_heads=2, n_docs=400, lo=128, hi=192, layers=4, prefix=64, iters=10):
    """cf_document_prefill_attn (offline cache construction, Sec. 2.2): documents shaped like the benchmark's attend a
    shared prefix and themselves under the causal mask.  Flops = 4 * head_dim * visible (row, key) pairs per query head
    (QK^T and PV, the masked half of the square not counted); bytes = every tensor once.  The roofline is the longer of
    the two times: with six query heads per kv head and 64 + ~80 visible keys per row the pass is bound by memory."""
    rng = np.random.default_rng(0)
    lens = rng.integers(lo, hi + 1, size=n_docs)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    total = int(off[-1])
    geom = cf.make_geom(n_q_heads, n_kv_heads, 128, torch.bfloat16, 32768, 1e6)
    q = torch.empty((layers, total, n_q_heads, 128), dtype=torch.bfloat16, device=device).normal_()
    k = torch.empty((layers, total, n_kv_heads, 128), dtype=torch.bfloat16, device=device).normal_()
    v = torch.empty_like(k).normal_()
    kp = torch.empty((layers, prefix, n_kv_heads, 128), dtype=torch.bfloat16, device=device).normal_()
    vp = torch.empty_like(kp).normal_()
    out = torch.empty_like(q)
    off_d = torch.from_numpy(off).to(device)
    status = torch.zeros(1, dtype=torch.int32, device=device)

    def step():
        cf.cf_document_prefill_attn(geom, off_d, int(lens.max()), q, k, v, out, kp, vp, None, status=status)

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(iters):
        step()
    stop.record()
    torch.cuda.synchronize()
    ms = start.elapsed_time(stop) / iters
    assert int(status.item()) == 0
    pairs = float(sum(int(n) * prefix + int(n) * (int(n) + 1) // 2 for n in lens))
    flops = 4.0 * 128 * pairs * n_q_heads * layers
    # algorithmic bytes: queries read and outputs written once, the documents' keys and values and the prefix cache read once
    nbytes = float(2 * q.numel() * 2 + (k.numel() + v.numel() + kp.numel() + vp.numel()) * 2)
    t_tensor, t_hbm = flops / (peaks["tflops"] * 1e12), nbytes / (peaks["hbm_gbs"] * 1e9)
    tfs, gbs = flops / ms / 1e9, nbytes / ms / 1e6
    hbm_bound = t_hbm >= t_tensor
    return {"kernel": "cf_document_prefill_attn", "workload": f"{n_docs} documents of {lo}-{hi} tokens behind a {prefix}-token "
            f"prefix, {n_q_heads}/{n_kv_heads} heads, {layers} layers per call", "bound": "hbm" if hbm_bound else "tensor",
            "flops_per_launch": flops, "bytes_per_launch": nbytes, "ms_per_launch": ms,
            "achieved": gbs if hbm_bound else tfs, "peak": peaks["hbm_gbs"] if hbm_bound else peaks["tflops"],
            "unit": "GB/s" if hbm_bound else "TFLOP/s", "frac": max(t_tensor, t_hbm) / (ms * 1e-3),
            "tflops": tfs, "tensor_frac": tfs / peaks["tflops"], "gbs": gbs, "hbm_frac": gbs / peaks["hbm_gbs"],
            "tokens_per_s": total * layers / (ms * 1e-3), "peak_source": peaks["source"]}


def whole_job(ms, tokens_per_step, steps, world, device):
    """Whole-job numbers of a replica run: every rank processed `tokens_per_step` tokens per step in `ms`
    milliseconds for `steps` steps; the job's time is the slowest rank's, its work the sum over ranks.
    Returns (ms_max, tokens_all_per_step, tokens_per_second)."""
    stats = torch.tensor([ms, float(tokens_per_step)], dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        mx, sm = stats.clone(), stats.clone()
        dist.all_reduce(mx, op=dist.ReduceOp.MAX)
        dist.all_reduce(sm, op=dist.ReduceOp.SUM)
        ms_max, tokens_all = float(mx[0]), float(sm[1])
    else:
        ms_max, tokens_all = float(ms), float(tokens_per_step)
    return ms_max, tokens_all, tokens_all * steps / (ms_max * 1e-3)


def oracle_sample(cfg, seed):
    """The oracle, as it stands, on one request of the workload (all layers, pruning schedule)."""
    import oracle
    one = W.scaled_config(cfg, batch=1)
    meta = W.make_meta(one, seed)
    q = W.make_q(meta).double().numpy()
    k, v = W.make_kv(meta)
    k, v = k.double().numpy(), v.double().numpy()
    t0 = time.perf_counter()
    res = oracle.run_stack(q[:, 0], k, v, meta.doc_len, meta.doc_offsets, meta.doc_src_start, one.rope_theta,
                           one.pos_range, one.schedule, STRATEGY_ALIGN, tail_reserve=one.q_len)
    dt = time.perf_counter() - t0
    tokens = sum(int(sum(int(meta.doc_len[i]) for i in rec["order_in"])) for rec in res["layers"])
    return dt, tokens


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, cfg, rank):
    if rank != 0:
        return
    times, tokens = [], []
    for i in range(args.warmup):
        oracle_sample(cfg, 100 + i)
    for i in range(args.steps):
        dt, tk = oracle_sample(cfg, i)
        times.append(dt)
        tokens.append(tk)
    value = sum(tokens) / sum(times)
    sample = f"one request of workload {args.workload} per step (all {cfg.n_layers} layers, pruning schedule), fp64"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"configs[{args.workload - 1}] {cfg.name}", "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def kernel_source_sha():
    """Digest of the attention kernel's sources: an ncu capture is only quoted for the kernel it was taken on."""
    import hashlib
    h = hashlib.sha256()
    for name in ("cf_attn_tc.cu", "cf_tc_util.cuh"):
        with open(os.path.join(ROOT, "paper_2502_11101_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def time_blocks(fn, steps, warmup, world, min_seconds=0.3, max_blocks=400):
    """W warm-up steps, then blocks of exactly `steps` steps, each bracketed by a barrier and a device
    synchronisation and timed with CUDA events, repeated until `min_seconds` have passed so that the clock
    sampler sees the timed work.  Returns (median block ms, wall start, wall end, blocks)."""
    import torch.distributed as dist
    for i in range(warmup):
        fn(i)
    times = []
    t0 = time.time()
    it = warmup
    while True:
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        for i in range(steps):
            fn(it + i)
        stop.record()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        it += steps
        times.append(start.elapsed_time(stop))
        enough = time.time() - t0 >= min_seconds or len(times) >= max_blocks
        if world > 1:                                        # every rank must leave the loop together
            flag = torch.tensor([1.0 if enough else 0.0], device="cuda")
            dist.all_reduce(flag, op=dist.ReduceOp.MIN)
            enough = bool(flag.item() > 0.5)
        if enough:
            break
    return float(np.median(times)), t0, time.time(), len(times)


def attention_roofline(cf, wl, cfg, per_layer_tokens, peaks, prof_steps):
    """Event pairs around every attention-kernel launch of a few eagerly issued steps.  A spin kernel
    queued first keeps the GPU busy until the host has enqueued the whole step, so the pairs time kernels
    running back to back and not the host's launch latency."""
    host_s = []
    for i in range(3):
        torch.cuda.synchronize()
        t_host = time.perf_counter()
        wl.step(i)
        host_s.append(time.perf_counter() - t_host)
    torch.cuda.synchronize()
    spin_cycles = int(max(host_s) * 1.5 * 2.0e9)
    calls = wl.calls()
    cf.cf_profile_begin(prof_steps * len(calls))
    for i in range(prof_steps):
        torch.cuda._sleep(spin_cycles)
        wl.step(3 + i)
        torch.cuda.synchronize()
    durations = cf.cf_profile_end(prof_steps * len(calls)).astype(np.float64)
    per_call_tokens = [sum(per_layer_tokens[lo:hi]) for lo, hi in calls]
    kv_bytes_per_token = 2 * cfg.head_dim * (2 if cfg.dtype == "bf16" else 4) * cfg.n_kv_heads
    flops_per_token = 4 * cfg.group_size * cfg.q_len * cfg.head_dim * cfg.n_kv_heads
    launch_bytes = np.tile(np.array(per_call_tokens, dtype=np.float64) * kv_bytes_per_token, prof_steps)
    launch_flops = np.tile(np.array(per_call_tokens, dtype=np.float64) * flops_per_token, prof_steps)
    n = min(len(durations), len(launch_bytes))
    per_call_us = None
    if n == prof_steps * len(calls):
        per_call_us = [float(x) for x in durations[:n].reshape(prof_steps, len(calls)).mean(axis=0) * 1e3]
    dur_s = durations[:n].sum() * 1e-3
    gbs = launch_bytes[:n].sum() / dur_s / 1e9
    tfs = launch_flops[:n].sum() / dur_s / 1e12
    t_hbm = launch_bytes[:n].sum() / (peaks["hbm_gbs"] * 1e9)
    t_tc = launch_flops[:n].sum() / (peaks["tflops"] * 1e12)
    if t_tc > t_hbm:
        roofline = {"bound": "tensor", "achieved": tfs, "peak": peaks["tflops"], "unit": "TFLOP/s",
                    "frac": tfs / peaks["tflops"]}
    else:
        roofline = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": gbs / peaks["hbm_gbs"]}
    roofline.update({"algorithmic_bytes_per_launch": float(launch_bytes[:n].mean()),
                     "kernel": "fused re-position + query-prefill attention", "peak_source": peaks["source"],
                     "avg_launch_us": 1e3 * durations[:n].mean(), "launches_timed": int(n),
                     "attention_us_per_step": 1e3 * durations[:n].sum() / prof_steps, "hbm_gbs": gbs, "tflops": tfs,
                     "frac_of_applicable_roofline": max(t_hbm, t_tc) / dur_s})
    if per_call_us is not None:
        roofline["launch_us_by_call"] = [{"layers": f"{lo + 1}-{hi}", "us": us} for (lo, hi), us in zip(calls, per_call_us)]
    return roofline


def capture_graphs(wl, ring, no_graph):
    """One CUDA graph of the whole step per ring slot (the pointers differ)."""
    if no_graph:
        return None
    try:
        wl.step(0)
        torch.cuda.synchronize()
        made = []
        side = torch.cuda.Stream()
        for r in range(ring):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                wl.step(r)
            made.append(g)
        return made
    except Exception as exc:  # capture not possible: time eager launches and say so
        sys.stderr.write(f"[bench] graph capture failed, timing eager launches: {exc}\n")
        torch.cuda.synchronize()
        return None


def other_workload(cf, number, cfg, device, peaks, local, note):
    """One more configuration in the same line: whole step as a CUDA graph, the attention kernel's
    roofline fraction, and the SM clock seen while it ran."""
    t_begin = time.time()
    wl = GpuWorkload(cfg, 0, device, ring=1, batch_layers=True)
    kept, _ = wl.kept_per_layer()
    per_layer_tokens = token_layers(cfg, wl.meta, kept)
    tokens = sum(per_layer_tokens)
    graphs = capture_graphs(wl, 1, False)

    def run(i):
        if graphs is not None:
            graphs[0].replay()
        else:
            wl.step(i)

    sampler = ClockSampler(local)
    steps = 5
    ms, t0, t1, blocks = time_blocks(run, steps, 3, 1, min_seconds=0.4, max_blocks=200)
    clocks = sampler.stop(t0, t1)
    assert wl.sess.status() == 0
    roof = attention_roofline(cf, wl, cfg, per_layer_tokens, peaks, prof_steps=3)
    assert wl.sess.status() == 0
    slot_mb = sum(t.numel() * t.element_size() for t in wl.slots[0]) / 1e6
    out = {"workload": f"configs[{number - 1}] {cfg.name}", "n_layers": cfg.n_layers, "requests": cfg.batch,
           "note": note, "ms_per_step": ms / steps, "value": tokens * steps / (ms * 1e-3), "unit": UNIT,
           "tokens_per_step": tokens, "resident_input_mb": slot_mb, "blocks_timed": blocks,
           "attention_calls_per_step": len(wl.calls()), "gpu_launches_per_step": wl.launches_per_step(),
           "roofline": {k: roof[k] for k in ("bound", "achieved", "peak", "unit", "frac", "avg_launch_us",
                                             "attention_us_per_step", "hbm_gbs", "tflops")},
           "sm_mhz": clocks["sm_mhz"], "clock_reasons": clocks["reasons"], "seconds": None}
    del wl, graphs
    torch.cuda.empty_cache()
    out["seconds"] = time.time() - t_begin
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=3, help="1-based index into the named configurations")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--ring", type=int, default=3, help="distinct resident input sets cycled between steps")
    ap.add_argument("--no-graph", action="store_true", help="launch every call eagerly instead of replaying CUDA graphs")
    ap.add_argument("--force-simt", action="store_true", help="use the CUDA-core attention kernel")
    ap.add_argument("--per-layer", action="store_true",
                    help="one attention call per layer instead of one per run of layers between two pruning layers")
    ap.add_argument("--skip-per-layer", action="store_true",
                    help="do not also time the step with one attention call per layer")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--skip-reposition", action="store_true", help="do not time the standalone re-positioning kernel")
    ap.add_argument("--skip-others", action="store_true", help="do not also measure the other configurations")
    ap.add_argument("--skip-e2e", action="store_true", help="do not time the step from pinned host memory")
    ap.add_argument("--layers", type=int, default=0, help="experiment only: truncate the stack to this many layers")
    ap.add_argument("--q-len", type=int, default=0, help="variant: query rows per request (1 = the shape of a decoding step)")
    ap.add_argument("--self-block", action="store_true",
                    help="variant: every layer also attends the query tokens themselves (cf_query_prefill_attn_full)")
    ap.add_argument("--only", default=None, choices=["reposition", "assemble", "decode", "document_prefill"],
                    help="run one of the side measurements alone and print its JSON (profiling aid)")
    ap.add_argument("--prefix", type=int, default=0,
                    help="variant: every layer also attends a shared prefix cache of this many tokens "
                         "(cf_query_prefill_attn_prefix)")
    ap.add_argument("--schedule", default="config", choices=["config", "linear"],
                    help="pruning schedule: the workload's own, or the paper's linear one (App. C: every 4 layers, "
                         "a constant number of documents, down to 5)")
    ap.add_argument("--n-reuse", default="eq6", choices=["eq6", "k", "1", "k/5", "5"],
                    help="number of parallel windows (Sec. 3.3): Eq. 6, one window per document, a single window, "
                         "a fifth of the documents, or five")
    args = ap.parse_args()
    cfg = W.CONFIGS[args.workload]
    if args.layers:
        cfg = W.scaled_config(cfg, n_layers=args.layers,
                              schedule=tuple(s for s in cfg.schedule if s[0] <= args.layers))
    if args.q_len:
        cfg = W.scaled_config(cfg, q_len=args.q_len)
    rank, world, local = dist_env()

    if args.impl == "reference":
        args.steps = 10 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        if args.schedule == "linear":
            import oracle
            cfg = W.scaled_config(cfg, schedule=tuple(oracle.prune_schedule_linear(cfg.n_layers, 4, cfg.n_docs, 5)))
        run_reference(args, cfg, rank)
        return

    args.steps = 200 if args.steps is None else args.steps
    args.warmup = 10 if args.warmup is None else max(3, args.warmup)
    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(device))
    import paper_2502_11101_b200 as cf
    from paper_2502_11101_b200 import build as cf_build
    if rank == 0:
        cf_build.build()
    if world > 1:
        dist.barrier()
    cf.load_library()
    if args.schedule == "linear":                             # App. C, from the library
        cfg = W.scaled_config(cfg, schedule=tuple(cf.cf_schedule_linear(cfg.n_layers, 4, cfg.n_docs, 5)))
    if args.force_simt:
        cf.cf_set_attn_path(1)
    peaks = load_peaks()
    if args.only:
        one = {"reposition": lambda: reposition_roofline(device, peaks),
               "assemble": lambda: assemble_roofline(device, peaks),
               "decode": lambda: decode_roofline(cf, device, peaks, "configs[3]-shaped final caches, one call per layer",
                                                 28, 4, 4, 16000, 8, 1),
               "document_prefill": lambda: docattn_roofline(cf, device, peaks)}[args.only]()
        if rank == 0:
            print(json.dumps(one), flush=True)
        return
    n_reuse = {"eq6": 0, "k": cfg.n_docs, "1": 1, "k/5": max(1, cfg.n_docs // 5), "5": 5}[args.n_reuse]

    wl = GpuWorkload(cfg, args.seed + 7919 * rank, device, args.ring, batch_layers=not args.per_layer,
                     self_block=args.self_block, n_reuse=n_reuse, prefix=args.prefix)
    wl.self_kernel = args.self_block and (args.force_simt or not _tc_used(cf, wl))
    kept, survivors = wl.kept_per_layer()
    per_layer_tokens = token_layers(cfg, wl.meta, kept)
    tokens_per_step = sum(per_layer_tokens)
    final_tokens = sum(int(wl.meta.doc_len[int(wl.meta.req_doc_begin[b]) + i]) for b in range(cfg.batch)
                       for i in survivors[b]) * cfg.n_layers
    assert wl.sess.status() == 0, f"device status {wl.sess.status()}"
    windows = [int(x) for x in wl.sess.read_plan()["n_reuse"]]

    graphs = capture_graphs(wl, args.ring, args.no_graph)

    def run(i):
        if graphs is not None:
            graphs[i % args.ring].replay()
        else:
            wl.step(i)

    sampler = ClockSampler(local) if rank == 0 else None
    ms, t0, t1, blocks = time_blocks(run, args.steps, args.warmup, world)
    clocks = sampler.stop(t0, t1) if sampler else None
    assert wl.sess.status() == 0

    ms_max, tokens_all, value = whole_job(ms, tokens_per_step, args.steps, world, device)

    # ---- the same step with one attention call per layer (what a running model can issue) ------
    per_layer = None
    if wl.batch_layers and world == 1 and not args.skip_per_layer:
        main_graphs = graphs
        wl.batch_layers = False
        graphs = capture_graphs(wl, args.ring, args.no_graph)
        pl_steps = max(1, min(args.steps, 50))
        pl_ms, _, _, _ = time_blocks(run, pl_steps, 3, world, min_seconds=0.1)
        assert wl.sess.status() == 0
        per_layer = {"value": tokens_per_step * pl_steps / (pl_ms * 1e-3), "unit": UNIT, "ms_per_step": pl_ms / pl_steps,
                     "steps": pl_steps, "gpu_launches_per_step": wl.launches_per_step(),
                     "note": "one attention call per layer (cf_query_prefill_attn_slot); document scores added to S before each pruning layer (cf_accumulate_scores)"}
        wl.batch_layers = True
        graphs, main_graphs = main_graphs, None

    # ---- the dominant kernel alone --------------------------------------------------------------
    roofline = attention_roofline(cf, wl, cfg, per_layer_tokens, peaks, max(1, min(args.steps, 20)))
    if "launch_us_by_call" in roofline:
        sys.stderr.write("[bench] attention launches of a step, mean us (layers first-last): " +
                         " ".join(f"{c['layers']}:{c['us']:.1f}" for c in roofline["launch_us_by_call"]) + "\n")
    attn_kernel = "cuda-core" if args.force_simt or not _tc_used(cf, wl) else "tcgen05"
    traffic_key = (f"configs[{args.workload - 1}]", "layer-batched" if wl.batch_layers else "per-layer", attn_kernel)
    default_variant = not (args.layers or args.q_len or args.self_block or args.prefix or args.schedule != "config" or args.n_reuse != "eq6")
    capture = NCU_TRAFFIC.get(traffic_key) if default_variant else None
    sha = kernel_source_sha()
    roofline.update({"traffic": capture["bytes_per_launch"] if capture and capture["kernel_sha"] == sha else None,
                     "traffic_unit": "bytes per launch (ncu dram read + write)", "kernel_sha": sha,
                     "traffic_note": None if capture and capture["kernel_sha"] == sha else
                     "no ncu capture of this kernel state is on record (profiles/ holds the last one)"})

    # ---- end to end: query and cache store start in pinned host memory every step --------------
    e2e = None
    if not args.skip_e2e:
        q0, k0, v0 = wl.slots[0]
        resident = [q0, k0, v0] + [t for t in wl.self_kv[0] if t is not None]
        host = [t.cpu().pin_memory() for t in resident]
        out_h = torch.empty(wl.out.shape, dtype=wl.out.dtype).pin_memory()
        acc_h = torch.empty(wl.sess.score_accum.shape, dtype=torch.float32).pin_memory()
        kept_h = torch.empty(wl.sess.n_docs_total, dtype=torch.int32).pin_memory()

        def e2e_step(_):
            for src, dst in zip(host, resident):
                dst.copy_(src, non_blocking=True)
            wl.step(0)
            out_h.copy_(wl.out, non_blocking=True)
            acc_h.copy_(wl.sess.score_accum, non_blocking=True)
            kept_h.copy_(wl.sess.field("kept", wl.sess.n_docs_total), non_blocking=True)

        e2e_steps = max(1, min(args.steps, 20))
        e2e_ms, _, _ = time_steps(e2e_step, e2e_steps, 3, world)
        e2e_ms_max, _, e2e_value = whole_job(e2e_ms, tokens_per_step, e2e_steps, world, device)
        h2d = sum(t.numel() * t.element_size() for t in host)
        d2h = sum(t.numel() * t.element_size() for t in (out_h, acc_h, kept_h))
        e2e = {"value": e2e_value, "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps}
        del host, q0, k0, v0, resident

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    launches = wl.launches_per_step() * args.steps * blocks
    n_calls = len(wl.calls())
    slot_mb = sum(t.numel() * t.element_size() for t in wl.slots[0]) / 1e6
    launch_mode = "cuda graph per ring slot" if graphs is not None else "eager"
    call_mode = ("one attention call per run of layers between two pruning layers (every layer's query states "
                 "are inputs of the step)") if wl.batch_layers else "one attention call per layer"
    launches_per_step = wl.launches_per_step()
    del wl, graphs
    torch.cuda.empty_cache()
    repo = assemble = None
    if world == 1 and not args.skip_reposition:
        repo = reposition_roofline(device, peaks)
        torch.cuda.empty_cache()
        assemble = assemble_roofline(device, peaks)
        torch.cuda.empty_cache()

    decode = None
    if world == 1 and not args.skip_reposition:
        # the decoding step (one query row per head) over final caches with every document of the configuration kept
        decode = [decode_roofline(cf, device, peaks, "configs[4]-shaped final caches, one call per layer", 32, 32, 8, 21600, 4, 1),
                  decode_roofline(cf, device, peaks, "configs[3]-shaped final caches, one call per layer", 28, 4, 4, 16000, 8, 1),
                  decode_roofline(cf, device, peaks, "configs[3]-shaped final caches, eight layers per call", 28, 4, 4, 16000, 8, 8)]
        torch.cuda.empty_cache()
    docattn = docattn_roofline(cf, device, peaks) if world == 1 and not args.skip_reposition else None

    others = None
    if world == 1 and not args.skip_others and default_variant and args.workload == 3 and not args.force_simt:
        others = [other_workload(cf, 2, W.CONFIGS[2], device, peaks, local, "single layer; the whole configuration"),
                  other_workload(cf, 4, W.CONFIGS[4], device, peaks, local, "the whole configuration"),
                  other_workload(cf, 5, W.CONFIGS[5], device, peaks, local,
                                 "the whole configuration: 32 layers, 90.6 GB of keys and values plus 45.3 GB of final "
                                 "keys resident")]

    cpu = None
    if world == 1 and not args.skip_cpu_baseline:
        t_total, tok_total, reps = 0.0, 0, 0
        while t_total < 10.0 and reps < 24:
            dt, tk = oracle_sample(cfg, 50 + reps)
            t_total += dt
            tok_total += tk
            reps += 1
        cpu = {"value": tok_total / t_total, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
               "sample": f"{reps} x one request of workload {args.workload} (all {cfg.n_layers} layers, "
                         f"pruning schedule), {t_total:.1f} s of fp64 numpy"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_max / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": f"configs[{args.workload - 1}] {cfg.name}", "n_layers": cfg.n_layers,
                       "q_heads": cfg.n_q_heads, "kv_heads": cfg.n_kv_heads, "head_dim": cfg.head_dim,
                       "docs_per_request": cfg.n_docs, "requests": cfg.batch, "q_len": cfg.q_len,
                       "schedule": [list(s) for s in cfg.schedule], "schedule_kind": args.schedule, "strategy": "align",
                       "n_reuse_policy": args.n_reuse, "windows_at_init": windows,
                       "query_self_block": bool(args.self_block), "prefix_len": args.prefix,
                       "tokens_per_step": tokens_per_step, "final_reposition_tokens": final_tokens,
                       "l2": f"ring of {args.ring} resident input sets ({args.ring} x "
                             f"{slot_mb:.0f} MB) cycled between steps",
                       "timing": f"median of {blocks} blocks of {args.steps} steps, each block between device "
                                 "synchronisations, CUDA events",
                       "launch": launch_mode, "stack_driver": "cf_run_stack (C ABI)", "attention_calls": call_mode,
                       "attention_calls_per_step": n_calls, "gpu_launches_per_step": launches_per_step,
                       "attention_kernel": attn_kernel,
                       "parallelism": f"replicas x{world}"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
            "roofline": roofline, "per_layer_launch": per_layer, "reposition": repo, "assemble": assemble, "decode": decode, "document_prefill": docattn,
            "other_workloads": others, "cpu_baseline": cpu}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def _tc_used(cf, wl):
    return wl.cfg.dtype == "bf16" and wl.cfg.head_dim == 128 and getattr(cf, "TC_KERNEL_BUILT", False)


if __name__ == "__main__":
    main()
