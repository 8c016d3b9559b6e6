"""Buffer ownership and call sequencing around the C ABI (no arithmetic happens here).

A `Session` owns the device copies of a batch's integer description, the plan buffer, the
attention workspace and the score vectors, and issues the library calls of Algorithm 2 in
order on the current CUDA stream."""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

from . import binding as B


class Session:
    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, dtype: torch.dtype, pos_range: int,
                 rope_theta: float, q_len: int, doc_len: np.ndarray, req_doc_begin: np.ndarray,
                 doc_src_start: np.ndarray, tail_reserve: int, prefix_len: int = 0, n_reuse: int = 0,
                 rope_layout: int = B.CF_ROPE_HALF, token_stride: Optional[int] = None,
                 device: str = "cuda:0"):
        self.device = torch.device(device)
        self.doc_len = np.asarray(doc_len, dtype=np.int32)
        self.req_doc_begin_h = np.asarray(req_doc_begin, dtype=np.int32)
        doc_offsets = np.zeros(len(self.doc_len) + 1, dtype=np.int32)
        doc_offsets[1:] = np.cumsum(self.doc_len)
        self.doc_offsets_h = doc_offsets
        self.n_requests = len(self.req_doc_begin_h) - 1
        self.n_docs_total = len(self.doc_len)
        self.total_tokens = int(doc_offsets[-1])
        self.q_len = q_len
        self.geom = B.make_geom(n_q_heads, n_kv_heads, head_dim, dtype, pos_range, rope_theta, rope_layout)
        self._req_doc_begin = torch.from_numpy(self.req_doc_begin_h).to(self.device)
        self._doc_offsets = torch.from_numpy(doc_offsets).to(self.device)
        self._doc_src_start = torch.from_numpy(np.asarray(doc_src_start, dtype=np.int32)).to(self.device)
        stride = n_kv_heads * head_dim if token_stride is None else token_stride
        self.batch = B.make_batch(self.n_requests, q_len, self.total_tokens, stride, self._req_doc_begin,
                                  self._doc_offsets, self._doc_src_start, prefix_len, tail_reserve, n_reuse, 0)
        self.layout = B.cf_plan_layout_of(self.geom, self.batch)
        self.plan = torch.zeros(self.layout.total_bytes, dtype=torch.uint8, device=self.device)
        self.set_live_docs(int(np.diff(self.req_doc_begin_h).max()) if self.n_requests else 0)
        self.workspace = torch.empty(256, dtype=torch.uint8, device=self.device)
        self.reserve_workspace(1)
        self.doc_scores = torch.zeros(self.n_docs_total, dtype=torch.float32, device=self.device)
        self.score_accum = torch.zeros(self.n_docs_total, dtype=torch.float32, device=self.device)

    def set_live_docs(self, kept_per_request: int) -> None:
        """Tell the library how many documents a request can still hold (sizes kernel grids only):
        the hint is the tile count of the `kept_per_request` longest documents of any request."""
        worst = 1
        for b in range(self.n_requests):
            lens = self.doc_len[self.req_doc_begin_h[b]:self.req_doc_begin_h[b + 1]]
            tiles = np.sort((lens + B.CF_TILE_TOKENS - 1) // B.CF_TILE_TOKENS)[::-1]
            worst = max(worst, int(tiles[:kept_per_request].sum()))
        self.batch.tiles_hint = worst

    def reserve_workspace(self, n_layers: int, with_self: bool = False) -> None:
        """Grow the attention workspace to what a call over `n_layers` layers needs with the current
        live-document hint (allocation happens here, never inside a library call)."""
        need = (B.cf_attn_workspace_bytes_full if with_self else B.cf_attn_workspace_bytes_layers)(
            self.geom, self.batch, n_layers)
        if need > self.workspace.numel():
            self.workspace = torch.empty(need, dtype=torch.uint8, device=self.device)

    def init(self, order: Optional[torch.Tensor] = None, kept_count: Optional[torch.Tensor] = None,
             query_start: int = -1) -> None:
        self.score_accum.zero_()
        B.cf_plan_init(self.geom, self.batch, self.plan, order, kept_count, query_start)

    def attend(self, q: torch.Tensor, k_layer: torch.Tensor, v_layer: torch.Tensor, out: torch.Tensor,
               lse: Optional[torch.Tensor] = None, softmax_scale: float = 0.0) -> None:
        B.cf_query_prefill_attn(self.geom, self.batch, self.plan, q, k_layer, v_layer, out, self.workspace, lse,
                                self.doc_scores, self.score_accum, softmax_scale)

    def attend_layers(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor,
                      lse: Optional[torch.Tensor] = None, layer_scores: Optional[torch.Tensor] = None,
                      softmax_scale: float = 0.0, k_self: Optional[torch.Tensor] = None,
                      v_self: Optional[torch.Tensor] = None) -> None:
        """Consecutive layers that attend the same kept documents, in one library call: q, out
        [m, B, Lq, Hq, D]; k, v [m, T, Hkv, D]; lse [m, B, Hq, Lq]; layer_scores [m, n_docs_total].
        With `k_self`, `v_self` [m, B, Lq, Hkv, D] the causal query-self block is merged in."""
        self.reserve_workspace(q.shape[0], k_self is not None)
        if k_self is not None:
            B.cf_query_prefill_attn_full(self.geom, self.batch, self.plan, q, k, v, k_self, v_self, out, self.workspace,
                                         lse, layer_scores, self.score_accum, softmax_scale)
            return
        B.cf_query_prefill_attn_layers(self.geom, self.batch, self.plan, q, k, v, out, self.workspace, lse,
                                       layer_scores, self.score_accum, softmax_scale)

    def prune(self, keep: int, strategy: int) -> None:
        B.cf_prune_topk(self.geom, self.batch, self.plan, self.score_accum, keep, strategy)
        self.set_live_docs(keep)

    def reposition(self, k_in: torch.Tensor, k_out: torch.Tensor, n_layers: int = 1, layer_stride: int = 0) -> None:
        B.cf_reposition_keys(self.geom, self.batch, self.plan, k_in, k_out, n_layers, layer_stride)

    def assemble(self, k: torch.Tensor, v: torch.Tensor, k_self: torch.Tensor, v_self: torch.Tensor,
                 k_out: torch.Tensor, v_out: torch.Tensor, final_rows: torch.Tensor) -> None:
        """Phase 2 with the final caches packed per request: survivors in rank order, then the query rows."""
        B.cf_assemble_final_cache(self.geom, self.batch, self.plan, k, v, k_self, v_self, k_out, v_out, final_rows)

    def status(self) -> int:
        return B.cf_plan_status(self.geom, self.batch, self.plan)

    def field(self, name: str, count: int, dtype=torch.int32) -> torch.Tensor:
        return B.plan_field(self.plan, self.layout, name, count, dtype)

    def read_plan(self) -> Dict[str, object]:
        """Copy the integer state of the plan back to the host."""
        nd, nb = self.n_docs_total, self.n_requests
        kept = self.field("kept", nd).cpu().numpy()
        count = self.field("kept_count", nb).cpu().numpy()
        order = [list(map(int, kept[self.req_doc_begin_h[b]:self.req_doc_begin_h[b] + count[b]])) for b in range(nb)]
        return {"order": order, "dst_start": self.field("dst_start", nd).cpu().numpy(),
                "group": self.field("group", nd).cpu().numpy(), "n_reuse": self.field("n_reuse", nb).cpu().numpy(),
                "query_start": self.field("query_start", nb).cpu().numpy(),
                "n_tiles": self.field("n_tiles", nb).cpu().numpy()}

    def run_stack(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, schedule: Sequence[Tuple[int, int]],
                  strategy: int, out: torch.Tensor, lse: Optional[torch.Tensor] = None,
                  k_final: Optional[torch.Tensor] = None, layer_scores: Optional[torch.Tensor] = None,
                  batch_layers: bool = False, k_self: Optional[torch.Tensor] = None,
                  v_self: Optional[torch.Tensor] = None, driver: str = "library",
                  softmax_scale: float = 0.0, k_prefix: Optional[torch.Tensor] = None,
                  v_prefix: Optional[torch.Tensor] = None) -> None:
        """Algorithm 2, Phases 1 and 2: q, out [L, B, Lq, Hq, D]; k, v [L, T, Hkv, D];
        lse [L, B, Hq, Lq]; `layer_scores` [L, n_docs_total] receives each layer's document scores.

        With `batch_layers` the layers between two pruning layers go to the attention kernels in one
        launch (possible here because every layer's query states are given up front).  With `k_self`,
        `v_self` [L, B, Lq, Hkv, D] every layer also attends the query tokens themselves (causal).
        With `k_prefix`, `v_prefix` [L, P, Hkv, D] every layer also attends that shared prefix cache.
        `driver="library"`: one cf_run_stack call sequences the stack inside the library;
        `driver="calls"`: the same sequence issued from here, one library call per step."""
        if driver == "library":
            st, keepalive = B.make_stack(q, k, v, out, self.score_accum, schedule, strategy, batch_layers, lse,
                                         layer_scores, k_final, k_self, v_self, softmax_scale, self.doc_len,
                                         self.req_doc_begin_h, k_prefix, v_prefix)
            self.batch.tiles_hint = 0
            need = B.cf_run_stack_workspace_bytes(self.geom, self.batch, st)
            if need > self.workspace.numel():
                self.workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
            B.cf_run_stack(self.geom, self.batch, st, self.plan, self.workspace)
            del keepalive
            return
        assert driver == "calls" and k_prefix is None, "a prefix cache goes through the library's stack driver"
        sched = dict(schedule)
        n_layers = q.shape[0]
        self.set_live_docs(int(np.diff(self.req_doc_begin_h).max()))
        self.init()
        if batch_layers:
            cuts = sorted(l for l in sched if l < n_layers) + [n_layers]
            first = 0
            for last in cuts:                               # layers first+1 .. last (1-based) share one plan
                for lo in range(first, last, B.CF_MAX_LAYERS_PER_CALL):
                    hi = min(last, lo + B.CF_MAX_LAYERS_PER_CALL)
                    self.attend_layers(q[lo:hi], k[lo:hi], v[lo:hi], out[lo:hi], None if lse is None else lse[lo:hi],
                                       None if layer_scores is None else layer_scores[lo:hi], softmax_scale,
                                       k_self=None if k_self is None else k_self[lo:hi],
                                       v_self=None if v_self is None else v_self[lo:hi])
                if last in sched:
                    self.prune(sched[last], strategy)
                first = last
        else:
            n_slots, filled = min(8, n_layers), 0            # as cf_run_stack: the layers' scores wait in workspace slots
            if k_self is None:
                need = B.cf_attn_workspace_bytes_slots(self.geom, self.batch, n_slots)
                if need > self.workspace.numel():
                    self.workspace = torch.empty(need, dtype=torch.uint8, device=self.device)
            for layer in range(1, n_layers + 1):
                i = layer - 1
                if k_self is None:
                    B.cf_query_prefill_attn_slot(self.geom, self.batch, self.plan, filled, n_slots, q[i], k[i], v[i], out[i],
                                                 self.workspace, None if lse is None else lse[i], softmax_scale)
                    filled += 1
                    if layer in sched or filled == n_slots or layer == n_layers:
                        B.cf_accumulate_scores(self.geom, self.batch, self.plan, filled, n_slots, self.workspace,
                                               None if layer_scores is None else layer_scores[layer - filled:layer],
                                               self.score_accum)
                        filled = 0
                else:
                    self.attend_layers(q[i:i + 1], k[i:i + 1], v[i:i + 1], out[i:i + 1],
                                       None if lse is None else lse[i:i + 1],
                                       None if layer_scores is None else layer_scores[i:i + 1], softmax_scale,
                                       k_self=k_self[i:i + 1], v_self=v_self[i:i + 1])
                if layer in sched:
                    self.prune(sched[layer], strategy)
        if k_final is not None:
            self.reposition(k, k_final, n_layers, k.stride(0))
