"""Thin ctypes binding of libcachefocus.so: same names as the C ABI, argument marshalling only.

Tensors are torch tensors used purely as device (or host) buffers; every step of the path runs
in the library's kernels."""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

CF_OK, CF_ERR_INVALID_ARG, CF_ERR_RANGE, CF_ERR_UNSUPPORTED, CF_ERR_WORKSPACE, CF_ERR_CUDA, CF_ERR_TIMEOUT = range(7)
CF_BF16, CF_F32 = 0, 1
CF_ROPE_HALF, CF_ROPE_INTERLEAVED = 0, 1
CF_ALLOC_NONE, CF_ALLOC_ALIGN, CF_ALLOC_SORT = 0, 1, 2
CF_TILE_TOKENS = 128
CF_MAX_LAYERS_PER_CALL = 64
CF_MAX_SPLITS = 64
TC_KERNEL_BUILT = True      # bf16 / head_dim 128 batches take the tcgen05 attention kernel

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libcachefocus.so")

EXPORTS = ["cf_error_string", "cf_allocate_positions", "cf_schedule_linear", "cf_plan_layout_of",
           "cf_plan_init", "cf_plan_status", "cf_reposition_keys", "cf_attn_workspace_bytes",
           "cf_attn_workspace_bytes_layers", "cf_query_prefill_attn", "cf_query_prefill_attn_layers",
           "cf_attn_workspace_bytes_slots", "cf_query_prefill_attn_slot", "cf_accumulate_scores",
           "cf_attn_workspace_bytes_slots_full", "cf_query_prefill_attn_slot_full",
           "cf_attn_workspace_bytes_full", "cf_query_prefill_attn_full", "cf_query_prefill_attn_prefix", "cf_assemble_final_cache", "cf_merge_attn",
           "cf_query_prefill_attn_static", "cf_prune_topk", "cf_prune_topk_host", "cf_run_stack_workspace_bytes",
           "cf_run_stack", "cf_document_prefill_attn", "cf_decode_plan_bytes", "cf_decode_plan", "cf_decode_status",
           "cf_decode_workspace_bytes", "cf_decode_attn", "cf_decode_append", "cf_set_attn_path", "cf_profile_begin", "cf_profile_end", "cf_debug_wait_timeout"]
_SIZE_T_EXPORTS = ("cf_attn_workspace_bytes", "cf_attn_workspace_bytes_layers", "cf_attn_workspace_bytes_full",
                   "cf_attn_workspace_bytes_slots", "cf_attn_workspace_bytes_slots_full",
                   "cf_run_stack_workspace_bytes", "cf_decode_plan_bytes", "cf_decode_workspace_bytes")


class cf_geom(ctypes.Structure):
    _fields_ = [("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("rope_layout", ctypes.c_int32), ("pos_range", ctypes.c_int32),
                ("rope_theta", ctypes.c_double)]


class cf_batch(ctypes.Structure):
    _fields_ = [("n_requests", ctypes.c_int32), ("n_docs_total", ctypes.c_int32), ("q_len", ctypes.c_int32),
                ("prefix_len", ctypes.c_int32), ("tail_reserve", ctypes.c_int32), ("n_reuse", ctypes.c_int32),
                ("tiles_hint", ctypes.c_int32), ("reserved", ctypes.c_int32),
                ("total_tokens", ctypes.c_int64), ("token_stride", ctypes.c_int64),
                ("req_doc_begin", ctypes.c_void_p), ("doc_offsets", ctypes.c_void_p),
                ("doc_src_start", ctypes.c_void_p)]


class cf_plan_layout(ctypes.Structure):
    _fields_ = [(n, ctypes.c_size_t) for n in
                ("total_bytes", "status", "kept", "kept_count", "dst_start", "group", "n_reuse", "query_start",
                 "n_tiles", "tile_begin", "doc_tile_begin", "doc_tile_count", "tile_doc", "tile_row0", "tile_len", "trig")] + \
               [("max_tiles", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class cf_doc_batch(ctypes.Structure):
    _fields_ = [("n_docs", ctypes.c_int32), ("max_doc_len", ctypes.c_int32), ("prefix_len", ctypes.c_int32),
                ("reserved", ctypes.c_int32), ("total_tokens", ctypes.c_int64), ("token_stride", ctypes.c_int64),
                ("doc_offsets", ctypes.c_void_p)]


class cf_stack(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("n_prune", ctypes.c_int32),
                ("prune_layer", ctypes.c_void_p), ("prune_keep", ctypes.c_void_p),
                ("strategy", ctypes.c_int32), ("batch_layers", ctypes.c_int32),
                ("softmax_scale", ctypes.c_float), ("reserved", ctypes.c_int32),
                ("q", ctypes.c_void_p), ("q_layer_stride", ctypes.c_int64),
                ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p), ("kv_layer_stride", ctypes.c_int64),
                ("k_self", ctypes.c_void_p), ("v_self", ctypes.c_void_p), ("self_layer_stride", ctypes.c_int64),
                ("out", ctypes.c_void_p), ("out_layer_stride", ctypes.c_int64),
                ("lse", ctypes.c_void_p), ("layer_scores", ctypes.c_void_p), ("score_accum", ctypes.c_void_p),
                ("k_final", ctypes.c_void_p),
                ("doc_len_host", ctypes.c_void_p), ("req_doc_begin_host", ctypes.c_void_p),
                ("k_prefix", ctypes.c_void_p), ("v_prefix", ctypes.c_void_p), ("prefix_layer_stride", ctypes.c_int64),
                ("prefix_len", ctypes.c_int32), ("reserved2", ctypes.c_int32)]


class CacheFocusError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {cf_error_string(code)} (code {code})")


_LIB = None


def load_library() -> ctypes.CDLL:
    """Load libcachefocus.so (built by paper_2502_11101_b200.build); no fallback exists."""
    global _LIB
    if _LIB is not None:
        return _LIB
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2502_11101_b200.build` "
                           "(the CUDA library is the only implementation, there is no CPU path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    gp, bp = ctypes.POINTER(cf_geom), ctypes.POINTER(cf_batch)
    lib.cf_error_string.restype = ctypes.c_char_p
    lib.cf_error_string.argtypes = [ctypes.c_int]
    lib.cf_allocate_positions.argtypes = [gp, i32, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp]
    lib.cf_schedule_linear.argtypes = [i32, i32, i32, i32, i32, vp, vp, vp]
    lib.cf_plan_layout_of.argtypes = [gp, bp, ctypes.POINTER(cf_plan_layout)]
    lib.cf_plan_init.argtypes = [gp, bp, vp, vp, i32, vp, ctypes.c_size_t, vp]
    lib.cf_plan_status.argtypes = [gp, bp, vp, vp]
    lib.cf_reposition_keys.argtypes = [gp, bp, vp, i32, i64, vp, vp, vp]
    lib.cf_attn_workspace_bytes.restype = ctypes.c_size_t
    lib.cf_attn_workspace_bytes.argtypes = [gp, bp]
    lib.cf_query_prefill_attn.argtypes = [gp, bp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp, vp,
                                          ctypes.c_size_t, vp]
    lib.cf_attn_workspace_bytes_layers.restype = ctypes.c_size_t
    lib.cf_attn_workspace_bytes_layers.argtypes = [gp, bp, i32]
    lib.cf_query_prefill_attn_layers.argtypes = [gp, bp, vp, i32, vp, i64, vp, vp, i64, ctypes.c_float, vp, i64,
                                                 vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.cf_attn_workspace_bytes_slots.restype = ctypes.c_size_t
    lib.cf_attn_workspace_bytes_slots.argtypes = [gp, bp, i32]
    lib.cf_query_prefill_attn_slot.argtypes = [gp, bp, vp, i32, i32, vp, vp, vp, ctypes.c_float, vp, vp, vp,
                                               ctypes.c_size_t, vp]
    lib.cf_accumulate_scores.argtypes = [gp, bp, vp, i32, i32, vp, vp, vp, ctypes.c_size_t, vp]
    lib.cf_attn_workspace_bytes_slots_full.restype = ctypes.c_size_t
    lib.cf_attn_workspace_bytes_slots_full.argtypes = [gp, bp, i32]
    lib.cf_query_prefill_attn_slot_full.argtypes = [gp, bp, vp, i32, i32, vp, vp, vp, vp, vp, i32, vp, vp, ctypes.c_float,
                                                    vp, vp, vp, ctypes.c_size_t, vp]
    lib.cf_assemble_final_cache.argtypes = [gp, bp, vp, i32, i64, vp, vp, i64, vp, vp, i32, vp, vp, vp, vp]
    lib.cf_merge_attn.argtypes = [gp, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.cf_attn_workspace_bytes_full.restype = ctypes.c_size_t
    lib.cf_attn_workspace_bytes_full.argtypes = [gp, bp, i32]
    lib.cf_query_prefill_attn_full.argtypes = [gp, bp, vp, i32, vp, i64, vp, vp, i64, vp, vp, i64, ctypes.c_float,
                                               vp, i64, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.cf_query_prefill_attn_prefix.argtypes = [gp, bp, vp, i32, vp, i64, vp, vp, i64, vp, vp, i64, i32, vp, vp, i64,
                                                 ctypes.c_float, vp, i64, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.cf_query_prefill_attn_static.argtypes = [gp, bp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp, vp]
    lib.cf_prune_topk.argtypes = [gp, bp, vp, vp, i32, vp, i32, vp]
    lib.cf_prune_topk_host.argtypes = [i32, vp, vp, i32, i32, i32, vp, vp]
    sp = ctypes.POINTER(cf_stack)
    lib.cf_run_stack_workspace_bytes.restype = ctypes.c_size_t
    lib.cf_run_stack_workspace_bytes.argtypes = [gp, bp, sp]
    lib.cf_run_stack.argtypes = [gp, bp, sp, vp, ctypes.c_size_t, vp, ctypes.c_size_t, vp]
    lib.cf_debug_wait_timeout.argtypes = [gp, bp, vp, i64, vp]
    lib.cf_document_prefill_attn.argtypes = [gp, ctypes.POINTER(cf_doc_batch), i32, vp, i64, vp, vp, i64, vp, vp, i64,
                                             ctypes.c_float, vp, i64, vp, vp, vp]
    lib.cf_decode_plan_bytes.restype = ctypes.c_size_t
    lib.cf_decode_plan_bytes.argtypes = [gp, i32, i32]
    lib.cf_decode_plan.argtypes = [gp, i32, i32, vp, i32, vp, ctypes.c_size_t, vp]
    lib.cf_decode_status.argtypes = [gp, i32, i32, vp, vp]
    lib.cf_decode_workspace_bytes.restype = ctypes.c_size_t
    lib.cf_decode_workspace_bytes.argtypes = [gp, i32, i32, i32]
    lib.cf_decode_attn.argtypes = [gp, i32, i32, vp, i32, vp, i64, vp, vp, i64, ctypes.c_float, vp, i64, vp, vp,
                                   ctypes.c_size_t, vp]
    lib.cf_decode_append.argtypes = [gp, i32, i32, i32, vp, vp, i64, vp, i32, vp, vp, i64, vp, vp]
    lib.cf_set_attn_path.argtypes = [i32]
    lib.cf_profile_begin.argtypes = [i32]
    lib.cf_profile_end.argtypes = [vp, i32, vp]
    for name in EXPORTS:
        if name != "cf_error_string" and name not in _SIZE_T_EXPORTS:
            getattr(lib, name).restype = ctypes.c_int
    _LIB = lib
    return lib


def _check(code: int, where: str) -> None:
    if code != CF_OK:
        raise CacheFocusError(code, where)


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return int(t)


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def make_geom(n_q_heads: int, n_kv_heads: int, head_dim: int, dtype, pos_range: int, rope_theta: float,
              rope_layout: int = CF_ROPE_HALF) -> cf_geom:
    if isinstance(dtype, torch.dtype):
        dtype = {torch.bfloat16: CF_BF16, torch.float32: CF_F32}[dtype]
    return cf_geom(n_q_heads, n_kv_heads, head_dim, dtype, rope_layout, pos_range, float(rope_theta))


def make_batch(n_requests: int, q_len: int, total_tokens: int, token_stride: int,
               req_doc_begin: torch.Tensor, doc_offsets: torch.Tensor, doc_src_start: torch.Tensor,
               prefix_len: int = 0, tail_reserve: int = 0, n_reuse: int = 0, tiles_hint: int = 0) -> cf_batch:
    """`req_doc_begin`, `doc_offsets`, `doc_src_start` are int32 device tensors the caller keeps alive."""
    for t in (req_doc_begin, doc_offsets, doc_src_start):
        assert t.dtype == torch.int32 and t.is_contiguous()
    return cf_batch(n_requests, doc_src_start.numel(), q_len, prefix_len, tail_reserve, n_reuse, tiles_hint, 0,
                    total_tokens, token_stride, req_doc_begin.data_ptr(), doc_offsets.data_ptr(),
                    doc_src_start.data_ptr())


def cf_error_string(code: int) -> str:
    return load_library().cf_error_string(code).decode()


def cf_allocate_positions(geom: cf_geom, doc_len: Sequence[int], order: Sequence[int], prefix_len: int = 0,
                          tail_reserve: int = 0, n_reuse: int = 0, query_start: int = -1
                          ) -> Tuple[np.ndarray, np.ndarray, int, int]:
    """Host-side allocation for one request; returns (dst_start, group, n_reuse, query_start)."""
    doc_len, order = _i32(doc_len), _i32(order)
    dst, grp = np.empty(len(doc_len), np.int32), np.empty(len(doc_len), np.int32)
    used, qs = ctypes.c_int32(0), ctypes.c_int32(0)
    rc = load_library().cf_allocate_positions(ctypes.byref(geom), len(doc_len), doc_len.ctypes.data, order.ctypes.data,
                                              len(order), prefix_len, tail_reserve, n_reuse, query_start,
                                              dst.ctypes.data, grp.ctypes.data, ctypes.addressof(used),
                                              ctypes.addressof(qs))
    _check(rc, "cf_allocate_positions")
    return dst, grp, used.value, qs.value


def cf_schedule_linear(n_layers: int, every: int, k: int, k_finish: int) -> List[Tuple[int, int]]:
    cap = max(1, n_layers)
    layers, keeps = np.zeros(cap, np.int32), np.zeros(cap, np.int32)
    count = ctypes.c_int32(0)
    rc = load_library().cf_schedule_linear(n_layers, every, k, k_finish, cap, layers.ctypes.data, keeps.ctypes.data,
                                           ctypes.addressof(count))
    _check(rc, "cf_schedule_linear")
    return [(int(layers[i]), int(keeps[i])) for i in range(count.value)]


def cf_plan_layout_of(geom: cf_geom, batch: cf_batch) -> cf_plan_layout:
    layout = cf_plan_layout()
    _check(load_library().cf_plan_layout_of(ctypes.byref(geom), ctypes.byref(batch), ctypes.byref(layout)),
           "cf_plan_layout_of")
    return layout


def cf_plan_init(geom: cf_geom, batch: cf_batch, plan: torch.Tensor, order: Optional[torch.Tensor] = None,
                 kept_count: Optional[torch.Tensor] = None, query_start: int = -1, stream=None) -> None:
    rc = load_library().cf_plan_init(ctypes.byref(geom), ctypes.byref(batch), _ptr(order), _ptr(kept_count),
                                     query_start, plan.data_ptr(), plan.numel() * plan.element_size(), _stream(stream))
    _check(rc, "cf_plan_init")


def cf_plan_status(geom: cf_geom, batch: cf_batch, plan: torch.Tensor, stream=None) -> int:
    return load_library().cf_plan_status(ctypes.byref(geom), ctypes.byref(batch), plan.data_ptr(), _stream(stream))


def cf_reposition_keys(geom: cf_geom, batch: cf_batch, plan: torch.Tensor, k_in: torch.Tensor, k_out: torch.Tensor,
                       n_layers: int = 1, layer_stride: int = 0, stream=None) -> None:
    rc = load_library().cf_reposition_keys(ctypes.byref(geom), ctypes.byref(batch), plan.data_ptr(), n_layers,
                                           layer_stride, k_in.data_ptr(), k_out.data_ptr(), _stream(stream))
    _check(rc, "cf_reposition_keys")


def cf_attn_workspace_bytes(geom: cf_geom, batch: cf_batch) -> int:
    return int(load_library().cf_attn_workspace_bytes(ctypes.byref(geom), ctypes.byref(batch)))


def cf_query_prefill_attn(geom: cf_geom, batch: cf_batch, plan: torch.Tensor, q: torch.Tensor, k_cache: torch.Tensor,
                          v_cache: torch.Tensor, out: torch.Tensor, workspace: torch.Tensor,
                          lse: Optional[torch.Tensor] = None, doc_scores: Optional[torch.Tensor] = None,
                          score_accum: Optional[torch.Tensor] = None, softmax_scale: float = 0.0, stream=None) -> None:
    rc = load_library().cf_query_prefill_attn(ctypes.byref(geom), ctypes.byref(batch), plan.data_ptr(), q.data_ptr(),
                                              k_cache.data_ptr(), v_cache.data_ptr(), softmax_scale, out.data_ptr(),
                                              _ptr(lse), _ptr(doc_scores), _ptr(score_accum), workspace.data_ptr(),
                                              workspace.numel() * workspace.element_size(), _stream(stream))
    _check(rc, "cf_query_prefill_attn")


def cf_attn_workspace_bytes_layers(geom: cf_geom, batch: cf_batch, n_layers: int) -> int:
    return int(load_library().cf_attn_workspace_bytes_layers(ctypes.byref(geom), ctypes.byref(batch), n_layers))


def cf_query_prefill_attn_layers(geom: cf_geom, batch: cf_batch, plan: torch.Tensor, q: torch.Tensor,
                                 k_cache: torch.Tensor, v_cache: torch.Tensor, out: torch.Tensor,
                                 workspace: torch.Tensor, lse: Optional[torch.Tensor] = None,
                                 doc_scores: Optional[torch.Tensor] = None,
                                 score_accum: Optional[torch.Tensor] = None, softmax_scale: float = 0.0,
                                 stream=None) -> None:
    """`q`, `out` [n_layers, B, Lq, Hq, D]; `k_cache`, `v_cache` [n_layers, T, ...]; `lse` [n_layers, B, Hq, Lq];
    `doc_scores` [n_layers, n_docs_total].  Dimension 0 may be strided, the rest of a layer is dense."""
    n_layers = q.shape[0]
    assert k_cache.shape[0] == n_layers and v_cache.shape[0] == n_layers and out.shape[0] == n_layers
    assert k_cache.stride(0) == v_cache.stride(0)
    for t in (lse, doc_scores):
        assert t is None or (t.shape[0] == n_layers and t.is_contiguous())
    rc = load_library().cf_query_prefill_attn_layers(
        ctypes.byref(geom), ctypes.byref(batch), plan.data_ptr(), n_layers, q.data_ptr(), q.stride(0),
        k_cache.data_ptr(), v_cache.data_ptr(), k_cache.stride(0), softmax_scale, out.data_ptr(), out.stride(0),
        _ptr(lse), _ptr(doc_scores), _ptr(score_accum), workspace.data_ptr(),
        workspace.numel() * workspace.element_size(), _stream(stream))
    _check(rc, "cf_query_prefill_attn_layers")


def cf_attn_workspace_bytes_slots(geom: cf_geom, batch: cf_batch, n_slots: int) -> int:
    return int(load_library().cf_attn_workspace_bytes_slots(ctypes.byref(geom), ctypes.byref(batch), n_slots))


def cf_query_prefill_attn_slot(geom: cf_geom, batch: cf_batch, plan: torch.Tensor, slot: int, n_slots: int,
                               q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, out: torch.Tensor,
                               workspace: torch.Tensor, lse: Optional[torch.Tensor] = None, softmax_scale: float = 0.0,
                               stream=None) -> None:
    """One layer (tensors as in cf_query_prefill_attn) whose document scores are left for cf_accumulate_scores."""
    rc = load_library().cf_query_prefill_attn_slot(
        ctypes.byref(geom), ctypes.byref(batch), plan.data_ptr(), slot, n_slots, q.data_ptr(), k_cache.data_ptr(),
        v_cache.data_ptr(), softmax_scale, out.data_ptr(), _ptr(lse), workspace.data_ptr(),
        workspace.numel() * workspace.element_size(), _stream(stream))
    _check(rc, "cf_query_prefill_attn_slot")


def cf_attn_workspace_bytes_slots_full(geom: cf_geom, batch: cf_batch, n_slots: int) -> int:
    return int(load_library().cf_attn_workspace_bytes_slots_full(ctypes.byref(geom), ctypes.byref(batch), n_slots))


def cf_query_prefill_attn_slot_full(geom: cf_geom, batch: cf_batch, plan: torch.Tensor, slot: int, n_slots: int,
                                    q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, out: torch.Tensor,
                                    workspace: torch.Tensor, k_prefix: Optional[torch.Tensor] = None,
                                    v_prefix: Optional[torch.Tensor] = None, k_self: Optional[torch.Tensor] = None,
                                    v_self: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                                    softmax_scale: float = 0.0, stream=None) -> None:
    """One layer with a prefix cache `k_prefix`, `v_prefix` [P, Hkv, D] and / or the query tokens' own `k_self`,
    `v_self` [B, Lq, Hkv, D]; document scores left for cf_accumulate_scores."""
    rc = load_library().cf_query_prefill_attn_slot_full(
        ctypes.byref(geom), ctypes.byref(batch), plan.data_ptr(), slot, n_slots, q.data_ptr(), k_cache.data_ptr(),
        v_cache.data_ptr(), _ptr(k_prefix), _ptr(v_prefix), 0 if k_prefix is None else k_prefix.shape[0], _ptr(k_self),
        _ptr(v_self), softmax_scale, out.data_ptr(), _ptr(lse), workspace.data_ptr(),
        workspace.numel() * workspace.element_size(), _stream(stream))
    _check(rc, "cf_query_prefill_attn_slot_full")


def cf_accumulate_scores(geom: cf_geom, batch: cf_batch, plan: torch.Tensor, n_filled: int, n_slots: int,
                         workspace: torch.Tensor, doc_scores: Optional[torch.Tensor] = None,
                         score_accum: Optional[torch.Tensor] = None, stream=None) -> None:
    """`doc_scores` [n_filled, n_docs_total] (contiguous) and / or `score_accum` [n_docs_total]."""
    assert doc_scores is None or (doc_scores.shape[0] == n_filled and doc_scores.is_contiguous())
    rc = load_library().cf_accumulate_scores(
        ctypes.byref(geom), ctypes.byref(batch), plan.data_ptr(), n_filled, n_slots, _ptr(doc_scores), _ptr(score_accum),
        workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream(stream))
    _check(rc, "cf_accumulate_scores")


def cf_assemble_final_cache(geom: cf_geom, batch: cf_batch, plan: torch.Tensor, k_cache: torch.Tensor,
                            v_cache: torch.Tensor, k_self: torch.Tensor, v_self: torch.Tensor, k_out: torch.Tensor,
                            v_out: torch.Tensor, final_rows: torch.Tensor, stream=None) -> None:
    """k_cache, v_cache [L, T, Hkv, D]; k_self, v_self [L, B, Lq, Hkv, D]; k_out, v_out [L, B, out_rows, Hkv, D]
    (contiguous); final_rows int32 [B]."""
    assert k_out.is_contiguous() and v_out.is_contiguous() and k_out.shape == v_out.shape
    assert final_rows.dtype == torch.int32 and k_cache.stride(0) == v_cache.stride(0)
    rc = load_library().cf_assemble_final_cache(
        ctypes.byref(geom), ctypes.byref(batch), plan.data_ptr(), k_cache.shape[0], k_cache.stride(0),
        k_cache.data_ptr(), v_cache.data_ptr(), k_self.stride(0), k_self.data_ptr(), v_self.data_ptr(),
        k_out.shape[2], k_out.data_ptr(), v_out.data_ptr(), final_rows.data_ptr(), _stream(stream))
    _check(rc, "cf_assemble_final_cache")


def cf_merge_attn(geom: cf_geom, out_a: torch.Tensor, lse_a: torch.Tensor, out_b: torch.Tensor, lse_b: torch.Tensor,
                  out: torch.Tensor, lse: Optional[torch.Tensor] = None, stream=None) -> None:
    """out_* [..., Lq, Hq, D] and lse_* [..., Hq, Lq] with the same leading dimensions, all contiguous."""
    for t in (out_a, out_b, out, lse_a, lse_b):
        assert t.is_contiguous()
    q_len = out_a.shape[-3]
    n_blocks = out_a.numel() // (q_len * out_a.shape[-2] * out_a.shape[-1])
    rc = load_library().cf_merge_attn(ctypes.byref(geom), n_blocks, q_len, out_a.data_ptr(), lse_a.data_ptr(),
                                      out_b.data_ptr(), lse_b.data_ptr(), out.data_ptr(), _ptr(lse), _stream(stream))
    _check(rc, "cf_merge_attn")


def cf_attn_workspace_bytes_full(geom: cf_geom, batch: cf_batch, n_layers: int) -> int:
    return int(load_library().cf_attn_workspace_bytes_full(ctypes.byref(geom), ctypes.byref(batch), n_layers))


def cf_query_prefill_attn_full(geom: cf_geom, batch: cf_batch, plan: torch.Tensor, q: torch.Tensor,
                               k_cache: torch.Tensor, v_cache: torch.Tensor, k_self: torch.Tensor,
                               v_self: torch.Tensor, out: torch.Tensor, workspace: torch.Tensor,
                               lse: Optional[torch.Tensor] = None, doc_scores: Optional[torch.Tensor] = None,
                               score_accum: Optional[torch.Tensor] = None, softmax_scale: float = 0.0,
                               stream=None) -> None:
    """cf_query_prefill_attn_layers plus the causal block of the query tokens over themselves:
    `k_self`, `v_self` [n_layers, B, Lq, Hkv, D] (dimension 0 may be strided)."""
    n_layers = q.shape[0]
    assert k_cache.shape[0] == n_layers and v_cache.shape[0] == n_layers and out.shape[0] == n_layers
    assert k_self.shape[0] == n_layers and v_self.shape[0] == n_layers
    assert k_cache.stride(0) == v_cache.stride(0) and k_self.stride(0) == v_self.stride(0)
    for t in (lse, doc_scores):
        assert t is None or (t.shape[0] == n_layers and t.is_contiguous())
    rc = load_library().cf_query_prefill_attn_full(
        ctypes.byref(geom), ctypes.byref(batch), plan.data_ptr(), n_layers, q.data_ptr(), q.stride(0),
        k_cache.data_ptr(), v_cache.data_ptr(), k_cache.stride(0), k_self.data_ptr(), v_self.data_ptr(),
        k_self.stride(0), softmax_scale, out.data_ptr(), out.stride(0), _ptr(lse), _ptr(doc_scores),
        _ptr(score_accum), workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream(stream))
    _check(rc, "cf_query_prefill_attn_full")


def cf_query_prefill_attn_prefix(geom: cf_geom, batch: cf_batch, plan: torch.Tensor, q: torch.Tensor,
                                 k_cache: torch.Tensor, v_cache: torch.Tensor, k_prefix: torch.Tensor,
                                 v_prefix: torch.Tensor, out: torch.Tensor, workspace: torch.Tensor,
                                 k_self: Optional[torch.Tensor] = None, v_self: Optional[torch.Tensor] = None,
                                 lse: Optional[torch.Tensor] = None, doc_scores: Optional[torch.Tensor] = None,
                                 score_accum: Optional[torch.Tensor] = None, softmax_scale: float = 0.0,
                                 stream=None) -> None:
    """cf_query_prefill_attn_full with a shared prefix cache attended in the same call: `k_prefix`, `v_prefix`
    [n_layers, P, Hkv, D] dense; `k_self`, `v_self` [n_layers, B, Lq, Hkv, D] or None."""
    n_layers = q.shape[0]
    assert k_cache.shape[0] == n_layers and v_cache.shape[0] == n_layers and out.shape[0] == n_layers
    assert k_prefix.shape[0] == n_layers and v_prefix.shape == k_prefix.shape and k_prefix.stride(0) == v_prefix.stride(0)
    assert k_cache.stride(0) == v_cache.stride(0) and (k_self is None) == (v_self is None)
    for t in (lse, doc_scores):
        assert t is None or (t.shape[0] == n_layers and t.is_contiguous())
    rc = load_library().cf_query_prefill_attn_prefix(
        ctypes.byref(geom), ctypes.byref(batch), plan.data_ptr(), n_layers, q.data_ptr(), q.stride(0),
        k_cache.data_ptr(), v_cache.data_ptr(), k_cache.stride(0), k_prefix.data_ptr(), v_prefix.data_ptr(),
        k_prefix.stride(0), k_prefix.shape[1], _ptr(k_self), _ptr(v_self), 0 if k_self is None else k_self.stride(0),
        softmax_scale, out.data_ptr(), out.stride(0), _ptr(lse), _ptr(doc_scores), _ptr(score_accum),
        workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream(stream))
    _check(rc, "cf_query_prefill_attn_prefix")


def cf_query_prefill_attn_static(geom: cf_geom, batch: cf_batch, plan: torch.Tensor, q: torch.Tensor,
                                 k_cache: torch.Tensor, v_cache: torch.Tensor, out: torch.Tensor,
                                 lse: Optional[torch.Tensor] = None, doc_scores: Optional[torch.Tensor] = None,
                                 score_accum: Optional[torch.Tensor] = None, softmax_scale: float = 0.0,
                                 stream=None) -> None:
    """cf_query_prefill_attn without a workspace argument: the scratch is a fixed 32 MiB array inside
    the library, for callers that may not allocate device memory.  Raises CacheFocusError with
    CF_ERR_WORKSPACE when the batch needs more scratch than that."""
    rc = load_library().cf_query_prefill_attn_static(ctypes.byref(geom), ctypes.byref(batch), plan.data_ptr(),
                                                     q.data_ptr(), k_cache.data_ptr(), v_cache.data_ptr(), softmax_scale,
                                                     out.data_ptr(), _ptr(lse), _ptr(doc_scores), _ptr(score_accum),
                                                     _stream(stream))
    _check(rc, "cf_query_prefill_attn_static")


def cf_prune_topk(geom: cf_geom, batch: cf_batch, plan: torch.Tensor, score_accum: torch.Tensor, keep: int,
                  strategy: int, keep_per_request: Optional[torch.Tensor] = None, stream=None) -> None:
    rc = load_library().cf_prune_topk(ctypes.byref(geom), ctypes.byref(batch), plan.data_ptr(), score_accum.data_ptr(),
                                      keep, _ptr(keep_per_request), strategy, _stream(stream))
    _check(rc, "cf_prune_topk")


def cf_prune_topk_host(score_accum: Sequence[float], order: Sequence[int], keep: int, strategy: int) -> List[int]:
    """Host-side pruning step: `score_accum` float32 by local id, `order` the kept ids by rank."""
    scores = np.ascontiguousarray(np.asarray(score_accum, dtype=np.float32))
    order = _i32(order)
    out = np.zeros(max(1, len(order)), np.int32)
    n_out = ctypes.c_int32(0)
    rc = load_library().cf_prune_topk_host(len(scores), scores.ctypes.data, order.ctypes.data, len(order), keep,
                                           strategy, out.ctypes.data, ctypes.addressof(n_out))
    _check(rc, "cf_prune_topk_host")
    return [int(x) for x in out[:n_out.value]]


def make_stack(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, out: torch.Tensor,
               score_accum: torch.Tensor, schedule: Sequence[Tuple[int, int]], strategy: int, batch_layers: bool,
               lse: Optional[torch.Tensor] = None, layer_scores: Optional[torch.Tensor] = None,
               k_final: Optional[torch.Tensor] = None, k_self: Optional[torch.Tensor] = None,
               v_self: Optional[torch.Tensor] = None, softmax_scale: float = 0.0,
               doc_len: Optional[np.ndarray] = None, req_doc_begin: Optional[np.ndarray] = None,
               k_prefix: Optional[torch.Tensor] = None, v_prefix: Optional[torch.Tensor] = None):
    """A cf_stack over torch buffers (dimension 0 = layers, may be strided; the rest of a layer dense).
    Returns (struct, keepalive): the host arrays the struct points to live in `keepalive`."""
    n_layers = q.shape[0]
    assert k_cache.shape[0] == n_layers and v_cache.shape[0] == n_layers and out.shape[0] == n_layers
    assert k_cache.stride(0) == v_cache.stride(0)
    for t in (lse, layer_scores):
        assert t is None or (t.shape[0] == n_layers and t.is_contiguous())
    if k_final is not None:
        assert k_final.shape == k_cache.shape and k_final.stride(0) == k_cache.stride(0)
    if k_self is not None:
        assert k_self.shape[0] == n_layers and k_self.stride(0) == v_self.stride(0)
    sched = sorted((int(l), int(kp)) for l, kp in schedule)
    layers, keeps = _i32([l for l, _ in sched]), _i32([kp for _, kp in sched])
    keep = [layers, keeps]
    dl = rb = None
    if doc_len is not None and req_doc_begin is not None:
        dl, rb = _i32(doc_len), _i32(req_doc_begin)
        keep += [dl, rb]
    st = cf_stack(n_layers, len(sched), layers.ctypes.data if len(sched) else None,
                  keeps.ctypes.data if len(sched) else None, strategy, 1 if batch_layers else 0, softmax_scale, 0,
                  q.data_ptr(), q.stride(0), k_cache.data_ptr(), v_cache.data_ptr(), k_cache.stride(0),
                  _ptr(k_self), _ptr(v_self), 0 if k_self is None else k_self.stride(0),
                  out.data_ptr(), out.stride(0), _ptr(lse), _ptr(layer_scores), score_accum.data_ptr(),
                  _ptr(k_final), None if dl is None else dl.ctypes.data, None if rb is None else rb.ctypes.data,
                  _ptr(k_prefix), _ptr(v_prefix), 0 if k_prefix is None else k_prefix.stride(0),
                  0 if k_prefix is None else k_prefix.shape[1], 0)
    return st, keep


def cf_run_stack_workspace_bytes(geom: cf_geom, batch: cf_batch, stack: cf_stack) -> int:
    return int(load_library().cf_run_stack_workspace_bytes(ctypes.byref(geom), ctypes.byref(batch), ctypes.byref(stack)))


def cf_run_stack(geom: cf_geom, batch: cf_batch, stack: cf_stack, plan: torch.Tensor, workspace: torch.Tensor,
                 stream=None) -> None:
    rc = load_library().cf_run_stack(ctypes.byref(geom), ctypes.byref(batch), ctypes.byref(stack), plan.data_ptr(),
                                     plan.numel() * plan.element_size(), workspace.data_ptr(),
                                     workspace.numel() * workspace.element_size(), _stream(stream))
    _check(rc, "cf_run_stack")


def cf_document_prefill_attn(geom: cf_geom, doc_offsets: torch.Tensor, max_doc_len: int, q: torch.Tensor,
                             k: torch.Tensor, v: torch.Tensor, out: torch.Tensor,
                             k_prefix: Optional[torch.Tensor] = None, v_prefix: Optional[torch.Tensor] = None,
                             lse: Optional[torch.Tensor] = None, softmax_scale: float = 0.0,
                             token_stride: Optional[int] = None, status: Optional[torch.Tensor] = None,
                             stream=None) -> None:
    """Attention of the offline cache construction.  q, out [L, T, Hq, D]; k, v [L, T, Hkv, D] (rows may be
    padded to `token_stride`); k_prefix, v_prefix [L, P, Hkv, D] dense; lse [L, Hq, T]; doc_offsets int32
    device [n_docs + 1].  Dimension 0 may be strided."""
    n_layers, total = q.shape[0], q.shape[1]
    assert doc_offsets.dtype == torch.int32 and doc_offsets.is_contiguous()
    assert k.shape[0] == n_layers and v.shape[0] == n_layers and out.shape[0] == n_layers
    assert k.stride(0) == v.stride(0) and (lse is None or lse.is_contiguous())
    prefix_len = 0 if k_prefix is None else k_prefix.shape[1]
    if prefix_len:
        assert k_prefix.stride(0) == v_prefix.stride(0)
    stride = k.shape[2] * k.shape[3] if token_stride is None else token_stride
    docs = cf_doc_batch(doc_offsets.numel() - 1, max_doc_len, prefix_len, 0, total, stride, doc_offsets.data_ptr())
    rc = load_library().cf_document_prefill_attn(
        ctypes.byref(geom), ctypes.byref(docs), n_layers, q.data_ptr(), q.stride(0), k.data_ptr(), v.data_ptr(),
        k.stride(0), _ptr(k_prefix) if prefix_len else None, _ptr(v_prefix) if prefix_len else None,
        k_prefix.stride(0) if prefix_len else 0, softmax_scale, out.data_ptr(), out.stride(0), _ptr(lse),
        _ptr(status), _stream(stream))
    _check(rc, "cf_document_prefill_attn")


def cf_debug_wait_timeout(geom: cf_geom, batch: cf_batch, plan: torch.Tensor, limit_cycles: int, stream=None) -> None:
    _check(load_library().cf_debug_wait_timeout(ctypes.byref(geom), ctypes.byref(batch), plan.data_ptr(),
                                                limit_cycles, _stream(stream)), "cf_debug_wait_timeout")


def cf_set_attn_path(path: int) -> None:
    _check(load_library().cf_set_attn_path(path), "cf_set_attn_path")


def cf_profile_begin(max_records: int) -> None:
    _check(load_library().cf_profile_begin(max_records), "cf_profile_begin")


def cf_profile_end(capacity: int) -> np.ndarray:
    """Durations (ms) of the attention kernel launches recorded since cf_profile_begin."""
    ms = np.zeros(max(1, capacity), np.float32)
    count = ctypes.c_int32(0)
    _check(load_library().cf_profile_end(ms.ctypes.data, capacity, ctypes.addressof(count)), "cf_profile_end")
    return ms[:min(capacity, count.value)]


def cf_decode_plan_bytes(geom: cf_geom, n_requests: int, cache_rows: int) -> int:
    return int(load_library().cf_decode_plan_bytes(ctypes.byref(geom), n_requests, cache_rows))


def cf_decode_workspace_bytes(geom: cf_geom, n_requests: int, cache_rows: int, n_layers: int) -> int:
    return int(load_library().cf_decode_workspace_bytes(ctypes.byref(geom), n_requests, cache_rows, n_layers))


def cf_decode_plan(geom: cf_geom, n_requests: int, cache_rows: int, rows: torch.Tensor, extra_rows: int,
                   decode_plan: torch.Tensor, stream=None) -> None:
    """One decoding step's description: request b attends rows 0 .. rows[b] + extra_rows - 1 of its slot."""
    rc = load_library().cf_decode_plan(ctypes.byref(geom), n_requests, cache_rows, rows.data_ptr(), extra_rows,
                                       decode_plan.data_ptr(), decode_plan.numel() * decode_plan.element_size(),
                                       _stream(stream))
    _check(rc, "cf_decode_plan")


def cf_decode_status(geom: cf_geom, n_requests: int, cache_rows: int, decode_plan: torch.Tensor, stream=None) -> int:
    return int(load_library().cf_decode_status(ctypes.byref(geom), n_requests, cache_rows, decode_plan.data_ptr(),
                                               _stream(stream)))


def cf_decode_attn(geom: cf_geom, n_requests: int, cache_rows: int, decode_plan: torch.Tensor, q: torch.Tensor,
                   k_final: torch.Tensor, v_final: torch.Tensor, out: torch.Tensor, workspace: torch.Tensor,
                   lse: Optional[torch.Tensor] = None, softmax_scale: float = 0.0, stream=None) -> None:
    """q, out [n_layers, B, Hq, D]; k_final, v_final [n_layers, B, cache_rows, Hkv, D]; lse [n_layers, B, Hq]."""
    n_layers = q.shape[0]
    assert k_final.shape[0] == n_layers and v_final.shape[0] == n_layers and out.shape[0] == n_layers
    assert k_final.stride(0) == v_final.stride(0) and (lse is None or lse.is_contiguous())
    rc = load_library().cf_decode_attn(ctypes.byref(geom), n_requests, cache_rows, decode_plan.data_ptr(), n_layers,
                                       q.data_ptr(), q.stride(0), k_final.data_ptr(), v_final.data_ptr(),
                                       k_final.stride(0), softmax_scale, out.data_ptr(), out.stride(0), _ptr(lse),
                                       workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                       _stream(stream))
    _check(rc, "cf_decode_attn")


def cf_decode_append(geom: cf_geom, n_requests: int, cache_rows: int, k_final: torch.Tensor, v_final: torch.Tensor,
                     rows: torch.Tensor, step: int, k_new: torch.Tensor, v_new: torch.Tensor,
                     status: Optional[torch.Tensor] = None, stream=None) -> None:
    """k_new, v_new [n_layers, B, Hkv, D] become row rows[b] + step of request b's slot in every layer."""
    n_layers = k_final.shape[0]
    assert v_final.shape[0] == n_layers and k_new.shape[0] == n_layers and v_new.shape[0] == n_layers
    assert k_final.stride(0) == v_final.stride(0) and k_new.stride(0) == v_new.stride(0)
    rc = load_library().cf_decode_append(ctypes.byref(geom), n_requests, cache_rows, n_layers, k_final.data_ptr(),
                                         v_final.data_ptr(), k_final.stride(0), rows.data_ptr(), step,
                                         k_new.data_ptr(), v_new.data_ptr(), k_new.stride(0), _ptr(status),
                                         _stream(stream))
    _check(rc, "cf_decode_append")


def plan_field(plan: torch.Tensor, layout: cf_plan_layout, name: str, count: int, dtype=torch.int32) -> torch.Tensor:
    """View of one field of a plan buffer (a uint8 device tensor)."""
    off = getattr(layout, name)
    size = count * torch.empty((), dtype=dtype).element_size()
    return plan[off:off + size].view(dtype)
