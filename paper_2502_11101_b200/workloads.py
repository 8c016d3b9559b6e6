"""Seeded synthetic workloads shaped like the paper's retrieval-augmented settings.

This module only *draws inputs*: document lengths, a query tensor, and a key/value
cache store.  It contains none of the method's arithmetic (no rotary embedding, no
attention, no allocation, no pruning), so the CPU oracle and the CUDA path can both be
fed from it without sharing any computation.

Shapes follow the paper's experiments (Sec. 3.1, App. B): passages of roughly one
hundred words (about 120-200 tokens), tens to 100+ passages per query, LLaMA-2-7B and
Qwen2 head geometry.  Contents are synthetic: a counter-based integer hash gives every
tensor element a reproducible, device-independent value (integer arithmetic only, one
fp32 multiply, one rounding to the storage type), so a tensor generated on the CPU and
the same tensor generated on a GPU are bit-identical.

Relevance is planted through the *norm* of a document's cached keys: a rotation of the
two-dimensional slices of a key (Eq. 2) preserves that norm, hence the planted ranking
does not depend on where a document is later placed in the positional range.  Planted
documents get the largest key scale; the remaining documents get a strictly decreasing
ladder of scales so that no cut of a pruning schedule falls between two statistically
identical documents.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB

TENSOR_Q = 1
TENSOR_K = 2
TENSOR_V = 3
TENSOR_META = 4
TENSOR_K_SELF = 5
TENSOR_V_SELF = 6


def _signed(x: int) -> int:
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


def _mix_py(z: int) -> int:
    """splitmix64 finaliser on a Python integer (used for the small metadata draws)."""
    z = (z + _GOLDEN) & _MASK64
    z = ((z ^ (z >> 30)) * _C1) & _MASK64
    z = ((z ^ (z >> 27)) * _C2) & _MASK64
    return z ^ (z >> 31)


def _stream_key(seed: int, tensor_id: int) -> int:
    return _mix_py(_mix_py(seed & _MASK64) ^ (tensor_id * 0xD1342543DE82EF95 & _MASK64))


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    return (z >> s) & ((1 << (64 - s)) - 1)


def _mix_torch(z: torch.Tensor) -> torch.Tensor:
    """The same finaliser on an int64 tensor (two's-complement wrap-around)."""
    z = z + _signed(_GOLDEN)
    z = (z ^ _lsr(z, 30)) * _signed(_C1)
    z = (z ^ _lsr(z, 27)) * _signed(_C2)
    return z ^ _lsr(z, 31)


_NORMAL_SCALE = math.sqrt(3.0) / 65536.0


def hashed_normal(seed: int, tensor_id: int, base_index: int, count: int,
                  device: torch.device | str = "cpu") -> torch.Tensor:
    """`count` approximately standard-normal fp32 values for flat element indices
    `base_index .. base_index+count-1` of tensor `tensor_id`.

    Each value is the centred sum of the four 16-bit fields of one 64-bit hash (an
    Irwin-Hall variate with unit variance, bounded by +-3.47)."""
    idx = torch.arange(base_index, base_index + count, dtype=torch.int64, device=device)
    h = _mix_torch(idx ^ _signed(_stream_key(seed, tensor_id)))
    s = (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + (_lsr(h, 48) & 0xFFFF)
    return (s - 131070).to(torch.float32) * _NORMAL_SCALE


def _hashed_ints(seed: int, tensor_id: int, count: int) -> List[int]:
    key = _stream_key(seed, tensor_id)
    return [_mix_py(key ^ i) for i in range(count)]


@dataclasses.dataclass(frozen=True)
class WorkloadConfig:
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str                      # "f32" or "bf16": storage type of Q, K, V
    rope_theta: float
    pos_range: int
    n_docs: int                     # retrieved documents per request
    doc_len_lo: int
    doc_len_hi: int
    q_len: int
    batch: int                      # independent requests with distinct document sets
    n_planted: int
    schedule: Tuple[Tuple[int, int], ...]   # (layer, keep): after 1-based `layer` keep top-`keep`

    @property
    def group_size(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    def kept_at_layer(self, layer: int) -> int:
        """Documents attended by 1-based `layer` under the schedule."""
        kept = self.n_docs
        for at, keep in self.schedule:
            if layer > at:
                kept = keep
        return kept


CONFIGS: Dict[int, WorkloadConfig] = {
    1: WorkloadConfig("tiny-mha-f32", 1, 4, 4, 64, "f32", 1.0e4, 256, 8, 32, 32, 16, 1, 2,
                      ((1, 4),)),
    2: WorkloadConfig("llama2-7b-layer", 1, 32, 32, 128, "bf16", 1.0e4, 4096, 20, 120, 200, 32, 1, 4,
                      ((1, 10),)),
    3: WorkloadConfig("qwen2-1.5b-stack", 28, 12, 2, 128, "bf16", 1.0e6, 32768, 50, 128, 192, 48, 1, 6,
                      ((4, 25), (12, 12), (20, 6))),
    4: WorkloadConfig("qwen2-7b-stack-b4", 28, 28, 4, 128, "bf16", 1.0e6, 32768, 100, 128, 192, 64, 4, 12,
                      ((4, 50), (12, 25), (20, 12))),
    5: WorkloadConfig("llama2-7b-stack-b8", 32, 32, 32, 128, "bf16", 1.0e4, 4096, 120, 160, 200, 64, 8, 15,
                      ((4, 60), (12, 30), (24, 15))),
}

PLANTED_SCALE = 1.5
LADDER_HI = 1.15
LADDER_LO = 0.65


@dataclasses.dataclass
class WorkloadMeta:
    """Integer description of a batch: every request's documents laid end to end in one
    packed store of `total_tokens` rows."""
    cfg: WorkloadConfig
    seed: int
    doc_len: np.ndarray          # int32 [n_docs_total]
    doc_offsets: np.ndarray      # int32 [n_docs_total+1]  first store row of each document
    req_doc_begin: np.ndarray    # int32 [batch+1]
    doc_src_start: np.ndarray    # int32 [n_docs_total]    position the document was cached at
    key_scale: np.ndarray        # float32 [n_docs_total]  planted relevance (key norm scale)
    planted: List[List[int]]     # per request: local ids of the planted documents

    @property
    def n_docs_total(self) -> int:
        return int(self.doc_len.shape[0])

    @property
    def total_tokens(self) -> int:
        return int(self.doc_offsets[-1])


def make_meta(cfg: WorkloadConfig, seed: int, doc_len_override: Optional[Sequence[int]] = None
              ) -> WorkloadMeta:
    n_total = cfg.n_docs * cfg.batch
    draws = _hashed_ints(seed, TENSOR_META, 3 * n_total)
    span = cfg.doc_len_hi - cfg.doc_len_lo + 1
    if doc_len_override is not None:
        assert len(doc_len_override) == n_total
        doc_len = np.asarray(doc_len_override, dtype=np.int32)
    else:
        doc_len = np.array([cfg.doc_len_lo + draws[i] % span for i in range(n_total)], dtype=np.int32)
    doc_offsets = np.zeros(n_total + 1, dtype=np.int32)
    doc_offsets[1:] = np.cumsum(doc_len)
    req_doc_begin = np.arange(cfg.batch + 1, dtype=np.int32) * cfg.n_docs
    key_scale = np.zeros(n_total, dtype=np.float32)
    planted: List[List[int]] = []
    for b in range(cfg.batch):
        base = b * cfg.n_docs
        by_hash = sorted(range(cfg.n_docs), key=lambda i: draws[n_total + base + i])
        chosen = sorted(by_hash[:cfg.n_planted])
        rest = sorted(by_hash[cfg.n_planted:], key=lambda i: draws[2 * n_total + base + i])
        planted.append(chosen)
        for i in chosen:
            key_scale[base + i] = PLANTED_SCALE
        for k, i in enumerate(rest):
            frac = k / max(1, len(rest) - 1)
            key_scale[base + i] = LADDER_HI - (LADDER_HI - LADDER_LO) * frac
    return WorkloadMeta(cfg, seed, doc_len, doc_offsets, req_doc_begin,
                        np.zeros(n_total, dtype=np.int32), key_scale, planted)


def make_q(meta: WorkloadMeta, device: torch.device | str = "cpu",
           layers: Optional[range] = None) -> torch.Tensor:
    """Query states [n_layers, batch, q_len, n_q_heads, head_dim] in the storage type.
    The library treats them as already position-encoded at `query_start + j`."""
    cfg = meta.cfg
    layers = range(cfg.n_layers) if layers is None else layers
    per_layer = cfg.batch * cfg.q_len * cfg.n_q_heads * cfg.head_dim
    out = torch.empty((len(layers), cfg.batch, cfg.q_len, cfg.n_q_heads, cfg.head_dim),
                      dtype=cfg.torch_dtype, device=device)
    for n, layer in enumerate(layers):
        vals = hashed_normal(meta.seed, TENSOR_Q, layer * per_layer, per_layer, device)
        out[n] = vals.view(out.shape[1:]).to(cfg.torch_dtype)
    return out


def fill_kv_layer(meta: WorkloadMeta, layer: int, k_out: torch.Tensor, v_out: torch.Tensor,
                  chunk_tokens: int = 1 << 14) -> None:
    """Write one layer of the cache store: `k_out`, `v_out` are [total_tokens, n_kv_heads,
    head_dim] views in the storage type.  Keys carry the per-document relevance scale."""
    cfg = meta.cfg
    device = k_out.device
    row = cfg.n_kv_heads * cfg.head_dim
    total = meta.total_tokens
    token_scale = torch.from_numpy(np.repeat(meta.key_scale, meta.doc_len)).to(device)
    for t0 in range(0, total, chunk_tokens):
        t1 = min(total, t0 + chunk_tokens)
        base = (layer * total + t0) * row
        count = (t1 - t0) * row
        kv = hashed_normal(meta.seed, TENSOR_K, base, count, device).view(t1 - t0, row)
        kv = kv * token_scale[t0:t1, None]
        k_out[t0:t1] = kv.view(t1 - t0, cfg.n_kv_heads, cfg.head_dim).to(cfg.torch_dtype)
        vv = hashed_normal(meta.seed, TENSOR_V, base, count, device)
        v_out[t0:t1] = vv.view(t1 - t0, cfg.n_kv_heads, cfg.head_dim).to(cfg.torch_dtype)


def make_kv(meta: WorkloadMeta, device: torch.device | str = "cpu",
            layers: Optional[range] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Cache store K, V: [n_layers, total_tokens, n_kv_heads, head_dim]."""
    cfg = meta.cfg
    layers = range(cfg.n_layers) if layers is None else layers
    shape = (len(layers), meta.total_tokens, cfg.n_kv_heads, cfg.head_dim)
    k = torch.empty(shape, dtype=cfg.torch_dtype, device=device)
    v = torch.empty(shape, dtype=cfg.torch_dtype, device=device)
    for n, layer in enumerate(layers):
        fill_kv_layer(meta, layer, k[n], v[n])
    return k, v


def make_kv_self(meta: WorkloadMeta, device: torch.device | str = "cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """Key and value states of the query tokens themselves, [n_layers, batch, q_len, n_kv_heads,
    head_dim] in the storage type; like the query states they count as already position-encoded."""
    cfg = meta.cfg
    shape = (cfg.n_layers, cfg.batch, cfg.q_len, cfg.n_kv_heads, cfg.head_dim)
    count = int(np.prod(shape))
    k = hashed_normal(meta.seed, TENSOR_K_SELF, 0, count, device).view(shape).to(cfg.torch_dtype)
    v = hashed_normal(meta.seed, TENSOR_V_SELF, 0, count, device).view(shape).to(cfg.torch_dtype)
    return k, v


def scaled_config(cfg: WorkloadConfig, **changes) -> WorkloadConfig:
    """A copy of `cfg` with some fields replaced (reduced cases for parity tests)."""
    return dataclasses.replace(cfg, **changes)
