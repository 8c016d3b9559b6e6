"""Parity of cf_document_prefill_attn (attention of the offline cache construction, Sec. 2.2) with the
oracle's document_prefill_attn, document by document, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_11101_b200 as cf
from paper_2502_11101_b200 import workloads as W
from tests import harness

pytestmark = pytest.mark.gpu

RAGGED = [1, 63, 64, 65, 129, 200]


@pytest.fixture(scope="module", autouse=True)
def _library():
    assert torch.cuda.is_available()
    from paper_2502_11101_b200 import build
    build.build()
    cf.load_library()


def _inputs(seed, lens, n_layers, hq, hkv, d, dtype, prefix_len):
    total = int(sum(lens))
    n = lambda tid, *shape: W.hashed_normal(seed, tid, 0, int(np.prod(shape))).view(*shape).to(dtype)
    q = n(W.TENSOR_Q, n_layers, total, hq, d)
    k = n(W.TENSOR_K, n_layers, total, hkv, d)
    v = n(W.TENSOR_V, n_layers, total, hkv, d)
    kp = n(W.TENSOR_K_SELF, n_layers, prefix_len, hkv, d) if prefix_len else None
    vp = n(W.TENSOR_V_SELF, n_layers, prefix_len, hkv, d) if prefix_len else None
    return q, k, v, kp, vp


def _check(lens, n_layers, hq, hkv, d, dtype, prefix_len, scale=0.0, token_stride=None, seed=0, force_simt=False,
           sample=None):
    q, k, v, kp, vp = _inputs(seed, lens, n_layers, hq, hkv, d, dtype, prefix_len)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    total = int(off[-1])
    geom = cf.make_geom(hq, hkv, d, dtype, 4096, 1e4)
    dev = "cuda"
    qg = q.to(dev)
    if token_stride is None:
        kg, vg = k.to(dev), v.to(dev)
    else:
        kg, vg = harness.padded_store(k, token_stride, dev), harness.padded_store(v, token_stride, dev)
    out = torch.full_like(qg, float("nan"))
    lse = torch.full((n_layers, hq, total), float("nan"), device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    cf.cf_set_attn_path(1 if force_simt else 0)
    try:
        cf.cf_document_prefill_attn(geom, torch.from_numpy(off).to(dev), max(lens), qg, kg, vg, out,
                                    None if kp is None else kp.to(dev), None if vp is None else vp.to(dev), lse,
                                    softmax_scale=scale, token_stride=token_stride, status=status)
        torch.cuda.synchronize()
    finally:
        cf.cf_set_attn_path(0)
    assert int(status[0]) == 0
    o_got, l_got = out.float().cpu().numpy(), lse.cpu().numpy()
    tight = dtype == torch.float32
    assert not np.isnan(o_got).any() and not np.isnan(l_got).any()      # every row of every document was written
    for l in range(n_layers):
        for i, n_tok in enumerate(lens):
            if sample is not None and (l, i) not in sample:
                continue
            a, b = int(off[i]), int(off[i + 1])
            o_ref, lse_ref = oracle.document_prefill_attn(
                q[l, a:b].double().numpy(), k[l, a:b].double().numpy(), v[l, a:b].double().numpy(),
                None if kp is None else kp[l].double().numpy(), None if vp is None else vp[l].double().numpy(),
                scale if scale else None)
            err = np.abs(o_got[l, a:b] - o_ref)
            assert np.all(err <= (1e-4 if tight else 1e-2 + 2e-2 * np.abs(o_ref))), (l, i, float(err.max()))
            assert np.all(np.abs(l_got[l, :, a:b] - lse_ref) <= (1e-4 if tight else 1e-2)), (l, i)
    if token_stride is not None:
        assert bool(torch.all(harness.padding_of(kg, token_stride) == harness.PAD_SENTINEL))


@pytest.mark.parametrize("force_simt", [False, True])
@pytest.mark.parametrize("prefix_len", [0, 40, 64, 130, 160])
@pytest.mark.parametrize("heads", [(12, 2), (4, 4), (28, 4)])
def test_ragged_documents_bf16(heads, prefix_len, force_simt):
    """Documents of 1, 63, 64, 65, 129 and 200 tokens behind a shared prefix of 0, 40, 64, 130 or 160 tokens (a
    prefix of a whole number of 32-row copy boxes shares key tiles with the document, any other has tiles of its own);
    grouped-query (6 and 7 query heads per kv head: items of 126 rows) and multi-head geometry; both kernels of the library."""
    _check(RAGGED, 2, heads[0], heads[1], 128, torch.bfloat16, prefix_len, force_simt=force_simt)


@pytest.mark.parametrize("dtype,d", [(torch.float32, 64), (torch.float32, 128), (torch.bfloat16, 64)])
def test_ragged_documents_other_storage_types(dtype, d):
    _check(RAGGED, 1, 8, 2, d, dtype, 17)


def test_softmax_scale_and_padded_rows():
    _check([150, 33, 128], 2, 8, 2, 128, torch.bfloat16, 24, scale=0.2, token_stride=2 * 128 + 64)
    _check([150, 33, 128], 1, 8, 2, 64, torch.float32, 24, scale=0.05, token_stride=2 * 64 + 64)


def test_workload_shaped_batch():
    """Fifty passages of 128-192 tokens, Qwen2-1.5B head geometry (the documents of configs[2]), four layers."""
    cfg = W.CONFIGS[3]
    meta = W.make_meta(cfg, 0)
    _check([int(x) for x in meta.doc_len], 4, cfg.n_q_heads, cfg.n_kv_heads, 128, torch.bfloat16, 32, seed=3)


def test_empty_batch_and_argument_errors():
    geom = cf.make_geom(4, 2, 128, cf.CF_BF16, 4096, 1e4)
    z = torch.zeros((1, 0, 4, 128), dtype=torch.bfloat16, device="cuda")
    zk = torch.zeros((1, 0, 2, 128), dtype=torch.bfloat16, device="cuda")
    off = torch.zeros(1, dtype=torch.int32, device="cuda")
    cf.cf_document_prefill_attn(geom, off, 0, z, zk, zk, z)            # nothing to do is not an error
    q = torch.zeros((1, 8, 4, 128), dtype=torch.bfloat16, device="cuda")
    kk = torch.zeros((1, 8, 2, 128), dtype=torch.bfloat16, device="cuda")
    off = torch.tensor([0, 8], dtype=torch.int32, device="cuda")
    with pytest.raises(cf.CacheFocusError) as e:                       # a row stride shorter than a row
        cf.cf_document_prefill_attn(geom, off, 8, q, kk, kk, q, token_stride=128)
    assert e.value.code == cf.CF_ERR_INVALID_ARG
    shifted = torch.zeros(q.numel() + 8, dtype=torch.bfloat16, device="cuda")[1:q.numel() + 1].view(q.shape)
    with pytest.raises(cf.CacheFocusError) as e:                       # a query pointer off the 16-byte grid
        cf.cf_document_prefill_attn(geom, off, 8, shifted, kk, kk, q)
    assert e.value.code == cf.CF_ERR_INVALID_ARG
    with pytest.raises(cf.CacheFocusError) as e:                       # a prefix length without a prefix cache
        docs = cf.cf_doc_batch(1, 8, 4, 0, 8, 2 * 128, off.data_ptr())
        import ctypes
        rc = cf.load_library().cf_document_prefill_attn(ctypes.byref(geom), ctypes.byref(docs), 1, q.data_ptr(), 0,
                                                        kk.data_ptr(), kk.data_ptr(), 0, None, None, 0, 0.0,
                                                        q.data_ptr(), 0, None, None, None)
        raise cf.CacheFocusError(rc, "cf_document_prefill_attn")
    assert e.value.code == cf.CF_ERR_INVALID_ARG
    torch.cuda.synchronize()


def test_bench_sized_batch_sampled():
    """The batch bench.py times (400 passages of 128-192 tokens behind a 64-token prefix, 12/2 heads, four layers: each
    persistent CTA walks some ninety work items), a dozen (layer, document) pairs compared with the oracle, every
    output checked to have been written."""
    rng = np.random.default_rng(0)
    lens = [int(x) for x in rng.integers(128, 193, size=400)]
    picks = {(int(l), int(i)) for l, i in zip(rng.integers(0, 4, size=12), rng.integers(0, 400, size=12))}
    picks |= {(0, 0), (3, 399), (1, int(np.argmax(lens))), (2, int(np.argmin(lens)))}
    _check(lens, 4, 12, 2, 128, torch.bfloat16, 64, seed=4, sample=picks)
