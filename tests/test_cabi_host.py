"""Host-side checks that need no GPU: the library loads, exports every declared symbol, and its
integer steps agree bit for bit with the oracle."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2502_11101_b200 as cf
from paper_2502_11101_b200 import build as cf_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    cf_build.build()
    return cf.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = "".join(open(os.path.join(ROOT, "include", name)).read()
                     for name in sorted(os.listdir(os.path.join(ROOT, "include"))) if name.endswith(".h"))
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(cf_[a-z_0-9]+)\s*\(", header))
    assert declared == set(cf.EXPORTS), declared ^ set(cf.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_struct_sizes_match_the_header(lib):
    assert ctypes.sizeof(cf.cf_geom) == 32
    assert ctypes.sizeof(cf.cf_batch) == 72
    assert ctypes.sizeof(cf.cf_plan_layout) == 16 * 8 + 8
    assert cf.cf_error_string(cf.CF_ERR_RANGE).startswith("kept documents")


def _geom(pos_range):
    return cf.make_geom(4, 2, 64, cf.CF_BF16, pos_range, 1e4)


@pytest.mark.parametrize("seed", range(30))
def test_allocation_matches_oracle(lib, seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 60))
    doc_len = rng.integers(1, 200, size=n)
    order = list(rng.permutation(n)[: int(rng.integers(1, n + 1))])
    prefix, tail = int(rng.integers(0, 40)), int(rng.integers(0, 64))
    pos_range = int(prefix + tail + doc_len.max() * rng.integers(1, 8) + rng.integers(0, 100))
    n_reuse = int(rng.choice([0, 0, 1, 2, 5, len(order)]))
    qs_arg = -1 if rng.random() < 0.7 else pos_range - tail - int(rng.integers(0, 20))
    try:
        ref = oracle.allocate_positions(doc_len, order, pos_range, prefix, tail, n_reuse, qs_arg)
    except oracle.RangeError:
        with pytest.raises(cf.CacheFocusError) as e:
            cf.cf_allocate_positions(_geom(pos_range), doc_len, order, prefix, tail, n_reuse, qs_arg)
        assert e.value.code == cf.CF_ERR_RANGE
        return
    dst, grp, used, qs = cf.cf_allocate_positions(_geom(pos_range), doc_len, order, prefix, tail, n_reuse, qs_arg)
    assert np.array_equal(dst, ref[0]) and np.array_equal(grp, ref[1]) and used == ref[2] and qs == ref[3]


def test_allocation_rejects_bad_input(lib):
    g = _geom(256)
    for bad in ([0, 0], [0, 5], [-1]):
        with pytest.raises(cf.CacheFocusError) as e:
            cf.cf_allocate_positions(g, [10, 10], bad)
        assert e.value.code == cf.CF_ERR_INVALID_ARG
    with pytest.raises(cf.CacheFocusError) as e:
        cf.cf_allocate_positions(g, [300], [0])
    assert e.value.code == cf.CF_ERR_RANGE
    dst, grp, used, qs = cf.cf_allocate_positions(g, [10, 10], [], tail_reserve=16)
    assert list(dst) == [-1, -1] and qs == 240


def test_schedule_matches_oracle_and_printed_example(lib, golden):
    ex = golden("kprune_example.txt")
    sched = cf.cf_schedule_linear(ex["n_layers"], ex["every"], ex["k"], ex["k_finish"])
    assert sched == oracle.prune_schedule_linear(28, 4, 40, 5)
    assert [k for _, k in sched] == [35, 30, 25, 20, 15, 10, 5]
    for L, n, k, kf in [(28, 4, 50, 5), (32, 4, 120, 15), (3, 4, 10, 2), (28, 7, 33, 4)]:
        assert cf.cf_schedule_linear(L, n, k, kf) == oracle.prune_schedule_linear(L, n, k, kf)


def test_workspace_size_of_layer_batched_calls(lib):
    """Host arithmetic only: the descriptor's device pointers are never dereferenced by these calls."""
    geom = cf.make_geom(12, 2, 128, cf.CF_BF16, 32768, 1e6)
    fake = 256                                            # any non-null address
    batch = cf.cf_batch(1, 50, 48, 0, 48, 0, 0, 0, 8000, 2 * 128, fake, fake, fake)
    one = cf.cf_attn_workspace_bytes(geom, batch)
    assert one > 0 and one == cf.cf_attn_workspace_bytes_layers(geom, batch, 1)
    for n_layers in (2, 8, cf.CF_MAX_LAYERS_PER_CALL):
        need = cf.cf_attn_workspace_bytes_layers(geom, batch, n_layers)
        assert need > 0 and need % 256 == 0
        # per layer: the merged log-sum-exp of every row and one value per (tile slot, row)
        rows, tile_slots = 12 * 48, 50 + 8000 // 128 + 1
        assert need >= n_layers * 4 * (rows + tile_slots * rows)
        # with further key blocks: one more part per row (reference, sum, fp32 row) and one more sum per part and row
        full = cf.cf_attn_workspace_bytes_full(geom, batch, n_layers)
        assert need < full <= need + n_layers * rows * 4 * (128 + 2 + cf.CF_MAX_SPLITS) + 4 * 256
    assert cf.cf_attn_workspace_bytes_full(geom, batch, 0) == 0
    assert cf.cf_attn_workspace_bytes_layers(geom, batch, 0) == 0
    assert cf.cf_attn_workspace_bytes_layers(geom, batch, cf.CF_MAX_LAYERS_PER_CALL + 1) == 0


@pytest.mark.parametrize("seed", range(20))
def test_host_pruning_step_matches_oracle(lib, seed):
    """cf_prune_topk_host against the oracle's prune_topk: kept set and order bit-exact, ties included."""
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(1, 80))
    n_kept = int(rng.integers(1, n + 1))
    order = [int(i) for i in rng.permutation(n)[:n_kept]]
    # scores drawn from a handful of float32 values so that ties are common
    scores = rng.choice(np.array([0.0, 0.125, 0.25, 0.3, 0.7, 1.5], dtype=np.float32), size=n).astype(np.float32)
    if seed % 3 == 0:
        scores = rng.random(n).astype(np.float32)
    for strategy in (oracle.ALLOC_NONE, oracle.ALLOC_ALIGN, oracle.ALLOC_SORT):
        for keep in (0, 1, n_kept // 2, n_kept, n_kept + 3):
            want = oracle.prune_topk(scores, order, keep, strategy)
            assert cf.cf_prune_topk_host(scores, order, keep, strategy) == want


def test_host_pruning_step_rejects_bad_input(lib):
    for bad in ([0, 0], [3], [-1]):
        with pytest.raises(cf.CacheFocusError) as e:
            cf.cf_prune_topk_host([0.1, 0.2, 0.3], bad, 1, oracle.ALLOC_ALIGN)
        assert e.value.code == cf.CF_ERR_INVALID_ARG
    with pytest.raises(cf.CacheFocusError):
        cf.cf_prune_topk_host([0.1, 0.2], [0, 1], 1, 7)
    assert cf.cf_prune_topk_host([], [], 3, oracle.ALLOC_SORT) == []


def test_stack_driver_checks_its_arguments_on_the_host(lib):
    """cf_run_stack and its workspace query through ctypes; every case returns before anything is launched
    (the device pointers of the descriptors are never dereferenced)."""
    geom = cf.make_geom(12, 2, 128, cf.CF_BF16, 32768, 1e6)
    fake = 256
    batch = cf.cf_batch(1, 50, 48, 0, 48, 0, 0, 0, 8000, 2 * 128, fake, fake, fake)

    def stack(layers, keeps, n_layers=28, strategy=cf.CF_ALLOC_ALIGN, batch_layers=1, q=fake):
        la, ke = np.asarray(layers, np.int32), np.asarray(keeps, np.int32)
        st = cf.cf_stack(n_layers, len(la), la.ctypes.data if len(la) else None, ke.ctypes.data if len(ke) else None,
                         strategy, batch_layers, 0.0, 0, q, 1 << 20, fake, fake, 1 << 22, None, None, 0, fake, 1 << 20,
                         None, None, fake, None, None, None)
        return st, (la, ke)

    good, keep = stack([4, 12, 20], [25, 12, 6])
    per_call = [cf.cf_attn_workspace_bytes_layers(geom, batch, m) for m in (4, 8)]
    assert cf.cf_run_stack_workspace_bytes(geom, batch, good) == max(per_call) > 0
    one_by_one, keep2 = stack([4, 12, 20], [25, 12, 6], batch_layers=0)
    # one call per layer: partial results of one layer, the scores of up to eight layers waiting in slots
    assert cf.cf_run_stack_workspace_bytes(geom, batch, one_by_one) == cf.cf_attn_workspace_bytes_slots(geom, batch, 8)
    # document lengths on the host let the call shrink its grids to the documents still kept
    lens = np.full(50, 160, np.int32)
    begin = np.array([0, 50], np.int32)
    hinted, keep3 = stack([4, 12, 20], [25, 12, 6])
    hinted.doc_len_host, hinted.req_doc_begin_host = lens.ctypes.data, begin.ctypes.data
    assert 0 < cf.cf_run_stack_workspace_bytes(geom, batch, hinted) <= max(per_call)
    for st, _ in (stack([4, 4], [25, 12]), stack([12, 4], [25, 12]), stack([0], [5]), stack([4], [-1]),
                  stack([4], [5], n_layers=0), stack([4], [5], strategy=9)):
        assert cf.cf_run_stack_workspace_bytes(geom, batch, st) == 0
        rc = lib.cf_run_stack(ctypes.byref(geom), ctypes.byref(batch), ctypes.byref(st), fake, 1 << 20, fake, 1 << 20, None)
        assert rc == cf.CF_ERR_INVALID_ARG
    null_q, _ = stack([4], [5], q=None)
    assert lib.cf_run_stack(ctypes.byref(geom), ctypes.byref(batch), ctypes.byref(null_q), fake, 1 << 20, fake,
                            1 << 20, None) == cf.CF_ERR_INVALID_ARG
    assert lib.cf_debug_wait_timeout(ctypes.byref(geom), ctypes.byref(batch), fake, 0, None) == cf.CF_ERR_INVALID_ARG
    assert lib.cf_debug_wait_timeout(ctypes.byref(geom), ctypes.byref(batch), fake + 8, 1000, None) == cf.CF_ERR_WORKSPACE


def test_decoding_calls_check_their_arguments_on_the_host(lib):
    """Sizes are host arithmetic; every failing case returns before anything is launched."""
    geom = cf.make_geom(28, 4, 128, cf.CF_BF16, 32768, 1e6)
    fake = 256
    need = cf.cf_decode_plan_bytes(geom, 4, 16064)
    assert need > 0 and need % 256 == 0
    assert cf.cf_decode_plan_bytes(geom, 8, 16064) > need                  # grows with the batch
    assert cf.cf_decode_plan_bytes(geom, 0, 16064) == 0 and cf.cf_decode_plan_bytes(geom, 4, 0) == 0
    one, eight = cf.cf_decode_workspace_bytes(geom, 4, 16064, 1), cf.cf_decode_workspace_bytes(geom, 4, 16064, 8)
    assert 0 < one < eight and cf.cf_decode_workspace_bytes(geom, 4, 16064, 0) == 0
    g = ctypes.byref(geom)
    assert lib.cf_decode_plan(g, 4, 16064, None, 1, fake, need, None) == cf.CF_ERR_INVALID_ARG          # no row counts
    assert lib.cf_decode_plan(g, 4, 16064, fake, 1, fake + 8, need, None) == cf.CF_ERR_WORKSPACE        # misaligned
    assert lib.cf_decode_plan(g, 4, 16064, fake, 1, fake, need - 1, None) == cf.CF_ERR_WORKSPACE        # too small
    assert lib.cf_decode_plan(g, 1 << 21, 16064, fake, 1, fake, need, None) == cf.CF_ERR_INVALID_ARG    # batch too large
    assert lib.cf_decode_attn(g, 4, 16064, None, 1, fake, 0, fake, fake, 0, 0.0, fake, 0, None, fake, 1 << 20,
                              None) == cf.CF_ERR_INVALID_ARG
    assert lib.cf_decode_append(g, 4, 16064, 1, fake, fake, 0, fake, -1, fake, fake, 0, None, None) == cf.CF_ERR_INVALID_ARG
    assert lib.cf_decode_append(g, 4, 16064, 1, fake + 2, fake, 0, fake, 0, fake, fake, 0, None, None) == cf.CF_ERR_INVALID_ARG
    assert lib.cf_decode_append(g, 4, 16064, 2, fake, fake, 8, fake, 0, fake, fake, 8, None, None) == cf.CF_ERR_INVALID_ARG


def test_prefix_call_checks_its_arguments_on_the_host(lib):
    geom = cf.make_geom(12, 2, 128, cf.CF_BF16, 32768, 1e6)
    fake = 256
    batch = cf.cf_batch(1, 50, 48, 64, 48, 0, 0, 0, 8000, 2 * 128, fake, fake, fake)          # 64 positions reserved
    g, b = ctypes.byref(geom), ctypes.byref(batch)
    ws = cf.cf_attn_workspace_bytes_full(geom, batch, 1)

    def call(prefix_len=64, k_prefix=fake, v_prefix=fake, k_self=None, v_self=None):
        return lib.cf_query_prefill_attn_prefix(g, b, fake, 1, fake, 0, fake, fake, 0, k_prefix, v_prefix, 0, prefix_len,
                                                k_self, v_self, 0, 0.0, fake, 0, None, None, None, fake, ws, None)

    assert call(prefix_len=0) == cf.CF_ERR_INVALID_ARG
    assert call(k_prefix=None) == cf.CF_ERR_INVALID_ARG
    assert call(prefix_len=65) == cf.CF_ERR_INVALID_ARG                     # beyond the positions kept clear of documents
    assert call(k_self=fake) == cf.CF_ERR_INVALID_ARG                       # keys of the query tokens without their values


def test_deferred_score_calls_check_their_arguments_on_the_host(lib):
    geom = cf.make_geom(12, 2, 128, cf.CF_BF16, 32768, 1e6)
    fake = 256
    batch = cf.cf_batch(1, 50, 48, 0, 48, 0, 0, 0, 8000, 2 * 128, fake, fake, fake)
    g, b = ctypes.byref(geom), ctypes.byref(batch)
    one, eight = cf.cf_attn_workspace_bytes_slots(geom, batch, 1), cf.cf_attn_workspace_bytes_slots(geom, batch, 8)
    assert cf.cf_attn_workspace_bytes(geom, batch) == one < eight                  # partial results of one layer only
    assert cf.cf_attn_workspace_bytes_slots(geom, batch, 0) == 0 and cf.cf_attn_workspace_bytes_slots(geom, batch, 65) == 0
    slot = lambda s, n, bytes_=eight: lib.cf_query_prefill_attn_slot(g, b, fake, s, n, fake, fake, fake, 0.0, fake, None,
                                                                      fake, bytes_, None)
    assert slot(-1, 8) == cf.CF_ERR_INVALID_ARG and slot(8, 8) == cf.CF_ERR_INVALID_ARG and slot(0, 0) == cf.CF_ERR_INVALID_ARG
    assert slot(0, 8, eight - 1) == cf.CF_ERR_WORKSPACE
    acc = lambda f, n, bytes_=eight: lib.cf_accumulate_scores(g, b, fake, f, n, None, fake, fake, bytes_, None)
    assert acc(0, 8) == cf.CF_ERR_INVALID_ARG and acc(9, 8) == cf.CF_ERR_INVALID_ARG and acc(1, 65) == cf.CF_ERR_INVALID_ARG
    assert acc(8, 8, eight - 1) == cf.CF_ERR_WORKSPACE


def test_slot_call_with_further_key_blocks_checks_its_arguments_on_the_host(lib):
    geom = cf.make_geom(12, 2, 128, cf.CF_BF16, 32768, 1e6)
    fake = 256
    batch = cf.cf_batch(1, 50, 48, 64, 48, 0, 0, 0, 8000, 2 * 128, fake, fake, fake)          # 64 positions kept for a prefix
    g, b = ctypes.byref(geom), ctypes.byref(batch)
    plain, full = cf.cf_attn_workspace_bytes_slots(geom, batch, 4), cf.cf_attn_workspace_bytes_slots_full(geom, batch, 4)
    assert 0 < plain < full and cf.cf_attn_workspace_bytes_slots_full(geom, batch, 0) == 0

    def call(slot=0, n_slots=4, k_prefix=fake, prefix_len=64, k_self=fake, v_self=fake, nbytes=full):
        return lib.cf_query_prefill_attn_slot_full(g, b, fake, slot, n_slots, fake, fake, fake, k_prefix, fake, prefix_len,
                                                   k_self, v_self, 0.0, fake, None, fake, nbytes, None)

    assert call(prefix_len=0, k_self=None, v_self=None) == cf.CF_ERR_INVALID_ARG      # neither block: the plain slot call
    assert call(v_self=None) == cf.CF_ERR_INVALID_ARG                                 # keys of the query tokens without values
    assert call(prefix_len=65) == cf.CF_ERR_INVALID_ARG                               # beyond the positions kept clear
    assert call(k_prefix=None) == cf.CF_ERR_INVALID_ARG
    assert call(slot=4) == cf.CF_ERR_INVALID_ARG and call(prefix_len=-1) == cf.CF_ERR_INVALID_ARG
    assert call(nbytes=full - 1) == cf.CF_ERR_WORKSPACE
