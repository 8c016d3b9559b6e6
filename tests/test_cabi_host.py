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
    header = open(os.path.join(ROOT, "include", "cachefocus.h")).read()
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
        # with a query-self block: one more part per row (reference, sum, fp32 row) at most
        full = cf.cf_attn_workspace_bytes_full(geom, batch, n_layers)
        assert need < full <= need + n_layers * rows * 4 * (128 + 2) + 3 * 256
    assert cf.cf_attn_workspace_bytes_full(geom, batch, 0) == 0
    assert cf.cf_attn_workspace_bytes_layers(geom, batch, 0) == 0
    assert cf.cf_attn_workspace_bytes_layers(geom, batch, cf.CF_MAX_LAYERS_PER_CALL + 1) == 0
