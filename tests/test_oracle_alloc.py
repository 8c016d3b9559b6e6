"""Pins for the oracle's positional allocation (Eq. 6, Sec. 2.3.1, Sec. 2.5) and pruning (Algorithm 2, App. C)."""
import itertools
import math

import numpy as np
import pytest

import oracle
from oracle import ALLOC_ALIGN, ALLOC_NONE, ALLOC_SORT


def _check_invariants(doc_len, order, dst, group, n_reuse, qs, prefix_len, pos_range, tail_reserve):
    kept = list(order)
    # every kept document lies inside [prefix_len, qs); the query and its reserve fit the range
    for i in kept:
        assert prefix_len <= dst[i] and dst[i] + doc_len[i] <= qs
        assert 0 <= group[i] < n_reuse
    assert qs + tail_reserve <= pos_range
    for i in range(len(doc_len)):
        if i not in kept:
            assert dst[i] == -1 and group[i] == -1
    # inside a window: no overlap, no holes, the window ends at the query start
    for g in range(n_reuse):
        members = [i for i in kept if group[i] == g]
        spans = sorted((dst[i], dst[i] + doc_len[i]) for i in members)
        for (a0, a1), (b0, b1) in zip(spans, spans[1:]):
            assert a1 == b0
        if spans:
            assert spans[-1][1] == qs
        # earlier rank = closer to the query
        ranks = [kept.index(i) for i in sorted(members, key=lambda i: -dst[i])]
        assert ranks == sorted(ranks)
    sizes = [sum(1 for i in kept if group[i] == g) for g in range(n_reuse)]
    assert max(sizes) - min(sizes) <= 1


def test_eq6_closed_form():
    # ceil(k / floor(L / l_C))
    assert oracle.n_reuse_eq6(120, 4032, 200) == 6      # 20 caches per window, 120 caches
    assert oracle.n_reuse_eq6(20, 4064, 200) == 1
    assert oracle.n_reuse_eq6(8, 240, 32) == 2          # 7 per window
    assert oracle.n_reuse_eq6(21, 4000, 200) == 2
    assert oracle.n_reuse_eq6(1, 200, 200) == 1
    with pytest.raises(oracle.RangeError):
        oracle.n_reuse_eq6(3, 100, 101)
    for k, cap, lc in itertools.product([1, 7, 40, 100], [256, 4096, 32768], [32, 100, 200]):
        assert oracle.n_reuse_eq6(k, cap, lc) == math.ceil(k / math.floor(cap / lc))


def test_printed_example_k20(golden):
    # Sec. 3.3: k = 20, N_reuse = k/5 -> 5 windows in continuous positions, each position used 4 times.
    ex = golden("nreuse_example.txt")
    k, n_reuse = ex["k"], ex["n_reuse"]
    doc_len = [100] * k
    dst, group, used, qs = oracle.allocate_positions(doc_len, range(k), 4096, n_reuse=n_reuse)
    assert used == n_reuse
    per_group = [sum(1 for i in range(k) if group[i] == g) for g in range(n_reuse)]
    assert per_group == [ex["windows_in_continuous_positions"]] * n_reuse
    assert qs == 4096
    coverage = np.zeros(qs, dtype=int)
    for i in range(k):
        coverage[dst[i]:dst[i] + 100] += 1
    window = 100 * ex["windows_in_continuous_positions"]
    assert np.all(coverage[qs - window:] == ex["times_each_position_is_used"])
    assert np.all(coverage[:qs - window] == 0)
    _check_invariants(doc_len, list(range(k)), dst, group, used, qs, 0, 4096, 0)


def test_parallel_and_sequential_special_cases():
    doc_len = [30, 50, 20, 40]
    # N_reuse = k: every document is its own window, all end at the query (Sec. 3.3, first policy)
    dst, group, used, qs = oracle.allocate_positions(doc_len, [0, 1, 2, 3], 4096, n_reuse=4, query_start=50)
    assert qs == 50 and list(dst) == [20, 0, 30, 10] and sorted(group) == [0, 1, 2, 3]
    # N_reuse = 1: unique positions, one contiguous sequence ending at the query (second policy)
    dst, group, used, qs = oracle.allocate_positions(doc_len, [2, 0, 3, 1], 4096, n_reuse=1, query_start=140)
    assert qs == 140 and used == 1
    assert [int(dst[i]) for i in (1, 3, 0, 2)] == [0, 50, 90, 120]   # rank 0 (doc 2) next to the query


def test_small_case_worked_by_hand():
    # range 256, 16 query tokens reserved: capacity 240, l_C = 32 -> 7 per window -> 2 windows
    doc_len = [32] * 8
    dst, group, used, qs = oracle.allocate_positions(doc_len, range(8), 256, tail_reserve=16)
    assert used == 2 and qs == 240                     # the query closes the usable range
    assert list(group) == [0, 1, 0, 1, 0, 1, 0, 1]
    assert list(dst) == [208, 208, 176, 176, 144, 144, 112, 112]
    # default anchor: every window fits whatever subset survives a later pruning
    dst, group, used, qs = oracle.allocate_positions(doc_len, [0, 3, 5], 256, tail_reserve=16, query_start=240)
    assert used == 1 and [int(dst[i]) for i in (0, 3, 5)] == [208, 176, 144]


@pytest.mark.parametrize("seed", range(20))
def test_invariants_random(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 40))
    doc_len = rng.integers(1, 60, size=n)
    kept = list(rng.permutation(n)[: int(rng.integers(1, n + 1))])
    prefix = int(rng.integers(0, 20))
    tail = int(rng.integers(0, 30))
    pos_range = int(prefix + tail + doc_len.max() * rng.integers(1, 6) + rng.integers(0, 50))
    dst, group, used, qs = oracle.allocate_positions(doc_len, kept, pos_range, prefix, tail)
    lc = max(doc_len[i] for i in kept)
    assert used == math.ceil(len(kept) / ((pos_range - prefix - tail) // lc))
    _check_invariants(doc_len, kept, dst, group, used, qs, prefix, pos_range, tail)
    # a later call with the query start fixed and fewer documents still ends every window at the query
    fewer = kept[: max(1, len(kept) // 2)]
    dst2, group2, used2, qs2 = oracle.allocate_positions(doc_len, fewer, pos_range, prefix, tail, 0, qs)
    assert qs2 == qs
    _check_invariants(doc_len, fewer, dst2, group2, used2, qs, prefix, pos_range, tail)


def test_range_errors():
    with pytest.raises(oracle.RangeError):
        oracle.allocate_positions([300], [0], 256)
    with pytest.raises(oracle.RangeError):          # forced single window that overflows the range
        oracle.allocate_positions([100] * 5, range(5), 256, n_reuse=1)
    with pytest.raises(oracle.RangeError):          # query start beyond the range
        oracle.allocate_positions([10], [0], 256, tail_reserve=16, query_start=250)
    with pytest.raises(oracle.RangeError):          # fixed query start too small for the window
        oracle.allocate_positions([100, 100], [0, 1], 4096, n_reuse=1, query_start=150)
    with pytest.raises(ValueError):
        oracle.allocate_positions([10, 10], [0, 0], 256)


def test_prune_against_brute_force():
    rng = np.random.default_rng(0)
    for _ in range(50):
        n = int(rng.integers(2, 12))
        scores = rng.integers(0, 5, size=n).astype(float)          # many exact ties
        order = list(rng.permutation(n)[: int(rng.integers(1, n + 1))])
        keep = int(rng.integers(1, len(order) + 1))
        # brute force: repeatedly remove the worst (lowest score; among equals the higher id)
        alive = list(order)
        while len(alive) > keep:
            worst = max(alive, key=lambda i: (-scores[i], i))
            alive.remove(worst)
        got_align = oracle.prune_topk(scores, order, keep, ALLOC_ALIGN)
        got_none = oracle.prune_topk(scores, order, keep, ALLOC_NONE)
        got_sort = oracle.prune_topk(scores, order, keep, ALLOC_SORT)
        assert got_align == alive == got_none                       # previous order kept
        assert sorted(got_sort) == sorted(alive)
        keys = [(-scores[i], i) for i in got_sort]
        assert keys == sorted(keys)                                  # best first, ties by id


def test_prune_tie_goes_to_lower_id():
    assert oracle.prune_topk([1.0, 2.0, 2.0, 2.0], [3, 2, 1, 0], 2, ALLOC_ALIGN) == [2, 1]
    assert oracle.prune_topk([1.0, 2.0, 2.0, 2.0], [3, 2, 1, 0], 2, ALLOC_SORT) == [1, 2]


def test_printed_schedule_example(golden):
    ex = golden("kprune_example.txt")
    sched = oracle.prune_schedule_linear(ex["n_layers"], ex["every"], ex["k"], ex["k_finish"])
    layers = [l for l, _ in sched]
    keeps = [k for _, k in sched]
    assert layers == [4, 8, 12, 16, 20, 24, 28]                     # l mod n = 0, l from 1
    removed = [a - b for a, b in zip([ex["k"]] + keeps, keeps)]
    assert removed == [ex["k_prune"]] * 7
    assert keeps[-1] == ex["k_finish"]


def test_schedule_remainder_goes_to_last_layer():
    sched = oracle.prune_schedule_linear(28, 4, 50, 5)              # 45 / 7 = 6 remainder 3
    keeps = [k for _, k in sched]
    assert keeps == [44, 38, 32, 26, 20, 14, 5]
    assert oracle.prune_schedule_linear(3, 4, 50, 5) == []
