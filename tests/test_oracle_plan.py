"""Pins for the oracle's routing plan: invariants, a library stable sort, brute force."""
import os

import numpy as np
import pytest

from oracle import grouter_oracle as orc
from paper_2603_06626_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _check_invariants(idx, fold_map, E_tgt, counts, offsets, row_to_slot, slot_to_row):
    R = idx.size
    e = idx.astype(np.int64).ravel()
    if fold_map is not None:
        e = fold_map.astype(np.int64)[e]
    assert counts.sum() == R
    assert offsets[0] == 0 and offsets[-1] == R
    assert np.all(np.diff(offsets) == counts)
    # bijection, mutual inverses
    assert np.array_equal(np.sort(slot_to_row), np.arange(R))
    assert np.array_equal(row_to_slot[slot_to_row], np.arange(R))
    # rows are grouped by expert in ascending order, and each group is the expert's segment
    e_rows = e[row_to_slot]
    assert np.all(np.diff(e_rows) >= 0)
    for x in range(E_tgt):
        seg = row_to_slot[offsets[x]:offsets[x + 1]]
        assert np.all(e[seg] == x)
        assert np.all(np.diff(seg) > 0)          # stability: slot order kept inside an expert


@pytest.mark.parametrize("name", ["tiny", "small", "fine_fold", "skewed"])
def test_plan_matches_library_stable_sort(name):
    w = synth.WORKLOADS[name]
    idx = synth.make_idx(w)
    fm = synth.make_fold_map(w)
    counts, offsets, r2s, s2r = orc.plan(idx, fm, w.E_tgt)
    _check_invariants(idx, fm, w.E_tgt, counts, offsets, r2s, s2r)
    e = idx.astype(np.int64).ravel()
    if fm is not None:
        e = fm.astype(np.int64)[e]
    order = np.argsort(e, kind="stable")
    assert np.array_equal(r2s, order.astype(np.int32))
    assert np.array_equal(counts, np.bincount(e, minlength=w.E_tgt))
    assert np.array_equal(offsets[1:], np.cumsum(np.bincount(e, minlength=w.E_tgt)))
    if name == "skewed":
        assert (counts == 0).sum() == 4           # the recipe's four unrouted experts
    if name == "fine_fold":
        # each target expert folds exactly floor(E_S/E_T) = 4 sources (section "Expert Folding")
        assert np.all(np.bincount(fm, minlength=16) == 4)


def test_plan_bruteforce_rank_tiny():
    rng = np.random.default_rng(7)
    for T, k, E in [(1, 1, 1), (5, 2, 3), (17, 3, 4), (33, 1, 2), (40, 4, 7)]:
        idx = rng.integers(0, E, size=(T, k)).astype(np.uint8)
        counts, offsets, r2s, s2r = orc.plan(idx, None, E)
        e = idx.ravel().astype(int)
        R = T * k
        for s in range(R):
            smaller = sum(1 for s2 in range(R) if e[s2] < e[s])
            earlier_same = sum(1 for s2 in range(s) if e[s2] == e[s])
            assert s2r[s] == smaller + earlier_same
        _check_invariants(idx, None, E, counts, offsets, r2s, s2r)


def test_plan_identity_fold_is_no_fold():
    w = synth.WORKLOADS["tiny"]
    idx = synth.make_idx(w)
    a = orc.plan(idx, None, w.E_tgt)
    b = orc.plan(idx, np.arange(w.E_src, dtype=np.int32), w.E_tgt)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


def test_plan_degenerate_cases():
    # all slots on one expert; E=1; empty experts
    idx = np.full((9, 2), 3, dtype=np.uint8)
    counts, offsets, r2s, s2r = orc.plan(idx, None, 5)
    assert counts.tolist() == [0, 0, 0, 18, 0]
    assert offsets.tolist() == [0, 0, 0, 0, 18, 18]
    assert np.array_equal(s2r, np.arange(18)) and np.array_equal(r2s, np.arange(18))
    counts, offsets, r2s, s2r = orc.plan(np.zeros((4, 1), dtype=np.int32), None, 1)
    assert counts.tolist() == [4] and offsets.tolist() == [0, 4]
    # fold collisions: a token may own several rows of one target expert
    idx = np.array([[0, 2], [1, 3]], dtype=np.uint8)
    fm = np.array([0, 1, 0, 1], dtype=np.int32)
    counts, offsets, r2s, s2r = orc.plan(idx, fm, 2)
    assert counts.tolist() == [2, 2]
    assert r2s.tolist() == [0, 1, 2, 3]
    with pytest.raises(ValueError):
        orc.plan(np.array([[5]], dtype=np.uint8), None, 4)


def test_cache_format_bytes_per_token():
    """uint8 id + bf16 score per active expert: k*3 bytes per token (24 at k=8)."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "cache_format.txt")) if l.strip() and not l.startswith("#")]
    for k, nbytes in rows:
        k, nbytes = int(k), int(nbytes)
        w = synth.custom_workload("c", T=16, d=8, ffn=8, E=max(8, k), k=k)
        idx, gates = synth.make_idx(w), synth.make_gates(w)
        assert idx.dtype == np.uint8 and gates.dtype == np.uint16
        assert (idx.nbytes + gates.nbytes) // w.T == nbytes
