"""Pins for the router-head oracle (Eq. 2 and matrix folding): group sums written out, library argsort / softmax,
invariants of a binary fold, a hand-worked token, bfloat16 rounding against torch."""
import numpy as np
import pytest
import torch
from scipy.special import softmax as scipy_softmax

from oracle import router_oracle as ro
from paper_2603_06626_b200 import synth


def _rand(seed, T=37, dh=24, E_S=12, E_T=5):
    rng = np.random.default_rng(seed)
    H = rng.standard_normal((T, dh))
    W = rng.standard_normal((E_S, dh))
    fm = rng.integers(0, E_T, size=E_S).astype(np.int32)
    return H, W, fm


def test_fold_matrix_is_binary_with_one_target_per_source():
    fm = np.array([2, 0, 2, 1, 0], dtype=np.int32)
    M = ro.fold_matrix(fm, 3)
    assert set(np.unique(M)) <= {0.0, 1.0} and np.array_equal(M.sum(axis=1), np.ones(5))
    assert np.array_equal(M.argmax(axis=1), fm)
    with pytest.raises(ValueError):
        ro.fold_matrix(np.array([0, 3]), 3)


def test_folded_layer_sums_the_source_rows_of_each_group():
    H, W, fm = _rand(1)
    Wf = ro.folded_score_layer(W, fm, 5)
    for j in range(5):                                   # W~_s column j = sum of the W_s columns mapped to j
        want = np.zeros(W.shape[1])
        for i in range(W.shape[0]):
            if fm[i] == j:
                want += W[i]
        assert np.allclose(Wf[j], want, rtol=0, atol=1e-14)
    # folded scores = source scores summed per group (linearity): logits are folded BEFORE top-k
    S_src = H @ W.T
    S = ro.scores(H, W, fm, 5)
    for j in range(5):
        assert np.allclose(S[:, j], S_src[:, fm == j].sum(axis=1), atol=1e-12)
    # identity fold and no fold agree
    assert np.array_equal(ro.scores(H, W, np.arange(12, dtype=np.int32), 12), ro.scores(H, W, None, 12))


def test_top_k_against_library_sort_and_tie_break():
    rng = np.random.default_rng(2)
    S = rng.standard_normal((50, 17))
    for k in (1, 4, 17):
        want = np.argsort(-S, axis=1, kind="stable")[:, :k]
        assert np.array_equal(ro.top_k(S, k), want)
    S = np.array([[1.0, 3.0, 3.0, 0.5, 3.0]])
    assert ro.top_k(S, 3).tolist() == [[1, 2, 4]]       # equal scores: lower id first
    ids = ro.top_k(rng.standard_normal((20, 9)), 4)
    assert all(len(set(r)) == 4 for r in ids.tolist())   # a token never picks one expert twice


def test_normalisation_against_library_and_closed_forms():
    rng = np.random.default_rng(3)
    kept = rng.standard_normal((30, 6)) * 3
    r = ro.normalise(kept, ro.SOFTMAX)
    assert np.allclose(r, scipy_softmax(kept, axis=1), atol=1e-15) and np.allclose(r.sum(axis=1), 1.0)
    assert np.allclose(ro.normalise(kept + 100.0, ro.SOFTMAX), r, atol=1e-13)          # shift invariance
    s = ro.normalise(kept, ro.SIGMOID)
    assert np.allclose(s, torch.sigmoid(torch.from_numpy(kept)).numpy(), atol=1e-15)
    assert np.allclose(s + ro.normalise(-kept, ro.SIGMOID), 1.0)


def test_hand_worked_token():
    # h = [1, -1]; W_s rows: e0 [2,0] e1 [0,1] e2 [1,1] e3 [0,-3]; fold 0,1 -> 0 ; 2 -> 1 ; 3 -> 2
    H = np.array([[1.0, -1.0]])
    W = np.array([[2.0, 0.0], [0.0, 1.0], [1.0, 1.0], [0.0, -3.0]])
    fm = np.array([0, 0, 1, 2], dtype=np.int32)
    ids, r, S = ro.route(H, W, fm, 3, 2, ro.SOFTMAX)
    assert S.tolist() == [[1.0, 0.0, 3.0]]               # source scores 2, -1, 0, 3 ; folded 2-1, 0, 3
    assert ids.tolist() == [[2, 0]]
    e2 = np.exp(-2.0)                                    # softmax over (3, 1): 1/(1+e^-2), e^-2/(1+e^-2)
    assert np.allclose(r, [[1 / (1 + e2), e2 / (1 + e2)]], atol=1e-15)
    _, rs, _ = ro.route(H, W, fm, 3, 2, ro.SIGMOID)
    assert np.allclose(rs, [[1 / (1 + np.exp(-3.0)), 1 / (1 + np.exp(-1.0))]], atol=1e-15)


def test_routing_is_invariant_to_relabelling_the_source_experts():
    H, W, fm = _rand(4)
    perm = np.random.default_rng(5).permutation(12)
    ids1, r1, _ = ro.route(H, W, fm, 5, 3)
    ids2, r2, _ = ro.route(H, W[perm], fm[perm], 5, 3)
    assert np.array_equal(ids1, ids2) and np.allclose(r1, r2, atol=1e-13)


def test_bf16_rounding_and_cache_record():
    rng = np.random.default_rng(6)
    a = np.concatenate([rng.random(5000), [0.0, 1.0, 0.5, 2.0 ** -9 + 2.0 ** -17, 1 - 2.0 ** -9]])
    got = ro.to_bf16_bits(a)
    # float32 values: torch's float32 -> bfloat16 conversion is round-to-nearest-even
    a32 = a.astype(np.float32)
    want = torch.from_numpy(a32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ro.to_bf16_bits(a32.astype(np.float64)), want)
    assert np.array_equal(ro.to_bf16_bits(a32.astype(np.float64)), synth.f32_to_bf16_bits(a32))
    # exact ties go to the even neighbour; float64 inputs are rounded once, not via float32
    assert ro.to_bf16_bits(np.array([1.0 + 2.0 ** -8]))[0] == 0x3F80 and ro.to_bf16_bits(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 0x3F82
    assert ro.to_bf16_bits(np.array([1.0 + 2.0 ** -8 + 2.0 ** -40]))[0] == 0x3F81   # float32 would see an exact tie here
    err = np.abs(synth.bf16_bits_to_f64(got) - a)
    assert np.all(err <= np.maximum(a, 1e-30) * 2.0 ** -8)
    ids, bits = ro.pack_cache(np.array([[3, 255]]), np.array([[0.25, 0.75]]))
    assert ids.dtype == np.uint8 and bits.dtype == np.uint16 and ids.nbytes + bits.nbytes == 3 * 2   # 3k bytes per token
