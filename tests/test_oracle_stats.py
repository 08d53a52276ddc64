"""Pins for the routing-statistics oracle: matrix identities, library routines, brute force and hand-worked cases."""
import itertools

import numpy as np
import pytest

from oracle import stats_oracle as so


def _idx(seed, T=240, E=12, k=3):
    rng = np.random.default_rng(seed)
    return np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.uint8)


def test_coactivation_is_a_gram_matrix_of_the_activation_vectors():
    idx = _idx(0)
    a = so.activation(idx, 12)
    P = so.coactivation(idx, 12)
    assert np.array_equal(P, a.T @ a)                            # sum_t a_t a_t^T with a library matmul
    assert np.array_equal(P, P.T) and np.array_equal(np.diag(P), so.loads(idx, 12))
    assert P.sum() == idx.shape[0] * 3 * 3                       # k*k ordered pairs per token
    assert np.array_equal(so.loads(idx, 12), np.bincount(idx.ravel().astype(np.int64), minlength=12))
    # brute force over pairs
    for i, j in itertools.combinations(range(12), 2):
        assert P[i, j] == sum(1 for row in idx.tolist() if i in row and j in row)
    # a repeated id activates its expert once
    assert so.coactivation(np.array([[2, 2, 5]]), 6)[2, 2] == 1 and so.coactivation(np.array([[2, 2, 5]]), 6)[2, 5] == 1


def test_affinity_vectors_and_maxvio():
    idx = _idx(1, T=200, E=10, k=2)
    phi = so.affinity_vectors(idx, 10, 50)
    assert phi.shape == (4, 10) and np.allclose(phi.sum(axis=1), 2.0)            # k experts per token
    assert np.allclose(phi.mean(axis=0) * 200, so.loads(idx, 10))                  # samples of equal length average to the global load
    one = np.tile(np.array([[3, 7]]), (50, 1))
    assert so.affinity_vectors(one, 10, 50).tolist() == [[0, 0, 0, 1.0, 0, 0, 0, 1.0, 0, 0]]
    assert so.max_vio(np.array([5, 5, 5, 5])) == 0.0
    assert so.max_vio(np.array([8, 0, 0, 0])) == 3.0             # (8 - 2) / 2
    with pytest.raises(ValueError):
        so.affinity_vectors(idx, 10, 7)


def test_greedy_fold_group_sizes_and_hand_example():
    # 5 sources, 2 targets: sizes 3 and 2.  Affinities make 0-3-4 one group and 1-2 the other.
    P = np.zeros((5, 5), dtype=np.int64)
    for (i, j), v in {(0, 3): 9, (0, 4): 1, (3, 4): 8, (1, 2): 7, (0, 1): 2, (0, 2): 0}.items():
        P[i, j] = P[j, i] = v
    fold = so.greedy_fold(P, 2)
    # seed 0; best partner 3 (9); then 4: P[0,4]+P[3,4] = 9 beats 1: 2 and 2: 0.  Second group: seed 1, partner 2.
    assert fold.tolist() == [0, 1, 1, 0, 0]
    rng = np.random.default_rng(3)
    A = rng.integers(0, 50, size=(23, 23))
    P = A + A.T
    for E_T in (1, 4, 5, 23):
        f = so.greedy_fold(P, E_T)
        sizes = np.bincount(f, minlength=E_T)
        assert f.min() == 0 and f.max() == E_T - 1                 # a total map onto the targets
        assert sorted(sizes.tolist(), reverse=True) == [23 // E_T + 1] * (23 % E_T) + [23 // E_T] * (E_T - 23 % E_T)
        assert np.array_equal(sizes[: 23 % E_T], np.full(23 % E_T, 23 // E_T + 1))   # the first groups are the larger ones
    assert so.greedy_fold(P, 23).tolist() == list(range(23))       # one source per target: seeds in id order
    # relabelling-free sanity: equal affinities everywhere -> consecutive ids are grouped
    assert so.greedy_fold(np.ones((6, 6), dtype=np.int64), 3).tolist() == [0, 0, 1, 1, 2, 2]
    with pytest.raises(ValueError):
        so.greedy_fold(P, 24)


def test_local_tokens_and_placement():
    # 2 samples of 3 tokens, 4 experts on 2 nodes (experts 0,1 -> node 0; 2,3 -> node 1), k = 2
    idx = np.array([[0, 1], [0, 2], [2, 3], [2, 3], [3, 2], [1, 3]])
    node = np.array([0, 0, 1, 1])
    comm = so.local_tokens(idx, node, 2, 3)
    assert comm.tolist() == [[2, 2], [1, 3]]
    assert so.place_samples(comm).tolist() == [0, 1]               # a draw goes to the lower-numbered node
    rng = np.random.default_rng(5)
    idx = _idx(6, T=300, E=16, k=4)
    node = rng.integers(0, 4, size=16)
    comm = so.local_tokens(idx, node, 4, 60)
    a = so.activation(idx, 16)
    on_node = np.stack([(a[:, node == n].sum(axis=1) > 0) for n in range(4)], axis=1)     # [T, N] via the activation matrix
    assert np.array_equal(comm, on_node.reshape(5, 60, 4).sum(axis=1))
    assert np.all(comm <= 60) and np.all(comm.sum(axis=1) >= 60)   # every token is local to at least one node
    best = so.place_samples(comm)                                  # defining property, checked node by node
    for s_, b in enumerate(best.tolist()):
        assert all(comm[s_, b] >= comm[s_, n] for n in range(4)) and all(comm[s_, b] > comm[s_, n] for n in range(b))
    assert so.place_samples(np.array([[5, 9, 9, 1], [7, 7, 7, 7], [0, 0, 0, 3]])).tolist() == [1, 0, 3]
    # with every expert on one node every token is local there
    assert so.local_tokens(idx, np.zeros(16, dtype=int), 2, 60).tolist() == [[60, 0]] * 5
