"""CPU oracle for the routing statistics the offline stages of the method are built on.

TEST INFRASTRUCTURE ONLY: imported by the test suite, never by the product; no code shared with the CUDA path.

What it follows
  * Expert co-activation affinity matrix P (section "Expert Folding", Expert Folding Mapping): P_ij counts how often
    source experts i and j are activated for the same token.
  * Greedy affinity folding (same passage): target groups of floor(E_S/E_T) source experts, E_S mod E_T of them one
    larger; a group is seeded with an unassigned expert and grown by the unassigned expert with the largest summed
    affinity to the group's members.  The groups are the columns of the binary fold matrix M.
  * Routing affinity vector (section "Decoupling Communication Optimization"):
        phi(X)_i = (1/|X|) sum_{t in X} 1[e_i in TopK(G*(x_t), k)]
  * MaxVio_Global = (max_i L_i - mean L) / mean L (appendix "Maximal Violation").
  * Sample placement, Algorithm 1 (appendix "Efficiency Experiment Detail"): per sample and node, the number of the
    sample's tokens with at least one kept expert on the node; the sample goes to the node where that number is largest.

Readings where the paper is silent or loose:
  * P is the sum over tokens of a a^T with a the token's 0/1 activation vector: off-diagonal entries are pair counts,
    the diagonal holds each expert's activation count (never used by the folding rule, which only looks at other experts).
  * A token that lists one id twice activates that expert once (ids are distinct in the cache the router head writes).
  * Seeds: the lowest-numbered unassigned expert; the first E_S mod E_T groups are the larger ones; equal affinity sums
    go to the lower id; target j is group j.
  * Algorithm 1 names its running maximum "max_comm" but maximises the tokens that stay local; with the strict
    comparison the lowest-numbered node wins among equals.
  * |X| is the sample's token count; samples are consecutive runs of `seq_len` tokens of the routing table.

Integer results are exact; phi is a float64 quotient.  Parity pins: tests/test_oracle_stats.py.
"""
from __future__ import annotations

import numpy as np


def activation(idx: np.ndarray, E: int) -> np.ndarray:
    """0/1 matrix [T, E]: a[t, i] = 1 iff expert i is among token t's kept experts."""
    idx = np.asarray(idx).astype(np.int64)
    T = idx.shape[0]
    a = np.zeros((T, E), dtype=np.int64)
    for t in range(T):
        for e in idx[t]:
            a[t, e] = 1
    return a


def coactivation(idx: np.ndarray, E: int) -> np.ndarray:
    """P [E, E] int64: P[i, j] = number of tokens that activate both i and j (diagonal: activation counts)."""
    P = np.zeros((E, E), dtype=np.int64)
    idx = np.asarray(idx).astype(np.int64)
    for t in range(idx.shape[0]):
        ids = sorted(set(idx[t].tolist()))
        for i in ids:
            for j in ids:
                P[i, j] += 1
    return P


def loads(idx: np.ndarray, E: int) -> np.ndarray:
    """L [E]: tokens afforded to each expert."""
    return activation(idx, E).sum(axis=0)


def max_vio(L: np.ndarray) -> float:
    L = np.asarray(L, dtype=np.float64)
    mean = L.sum() / L.shape[0]
    return float((L.max() - mean) / mean)


def affinity_vectors(idx: np.ndarray, E: int, seq_len: int) -> np.ndarray:
    """phi [S, E] float64 for the S = T / seq_len samples."""
    a = activation(idx, E)
    T = a.shape[0]
    if T % seq_len:
        raise ValueError("T must be a whole number of samples")
    return a.reshape(T // seq_len, seq_len, E).sum(axis=1) / float(seq_len)


def greedy_fold(P: np.ndarray, E_tgt: int) -> np.ndarray:
    """fold_map [E_S] -> [0, E_T) from the co-activation matrix by greedy affinity merging."""
    P = np.asarray(P)
    E_S = P.shape[0]
    g_avg, n_extra = E_S // E_tgt, E_S % E_tgt
    if g_avg < 1:
        raise ValueError("more targets than sources")
    assigned = np.zeros(E_S, dtype=bool)
    fold = np.full(E_S, -1, dtype=np.int32)
    for k in range(E_tgt):
        size = g_avg + (1 if k < n_extra else 0)
        seed = int(np.nonzero(~assigned)[0][0])
        group = [seed]
        assigned[seed] = True
        while len(group) < size:
            best, best_aff = -1, None
            for j in range(E_S):
                if assigned[j]:
                    continue
                aff = sum(int(P[m, j]) for m in group)
                if best < 0 or aff > best_aff:
                    best, best_aff = j, aff
            group.append(best)
            assigned[best] = True
        for i in group:
            fold[i] = k
    return fold


def local_tokens(idx: np.ndarray, node_of_expert: np.ndarray, n_nodes: int, seq_len: int) -> np.ndarray:
    """comm [S, N]: tokens of sample s with at least one kept expert placed on node n (|T_s(n)| of Algorithm 1)."""
    idx = np.asarray(idx).astype(np.int64)
    node_of_expert = np.asarray(node_of_expert).astype(np.int64)
    T = idx.shape[0]
    S = T // seq_len
    comm = np.zeros((S, n_nodes), dtype=np.int64)
    for t in range(T):
        for n in set(node_of_expert[idx[t]].tolist()):
            comm[t // seq_len, n] += 1
    return comm


def place_samples(comm: np.ndarray) -> np.ndarray:
    """best_node [S]: for every sample the node holding most of its local tokens, argmax_n |T_s(n)| (Algorithm 1);
    among nodes with equal counts the lowest-numbered one (np.argmax returns the first maximum)."""
    return np.asarray(comm).argmax(axis=1).astype(np.int32)
