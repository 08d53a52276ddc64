"""CPU oracle for the router head that produces the pre-dispatch routing cache.

TEST INFRASTRUCTURE ONLY: imported by the test suite (and the benchmark's CPU leg), never by the product, and it
shares no code with the CUDA path.

What it follows
  * Routing function, Eq. 2 (section "Mixture-of-Experts"):  r(x) = g(TopK(s(x), k)), with s(x) the router's raw
    scores over the experts, TopK keeping the k highest, and g a normalisation (softmax or sigmoid) applied to the
    kept scores.
  * Matrix folding (section "Expert Folding", Matrix Folding Implementation): the score layer of a router distilled
    for E_S source experts serves a model with E_T experts through  W~_s = W_s M,  M in {0,1}^{E_S x E_T} with one 1
    per row.  Folding therefore happens on the scores, before TopK: a token never picks one target expert twice.
  * Pre-dispatch cache (appendix "Efficiency Experiment Detail"): per token, k expert ids as uint8 and k routing
    scores as bfloat16.

Readings where the paper is silent:
  * s(x) = W_s^T h with h the router's last hidden state of the token; no bias.
  * TopK order: scores descending, equal scores by ascending expert id; the cache keeps that order.
  * softmax runs over the k kept scores only (the usual "softmax after top-k"); sigmoid is applied to each kept score.
  * the cached score is the normalised coefficient r(x)_i rounded to bfloat16, round-to-nearest-even.

All arithmetic is float64; np.matmul is the only library primitive.
Parity pins: tests/test_oracle_router.py (column-group sums, library argsort and softmax, permutation and identity
fold invariants, hand-worked example).
"""
from __future__ import annotations

from typing import Optional

import numpy as np

SOFTMAX, SIGMOID = 0, 1


def fold_matrix(fold_map: np.ndarray, E_tgt: int) -> np.ndarray:
    """Binary M [E_S, E_T]: M[i, j] = 1 iff source expert i is mapped to target expert j."""
    fold_map = np.asarray(fold_map).astype(np.int64)
    M = np.zeros((fold_map.shape[0], E_tgt), dtype=np.float64)
    for i, j in enumerate(fold_map):
        if not 0 <= j < E_tgt:
            raise ValueError("fold target out of range")
        M[i, j] = 1.0
    return M


def folded_score_layer(W_s: np.ndarray, fold_map: Optional[np.ndarray], E_tgt: int) -> np.ndarray:
    """W~_s = W_s M.  W_s is stored [E_S, d_h] (one row per source expert), so the result is M^T W_s, [E_T, d_h]."""
    W_s = np.asarray(W_s, dtype=np.float64)
    if fold_map is None:
        if W_s.shape[0] != E_tgt:
            raise ValueError("no fold map: E_src must equal E_tgt")
        return W_s
    return fold_matrix(fold_map, E_tgt).T @ W_s


def scores(H: np.ndarray, W_s: np.ndarray, fold_map: Optional[np.ndarray], E_tgt: int) -> np.ndarray:
    """s(x) for every token: H [T, d_h] times the folded score layer -> [T, E_T]."""
    return np.asarray(H, dtype=np.float64) @ folded_score_layer(W_s, fold_map, E_tgt).T


def top_k(S: np.ndarray, k: int) -> np.ndarray:
    """Ids of the k highest scores per row, scores descending, ties by ascending id.  [T, k] int64."""
    T, E = S.shape
    out = np.empty((T, k), dtype=np.int64)
    for t in range(T):
        taken = np.zeros(E, dtype=bool)
        for j in range(k):
            best = -1
            for e in range(E):
                if not taken[e] and (best < 0 or S[t, e] > S[t, best]):
                    best = e
            taken[best] = True
            out[t, j] = best
    return out


def normalise(kept: np.ndarray, norm: int) -> np.ndarray:
    """g of Eq. 2 on the kept scores [T, k]."""
    if norm == SOFTMAX:
        z = kept - kept.max(axis=1, keepdims=True)
        e = np.exp(z)
        return e / e.sum(axis=1, keepdims=True)
    if norm == SIGMOID:
        return 1.0 / (1.0 + np.exp(-kept))
    raise ValueError("norm")


def route(H, W_s, fold_map, E_tgt: int, k: int, norm: int = SOFTMAX):
    """Eq. 2 for every token.  Returns (ids [T,k] int64, r [T,k] float64, S [T,E_T] float64)."""
    S = scores(H, W_s, fold_map, E_tgt)
    ids = top_k(S, k)
    kept = np.take_along_axis(S, ids, axis=1)
    return ids, normalise(kept, norm), S


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float64 -> bfloat16 bit patterns (uint16), round-to-nearest-even in ONE rounding: the float64 mantissa is cut to
    bfloat16's 7 bits directly on the integer representation (a carry moves into the exponent by itself).  Valid for
    zeros and for magnitudes in float32's normal range, which covers routing coefficients."""
    a = np.ascontiguousarray(a, dtype=np.float64)
    if np.any((a != 0) & ((np.abs(a) < 1e-37) | (np.abs(a) > 3e38))):
        raise ValueError("outside the range this rounding handles")
    x = a.view(np.uint64)
    drop = np.uint64(52 - 7)
    rem = x & ((np.uint64(1) << drop) - np.uint64(1))
    base = x >> drop
    half = np.uint64(1) << (drop - np.uint64(1))
    up = (rem > half) | ((rem == half) & ((base & np.uint64(1)) == np.uint64(1)))
    rounded = ((base + up.astype(np.uint64)) << drop).view(np.float64)      # exactly representable in bfloat16
    return (rounded.astype(np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def pack_cache(ids: np.ndarray, r: np.ndarray):
    """The cache record of the paper: uint8 ids and bfloat16 scores, 3*k bytes per token."""
    if ids.max() > 255:
        raise ValueError("uint8 ids address at most 256 experts")
    return ids.astype(np.uint8), to_bf16_bits(r)
