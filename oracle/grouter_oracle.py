"""CPU oracle for the routed expert layer under preemptive routing.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of
what the layer computes, written from the paper's definitions.  Only the test
suite, the smoke check and the benchmark's CPU-baseline leg may import it; the
product (the CUDA library and its Python binding) never does, and it shares
no code with the CUDA path.

What it follows
  * MoE layer output, Eq. 1 (section "Mixture-of-Experts"):
        y = sum_{i=1..E} r(x)_i * f_i(x)
    where r(x) is *given* (Eq. 2 is evaluated offline by the frozen router and
    cached as k expert ids + k scores per token; section "Decoupling
    Preemptive Routing").  r(x)_i is the sum of the token's cached scores whose
    (folded) id equals i, and 0 for every other expert.
  * Expert gradient (appendix on joint optimisation, "observed expert
    gradient"):  dL/dtheta_e = dL/dy * sum_i r(x)_i * grad_theta f_i(x).
  * Expert folding (section "Expert Folding", Matrix Folding): the binary
    map M in its compact form fold_map[source id] -> target id.

Readings where the paper is silent:
  * f_i is a bias-free SwiGLU FFN:  f(x) = W_d ( silu(W_g x) * (W_u x) ),
    silu(z) = z / (1 + exp(-z)).
  * gates are used as given: never renormalised, leaf inputs, so
    dgate_{t,j} = <dY_t, f_{e(t,j)}(x_t)>.
  * folding remaps ids *after* top-k; colliding slots stay separate rows.
  * the plan is a stable counting sort: key = target expert id ascending,
    ties by flat slot index s = t*k + j ascending.

Every function works on float64 arrays; callers widen bf16 bits exactly before
calling.  Nothing here rounds an intermediate.  np.matmul (a library matmul) is
the only non-elementwise primitive used.

Parity pins: every function in this file is pinned by tests/test_oracle_*.py
(library stable argsort, O(R^2) brute-force ranks, hand-worked example, dense
SwiGLU special case, torch autograd, finite differences, adjoint identity, a
slot-by-slot scalar-loop restatement on tiny inputs; the two error measures
rel_frobenius and rel_rows by hand-worked numbers).
"""
from __future__ import annotations

from typing import Iterable, Optional, Sequence

import numpy as np


# --------------------------------------------------------------------------
# Routing plan (exact integer work)
# --------------------------------------------------------------------------

def fold_ids(idx: np.ndarray, fold_map: Optional[np.ndarray]) -> np.ndarray:
    """e_s = m[idx_s]: target expert of every slot, int64 [T*k] in slot order."""
    e = np.asarray(idx).astype(np.int64).reshape(-1)
    if fold_map is not None:
        e = np.asarray(fold_map).astype(np.int64)[e]
    return e


def plan(idx: np.ndarray, fold_map: Optional[np.ndarray], E_tgt: int):
    """Stable counting sort of the slots by target expert.

    Returns (counts[E_tgt], offsets[E_tgt+1], row_to_slot[R], slot_to_row[R]),
    all int32.  counts[e] = number of slots routed to e; offsets is its
    exclusive prefix sum with offsets[E_tgt] = R; slot s sits at row
    offsets[e_s] + (number of slots s' < s with e_s' == e_s).
    """
    e = fold_ids(idx, fold_map)
    R = e.shape[0]
    if R and (e.min() < 0 or e.max() >= E_tgt):
        raise ValueError("expert id out of range")
    counts = [0] * E_tgt
    for s in range(R):
        counts[e[s]] += 1
    offsets = [0] * (E_tgt + 1)
    for i in range(E_tgt):
        offsets[i + 1] = offsets[i] + counts[i]
    cursor = offsets[:E_tgt]
    slot_to_row = np.empty(R, dtype=np.int32)
    row_to_slot = np.empty(R, dtype=np.int32)
    for s in range(R):
        row = cursor[e[s]]
        cursor[e[s]] = row + 1
        slot_to_row[s] = row
        row_to_slot[row] = s
    return (np.asarray(counts, dtype=np.int32), np.asarray(offsets, dtype=np.int32), row_to_slot, slot_to_row)


# --------------------------------------------------------------------------
# Layer (floating point, fp64)
# --------------------------------------------------------------------------

def sigmoid(z: np.ndarray) -> np.ndarray:
    return 1.0 / (1.0 + np.exp(-z))


def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def expert_ffn(x: np.ndarray, W_g: np.ndarray, W_u: np.ndarray, W_d: np.ndarray) -> np.ndarray:
    """f(x) for a batch of rows x [n,d]; W_g, W_u [F,d]; W_d [d,F] -> [n,d]."""
    a = x @ W_g.T
    u = x @ W_u.T
    return (silu(a) * u) @ W_d.T


def routing_coefficients(idx, gates, fold_map, E_tgt: int, tokens: np.ndarray, e: int) -> np.ndarray:
    """r(x_t)_e for the listed tokens: sum of the token's gates whose folded id is e."""
    k = idx.shape[1]
    ids = fold_ids(idx[tokens], fold_map).reshape(-1, k)
    return np.where(ids == e, gates[tokens], 0.0).sum(axis=1)


class Weights:
    """Access to per-expert fp64 weights, either from arrays or from a callback
    (so a large layer can be streamed one expert at a time)."""

    def __init__(self, W_gu=None, W_d=None, getter=None, ffn: Optional[int] = None):
        self._W_gu, self._W_d, self._getter = W_gu, W_d, getter
        self.ffn = ffn if ffn is not None else (W_gu.shape[1] // 2)

    def get(self, e: int):
        """-> (W_g [F,d], W_u [F,d], W_d [d,F]) float64"""
        if self._getter is not None:
            W_gu, W_d = self._getter(e)
        else:
            W_gu, W_d = self._W_gu[e], self._W_d[e]
        W_gu = np.asarray(W_gu, dtype=np.float64)
        return W_gu[: self.ffn], W_gu[self.ffn:], np.asarray(W_d, dtype=np.float64)


def moe_forward(X, idx, gates, weights: Weights, E_tgt: int, fold_map=None,
                tokens: Optional[Sequence[int]] = None) -> np.ndarray:
    """Eq. 1 for the listed tokens (all if None): Y[i] = sum_e r(x_t)_e f_e(x_t).

    X [T,d] f64, idx [T,k] int, gates [T,k] f64.  Experts with r_e = 0 for a
    token contribute exactly nothing and are skipped for that token.
    """
    tokens = np.arange(X.shape[0]) if tokens is None else np.asarray(tokens, dtype=np.int64)
    Y = np.zeros((tokens.shape[0], X.shape[1]), dtype=np.float64)
    k = idx.shape[1]
    ids = fold_ids(idx[tokens], fold_map).reshape(-1, k)
    for e in range(E_tgt):
        hit = (ids == e).any(axis=1)
        if not hit.any():
            continue
        sel = np.nonzero(hit)[0]
        W_g, W_u, W_d = weights.get(e)
        r_e = routing_coefficients(idx, gates, fold_map, E_tgt, tokens[sel], e)
        Y[sel] += r_e[:, None] * expert_ffn(X[tokens[sel]], W_g, W_u, W_d)
    return Y


def moe_backward_tokens(dY, X, idx, gates, weights: Weights, E_tgt: int, fold_map=None,
                        tokens: Optional[Sequence[int]] = None):
    """Input-side gradients for the listed tokens: (dX [n,d], dgates [n,k]).

    With L = sum(Y * dY):  per token t and expert e with coefficient r_e,
    a = W_g x, u = W_u x, h = silu(a)*u, o = W_d h:
      dgate_{t,j} = <dY_t, o>            for every slot j of t whose folded id is e
      dh = r_e * W_d^T dY_t
      da = dh * u * sigma(a) * (1 + a*(1 - sigma(a)));  du = dh * silu(a)
      dX_t += W_g^T da + W_u^T du
    """
    tokens = np.arange(X.shape[0]) if tokens is None else np.asarray(tokens, dtype=np.int64)
    k = idx.shape[1]
    n = tokens.shape[0]
    dX = np.zeros((n, X.shape[1]), dtype=np.float64)
    dgates = np.zeros((n, k), dtype=np.float64)
    ids = fold_ids(idx[tokens], fold_map).reshape(-1, k)
    for e in range(E_tgt):
        hit = (ids == e).any(axis=1)
        if not hit.any():
            continue
        sel = np.nonzero(hit)[0]
        W_g, W_u, W_d = weights.get(e)
        x = X[tokens[sel]]
        dy = dY[tokens[sel]]
        r_e = routing_coefficients(idx, gates, fold_map, E_tgt, tokens[sel], e)
        a = x @ W_g.T
        u = x @ W_u.T
        sa = sigmoid(a)
        h = a * sa * u
        o = h @ W_d.T
        dg = (dy * o).sum(axis=1)
        dgates[sel] += np.where(ids[sel] == e, dg[:, None], 0.0)
        dh = (r_e[:, None] * dy) @ W_d
        da = dh * u * sa * (1.0 + a * (1.0 - sa))
        du = dh * a * sa
        dX[sel] += da @ W_g + du @ W_u
    return dX, dgates


def moe_backward_expert(dY, X, idx, gates, weights: Weights, E_tgt: int, e: int, fold_map=None):
    """Parameter gradients of one expert: (dW_gu [2F,d], dW_d [d,F]), fp64.

    dW_d = sum_t (r_e dY_t) (x) h_t ; dW_g = sum_t da_t (x) x_t ; dW_u = sum_t du_t (x) x_t,
    the sums running over the tokens with r(x_t)_e != 0 routed to e.  An expert
    that receives no slot gets exact zeros.
    """
    k = idx.shape[1]
    ids = fold_ids(idx, fold_map).reshape(-1, k)
    W_g, W_u, W_d = weights.get(e)
    F, d = W_g.shape
    sel = np.nonzero((ids == e).any(axis=1))[0]
    if sel.shape[0] == 0:
        return np.zeros((2 * F, d)), np.zeros((d, F))
    x = X[sel]
    dy = dY[sel]
    r_e = routing_coefficients(idx, gates, fold_map, E_tgt, sel, e)
    a = x @ W_g.T
    u = x @ W_u.T
    sa = sigmoid(a)
    h = a * sa * u
    do = r_e[:, None] * dy
    dW_d = do.T @ h
    dh = do @ W_d
    da = dh * u * sa * (1.0 + a * (1.0 - sa))
    du = dh * a * sa
    dW_gu = np.concatenate([da.T @ x, du.T @ x], axis=0)
    return dW_gu, dW_d


def moe_backward(dY, X, idx, gates, weights: Weights, E_tgt: int, fold_map=None,
                 experts: Optional[Iterable[int]] = None):
    """Full backward: dX [T,d], dgates [T,k], and {e: (dW_gu, dW_d)} for the listed experts (all if None)."""
    dX, dgates = moe_backward_tokens(dY, X, idx, gates, weights, E_tgt, fold_map)
    experts = range(E_tgt) if experts is None else experts
    dW = {int(e): moe_backward_expert(dY, X, idx, gates, weights, E_tgt, int(e), fold_map) for e in experts}
    return dX, dgates, dW


def rel_frobenius(a: np.ndarray, ref: np.ndarray) -> float:
    """||a - ref||_F / ||ref||_F in fp64 (exact match required where ref is all zero)."""
    a = np.asarray(a, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref.ravel())
    num = np.linalg.norm((a - ref).ravel())
    if den == 0.0:
        return 0.0 if num == 0.0 else float("inf")
    return float(num / den)


def rel_rows(a: np.ndarray, ref: np.ndarray) -> np.ndarray:
    """Per-row error of a 2-D comparison: e_i = ||a_i - ref_i||_2 / max(||ref_i||_2, rho), where rho is the root mean
    square of the rows' norms ||ref_j||_2.  The floor rho keeps a row that is small by cancellation from dividing by
    almost nothing; a row of an all-zero reference must match exactly (0 if it does, inf if not)."""
    a = np.asarray(a, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    a = a.reshape(a.shape[0], -1)
    ref = ref.reshape(ref.shape[0], -1)
    num = np.sqrt(((a - ref) ** 2).sum(axis=1))
    norms = np.sqrt((ref ** 2).sum(axis=1))
    rho = np.sqrt((norms ** 2).mean()) if norms.size else 0.0
    den = np.maximum(norms, rho)
    out = np.zeros_like(num)
    nz = den > 0.0
    out[nz] = num[nz] / den[nz]
    out[~nz & (num > 0.0)] = np.inf
    return out

