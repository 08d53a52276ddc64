"""Pins for the oracle's forward/backward: a hand-worked example, the dense-FFN
special case against torch, torch autograd over the dense-r form of Eq. 1,
finite differences, the adjoint identity and structural invariants."""
import os

import numpy as np
import pytest
import torch

from oracle import grouter_oracle as orc
from paper_2603_06626_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_layer(seed, T, d, F, E, k, fold_to=None, distinct=True):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((T, d))
    dY = rng.standard_normal((T, d))
    W_gu = rng.standard_normal((fold_to or E, 2 * F, d)) * 0.5
    W_d = rng.standard_normal((fold_to or E, d, F)) * 0.5
    if distinct:
        idx = np.stack([rng.permutation(E)[:k] for _ in range(T)]).astype(np.uint8)
    else:
        idx = rng.integers(0, E, size=(T, k)).astype(np.uint8)
    gates = rng.random((T, k)) + 0.1
    fm = None if fold_to is None else (np.arange(E) % fold_to).astype(np.int32)
    return X, dY, W_gu, W_d, idx, gates, fm


def _torch_dense_r(X, W_gu, W_d, idx, gates, fm, E_tgt):
    """Eq. 1 with a dense coefficient matrix r [T,E] and *every* expert evaluated on *every* token,
    in torch fp64 so autograd supplies independent gradients."""
    T, k = idx.shape
    F = W_gu.shape[1] // 2
    ids = torch.as_tensor(idx.astype(np.int64))
    if fm is not None:
        ids = torch.as_tensor(fm.astype(np.int64))[ids]
    r = torch.zeros(T, E_tgt, dtype=torch.float64).scatter_add(1, ids, gates)
    Y = torch.zeros_like(X)
    for e in range(E_tgt):
        a = X @ W_gu[e, :F].T
        u = X @ W_gu[e, F:].T
        Y = Y + r[:, e:e + 1] * ((torch.nn.functional.silu(a) * u) @ W_d[e].T)
    return Y


def test_hand_worked_example():
    vals = {}
    for line in open(os.path.join(GOLDEN, "eq1_hand_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        p = line.split()
        vals[p[0]] = [float(v) for v in p[1:]]
    X = np.array([[1.0, 2.0]])
    W_gu = np.array([[[1.0, 0.0], [0.0, 1.0]], [[0.0, -1.0], [3.0, 0.0]]])
    W_d = np.array([[[1.0], [-1.0]], [[2.0], [0.5]]])
    idx = np.array([[0, 1]], dtype=np.uint8)
    gates = np.array([[0.25, 0.75]])
    Wt = orc.Weights(W_gu, W_d)
    Y = orc.moe_forward(X, idx, gates, Wt, 2)
    np.testing.assert_allclose(Y[0], vals["y"], rtol=1e-14)
    _, dg = orc.moe_backward_tokens(np.ones((1, 2)), X, idx, gates, Wt, 2)
    np.testing.assert_allclose(dg[0], vals["dgates"], rtol=1e-14, atol=1e-15)


def test_dense_ffn_special_case_forward_backward():
    """E=1, k=1, gate=1 reduces to a dense SwiGLU FFN (torch ops + autograd as the textbook routine)."""
    T, d, F = 37, 24, 40
    X, dY, W_gu, W_d, _, _, _ = _rand_layer(1, T, d, F, 1, 1)
    idx = np.zeros((T, 1), dtype=np.uint8)
    gates = np.ones((T, 1))
    Wt = orc.Weights(W_gu, W_d)
    Y = orc.moe_forward(X, idx, gates, Wt, 1)
    dX, dg, dW = orc.moe_backward(dY, X, idx, gates, Wt, 1)
    tX = torch.tensor(X, requires_grad=True)
    tg = torch.tensor(W_gu[0, :F], requires_grad=True)
    tu = torch.tensor(W_gu[0, F:], requires_grad=True)
    td = torch.tensor(W_d[0], requires_grad=True)
    tY = (torch.nn.functional.silu(tX @ tg.T) * (tX @ tu.T)) @ td.T
    (tY * torch.tensor(dY)).sum().backward()
    np.testing.assert_allclose(Y, tY.detach().numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dX, tX.grad.numpy(), rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(dW[0][0][:F], tg.grad.numpy(), rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(dW[0][0][F:], tu.grad.numpy(), rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(dW[0][1], td.grad.numpy(), rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(dg[:, 0], (dY * Y).sum(1), rtol=1e-11)


@pytest.mark.parametrize("fold_to,distinct", [(None, True), (3, True), (None, False)])
def test_against_autograd_dense_r(fold_to, distinct):
    T, d, F, E, k = 23, 10, 6, 6, 3
    X, dY, W_gu, W_d, idx, gates, fm = _rand_layer(2, T, d, F, E, k, fold_to, distinct)
    E_tgt = fold_to or E
    Wt = orc.Weights(W_gu, W_d)
    Y = orc.moe_forward(X, idx, gates, Wt, E_tgt, fm)
    dX, dg, dW = orc.moe_backward(dY, X, idx, gates, Wt, E_tgt, fm)
    tX = torch.tensor(X, requires_grad=True)
    tWgu = torch.tensor(W_gu, requires_grad=True)
    tWd = torch.tensor(W_d, requires_grad=True)
    tgates = torch.tensor(gates, requires_grad=True)
    tY = _torch_dense_r(tX, tWgu, tWd, idx, tgates, fm, E_tgt)
    (tY * torch.tensor(dY)).sum().backward()
    np.testing.assert_allclose(Y, tY.detach().numpy(), rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(dX, tX.grad.numpy(), rtol=1e-10, atol=1e-10)
    np.testing.assert_allclose(dg, tgates.grad.numpy(), rtol=1e-10, atol=1e-10)
    for e in range(E_tgt):
        np.testing.assert_allclose(dW[e][0], tWgu.grad[e].numpy(), rtol=1e-10, atol=1e-10)
        np.testing.assert_allclose(dW[e][1], tWd.grad[e].numpy(), rtol=1e-10, atol=1e-10)


def test_finite_differences():
    T, d, F, E, k = 4, 3, 2, 3, 2
    X, dY, W_gu, W_d, idx, gates, fm = _rand_layer(3, T, d, F, E, k)

    def loss(X_, Wgu_, Wd_, g_):
        return float((orc.moe_forward(X_, idx, g_, orc.Weights(Wgu_, Wd_), E) * dY).sum())

    dX, dg, dW = orc.moe_backward(dY, X, idx, gates, orc.Weights(W_gu, W_d), E)
    dWgu = np.stack([dW[e][0] for e in range(E)])
    dWd = np.stack([dW[e][1] for e in range(E)])
    h = 1e-6
    for arr, grad, pos in [(X, dX, 0), (W_gu, dWgu, 1), (W_d, dWd, 2), (gates, dg, 3)]:
        fd = np.zeros_like(arr)
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            args = [X, W_gu, W_d, gates]
            p = arr.copy(); p[i] += h
            m = arr.copy(); m[i] -= h
            args[pos] = p; lp = loss(*args)
            args[pos] = m; lm = loss(*args)
            fd[i] = (lp - lm) / (2 * h)
        np.testing.assert_allclose(grad, fd, rtol=1e-6, atol=1e-7)


def test_adjoint_identity_medium():
    """<dY, J v> = <J^T dY, v> for a perturbation v of X (J v by central difference of the forward)."""
    T, d, F, E, k = 64, 32, 24, 8, 2
    X, dY, W_gu, W_d, idx, gates, _ = _rand_layer(4, T, d, F, E, k)
    Wt = orc.Weights(W_gu, W_d)
    v = np.random.default_rng(5).standard_normal(X.shape)
    h = 1e-6
    Jv = (orc.moe_forward(X + h * v, idx, gates, Wt, E) - orc.moe_forward(X - h * v, idx, gates, Wt, E)) / (2 * h)
    dX, _ = orc.moe_backward_tokens(dY, X, idx, gates, Wt, E)
    assert abs((dY * Jv).sum() - (dX * v).sum()) <= 1e-6 * abs((dX * v).sum())


def test_structural_invariants():
    T, d, F, E, k = 32, 16, 12, 6, 3
    X, dY, W_gu, W_d, idx, gates, _ = _rand_layer(6, T, d, F, E, k)
    Wt = orc.Weights(W_gu, W_d)
    Y = orc.moe_forward(X, idx, gates, Wt, E)
    # linear in the gates
    np.testing.assert_allclose(orc.moe_forward(X, idx, 2.5 * gates, Wt, E), 2.5 * Y, rtol=1e-12)
    # slot order inside a token does not matter for Y, dX; dgates permutes with it
    perm = np.array([2, 0, 1])
    Y2 = orc.moe_forward(X, idx[:, perm], gates[:, perm], Wt, E)
    np.testing.assert_allclose(Y2, Y, rtol=1e-12, atol=1e-13)
    dX1, dg1 = orc.moe_backward_tokens(dY, X, idx, gates, Wt, E)
    dX2, dg2 = orc.moe_backward_tokens(dY, X, idx[:, perm], gates[:, perm], Wt, E)
    np.testing.assert_allclose(dX2, dX1, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(dg2, dg1[:, perm], rtol=1e-12, atol=1e-13)
    # a zero gate removes the slot
    g0 = gates.copy(); g0[:, 1] = 0.0
    Y0 = orc.moe_forward(X, idx, g0, Wt, E)
    Y01 = orc.moe_forward(X, idx[:, [0, 2]], gates[:, [0, 2]], Wt, E)
    np.testing.assert_allclose(Y0, Y01, rtol=1e-12, atol=1e-13)
    # subset evaluation equals the rows of the full evaluation
    sub = np.array([3, 17, 4, 31])
    np.testing.assert_allclose(orc.moe_forward(X, idx, gates, Wt, E, tokens=sub), Y[sub], rtol=1e-13)
    dXs, dgs = orc.moe_backward_tokens(dY, X, idx, gates, Wt, E, tokens=sub)
    np.testing.assert_allclose(dXs, dX1[sub], rtol=1e-13)
    np.testing.assert_allclose(dgs, dg1[sub], rtol=1e-13)


def test_fold_semantics():
    T, d, F, E, k = 16, 8, 6, 4, 2
    X, dY, W_gu, W_d, idx, gates, _ = _rand_layer(8, T, d, F, E, k)
    # fold everything onto one expert with gates summing to 1 -> dense FFN of that expert
    fm = np.zeros(E, dtype=np.int32)
    g = gates / gates.sum(1, keepdims=True)
    Wt1 = orc.Weights(W_gu[:1], W_d[:1])
    Y = orc.moe_forward(X, idx, g, Wt1, 1, fm)
    np.testing.assert_allclose(Y, orc.expert_ffn(X, W_gu[0, :F], W_gu[0, F:], W_d[0]), rtol=1e-12, atol=1e-13)
    # a collision equals one slot carrying the merged gate; each colliding slot gets the same dgate
    idx2 = np.array([[0, 2]] * T, dtype=np.uint8)
    fm2 = np.array([0, 1, 0, 1], dtype=np.int32)
    Wt2 = orc.Weights(W_gu[:2], W_d[:2])
    Yc = orc.moe_forward(X, idx2, gates, Wt2, 2, fm2)
    Ym = orc.moe_forward(X, np.zeros((T, 1), dtype=np.uint8), gates.sum(1, keepdims=True), Wt2, 2)
    np.testing.assert_allclose(Yc, Ym, rtol=1e-12, atol=1e-13)
    _, dgc = orc.moe_backward_tokens(dY, X, idx2, gates, Wt2, 2, fm2)
    np.testing.assert_allclose(dgc[:, 0], dgc[:, 1], rtol=1e-13)


def test_empty_expert_zero_gradients():
    T, d, F, E, k = 12, 8, 6, 4, 2
    X, dY, W_gu, W_d, idx, gates, _ = _rand_layer(9, T, d, F, E, k)
    idx = (idx % 3).astype(np.uint8)               # expert 3 never used
    dWgu, dWd = orc.moe_backward_expert(dY, X, idx, gates, orc.Weights(W_gu, W_d), E, 3)
    assert not dWgu.any() and not dWd.any()
    assert dWgu.shape == (2 * F, d) and dWd.shape == (d, F)


def test_synth_bf16_roundtrip_and_rne():
    a = np.array([1.0, 1.00390625, 1.01171875, -2.5, 0.0, 3.140625], dtype=np.float32)
    bits = synth.f32_to_bf16_bits(a)
    # 1.00390625 = 1 + 2^-8 is a tie between 1.0 and 1.0078125 -> even mantissa (1.0);
    # 1.01171875 = 1 + 3*2^-8 is a tie between 1.0078125 and 1.015625 -> even (1.015625)
    np.testing.assert_array_equal(synth.bf16_bits_to_f32(bits),
                                  np.array([1.0, 1.0, 1.015625, -2.5, 0.0, 3.140625], dtype=np.float32))
    t = torch.tensor(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits, t)


def test_rel_frobenius_hand_worked():
    """The error measure every float parity test goes through, against numbers worked by hand."""
    assert orc.rel_frobenius([3.0, 4.0], [0.0, 0.0]) == float("inf")            # zero reference, non-zero input
    assert orc.rel_frobenius([0.0, 0.0], [0.0, 0.0]) == 0.0                     # zero against zero
    assert orc.rel_frobenius([1.0, 2.0, 2.0], [1.0, 2.0, 2.0]) == 0.0
    # a - ref = [0, 0, 2]: ||.|| = 2; ||ref|| = sqrt(1 + 4 + 0) = sqrt(5)
    assert orc.rel_frobenius([1.0, 2.0, 2.0], [1.0, 2.0, 0.0]) == pytest.approx(2.0 / 5.0 ** 0.5, rel=1e-15)
    # not symmetric: the reference is the denominator.  a - ref = [0, 0, -2]; ||ref|| = 3
    assert orc.rel_frobenius([1.0, 2.0, 0.0], [1.0, 2.0, 2.0]) == pytest.approx(2.0 / 3.0, rel=1e-15)
    # 2-D: differences 1, 0, 0, 2 -> sqrt(5); reference entries 1, 2, 3, 4 -> sqrt(30)
    assert orc.rel_frobenius([[2.0, 2.0], [3.0, 6.0]], [[1.0, 2.0], [3.0, 4.0]]) == pytest.approx((5.0 / 30.0) ** 0.5, rel=1e-15)
    # scale-free in the pair, first order in a uniform relative error
    ref = np.arange(1.0, 7.0).reshape(2, 3)
    assert orc.rel_frobenius(1.001 * ref, ref) == pytest.approx(1e-3, rel=1e-9)
    assert orc.rel_frobenius(7.0 * 1.001 * ref, 7.0 * ref) == pytest.approx(1e-3, rel=1e-9)
    # float32 input is widened, not the reference narrowed
    assert orc.rel_frobenius(np.array([1.0, 1.0], dtype=np.float32), np.array([1.0, 1.0 + 2.0 ** -40])) > 0.0


def test_rel_rows_hand_worked():
    ref = np.array([[3.0, 4.0], [0.0, 0.0], [6.0, 8.0]])          # row norms 5, 0, 10; rms = sqrt((25 + 0 + 100) / 3) = 6.4549...
    a = np.array([[3.0, 5.0], [0.3, 0.4], [6.0, 8.0]])            # row errors 1, 0.5, 0
    rho = (125.0 / 3.0) ** 0.5
    np.testing.assert_allclose(orc.rel_rows(a, ref), [1.0 / rho, 0.5 / rho, 0.0], rtol=1e-15)
    # a row above the floor is divided by its own norm: error 1 on the row of norm 10
    a2 = ref.copy(); a2[2, 0] += 1.0
    np.testing.assert_allclose(orc.rel_rows(a2, ref), [0.0, 0.0, 0.1], rtol=1e-15)
    # all-zero reference: exact match or inf
    z = np.zeros((2, 3))
    assert orc.rel_rows(z, z).tolist() == [0.0, 0.0]
    assert orc.rel_rows(np.array([[0.0, 0.0, 0.0], [0.0, 1e-30, 0.0]]), z).tolist() == [0.0, float("inf")]
    # trailing axes are flattened into the row: [2, 2, 2] is two rows of four
    r3 = np.arange(8.0).reshape(2, 2, 2)
    a3 = r3.copy(); a3[1, 1, 1] += 2.0                            # row norms sqrt(14), sqrt(126); rms = sqrt(70)
    np.testing.assert_allclose(orc.rel_rows(a3, r3), [0.0, 2.0 / 126.0 ** 0.5], rtol=1e-15)
    # one wrong row in a thousand stands out by orders of magnitude where the Frobenius ratio hardly moves
    rng = np.random.default_rng(0)
    big = rng.standard_normal((1000, 64))
    bad = big * (1.0 + 3e-3 * rng.standard_normal(big.shape))
    bad[417] = rng.standard_normal(64)
    assert orc.rel_frobenius(bad, big) < 5e-2 and orc.rel_rows(bad, big)[417] > 1.0
    assert np.delete(orc.rel_rows(bad, big), 417).max() < 1e-2


def _scalar_loop_layer(X, dY, W_gu, W_d, idx, gates, fm, E_tgt):
    """Eq. 1 and its gradients slot by slot with scalar loops only (no matmul, no masks, no grouping by expert):
    for every slot (t, j): e = m[idx], a = W_g x, u = W_u x, h = silu(a) u, o = W_d h, y_t += g o, and the chain rule
    written out element by element."""
    import math
    T, d = X.shape
    k = idx.shape[1]
    F = W_gu.shape[1] // 2
    Y = np.zeros((T, d)); dX = np.zeros((T, d)); dg = np.zeros((T, k))
    dWgu = np.zeros((E_tgt, 2 * F, d)); dWd = np.zeros((E_tgt, d, F))
    for t in range(T):
        for j in range(k):
            e = int(idx[t, j]) if fm is None else int(fm[int(idx[t, j])])
            g = gates[t, j]
            a = [sum(W_gu[e, f, c] * X[t, c] for c in range(d)) for f in range(F)]
            u = [sum(W_gu[e, F + f, c] * X[t, c] for c in range(d)) for f in range(F)]
            sg = [1.0 / (1.0 + math.exp(-a[f])) for f in range(F)]
            h = [a[f] * sg[f] * u[f] for f in range(F)]
            o = [sum(W_d[e, c, f] * h[f] for f in range(F)) for c in range(d)]
            for c in range(d):
                Y[t, c] += g * o[c]
            dg[t, j] = sum(dY[t, c] * o[c] for c in range(d))
            dh = [sum(g * dY[t, c] * W_d[e, c, f] for c in range(d)) for f in range(F)]
            for c in range(d):
                for f in range(F):
                    dWd[e, c, f] += g * dY[t, c] * h[f]
            for f in range(F):
                da = dh[f] * u[f] * sg[f] * (1.0 + a[f] * (1.0 - sg[f]))
                du = dh[f] * a[f] * sg[f]
                for c in range(d):
                    dWgu[e, f, c] += da * X[t, c]
                    dWgu[e, F + f, c] += du * X[t, c]
                    dX[t, c] += W_gu[e, f, c] * da + W_gu[e, F + f, c] * du
    return Y, dX, dg, dWgu, dWd


@pytest.mark.parametrize("fold_to,distinct", [(None, True), (2, True), (None, False)])
def test_against_scalar_loops(fold_to, distinct):
    """The oracle groups slots by expert and multiplies matrices with a library routine; the same quantities from
    scalar loops over single slots (no library contraction anywhere) must agree to rounding."""
    T, d, F, E, k = 7, 5, 3, 4, 2
    X, dY, W_gu, W_d, idx, gates, fm = _rand_layer(12, T, d, F, E, k, fold_to, distinct)
    E_tgt = fold_to or E
    Wt = orc.Weights(W_gu, W_d)
    Y = orc.moe_forward(X, idx, gates, Wt, E_tgt, fm)
    dX, dg, dW = orc.moe_backward(dY, X, idx, gates, Wt, E_tgt, fm)
    sY, sdX, sdg, sdWgu, sdWd = _scalar_loop_layer(X, dY, W_gu, W_d, idx, gates, fm, E_tgt)
    np.testing.assert_allclose(Y, sY, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dX, sdX, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dg, sdg, rtol=1e-12, atol=1e-12)
    for e in range(E_tgt):
        np.testing.assert_allclose(dW[e][0], sdWgu[e], rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(dW[e][1], sdWd[e], rtol=1e-12, atol=1e-12)

