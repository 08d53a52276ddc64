"""grouter_route against the router-head oracle (Eq. 2 with the score-layer fold).

The kept ids are an arg-max over floating-point scores: the CUDA path accumulates them in fp32, the oracle in fp64.
Where the oracle's k-th and (k+1)-th score (or two kept neighbours) are further apart than the fp32 error bound, the
ids must be identical, in order; on the few tokens that are closer, any order of the near-equal experts is accepted as
long as every kept expert's exact score is within the bound of the exact k-th score.  Folded scores are compared
element by element; coefficients to bf16 rounding.  Synthetic hidden states ~ N(0,1) and a score layer ~ N(0, 1/d_h)
stand in for the distilled router, whose weights are not available.
"""
import numpy as np
import pytest
import torch

from oracle import router_oracle as ro
from paper_2603_06626_b200 import synth
from tests.gpu_util import bits_to_bf16, to_dev

pytestmark = pytest.mark.gpu


def _inputs(seed, T, dh, E_src):
    rng = np.random.default_rng(seed)
    H = synth.f32_to_bf16_bits(rng.standard_normal((T, dh), dtype=np.float32))
    W = synth.f32_to_bf16_bits((rng.standard_normal((E_src, dh)) / np.sqrt(dh)).astype(np.float32))
    return H, W


def _check(T, dh, E_src, E_tgt, k, norm, fold, seed):
    from paper_2603_06626_b200 import binding
    H, W = _inputs(seed, T, dh, E_src)
    fm = None
    if fold == "mod":
        fm = (np.arange(E_src) % E_tgt).astype(np.int32)
    elif fold == "random":
        fm = np.random.default_rng(seed + 1).integers(0, E_tgt, size=E_src).astype(np.int32)
    idx, gates, S = binding.route(bits_to_bf16(H), bits_to_bf16(W), None if fm is None else to_dev(fm), E_tgt, k, norm, want_scores=True)
    idx = idx.cpu().numpy().astype(np.int64)
    gates = gates.float().cpu().numpy().astype(np.float64)
    S = S.cpu().numpy().astype(np.float64)

    ids_o, r_o, S_o = ro.route(synth.bf16_bits_to_f64(H), synth.bf16_bits_to_f64(W), fm, E_tgt, k, norm)
    # fp32 accumulation over d_h products and the group sum: |error| <= (d_h + group) * 2^-24 * sum |terms|, far below this
    bound = 4e-6 * max(1.0, np.abs(S_o).max())
    assert np.abs(S - S_o).max() < bound

    order = np.sort(S_o, axis=1)[:, ::-1]
    kth = order[:, k - 1]
    gaps = np.abs(np.diff(order[:, : min(k + 1, E_tgt)], axis=1)).min(axis=1)     # smallest gap among the top k+1 exact scores
    clear = gaps > 4 * bound
    assert clear.mean() > 0.6                            # most tokens have no near-tie (k = 32 of 256 has the most)
    assert np.array_equal(idx[clear], ids_o[clear])
    for t in np.nonzero(~clear)[0]:                      # near-ties: a valid top-k set in some order of the tied experts
        assert len(set(idx[t].tolist())) == k
        assert np.all(S_o[t, idx[t]] >= kth[t] - 4 * bound)
    # coefficients: bf16 of the normalised kept scores (one bf16 ulp of slack for the fp32/fp64 rounding boundary)
    assert np.abs(gates[clear] - r_o[clear]).max() <= 2.0 ** -8 * 1.01
    want_bits = ro.to_bf16_bits(r_o[clear]).astype(np.int64)
    got_bits = synth.f32_to_bf16_bits(gates[clear].astype(np.float32)).astype(np.int64)
    assert np.abs(got_bits - want_bits).max() <= 1 and (got_bits == want_bits).mean() > 0.98
    if norm == ro.SOFTMAX:
        assert np.abs(gates.sum(axis=1) - 1.0).max() < k * 2.0 ** -8


@pytest.mark.parametrize("T,dh,E_src,E_tgt,k,norm,fold", [
    (512, 64, 8, 8, 2, ro.SOFTMAX, None),
    (1000, 512, 128, 128, 8, ro.SOFTMAX, None),          # the paper's router width (512) and a Qwen3-like expert count
    (1000, 512, 128, 16, 4, ro.SOFTMAX, "mod"),          # 128 source experts folded onto 16
    (777 * 8, 256, 64, 24, 6, ro.SIGMOID, "random"),     # uneven groups, some targets possibly empty
    (264, 512, 256, 256, 32, ro.SOFTMAX, None),          # the widest id range and the largest k
    (128, 72, 1024, 7, 7, ro.SIGMOID, "mod"),            # k == E_tgt, E_tgt not a multiple of anything
])
def test_route_matches_oracle(T, dh, E_src, E_tgt, k, norm, fold):
    _check(T, dh, E_src, E_tgt, k, norm, fold, seed=T + dh + E_src)


def test_route_feeds_the_plan_and_reports_bad_fold_targets():
    from paper_2603_06626_b200 import binding
    T, dh, E_src, E_tgt, k = 2048, 128, 64, 16, 4
    H, W = _inputs(3, T, dh, E_src)
    fm = (np.arange(E_src) % E_tgt).astype(np.int32)
    idx, gates, _ = binding.route(bits_to_bf16(H), bits_to_bf16(W), to_dev(fm), E_tgt, k)
    assert int(idx.max()) < E_tgt
    rows = idx.cpu().numpy()
    assert all(len(set(r)) == k for r in rows.tolist())              # folded before top-k: no target twice
    layer = binding.GrouterLayer(T, 64, 64, E_tgt, k)
    counts, offsets, _, _ = layer.plan(idx)                          # the cache record is exactly what the plan consumes
    assert layer.status() == 0 and int(counts.sum()) == T * k
    layer.close()
    bad = fm.copy()
    bad[5] = E_tgt + 3
    with pytest.raises(binding.GrouterError) as e:
        binding.route(bits_to_bf16(H), bits_to_bf16(W), to_dev(bad), E_tgt, k)
    assert e.value.code == -6
    with pytest.raises(binding.GrouterError) as e:
        binding.route(bits_to_bf16(H), bits_to_bf16(W), None, E_tgt, k)      # E_src != E_tgt without a fold map
    assert e.value.code == -1
