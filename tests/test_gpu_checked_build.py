"""The checked build of the library (the same sources compiled with the index tests in, libgrouter_debug.so): on valid
inputs it computes what the release build computes, against the oracle, and reports nothing; an entry of the caller's
permutation arrays that points outside them is reported through the status word and not followed, and the context
works on afterwards."""
import numpy as np
import pytest
import torch

from oracle import grouter_oracle as orc
from paper_2603_06626_b200 import synth
from tests.gpu_util import bits_to_bf16, to_dev
from tests.test_gpu_layer import check_full, run_gpu

pytestmark = pytest.mark.gpu
ERR_BOUNDS = -9


def test_release_build_carries_no_index_tests(request):
    from paper_2603_06626_b200 import binding
    if request.config.getoption("--checked-build"):
        pytest.skip("the session runs on the checked build")
    assert binding.load_library().grouter_checked_build() == 0
    with binding.checked_build() as lib:
        assert lib.grouter_checked_build() == 1
        assert binding.strerror(ERR_BOUNDS).startswith("checked build")
    assert binding.load_library().grouter_checked_build() == 0


@pytest.mark.parametrize("case", ["tiny", "fold_dead", "fused_combine"])
def test_checked_build_matches_the_oracle_and_reports_nothing(case):
    from paper_2603_06626_b200 import binding
    flags = 0
    if case == "tiny":
        w = synth.WORKLOADS["tiny"]
    elif case == "fold_dead":     # fold collisions, experts without slots, ragged sizes
        w = synth.custom_workload("chk", T=700, d=264, ffn=200, E=24, k=4, load="zipf", zipf_s=1.3, n_dead=5, E_tgt=10, fold_mod=10, seed=31)
    else:
        w = synth.custom_workload("chk", T=900, d=512, ffn=384, E=12, k=3, seed=32)
        flags = binding.FLAG_FUSED_COMBINE
    li = synth.make_layer_inputs(w)
    with binding.checked_build():
        out = run_gpu(w, li, flags=flags)      # check_status inside: any reported index fails the test
    check_full(w, li, out)


def test_both_builds_give_the_same_bits(request):
    """No expert of this workload is split into chunks, so nothing depends on the order of atomic adds."""
    from paper_2603_06626_b200 import binding
    if request.config.getoption("--checked-build"):
        pytest.skip("the session runs on the checked build")
    w = synth.custom_workload("chk", T=1100, d=320, ffn=264, E=20, k=4, load="zipf", zipf_s=1.2, n_dead=3, seed=33)
    li = synth.make_layer_inputs(w)
    release = run_gpu(w, li)
    with binding.checked_build():
        checked = run_gpu(w, li)
    for name in ("Y", "dX", "dgates", "dW_gu", "dW_d"):
        assert torch.equal(release[name], checked[name]), name


@pytest.mark.parametrize("T,k,E", [(131203, 8, 128), (40000, 6, 200)])
def test_checked_plan_bit_exact(T, k, E):
    from paper_2603_06626_b200 import binding
    rng = np.random.default_rng(T + E)
    idx = (rng.random((T, k)) ** 3 * E).astype(np.uint8)
    with binding.checked_build():
        layer = binding.GrouterLayer(T, 8, 8, E, k, plan_only=True)
        got = [o.cpu().numpy() for o in layer.plan(to_dev(idx))]
        assert layer.status() == 0
        layer.close()
    for g, want in zip(got, orc.plan(idx, None, E)):
        assert np.array_equal(g, want)


def test_entry_outside_the_arrays_is_reported_and_not_followed():
    from paper_2603_06626_b200 import binding
    w = synth.WORKLOADS["tiny"]
    li = synth.make_layer_inputs(w)
    R = w.T * w.k
    with binding.checked_build():
        layer = binding.GrouterLayer(w.T, w.d, w.ffn, w.E_src, w.k, E_tgt=w.E_tgt)
        idx = to_dev(li.idx)
        gates, X, dY = bits_to_bf16(li.gates), bits_to_bf16(li.X), bits_to_bf16(li.dY)
        W_gu, W_d = bits_to_bf16(li.W_gu), bits_to_bf16(li.W_d)
        # slot_to_row is the caller's array, read again by the row movers of forward and backward
        layer.plan(idx)
        layer.slot_to_row[5] = R + 12345
        layer.slot_to_row[77] = -3
        Y = layer.forward(X, gates, W_gu, W_d)
        assert layer.status() == ERR_BOUNDS
        assert torch.isfinite(Y).all()
        assert layer.status() == 0                     # reading the status cleared it
        # row_to_slot is read by the GEMM epilogues (the slot's gate)
        layer.plan(idx)
        layer.row_to_slot[9] = 1 << 30
        layer.forward(X, gates, W_gu, W_d)
        assert layer.status() == ERR_BOUNDS
        # the context is none the worse: a fresh plan, a whole step, the oracle's results
        layer.plan(idx)
        Y = layer.forward(X, gates, W_gu, W_d)
        dX, dW_gu, dW_d, dgates = layer.backward(dY, X, gates, W_gu, W_d)
        layer.check_status()
        out = dict(Y=Y, dX=dX, dW_gu=dW_gu, dW_d=dW_d, dgates=dgates, counts=layer.counts.cpu().numpy())
        layer.close()
    check_full(w, li, out)
