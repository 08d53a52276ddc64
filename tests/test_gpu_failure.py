"""Failure reporting of the device side, made to happen without faulting or hanging anything.

Every wait inside the kernels (operand stage, accumulator, next tile number) is bounded: when it runs out the kernel
sets the timeout bit of the status word and returns.  The self-test kernel makes exactly that happen in isolation: one
thread waits on a barrier that nothing ever arrives at, with a limit of a millisecond."""
import time

import numpy as np
import pytest
import torch

from oracle import grouter_oracle as orc
from paper_2603_06626_b200 import synth
from tests.gpu_util import bits_to_bf16, to_dev

pytestmark = pytest.mark.gpu


def test_bounded_wait_runs_out_reports_timeout_and_leaves_the_context_usable():
    from paper_2603_06626_b200 import binding
    w = synth.WORKLOADS["tiny"]
    li = synth.make_layer_inputs(w)
    layer = binding.GrouterLayer(w.T, w.d, w.ffn, w.E_src, w.k, E_tgt=w.E_tgt)
    idx, gates, X, dY = to_dev(li.idx), bits_to_bf16(li.gates), bits_to_bf16(li.X), bits_to_bf16(li.dY)
    W_gu, W_d = bits_to_bf16(li.W_gu), bits_to_bf16(li.W_d)

    def step():
        layer.plan(idx)
        Y = layer.forward(X, gates, W_gu, W_d)
        return Y, layer.backward(dY, X, gates, W_gu, W_d)

    Y0, _ = step()
    assert layer.status() == 0
    torch.cuda.synchronize()
    t0 = time.time()
    waited = layer.wait_selftest(1000)                  # a 1 ms limit on a wait that cannot succeed
    wall = time.time() - t0
    assert 1000 <= waited < 100000, waited              # gave up at the limit (checked every 128 polls), not seconds later
    assert wall < 5.0
    assert layer.status() == -7                         # GROUTER_ERR_TIMEOUT, reported once ...
    assert "wait" in binding.strerror(-7)
    assert layer.status() == 0                          # ... and cleared
    # the context, its status word and its tile counter are in working order afterwards
    layer.set_wait_limit(2_000_000)
    Y1, (dX1, dW_gu1, dW_d1, dg1) = step()
    assert layer.status() == 0
    assert torch.equal(Y0, Y1)
    f64 = synth.bf16_bits_to_f64
    want = orc.moe_forward(f64(li.X), li.idx, f64(li.gates), orc.Weights(f64(li.W_gu), f64(li.W_d)), w.E_tgt)
    assert orc.rel_frobenius(Y1.double().cpu().numpy(), want) < 1e-2
    for bad in (0, -5, 2_000_000):
        with pytest.raises(binding.GrouterError):
            layer.wait_selftest(bad)
    with pytest.raises(binding.GrouterError):
        layer.set_wait_limit(0)
    layer.close()
