"""grouter_moe_step_host (host buffers in and out, copies pipelined against the compute) against the device-resident
calls: the same kernels run on the same bits, so the results must be identical, also when consecutive steps with
different inputs are in flight together and share the two device staging sets.  The last step's host results are also
checked against the oracle, so the host path does not rest on the device path alone."""
import numpy as np
import pytest
import torch

from paper_2603_06626_b200 import synth
from tests.gpu_util import bits_to_bf16, to_dev

pytestmark = pytest.mark.gpu


def _pinned(a):
    return torch.from_numpy(np.ascontiguousarray(a)).pin_memory()


@pytest.mark.parametrize("name,n_steps", [("tiny", 5), ("small", 4)])
def test_step_host_matches_device_calls_with_steps_in_flight(name, n_steps):
    from paper_2603_06626_b200 import binding
    base = synth.WORKLOADS[name]
    dev = "cuda:0"
    W_gu = bits_to_bf16(np.stack([synth.expert_W_gu(base, e) for e in range(base.E_tgt)]))
    W_d = bits_to_bf16(np.stack([synth.expert_W_d(base, e) for e in range(base.E_tgt)]))
    steps = [synth.make_layer_inputs(synth.reseeded(base, 100 + i), with_weights=False) for i in range(n_steps)]

    # expected: plan + fwd + bwd on device tensors, one step at a time
    ref_layer = binding.GrouterLayer(base.T, base.d, base.ffn, base.E_src, base.k, E_tgt=base.E_tgt)
    expected = []
    for li in steps:
        idx, gates, X, dY = to_dev(li.idx), bits_to_bf16(li.gates), bits_to_bf16(li.X), bits_to_bf16(li.dY)
        ref_layer.plan(idx)
        Y = ref_layer.forward(X, gates, W_gu, W_d)
        dX, dW_gu, dW_d, dg = ref_layer.backward(dY, X, gates, W_gu, W_d)
        ref_layer.check_status()
        expected.append([t.cpu() for t in (Y.view(torch.int16), dX.view(torch.int16), dg, dW_gu, dW_d)])
    ref_layer.close()

    layer = binding.GrouterLayer(base.T, base.d, base.ffn, base.E_src, base.k, E_tgt=base.E_tgt, host_staging=True)
    dW_gu = torch.empty(W_gu.shape, dtype=torch.float32, device=dev)
    dW_d = torch.empty(W_d.shape, dtype=torch.float32, device=dev)
    host = []
    for li in steps:      # every step has its own host buffers here, so all of them can be checked at the end
        host.append(dict(idx=_pinned(li.idx), gates=_pinned(li.gates.view(np.int16)), X=_pinned(li.X.view(np.int16)),
                         dY=_pinned(li.dY.view(np.int16)),
                         Y=torch.full((base.T, base.d), 0x7FC0, dtype=torch.int16).pin_memory(),
                         dX=torch.full((base.T, base.d), 0x7FC0, dtype=torch.int16).pin_memory(),
                         dg=torch.full((base.T, base.k), float("nan"), dtype=torch.float32).pin_memory()))
    for i, h in enumerate(host):
        layer.step_host(h["idx"], h["gates"], h["X"], h["dY"], None, W_gu, W_d, h["Y"], h["dX"], h["dg"], dW_gu, dW_d)
        layer.host_wait(1)
        if i >= 1:          # step i-1 is complete while step i may still be running
            p = host[i - 1]
            assert torch.equal(p["Y"], expected[i - 1][0]) and torch.equal(p["dX"], expected[i - 1][1])
            assert torch.equal(p["dg"], expected[i - 1][2])
    layer.host_wait(0)
    layer.check_status()
    h = host[-1]
    assert torch.equal(h["Y"], expected[-1][0]) and torch.equal(h["dX"], expected[-1][1]) and torch.equal(h["dg"], expected[-1][2])
    # an expert whose rows span several chunks has its gradient summed from partial tiles with fp32 atomics, whose order
    # is not fixed: equal up to that reordering
    for got, want in ((dW_gu.cpu(), expected[-1][3]), (dW_d.cpu(), expected[-1][4])):
        assert (got - want).double().norm() <= 1e-6 * want.double().norm()
    # the last step against the oracle (weights drawn from `base`, the step's other inputs from its own seed)
    from dataclasses import replace
    from tests.test_gpu_layer import check_full
    li = replace(steps[-1], W_gu=np.stack([synth.expert_W_gu(base, e) for e in range(base.E_tgt)]),
                 W_d=np.stack([synth.expert_W_d(base, e) for e in range(base.E_tgt)]))
    out = dict(Y=h["Y"].view(torch.bfloat16), dX=h["dX"].view(torch.bfloat16), dgates=h["dg"], dW_gu=dW_gu.cpu(), dW_d=dW_d.cpu(),
               counts=np.bincount(li.idx.reshape(-1), minlength=base.E_tgt))
    check_full(base, li, out)
    layer.close()
