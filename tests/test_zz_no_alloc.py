"""grouter_plan_noalloc against grouter_plan: the context-free, allocation-free plan build.

Some hosts cannot create a context because grouter_create calls cudaMalloc (all device memory already belongs
to a pooling allocator, a fixed memory budget, or a loop that cannot take an allocation's device-wide
synchronisation).  They call grouter_plan_noalloc, whose scratch is a fixed array inside the library.  This test
drives it through the C ABI with caller-owned outputs and checks that it returns exactly what the context-based
entry point returns (integer work: bit-exact, the same bar as the other plan tests), on two calls in a row so
that whatever the first call left in the shared scratch cannot leak into the second.

Collected last on purpose (file name): a run that stops at the first failure has then run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import grouter_oracle as orc
from paper_2603_06626_b200 import synth
from tests.gpu_util import to_dev

pytestmark = pytest.mark.gpu

NAMES = ["counts", "offsets", "row_to_slot", "slot_to_row"]


def _with_context(idx_np, fm_np, E_src, E_tgt):
    from paper_2603_06626_b200 import binding
    T, k = idx_np.shape
    layer = binding.GrouterLayer(T, 64, 64, E_src, k, E_tgt=E_tgt,
                                 idx_dtype=binding.IDX_U8 if idx_np.dtype == np.uint8 else binding.IDX_I32)
    fm = None if fm_np is None else to_dev(fm_np)
    out = [o.clone() for o in layer.plan(to_dev(idx_np), fm)]
    assert layer.status() == 0
    layer.close()
    return out


def test_noalloc_plan_matches_context_plan_twice_in_a_row():
    from paper_2603_06626_b200 import binding
    # first call: the largest benchmark routing table (R = 262144, E = 128); second: a smaller, folded, ragged one
    # that reuses the same scratch and must not see the first call's histograms, ticket or padded rows
    w1 = synth.WORKLOADS["large"]
    idx1 = synth.make_idx(w1)
    rng = np.random.default_rng(77)
    idx2 = rng.integers(0, 40, size=(2501, 3)).astype(np.uint8)
    fm2 = rng.integers(0, 6, size=40).astype(np.int32)
    cases = [(idx1, None, w1.E_src, w1.E_tgt), (idx2, fm2, 40, 6)]
    expected = [_with_context(*c) for c in cases]

    results = []
    for idx_np, fm_np, E_src, E_tgt in cases:                   # the two calls, back to back on one stream
        T, k = idx_np.shape
        i32 = dict(dtype=torch.int32, device="cuda:0")
        out = (torch.full((E_tgt,), -7, **i32), torch.full((E_tgt + 1,), -7, **i32),
               torch.full((T * k,), -7, **i32), torch.full((T * k,), -7, **i32))
        status = torch.full((1,), 99, **i32)                     # the call must clear it
        fm = None if fm_np is None else to_dev(fm_np)
        results.append(binding.plan_noalloc(to_dev(idx_np), fm, E_src, E_tgt, out=out, status=status))
    torch.cuda.synchronize()
    for got, want, (idx_np, fm_np, _, E_tgt) in zip(results, expected, cases):
        assert int(got[4].item()) == 0
        for g, w, name in zip(got[:4], want, NAMES):
            assert torch.equal(g, w), name
        for g, o, name in zip(got[:4], orc.plan(idx_np, fm_np, E_tgt), NAMES):      # and against the CPU oracle directly
            assert np.array_equal(g.cpu().numpy(), o), name

    # a bad id is reported through the caller's status word, nothing faults, every slot is still counted
    bad = np.zeros((100, 2), dtype=np.uint8)
    bad[7, 1] = 200
    got = binding.plan_noalloc(to_dev(bad), None, 8, 8)
    torch.cuda.synchronize()
    assert int(got[4].item()) == 1 and int(got[0].sum().item()) == 200
    # and the call after it starts clean again
    got = binding.plan_noalloc(to_dev(idx2), to_dev(fm2), 40, 6)
    torch.cuda.synchronize()
    assert int(got[4].item()) == 0
    for g, w, name in zip(got[:4], expected[1], NAMES):
        assert torch.equal(g, w), name


def test_noalloc_plan_at_the_limits_of_its_scratch_allocates_nothing():
    """The largest problem the fixed scratch is laid out for: T*k = 524288 slots over 256 experts, almost all of which
    get one or two rows (so the padded layout is at its longest), 32-bit ids, and no status word from the caller.
    Device memory in use must be the same before and after the call."""
    from paper_2603_06626_b200 import binding
    T, k, E = 65536, 8, 256
    rng = np.random.default_rng(5)
    idx_np = rng.integers(0, 2, size=(T, k)).astype(np.int32)           # two heavy experts ...
    light = rng.choice(T * k, size=380, replace=False)
    idx_np.reshape(-1)[light] = rng.integers(2, E, size=380)            # ... and 254 that get a row or two
    want = orc.plan(idx_np, None, E)
    assert (want[0][2:] <= 8).all() and (want[0] > 0).sum() > 150
    idx = to_dev(idx_np)
    i32 = dict(dtype=torch.int32, device="cuda:0")
    out = (torch.empty(E, **i32), torch.empty(E + 1, **i32), torch.empty(T * k, **i32), torch.empty(T * k, **i32))
    binding.plan_noalloc(idx, None, E, E, out=out, null_status=True)      # first call on the device: looks the scratch address up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for o in out:
        o.fill_(-7)
    got = binding.plan_noalloc(idx, None, E, E, out=out, null_status=True)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0 and got[4] is None
    for g, o, name in zip(got[:4], want, NAMES):
        assert np.array_equal(g.cpu().numpy(), o), name
    ctx = _with_context(idx_np, None, E, E)
    for g, c, name in zip(got[:4], ctx, NAMES):
        assert torch.equal(g, c), name


def test_noalloc_plan_rejects_sizes_beyond_its_scratch():
    from paper_2603_06626_b200 import binding
    idx = torch.zeros((65537, 8), dtype=torch.uint8, device="cuda:0")        # T*k = 524296 > 524288
    with pytest.raises(binding.GrouterError) as e:
        binding.plan_noalloc(idx, None, 16, 16)
    assert e.value.code == -3 and "unsupported" in str(e.value)
    idx = torch.zeros((64, 2), dtype=torch.int32, device="cuda:0")
    with pytest.raises(binding.GrouterError) as e:
        binding.plan_noalloc(idx, None, 300, 300)                               # E_tgt > 256
    assert e.value.code == -3
