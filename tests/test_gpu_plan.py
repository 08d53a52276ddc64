"""Plan kernels against the oracle: all four arrays bit-exact."""
import numpy as np
import pytest
import torch

from oracle import grouter_oracle as orc
from paper_2603_06626_b200 import synth
from tests.gpu_util import to_dev

pytestmark = pytest.mark.gpu


def _run_plan(idx, fold_map, E_src, E_tgt, idx_i32=False, plan_only=False):
    from paper_2603_06626_b200 import binding
    T, k = idx.shape
    idx_np = idx.astype(np.int32) if idx_i32 else idx.astype(np.uint8)
    layer = binding.GrouterLayer(T, 64, 64, E_src, k, E_tgt=E_tgt, plan_only=plan_only,
                                 idx_dtype=binding.IDX_I32 if idx_i32 else binding.IDX_U8)
    fm = None if fold_map is None else to_dev(fold_map.astype(np.int32))
    out = layer.plan(to_dev(idx_np), fm)
    st = layer.status()
    res = [o.cpu().numpy() for o in out]
    layer.close()
    return res, st


def _assert_equal(got, want):
    for g, w, name in zip(got, want, ["counts", "offsets", "row_to_slot", "slot_to_row"]):
        assert g.dtype == np.int32
        assert np.array_equal(g, w), name


@pytest.mark.parametrize("name", synth.WORKLOAD_ORDER)
def test_plan_workloads_bit_exact(name):
    w = synth.WORKLOADS[name]
    idx, fm = synth.make_idx(w), synth.make_fold_map(w)
    got, st = _run_plan(idx, fm, w.E_src, w.E_tgt)
    assert st == 0
    _assert_equal(got, orc.plan(idx, fm, w.E_tgt))


@pytest.mark.parametrize("T,k,E", [(1, 1, 1), (33, 1, 2), (1000, 3, 7), (4097, 2, 256), (777, 8, 128), (5000, 4, 1000)])
def test_plan_ragged_sizes(T, k, E):
    rng = np.random.default_rng(T + k + E)
    idx = rng.integers(0, E, size=(T, k))
    got, st = _run_plan(idx, None, E, E, idx_i32=E > 256)
    assert st == 0
    _assert_equal(got, orc.plan(idx, None, E))


@pytest.mark.parametrize("T,k,E,kind", [
    (131203, 8, 128, "u8"),        # just above 2^20 slots: runs of 32 slots per thread, ragged last block
    (131203, 8, 200, "fold_i32"),  # the same run length with 32-bit ids and a fold map onto 37 experts
    (524301, 8, 128, "u8"),        # just above 2^22 slots: runs of 64 slots per thread, ragged last block
    (600011, 7, 256, "skew"),      # 256 experts, most slots on a few of them (long runs of one expert inside a block)
])
def test_plan_longer_runs_per_thread_bit_exact(T, k, E, kind):
    """The permutation kernel gives a thread 16, 32 or 64 consecutive slots depending on the problem size; the two longer
    forms only appear above a million slots."""
    rng = np.random.default_rng(T + E)
    fm, E_tgt = None, E
    if kind == "skew":
        idx = (rng.random((T, k)) ** 6 * E).astype(np.int64)
    else:
        idx = rng.integers(0, E, size=(T, k))
    if kind == "fold_i32":
        E_tgt = 37
        fm = rng.integers(0, E_tgt, size=E)
    got, st = _run_plan(idx, fm, E, E_tgt, idx_i32=(kind == "fold_i32"))
    assert st == 0
    _assert_equal(got, orc.plan(idx, fm, E_tgt))


@pytest.mark.parametrize("T,k,E,kind", [
    (2500003, 8, 128, "u8"),       # 1221 chunks of 16384 slots, ragged last one
    (2600001, 8, 256, "skew_fold"),  # 8-bit ids folded onto 96 experts, most slots on a few of them
])
def test_plan_many_chunks_per_block_bit_exact(T, k, E, kind):
    """With more than eight chunks per SM the permutation kernel's blocks stay resident and take several chunks in turn,
    fetching the next one's ids while the current one is written out."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert -(-T * k // 16384) > 8 * sms, "the case no longer reaches the resident form on this GPU"
    rng = np.random.default_rng(T + E)
    fm, E_tgt = None, E
    if kind == "skew_fold":
        idx = (rng.random((T, k)) ** 5 * E).astype(np.int64)
        E_tgt = 96
        fm = rng.integers(0, E_tgt, size=E)
    else:
        idx = rng.integers(0, E, size=(T, k))
    got, st = _run_plan(idx, fm, E, E_tgt, plan_only=True)
    assert st == 0
    _assert_equal(got, orc.plan(idx, fm, E_tgt))


def test_plan_degenerate_and_i32():
    idx = np.full((3000, 2), 5)
    got, st = _run_plan(idx, None, 9, 9)
    assert st == 0
    _assert_equal(got, orc.plan(idx, None, 9))
    rng = np.random.default_rng(3)
    idx = rng.integers(0, 40, size=(2500, 4))
    fm = rng.integers(0, 6, size=40)
    for i32 in (False, True):
        got, st = _run_plan(idx, fm, 40, 6, idx_i32=i32)
        assert st == 0
        _assert_equal(got, orc.plan(idx, fm, 6))


def test_plan_reproducible_and_reusable():
    from paper_2603_06626_b200 import binding
    w = synth.WORKLOADS["skewed"]
    idx = to_dev(synth.make_idx(w))
    layer = binding.GrouterLayer(w.T, 64, 64, w.E_src, w.k)
    first = [o.clone() for o in layer.plan(idx)]
    for _ in range(3):
        again = layer.plan(idx)
        for a, b in zip(first, again):
            assert torch.equal(a, b)
    assert layer.status() == 0
    layer.close()


def test_plan_bad_index_sets_status_without_fault():
    from paper_2603_06626_b200 import binding
    idx = np.zeros((100, 2), dtype=np.uint8)
    idx[7, 1] = 200                                  # >= E_src
    got, st = _run_plan(idx, None, 8, 8)
    assert st == -6
    assert got[0].sum() == 200                        # every slot still counted (bad id treated as expert 0)
    got, st = _run_plan(np.zeros((100, 2), dtype=np.uint8), None, 8, 8)
    assert st == 0                                    # status is cleared by the previous read, and contexts are separate


def test_plan_range_checks_of_every_form():
    """Ids are range-checked four at a time when there is no fold map (two bounds: up to 128 ids, and above), one by one
    otherwise; a fold target out of range is reported only when a slot uses it; the ballot form serves more than 4096
    source ids.  Every bad slot counts as expert 0 and the rest of the plan is still exact."""
    rng = np.random.default_rng(9)
    for E in (100, 200):                                            # both branches of the four-at-a-time check
        idx = rng.integers(0, E, size=(3001, 4))
        good, st = _run_plan(idx, None, E, E)
        assert st == 0
        _assert_equal(good, orc.plan(idx, None, E))
        bad = idx.copy()
        bad[1234, 2] = E + 3                                         # in range of uint8, out of range of the experts
        got, st = _run_plan(bad, None, E, E)
        assert st == -6
        fixed = bad.copy(); fixed[1234, 2] = 0
        _assert_equal(got, orc.plan(fixed, None, E))
    # fold table with one bad target: harmless while no slot uses that source id, reported once one does
    idx = rng.integers(0, 30, size=(2000, 3))
    fm = rng.integers(0, 6, size=40)
    fm[35] = 9
    got, st = _run_plan(idx, fm, 40, 6)
    assert st == 0
    _assert_equal(got, orc.plan(idx, np.where(fm < 6, fm, 0), 6))
    idx[77, 1] = 35
    got, st = _run_plan(idx, fm, 40, 6)
    assert st == -6
    _assert_equal(got, orc.plan(idx, np.where(fm < 6, fm, 0), 6))
    # more source ids than the fold table in shared memory holds: the ballot form
    idx = rng.integers(0, 5000, size=(1500, 2))
    fm = rng.integers(0, 16, size=5000)
    got, st = _run_plan(idx, fm, 5000, 16, idx_i32=True)
    assert st == 0
    _assert_equal(got, orc.plan(idx, fm, 16))


def test_host_side_errors():
    from paper_2603_06626_b200 import binding
    with pytest.raises(binding.GrouterError) as e:
        binding.GrouterLayer(16, 60, 64, 4, 2)         # d % 8 != 0
    assert e.value.code == -3
    with pytest.raises(binding.GrouterError) as e:
        binding.GrouterLayer(16, 64, 64, 300, 2)       # uint8 ids cannot address 300 experts
    assert e.value.code == -3
    layer = binding.GrouterLayer(16, 64, 64, 4, 2)
    X = torch.zeros(16, 64, dtype=torch.bfloat16, device="cuda:0")
    g = torch.zeros(16, 2, dtype=torch.bfloat16, device="cuda:0")
    W_gu = torch.zeros(4, 128, 64, dtype=torch.bfloat16, device="cuda:0")
    W_d = torch.zeros(4, 64, 64, dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(binding.GrouterError) as e:
        layer.forward(X, g, W_gu, W_d)                 # no plan yet
    assert e.value.code == -4
    layer.close()


def test_kernel_timing_records_and_idle_gap():
    """The per-kernel timing aid: one event pair per launch, with or without idle time between launches."""
    import time
    from paper_2603_06626_b200 import binding
    w = synth.WORKLOADS["tiny"]
    idx = to_dev(synth.make_idx(w))
    layer = binding.GrouterLayer(w.T, 64, 64, w.E_src, w.k)
    layer.plan(idx)
    layer.timing_enable(8)
    layer.timing_gap(20000)                    # 20 ms after each of the three plan kernels
    torch.cuda.synchronize()
    t0 = time.time()
    layer.plan(idx)
    rec = layer.timing_read()
    waited = time.time() - t0
    assert rec["plan_hist"][1] == 1 and rec["plan_scan"][1] == 1 and rec["plan_permute"][1] == 1 and rec["plan_hist"][0] > 0
    assert rec["plan_hist"][0] < 5.0           # the idle time is not part of the kernel's own record
    assert waited >= 0.035
    layer.timing_gap(0)
    layer.plan(idx)
    assert layer.timing_read()["plan_permute"][1] == 1
    layer.timing_enable(0)
    with pytest.raises(binding.GrouterError):
        layer.timing_gap(-1)
    assert layer.status() == 0
    layer.close()


def test_weight_gradient_chunk_length_follows_the_problem_size():
    """Long chunks (few partial sums) when the batch gives every CTA pair tiles anyway, short ones for small problems."""
    from paper_2603_06626_b200 import binding
    got = {}
    for name in ("tiny", "small", "skewed", "large"):
        w = synth.WORKLOADS[name]
        layer = binding.GrouterLayer(w.T, w.d, w.ffn, w.E_src, w.k, E_tgt=w.E_tgt)
        got[name] = layer.wgrad_chunk_rows()
        layer.close()
    assert all(1024 <= v <= 16384 and v & (v - 1) == 0 for v in got.values()), got
    assert got["tiny"] == 1024 and got["large"] == 16384 and got["small"] <= got["skewed"], got
