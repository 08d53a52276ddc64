"""grouter_routing_stats against the statistics oracle: every integer result bit-exact, phi to float rounding."""
import numpy as np
import pytest
import torch

from oracle import stats_oracle as so
from paper_2603_06626_b200 import synth
from tests.gpu_util import to_dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,seq_len,n_nodes,i32", [("tiny", 64, 2, False), ("small", 512, 4, True), ("skewed", 2048, 8, False),
                                                       ("large", 4096, 16, False)])
def test_stats_match_oracle(name, seq_len, n_nodes, i32):
    from paper_2603_06626_b200 import binding
    w = synth.WORKLOADS[name]
    idx = synth.make_idx(w)
    if name in ("skewed", "large"):
        idx = idx[: 4 * seq_len]                      # the oracle is a pure-Python loop
    node = (np.random.default_rng(w.seed).permutation(w.E_src) % n_nodes).astype(np.int32)
    got = binding.routing_stats(to_dev(idx.astype(np.int32) if i32 else idx), w.E_src, seq_len, to_dev(node), n_nodes)
    assert got["status"] == 0
    L = so.loads(idx, w.E_src)
    assert np.array_equal(got["loads"].cpu().numpy(), L)
    assert np.array_equal(got["coact"].cpu().numpy(), so.coactivation(idx, w.E_src))
    phi = so.affinity_vectors(idx, w.E_src, seq_len)
    assert np.abs(got["phi"].cpu().numpy().astype(np.float64) - phi).max() <= 2.0 ** -24
    assert abs(float(got["max_vio"].item()) - so.max_vio(L)) <= 1e-6 * max(1.0, so.max_vio(L))
    comm = so.local_tokens(idx, node, n_nodes, seq_len)
    assert np.array_equal(got["local_tokens"].cpu().numpy(), comm)
    assert np.array_equal(got["best_node"].cpu().numpy(), so.place_samples(comm))


def test_stats_many_experts_repeated_ids_and_bad_ids():
    from paper_2603_06626_b200 import binding
    rng = np.random.default_rng(9)
    idx = rng.integers(0, 600, size=(1024, 5)).astype(np.int32)          # repeats within a token occur; P goes through global atomics
    idx[3] = [7, 7, 7, 9, 9]
    got = binding.routing_stats(to_dev(idx), 600, 128)
    assert got["status"] == 0
    assert np.array_equal(got["coact"].cpu().numpy(), so.coactivation(idx, 600))
    assert np.array_equal(got["loads"].cpu().numpy(), so.loads(idx, 600))
    bad = np.zeros((64, 2), dtype=np.uint8)
    bad[:, 1] = 1
    bad[5, 0] = 99
    got = binding.routing_stats(to_dev(bad), 8, 64)
    assert got["status"] == 1 and int(got["loads"].sum().item()) == 64 * 2 - 1      # the bad id is skipped, nothing faults
    with pytest.raises(binding.GrouterError):
        binding.routing_stats(to_dev(bad), 8, 48)                                    # T is not a whole number of samples


def test_greedy_fold_on_host_matches_oracle_and_feeds_the_router():
    from paper_2603_06626_b200 import binding
    w = synth.WORKLOADS["fine_fold"]
    idx = synth.make_idx(w)[:4096]
    P = binding.routing_stats(to_dev(idx), w.E_src, 1024)["coact"].cpu().numpy()
    P_oracle = so.coactivation(idx, w.E_src)              # the oracle folds its own matrix, never the CUDA path's
    assert np.array_equal(P, P_oracle)
    for E_T in (16, 24, 64, 1):
        fold = binding.fold_greedy(P, E_T)
        assert np.array_equal(fold, so.greedy_fold(P_oracle, E_T))
    rng = np.random.default_rng(1)
    A = rng.integers(0, 1000, size=(37, 37))
    assert np.array_equal(binding.fold_greedy(A + A.T, 5), so.greedy_fold(A + A.T, 5))
    with pytest.raises(binding.GrouterError):
        binding.fold_greedy(P_oracle, w.E_src + 1)
