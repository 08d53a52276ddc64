"""grouter_fold_greedy_host (host code of the library, no GPU needed) against the oracle's greedy affinity folding."""
import numpy as np
import pytest

from oracle import stats_oracle as so


@pytest.mark.parametrize("E_S,E_T,seed", [(5, 2, 0), (23, 4, 1), (64, 16, 2), (128, 24, 3), (9, 9, 4), (12, 1, 5)])
def test_host_fold_matches_oracle(E_S, E_T, seed):
    from paper_2603_06626_b200 import binding
    rng = np.random.default_rng(seed)
    A = rng.integers(0, 40, size=(E_S, E_S))            # small range: equal affinity sums do occur
    P = (A + A.T).astype(np.int32)
    fold = binding.fold_greedy(P, E_T)
    assert np.array_equal(fold, so.greedy_fold(P, E_T))
    sizes = np.bincount(fold, minlength=E_T)
    assert sizes.min() == E_S // E_T and sizes.max() == E_S // E_T + (1 if E_S % E_T else 0)


def test_host_fold_rejects_more_targets_than_sources():
    from paper_2603_06626_b200 import binding
    with pytest.raises(binding.GrouterError) as e:
        binding.fold_greedy(np.zeros((4, 4), dtype=np.int32), 5)
    assert e.value.code == -1
