"""Equivalent-steps cost report (Sec. 3.3): the oracle against closed forms and a hand-computed
trajectory at the paper's measured reductions (Appendix, hyper-parameter table: cache 0.95, sparse
candidates 0.05 / 0.07 / 0.10), then the library's host routine against the oracle."""
import numpy as np
import pytest

import oracle
from paper_2509_22323_b200 import binding

SKIP, REUSE, ATTEND = 0, 1, 2


def test_oracle_closed_forms():
    n = 28
    assert oracle.equivalent_steps([ATTEND] * n, [0.95] * n, [0.0] * n) == (28.0, 28)     # nothing saved
    assert oracle.equivalent_steps([SKIP] * n, [0.95] * n, [0.1] * n) == (0.0, 0)         # nothing runs
    k, kr = oracle.equivalent_steps([REUSE] * n, [0.95] * n, [0.1] * n)                   # sparse term plays no part
    assert k == pytest.approx(28 * (1 - float(np.float32(0.95))), abs=1e-12) and kr == 1
    k, _ = oracle.equivalent_steps([ATTEND] * n, [0.95] * n, [0.1] * n)                   # cache term plays no part
    assert k == pytest.approx(28 * (1 - float(np.float32(0.1))), abs=1e-12)
    assert oracle.equivalent_steps([], [], []) == (0.0, 0)


def test_oracle_hand_trajectory():
    # 28 scheduled steps: 6 skipped, 8 reuse the cache, 5 dense, 4 / 3 / 2 at the three candidates
    acts = [SKIP] * 6 + [REUSE] * 8 + [ATTEND] * 14
    c_sparse = [0.0] * 14 + [0.0] * 5 + [0.05] * 4 + [0.07] * 3 + [0.10] * 2
    k, kr = oracle.equivalent_steps(acts, [0.95] * 28, c_sparse)
    # 8 * 0.05 + 5 + 4 * 0.95 + 3 * 0.93 + 2 * 0.90 = 13.79
    assert k == pytest.approx(13.79, abs=1e-6) and kr == 14
    # order of the steps does not matter, and halves round upward
    perm = np.random.default_rng(0).permutation(28)
    k2, _ = oracle.equivalent_steps([acts[i] for i in perm], [0.95] * 28, [c_sparse[i] for i in perm])
    assert k2 == pytest.approx(k, abs=1e-12)
    assert oracle.equivalent_steps([ATTEND, ATTEND, ATTEND], [0.0] * 3, [0.5, 0.0, 0.0]) == (2.5, 3)


def test_library_matches_oracle():
    rng = np.random.default_rng(3)
    for n in (0, 1, 28, 50, 1000):
        acts = rng.integers(0, 3, n).tolist()
        cc = rng.uniform(0, 1, n).astype(np.float32).tolist()
        cs = rng.choice([0.0, 0.05, 0.07, 0.10], n).astype(np.float32).tolist()
        k, kr = binding.rapid3_equivalent_steps(acts, cc, cs)
        ko, kro = oracle.equivalent_steps(acts, cc, cs)
        assert k == pytest.approx(ko, rel=1e-13, abs=1e-13) and kr == kro
    for bad in (([3], [0.5], [0.5]), ([REUSE], [1.5], [0.0]), ([ATTEND], [0.0], [-0.1]), ([ATTEND], [0.0], [float("nan")])):
        with pytest.raises(binding.Rapid3Error) as e:
            binding.rapid3_equivalent_steps(*bad)
        assert e.value.code == -1
    assert binding.rapid3_equivalent_steps([SKIP], [7.0], [-3.0]) == (0.0, 0)            # a skipped step's entries are ignored
