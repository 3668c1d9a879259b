"""Pins of the oracle's cumulative-mass selection (the threshold variant of the block mask):
closed forms, the defining property checked with an independent computation, invariants, and
agreement with the (separately pinned) top-k selection at the count it arrives at."""
import math

import numpy as np
import pytest

import oracle


def free_candidates(nb, ntb, i):
    return [j for j in range(ntb, nb) if j != i]


@pytest.mark.parametrize("nb,n_text,tau", [(9, 64, 0.5), (12, 0, 0.3), (20, 130, 0.77), (70, 333, 0.123)])
def test_uniform_scores_keep_ceil_tau_n_lowest_indices(nb, n_text, tau):
    S = np.full((1, nb, nb), 0.37)
    mask, gap, k, margin = oracle.select_mask_mass(S, n_text, tau, 2.0)
    ntb = (n_text + 63) // 64
    for i in range(nb):
        free = free_candidates(nb, ntb, i)
        if i < ntb:
            assert mask[0, i].all() and k[0, i] == 0
            continue
        want = math.ceil(tau * len(free) - 1e-12)
        assert k[0, i] == want
        assert [j for j in free if mask[0, i, j]] == free[:want]      # equal scores: lowest block index first
        assert mask[0, i, :ntb].all() and mask[0, i, i]
        assert gap[0, i] == 0.0 or want == len(free)


def test_two_level_closed_form():
    # m candidates weigh twice the others (scores 1 and 0 at scale ln 2)
    nb, ntb, m = 14, 1, 4
    for tau in (0.1, 0.35, 0.55, 0.8, 0.97):
        S = np.zeros((1, nb, nb))
        i = 5
        free = free_candidates(nb, ntb, i)
        high = free[2:2 + m]
        S[0, i, high] = 1.0
        mask, _, k, _ = oracle.select_mask_mass(S, 64, tau, math.log(2.0))
        n = len(free)
        target = tau * (2 * m + (n - m))                              # in units of the low weight
        want = math.ceil(target / 2 - 1e-9) if target <= 2 * m else m + math.ceil(target - 2 * m - 1e-9)
        assert k[0, i] == want
        kept = [j for j in free if mask[0, i, j]]
        assert kept[:0] == [] and set(high[:min(want, m)]) <= set(kept)
        assert len(kept) == want


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_defining_property_independent_computation(seed):
    rng = np.random.default_rng(seed)
    nb, n_text, scale = 23, 100, 1.7
    ntb = 2
    S = rng.standard_normal((2, nb, nb)) * 2.0
    for tau in (0.05, 0.4, 0.75, 0.95):
        mask, gap, k, margin = oracle.select_mask_mass(S, n_text, tau, scale)
        for h in range(2):
            assert mask[h, :ntb].all()
            for i in range(ntb, nb):
                free = np.array(free_candidates(nb, ntb, i))
                s = S[h, i, free]
                w = np.exp(scale * (s - s.max()))
                kept = mask[h, i, free].astype(bool)
                assert kept.sum() == k[h, i] >= 1
                assert mask[h, i, :ntb].all() and mask[h, i, i]
                # enough mass, none to spare, and nothing dropped beats anything kept
                assert w[kept].sum() >= tau * w.sum() * (1 - 1e-12)
                weakest = s[kept].min()
                assert w[kept].sum() - math.exp(scale * (weakest - s.max())) < tau * w.sum() * (1 + 1e-12)
                if (~kept).any():
                    assert s[kept].min() >= s[~kept].max()
                    assert gap[h, i] == pytest.approx(s[kept].min() - s[~kept].max(), abs=1e-15)
                assert margin[h, i] >= 0


def test_nested_in_tau_and_limits():
    rng = np.random.default_rng(4)
    nb, n_text = 17, 64
    S = rng.standard_normal((1, nb, nb))
    prev = None
    for tau in (1e-9, 0.1, 0.3, 0.5, 0.7, 0.9, 0.999, 1.0):
        mask, _, k, margin = oracle.select_mask_mass(S, n_text, tau, 3.0)
        if prev is not None:
            assert ((prev == 1) <= (mask == 1)).all()
        prev = mask
        if tau == 1e-9:
            assert (k[0, 1:] == 1).all()                                  # the best candidate alone
            for i in range(1, nb):
                free = free_candidates(nb, 1, i)
                assert mask[0, i, free[int(np.argmax(S[0, i, free]))]]
    assert prev.all() and np.isinf(margin[0]).all()                       # tau = 1 keeps everything


def test_scale_limits_shift_invariance_and_topk_agreement():
    rng = np.random.default_rng(8)
    nb, n_text = 19, 70
    ntb = 2
    S = rng.standard_normal((1, nb, nb))
    m0, _, k0, _ = oracle.select_mask_mass(S, n_text, 0.6, 0.0)          # scale 0: every weight is 1
    assert (k0[0, ntb:] == math.ceil(0.6 * (nb - ntb - 1))).all()
    m1, _, k1, _ = oracle.select_mask_mass(S, n_text, 0.6, 1e4)          # one block holds all the mass
    assert (k1[0, ntb:] == 1).all()
    m2, _, k2, _ = oracle.select_mask_mass(S, n_text, 0.6, 2.5)
    shift = rng.standard_normal((1, nb, 1)) * 8                            # softmax weights ignore a row offset
    m3, _, k3, _ = oracle.select_mask_mass(S + shift, n_text, 0.6, 2.5)
    assert (m2 == m3).all() and (k2 == k3).all()
    # at the count it arrives at, the kept set is the top-k set of the pinned top-k oracle
    n_free = nb - ntb - 1
    for kk in np.unique(k2[0, ntb:]):
        mk, _ = oracle.select_mask(S, n_text, (kk - 0.5) / n_free)
        rows = [i for i in range(ntb, nb) if k2[0, i] == kk]
        assert (mk[0, rows] == m2[0, rows]).all()


def test_margin_flags_an_exact_hit():
    nb = 10                                                                # 8 free candidates, equal weights
    S = np.zeros((1, nb, nb))
    _, _, k, margin = oracle.select_mask_mass(S, 64, 0.5, 1.0)             # target = exactly 4 weights
    assert (k[0, 1:] == 4).all() and (margin[0, 1:] <= 1e-15).all()
    _, _, k, margin = oracle.select_mask_mass(S, 64, 0.55, 1.0)
    assert (k[0, 1:] == 5).all() and (margin[0, 1:] > 0.04).all()
