"""Pins for the expected-size / augmented-Lagrangian term (Eq. 3, Section 4.3)."""
import numpy as np

from oracle import flop_oracle as O

BETA, GAMMA, ZETA = 2.0 / 3.0, -0.1, 1.1


def _setup(seed=0):
    g = np.random.default_rng(seed)
    sizes = np.array([820.0, 2510.0, 2510.0, 820.0])
    counts = [5, 7, 3, 6]
    off = np.concatenate([[0], np.cumsum(counts)])
    a = g.normal(0.5, 1.0, size=off[-1])
    return a, off, sizes


def test_constraint_met_means_no_penalty():
    a, off, sizes = _setup()
    s = O.expected_l0_lagrangian(a, off, sizes, BETA, GAMMA, ZETA, 0.0, 0.0, 0.0)["s"]
    r = O.expected_l0_lagrangian(a, off, sizes, BETA, GAMMA, ZETA, s, 0.7, 1.9)
    assert r["g"] == 0.0 and r["dg_dlambda1"] == 0.0 and r["dg_dlambda2"] == 0.0
    # at s = t only the linear multiplier still pushes on alpha
    r0 = O.expected_l0_lagrangian(a, off, sizes, BETA, GAMMA, ZETA, s, 0.0, 1.9)
    assert np.all(r0["dlog_alpha"] == 0.0)


def test_limits_and_equal_sizes():
    a, off, sizes = _setup()
    r = O.expected_l0_lagrangian(np.full(21, 40.0), off, sizes, BETA, GAMMA, ZETA, 0.3, 1.0, 1.0)
    assert abs(r["s"] - 1.0) < 1e-12 and np.allclose(r["seg_expected"], [5, 7, 3, 6])
    r = O.expected_l0_lagrangian(np.full(21, -40.0), off, sizes, BETA, GAMMA, ZETA, 0.3, 1.0, 1.0)
    assert abs(r["s"]) < 1e-12
    eq = O.expected_l0_lagrangian(a, off, np.full(4, 512.0), BETA, GAMMA, ZETA, 0.5, 0.0, 0.0)
    assert abs(eq["s"] - np.mean(O.prob_nonzero(a, BETA, GAMMA, ZETA))) < 1e-14
    # s is the size-weighted mean of the per-matrix expected ranks
    r = O.expected_l0_lagrangian(a, off, sizes, BETA, GAMMA, ZETA, 0.5, 0.0, 0.0)
    counts = np.diff(off)
    assert abs(r["s"] - np.sum(r["seg_expected"] * sizes) / np.sum(counts * sizes)) < 1e-14


def test_penalty_is_linear_in_multipliers_and_matches_definition():
    a, off, sizes = _setup(1)
    t = 0.35
    base = O.expected_l0_lagrangian(a, off, sizes, BETA, GAMMA, ZETA, t, 0.0, 0.0)
    s = base["s"]
    for l1, l2 in ((0.3, 1.7), (-2.0, 0.25)):
        r = O.expected_l0_lagrangian(a, off, sizes, BETA, GAMMA, ZETA, t, l1, l2)
        assert abs(r["g"] - (l1 * (s - t) + l2 * (s - t) ** 2)) < 1e-15
        assert r["dg_dlambda1"] == s - t and r["dg_dlambda2"] == (s - t) ** 2
    assert base["g"] == 0.0 and np.all(base["dlog_alpha"] == 0.0)      # multipliers start at zero


def test_gradient_wrt_alpha_finite_differences():
    a, off, sizes = _setup(2)
    t, l1, l2 = 0.35, 0.3, 1.7
    grad = O.expected_l0_lagrangian(a, off, sizes, BETA, GAMMA, ZETA, t, l1, l2)["dlog_alpha"]
    eps = 1e-6
    for j in range(len(a)):
        ap, am = a.copy(), a.copy()
        ap[j] += eps; am[j] -= eps
        gp = O.expected_l0_lagrangian(ap, off, sizes, BETA, GAMMA, ZETA, t, l1, l2)["g"]
        gm = O.expected_l0_lagrangian(am, off, sizes, BETA, GAMMA, ZETA, t, l1, l2)["g"]
        assert abs((gp - gm) / (2 * eps) - grad[j]) < 1e-9
    # a gate of a larger block weighs more: same alpha, different segment
    a2 = np.zeros(21)
    g2 = O.expected_l0_lagrangian(a2, off, sizes, BETA, GAMMA, ZETA, t, 1.0, 0.0)["dlog_alpha"]
    assert abs(g2[5] / g2[0] - 2510.0 / 820.0) < 1e-12
