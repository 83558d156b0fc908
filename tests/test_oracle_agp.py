"""Pins for the FLOP-AGP gate rule (magnitude pruning of the diagonal mask, Section 5 baselines)."""
import numpy as np

from oracle import flop_oracle as O


def test_magnitude_rule_properties_and_brute_force():
    g = np.random.default_rng(0)
    vals = g.standard_normal(57)
    off = [0, 20, 20, 57]
    for s in (0.0, 0.25, 0.5, 0.9, 1.0):
        r = O.agp_gates(vals, off, s, 0.1)
        for lo, hi in ((0, 20), (20, 57)):
            n = hi - lo
            kept = r["mask"][lo:hi].astype(bool)
            assert kept.sum() == n - int(np.floor(s * n + 0.5))
            if 0 < kept.sum() < n:       # every kept magnitude is at least every pruned one
                assert np.abs(vals[lo:hi])[kept].min() >= np.abs(vals[lo:hi])[~kept].max()
        assert np.array_equal(r["z"], np.where(r["mask"] == 1, vals, 0.0))
        assert np.array_equal(r["dz_dg"], r["mask"])
    assert O.agp_gates(vals, off, 0.0, 0.0)["mask"].all() and not O.agp_gates(vals, off, 1.0, 0.0)["mask"].any()


def test_ties_and_l1_term():
    vals = np.array([0.5, -0.5, 0.5, 2.0, -0.5, 0.0])
    r = O.agp_gates(vals, [0, 6], 0.5, 0.3)          # prune 3 of 6: the zero, then the tied 0.5s from the highest index down
    assert list(r["mask"]) == [1, 1, 0, 1, 0, 0]
    assert abs(r["seg_l1"][0] - 4.0) < 1e-15
    # gradient of l1 * sum |g| by finite differences away from zero
    eps = 1e-6
    for k in (0, 1, 3):
        vp, vm = vals.copy(), vals.copy()
        vp[k] += eps; vm[k] -= eps
        fd = 0.3 * (np.abs(vp).sum() - np.abs(vm).sum()) / (2 * eps)
        assert abs(fd - r["l1_grad"][k]) < 1e-9
    assert r["l1_grad"][5] == 0.0
