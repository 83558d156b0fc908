"""Pins for the deterministic inference mask and the compaction (Sections 4.4, 4.1)."""
import numpy as np

from oracle import flop_oracle as O

BETA, GAMMA, ZETA = 2.0 / 3.0, -0.1, 1.1


def test_compaction_equals_brute_force_masking():
    g = np.random.default_rng(0)
    r, d, dp, T = 40, 12, 20, 9
    a = np.where(g.permutation(r) < 14, 4.0, -4.0) + g.normal(0, 0.1, r)
    P, Q, X = g.standard_normal((dp, r)), g.standard_normal((r, d)), g.standard_normal((T, d))
    k, idx, z_det = O.deterministic_mask(a, BETA, GAMMA, ZETA)
    pi = O.prob_nonzero(a, BETA, GAMMA, ZETA)
    assert k == int(np.floor(pi.sum() + 0.5)) == len(idx)
    assert list(idx) == [j for j in range(r) if z_det[j] > 0]
    assert np.all(np.diff(idx) > 0)
    # kept gates carry their Eq. 3 value; the kept set is the k largest
    assert np.array_equal(z_det[idx], pi[idx])
    assert k == 0 or k == r or a[idx].min() >= np.delete(a, idx).max()
    Pc, Qc = O.compact_ranks(P, Q, idx, z_det)
    assert Pc.shape == (dp, k) and Qc.shape == (k, d)
    Yc = O.compact_fwd(X, Qc, Pc)
    _, _, Y = O.gated_lowrank_fwd(X, Q, P, z_det)           # uncompacted layer with the same gates
    assert np.allclose(Yc, Y, rtol=0, atol=1e-12)
    # zeroing the pruned columns/rows by hand changes nothing either
    Pm, Qm = P.copy(), Q.copy()
    dead = z_det == 0
    Pm[:, dead] = 0; Qm[dead] = 0
    assert np.allclose(O.gated_lowrank_fwd(X, Qm, Pm, np.where(dead, 1.0, z_det))[2], Y, atol=1e-12)


def test_topk_ties_and_edges():
    a = np.array([1.0, 3.0, 1.0, 1.0, -9.0, 1.0])
    # pi: three of the four tied gates survive next to the clear winner -> ties go to the lower index
    k, idx, z = O.deterministic_mask(a, 1.0, GAMMA, ZETA)
    pi = O.prob_nonzero(a, 1.0, GAMMA, ZETA)
    assert k == int(np.floor(pi.sum() + 0.5))
    expect = sorted(sorted(range(6), key=lambda j: (-a[j], j))[:k])
    assert list(idx) == expect and (k < 5 or 5 in idx) and 4 not in idx
    k, idx, z = O.deterministic_mask(np.full(8, -30.0), BETA, GAMMA, ZETA)
    assert k == 0 and len(idx) == 0 and np.all(z == 0)
    k, idx, z = O.deterministic_mask(np.full(8, 30.0), BETA, GAMMA, ZETA)
    assert k == 8 and list(idx) == list(range(8)) and np.allclose(z, 1.0)


def test_active_ranks_rule_and_sampled_mask_compaction():
    """Keeping z_k > 0 of a sampled mask leaves the training forward unchanged."""
    g = np.random.default_rng(1)
    r, d, dp, T = 64, 10, 11, 5
    a = g.normal(-1.0, 2.0, r)
    z, mask, _ = O.gate_sample(a, BETA, GAMMA, ZETA, seed=0, offset=0)
    k, idx = O.active_ranks(z)
    assert k == int(mask.sum()) and np.array_equal(idx, np.nonzero(mask)[0])
    assert 0 < k < r
    P, Q, X = g.standard_normal((dp, r)), g.standard_normal((r, d)), g.standard_normal((T, d))
    Pc, Qc = O.compact_ranks(P, Q, idx, z)
    assert np.allclose(O.compact_fwd(X, Qc, Pc), O.gated_lowrank_fwd(X, Q, P, z)[2], atol=1e-12)
