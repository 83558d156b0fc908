"""Pins for the hard-concrete sampler and the closed-form L0 probability (Section 3, Eq. 3)."""
import math

import numpy as np

from oracle import flop_oracle as O

BETA, GAMMA, ZETA = 2.0 / 3.0, -0.1, 1.1
ALPHAS = [-3.0, -1.0, 0.0, 0.5, 1.0, 2.0, 3.0]


def _read_golden(name):
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", name)
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    return np.array(rows, dtype=np.float64)


def test_closed_form_values_golden():
    """Eq. 3 at beta=2/3, gamma=-0.1, zeta=1.1, evaluated by hand with the
    scalar math library (tests/golden/eq3_closed_form.txt)."""
    g = _read_golden("eq3_closed_form.txt")
    assert np.allclose(O.prob_nonzero(g[:, 0], BETA, GAMMA, ZETA), g[:, 1], atol=5e-7)
    thr = BETA * math.log(-GAMMA / ZETA)
    assert abs(thr - (-1.598597)) < 1e-6
    for a, p in zip(g[:, 0], g[:, 1]):
        assert abs(1.0 / (1.0 + math.exp(-(a - thr))) - p) < 5e-7


def test_monte_carlo_matches_eq3_and_upper_clamp():
    """P(z>0) from 4e6 sampled gates per alpha equals Eq. 3 within 1e-3, and
    P(z=1) equals sigmoid(alpha - beta log((1-gamma)/(zeta-1))), the same
    derivation applied to the upper clamp."""
    n = 4_000_000
    g = _read_golden("eq3_closed_form.txt")
    for i, a in enumerate(ALPHAS):
        u = O.gate_uniforms(n, seed=0, offset=i << 24)
        z, mask, _ = O.hard_concrete(np.full(n, a), u, BETA, GAMMA, ZETA)
        p_hat = mask.mean()
        assert abs(p_hat - O.prob_nonzero(a, BETA, GAMMA, ZETA)) < 1e-3
        assert abs(p_hat - g[i, 1]) < 1e-3
        p1 = 1.0 / (1.0 + math.exp(-(a - BETA * math.log((1 - GAMMA) / (ZETA - 1)))))
        assert abs((z == 1.0).mean() - p1) < 1e-3
        assert abs(p1 - g[i, 2]) < 5e-7
        assert z.min() >= 0.0 and z.max() <= 1.0
        assert np.array_equal(mask, (z > 0).astype(np.uint8))


def test_symmetric_stretch_identity():
    """For gamma = 1 - zeta, P(z=1 | alpha) = 1 - P(z>0 | -alpha)."""
    n = 1_000_000
    u = O.gate_uniforms(n, 5, 0)
    for a in (0.3, 1.7):
        z_pos, _, _ = O.hard_concrete(np.full(n, a), u, BETA, GAMMA, ZETA)
        _, m_neg, _ = O.hard_concrete(np.full(n, -a), 1.0 - u, BETA, GAMMA, ZETA)
        # exact pathwise: reflecting u and alpha reflects s about 1/2
        assert abs((z_pos == 1.0).mean() - (1.0 - m_neg.mean())) < 1e-12


def test_beta_one_is_the_papers_sampler():
    u = O.gate_uniforms(2000, 11, 3)
    a = np.linspace(-4, 4, 2000)
    z, _, _ = O.hard_concrete(a, u, 1.0, GAMMA, ZETA)
    for j in range(0, 2000, 37):
        s = 1.0 / (1.0 + math.exp(-(math.log(u[j]) - math.log(1 - u[j]) + a[j])))
        sb = s * (ZETA - GAMMA) + GAMMA
        assert abs(z[j] - min(1.0, max(0.0, sb))) < 1e-15
    # and Eq. 3 as printed (beta = 1)
    assert abs(O.prob_nonzero(0.7, 1.0, GAMMA, ZETA)
               - 1.0 / (1.0 + math.exp(-(0.7 - math.log(-GAMMA / ZETA))))) < 1e-15


def test_dz_dalpha_finite_differences():
    u = O.gate_uniforms(4000, 2, 0)
    a = np.random.default_rng(0).normal(0.5, 1.5, size=4000)
    z, mask, d = O.hard_concrete(a, u, BETA, GAMMA, ZETA)
    eps = 1e-6
    zp, _, _ = O.hard_concrete(a + eps, u, BETA, GAMMA, ZETA)
    zm, _, _ = O.hard_concrete(a - eps, u, BETA, GAMMA, ZETA)
    fd = (zp - zm) / (2 * eps)
    safe = (np.abs(z - 0.0) > 1e-3) & (np.abs(z - 1.0) > 1e-3) | (z == 0) & (zp == 0) & (zm == 0) | (z == 1) & (zp == 1) & (zm == 1)
    assert safe.mean() > 0.9
    assert np.allclose(d[safe], fd[safe], rtol=1e-6, atol=1e-8)
    assert np.all(d[(z == 0) | (z == 1)] == 0)           # no gradient on the clamp
    assert np.any(d > 0)
