"""Pins for the oracle's gated factorized layer, forward and backward (Section 4.1)."""
import numpy as np

from oracle import flop_oracle as O
from paper_1910_04732_b200 import inputs as I

BETA, GAMMA, ZETA = I.BETA, I.GAMMA, I.ZETA


def test_svd_factors_with_open_gates_reproduce_dense_layer():
    """z = 1 and P, Q from the SVD of W: y = W x."""
    m = I.Matrix("w", 256, 256, 256)
    g = np.random.default_rng(0)
    W = g.normal(0, 1 / 16, size=(256, 256))
    U, S, Vt = np.linalg.svd(W)
    P, Q = U * np.sqrt(S), np.sqrt(S)[:, None] * Vt
    X = g.standard_normal((64, 256))
    _, _, Y = O.gated_lowrank_fwd(X, Q, P, np.ones(256))
    assert np.allclose(Y, X @ W.T, rtol=0, atol=1e-12)
    # the generator used by the workloads does the same thing
    P2, Q2 = I.factors(m, "f32", 0, 0, 0, svd=True)
    assert np.linalg.matrix_rank(P2.astype(np.float64) @ Q2.astype(np.float64)) == 256


def test_input_feature_pruning_is_the_special_case_P_eq_W_Q_eq_I():
    """Footnote of Section 4.1: P = W, Q = I gives W G x (column masking)."""
    g = np.random.default_rng(1)
    W = g.standard_normal((7, 5))
    X = g.standard_normal((9, 5))
    z = np.array([0.0, 1.0, 0.3, 0.0, 0.8])
    _, _, Y = O.gated_lowrank_fwd(X, np.eye(5), W, z)
    assert np.allclose(Y, (X * z) @ W.T, atol=1e-14)
    Wm = W.copy(); Wm[:, z == 0] = 0
    _, _, Y2 = O.gated_lowrank_fwd(X, np.eye(5), Wm, np.where(z > 0, z, 1.0))
    assert np.allclose(Y, Y2, atol=1e-14)


def test_sum_of_rank_one_components():
    """W = sum_k z_k p_k q_k, written as the explicit sum."""
    g = np.random.default_rng(2)
    P, Q = g.standard_normal((6, 4)), g.standard_normal((4, 5))
    z = g.uniform(0, 1, 4); z[1] = 0
    X = g.standard_normal((3, 5))
    W = np.zeros((6, 5))
    for k in range(4):
        for i in range(6):
            for j in range(5):
                W[i, j] += z[k] * P[i, k] * Q[k, j]
    H, Hp, Y = O.gated_lowrank_fwd(X, Q, P, z)
    assert np.allclose(Y, X @ W.T, atol=1e-13)
    assert np.allclose(Hp, H * z, atol=0)
    assert H.shape == (3, 4)
    for t in range(3):
        for k in range(4):
            assert abs(H[t, k] - sum(X[t, j] * Q[k, j] for j in range(5))) < 1e-13


def _loss(X, Q, P, alpha, u, R):
    z, _, _ = O.hard_concrete(alpha, u, BETA, GAMMA, ZETA)
    return float(np.sum(O.gated_lowrank_fwd(X, Q, P, z)[2] * R))


def test_backward_matches_central_finite_differences():
    T, d, dp, r = 5, 4, 3, 6
    g = np.random.default_rng(3)
    X, Q, P = g.standard_normal((T, d)), g.standard_normal((r, d)), g.standard_normal((dp, r))
    R = g.standard_normal((T, dp))
    u = O.gate_uniforms(r, 0, 0)
    alpha = np.array([0.2, -1.5, 1.0, 3.5, -6.0, 0.6])     # gates 2,3 end on the upper clamp, gate 4 on the lower
    z, mask, dzda = O.hard_concrete(alpha, u, BETA, GAMMA, ZETA)
    inner = (z > 0) & (z < 1)
    assert np.any(z == 0) and np.any(z == 1) and inner.sum() >= 3
    assert np.all(z[inner] > 1e-3) and np.all(z[inner] < 1 - 1e-3)      # finite differences stay off the kinks
    G = O.gated_lowrank_bwd(R, X, Q, P, z, dzda)
    eps = 1e-6

    def fd(arr, name):
        out = np.zeros_like(arr)
        for i in np.ndindex(arr.shape):
            a0 = arr[i]
            arr[i] = a0 + eps; lp = _loss(X, Q, P, alpha, u, R)
            arr[i] = a0 - eps; lm = _loss(X, Q, P, alpha, u, R)
            arr[i] = a0
            out[i] = (lp - lm) / (2 * eps)
        return out

    for arr, name in ((X, "dX"), (Q, "dQ"), (P, "dP"), (alpha, "dlog_alpha")):
        num = fd(arr, name)
        assert np.allclose(G[name], num, rtol=1e-7, atol=1e-8), name
    assert np.count_nonzero(G["dlog_alpha"]) >= 3


def test_three_forms_of_dz_agree():
    """dz_k = sum_t H dH' = sum_i P[i,k] (dY^T H)[i,k] = sum_j Q[k,j] (dH'^T X)[k,j]."""
    g = np.random.default_rng(4)
    T, d, dp, r = 33, 12, 17, 9
    X, Q, P = g.standard_normal((T, d)), g.standard_normal((r, d)), g.standard_normal((dp, r))
    dY = g.standard_normal((T, dp))
    z = g.uniform(0, 1, r); z[2] = 0.0; z[5] = 1.0
    G = O.gated_lowrank_bwd(dY, X, Q, P, z, np.ones(r))
    H = X @ Q.T
    dHp = dY @ P
    f2 = np.sum(P * (dY.T @ H), axis=0)
    f3 = np.sum(Q * (dHp.T @ X), axis=1)
    assert np.allclose(G["dz"], f2, atol=1e-11) and np.allclose(G["dz"], f3, atol=1e-11)
    # dQ = diag(z) (dH'^T X): closed gates get no gradient in Q, open ones the full one
    assert np.allclose(G["dQ"], z[:, None] * (dHp.T @ X), atol=1e-11)
    assert np.all(G["dQ"][2] == 0) and np.all(G["dP"][:, 2] == 0)
    assert np.allclose(G["dX"], dY @ (P * z) @ Q, atol=1e-11)      # dX = dY W with W = P G Q
