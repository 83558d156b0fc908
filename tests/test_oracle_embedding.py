"""Pins for the gated adaptive embedding (Section 4.2): it is the gated low-rank layer applied to
one-hot inputs, so the already pinned layer functions fix it."""
import numpy as np

from oracle import flop_oracle as O


def test_embedding_equals_layer_on_one_hot_inputs():
    g = np.random.default_rng(0)
    n, d_i, d, T = 11, 6, 5, 23
    E, Om = g.standard_normal((n, d_i)), g.standard_normal((d_i, d))
    ids = g.integers(0, n, T); ids[:3] = 4                       # repeated words accumulate in dE
    z = g.uniform(0, 1, d_i); z[2] = 0.0
    dzd = g.uniform(0, 1, d_i)
    dY = g.standard_normal((T, d))
    X = np.zeros((T, n)); X[np.arange(T), ids] = 1.0
    # layer with Q = E^T (rank rows), P = O^T: y = P G Q x
    _, _, Y_layer = O.gated_lowrank_fwd(X, E.T, Om.T, z)
    H, Hp, Y = O.gated_embedding_fwd(ids, E, Om, z)
    assert np.allclose(Y, Y_layer, atol=1e-13) and np.array_equal(H, E[ids])
    G_layer = O.gated_lowrank_bwd(dY, X, E.T, Om.T, z, dzd)
    G = O.gated_embedding_bwd(dY, ids, E, Om, z, dzd)
    assert np.allclose(G["dE"], G_layer["dQ"].T, atol=1e-12)
    assert np.allclose(G["dO"], G_layer["dP"].T, atol=1e-12)
    assert np.allclose(G["dlog_alpha"], G_layer["dlog_alpha"], atol=1e-12)
    assert np.all(G["dE"][:, 2] == 0)                            # a pruned dimension gets no gradient
    unused = np.setdiff1d(np.arange(n), ids)
    assert np.all(G["dE"][unused] == 0)
