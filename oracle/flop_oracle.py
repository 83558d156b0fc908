"""CPU fp64 oracle for the FLOP gated low-rank layer (test infrastructure only).

This file is TEST INFRASTRUCTURE.  It is a plain, slow, obviously-correct
restatement of the definitions in "Structured Pruning of Large Language Models"
(FLOP, arXiv 1910.04732), written in numpy fp64.  It shares no code with the
CUDA path and never imports it.  Only the tests, the smoke check and the
CPU-baseline leg of the benchmark may call it; the product path must not.

Notation (the paper overloads r; here r is always the rank):
    X [T, d]   tokens are rows;  Q [r, d];  P [d', r];  z [r] gates
    W = P diag(z) Q                        (Section 4.1)
    alpha = log_alpha, the hard-concrete location (Section 3)
    gamma < 0 < 1 < zeta, the stretch limits (the paper calls them l and r)
    beta, the temperature; the paper's formulas are the beta = 1 case.

Every function cites the passage it follows.

Pins (tests/test_oracle_*.py), i.e. what fixes each function to something
other than itself:
    philox4x32_10         library cross-check against a vendor host generator
                          when one is loadable, statistical invariants,
                          counter-continuation; otherwise "parity unpinned"
                          for the constants only (any uniform stream serves
                          the method; both sides must merely agree).
    hard_concrete         Monte-Carlo against the closed forms of P(z>0) and
                          P(z=1); beta=1 reduces to the paper's sampler;
                          finite differences for dz/dalpha.
    gated_lowrank_fwd     dense W x with SVD factors and z=1; the footnote
                          identity P=W, Q=I (input-feature pruning).
    gated_lowrank_bwd     central finite differences; three algebraically
                          equal forms of dz.
    expected_l0_lagrangian  closed-form special cases (s=t, alpha->+inf,
                          equal sizes -> mean), finite differences.
    deterministic_mask / compact_ranks / compact_fwd
                          brute-force masking of the uncompacted layer.
    agp_gates             brute-force properties of the magnitude rule (counts, kept >= pruned,
                          tie order), finite differences of the L1 term.
    gated_embedding_fwd/bwd  equal to the (pinned) layer functions on one-hot inputs.
    The *choices* the paper leaves open (values of kept inference gates,
    top-k tie-break, which factor absorbs the gate) are "parity unpinned":
    several answers satisfy the paper, the oracle fixes one.
"""
from __future__ import annotations

import numpy as np

# ----------------------------------------------------------------------------
# Counter-based generator: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11).
# The paper only says u ~ U(0,1) (Section 3); a counter-based generator lets a
# CPU program and a GPU kernel draw the same u_j for gate j.
# ----------------------------------------------------------------------------
_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = np.uint64(0x9E3779B9)
_PHILOX_W1 = np.uint64(0xBB67AE85)
_MASK32 = np.uint64(0xFFFFFFFF)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten Philox-4x32 rounds on arrays of counters (c0..c3) with one key (k0,k1).

    One round: (hi0,lo0) = M0*c0, (hi1,lo1) = M1*c2 as 64-bit products;
    new counter = (hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0); then the key is
    bumped by the two Weyl constants.  Returns four uint32 arrays.
    """
    c0 = np.asarray(c0, dtype=np.uint64) & _MASK32
    c1 = np.asarray(c1, dtype=np.uint64) & _MASK32
    c2 = np.asarray(c2, dtype=np.uint64) & _MASK32
    c3 = np.asarray(c3, dtype=np.uint64) & _MASK32
    k0 = np.uint64(int(k0) & 0xFFFFFFFF)
    k1 = np.uint64(int(k1) & 0xFFFFFFFF)
    for _ in range(10):
        p0 = _PHILOX_M0 * c0            # < 2^64, exact in uint64
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK32
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0 = (k0 + _PHILOX_W0) & _MASK32
        k1 = (k1 + _PHILOX_W1) & _MASK32
    return (c0.astype(np.uint32), c1.astype(np.uint32),
            c2.astype(np.uint32), c3.astype(np.uint32))


def uniform_from_bits(x):
    """Map 32 random bits to u in the OPEN interval (0,1): ((x>>9)+1/2) * 2^-23.

    The paper writes U(0,1) and then takes log u and log(1-u) (Section 3), so
    both endpoints must be excluded.  The value has 24 significant bits, is
    exact in fp32 and fp64, and is symmetric about 1/2.
    """
    return ((np.asarray(x, dtype=np.uint32) >> np.uint32(9)).astype(np.float64) + 0.5) * 2.0 ** -23


def gate_uniforms(n, seed, offset):
    """u_j for gates j = 0..n-1.

    Gate j takes word (j mod 4) of the Philox block whose 128-bit counter is
    (offset + j // 4) in the two low words (the two high words are 0) and whose
    key is the 64-bit seed split into (low, high) 32-bit words.
    """
    j = np.arange(n, dtype=np.uint64)
    ctr = np.uint64(int(offset) & 0xFFFFFFFFFFFFFFFF) + (j >> np.uint64(2))
    w = philox4x32_10(ctr & _MASK32, ctr >> np.uint64(32), 0 * ctr, 0 * ctr,
                      int(seed) & 0xFFFFFFFF, (int(seed) >> 32) & 0xFFFFFFFF)
    bits = np.stack(w, axis=1)[np.arange(n), (j & np.uint64(3)).astype(np.int64)] if n else np.zeros(0, np.uint32)
    return uniform_from_bits(bits)


# ----------------------------------------------------------------------------
# Hard-concrete gates (Section 3: the inverse CDF G(u; alpha))
# ----------------------------------------------------------------------------
def sigmoid(x):
    x = np.asarray(x, dtype=np.float64)
    return 1.0 / (1.0 + np.exp(-x))


def hard_concrete(log_alpha, u, beta, gamma, zeta):
    """z, mask, dz/dalpha from uniforms u (Section 3, the four-line sampler).

        s     = sigmoid((log u - log(1-u) + alpha) / beta)
        s_bar = s (zeta - gamma) + gamma
        z     = min(1, max(0, s_bar))

    beta = 1 is the paper's formula verbatim.  For beta != 1 the division by
    beta is the form consistent with the closed form
    P(z>0) = sigmoid(alpha - beta log(-gamma/zeta)) (see prob_nonzero).
    mask = (z > 0).  dz/dalpha = (zeta-gamma) s (1-s) / beta strictly inside
    the clamp (0 < s_bar < 1) and 0 on and outside it.
    """
    a = np.asarray(log_alpha, dtype=np.float64)
    u = np.asarray(u, dtype=np.float64)
    s = sigmoid((np.log(u) - np.log(1.0 - u) + a) / beta)
    s_bar = s * (zeta - gamma) + gamma
    z = np.minimum(1.0, np.maximum(0.0, s_bar))
    mask = (z > 0.0).astype(np.uint8)
    inside = (s_bar > 0.0) & (s_bar < 1.0)
    dz_dla = np.where(inside, (zeta - gamma) * s * (1.0 - s) / beta, 0.0)
    return z, mask, dz_dla


def gate_sample(log_alpha, beta, gamma, zeta, seed, offset):
    """Sample all gates: Philox uniforms -> hard_concrete (Section 3)."""
    u = gate_uniforms(len(log_alpha), seed, offset)
    return hard_concrete(log_alpha, u, beta, gamma, zeta)


def prob_nonzero(log_alpha, beta, gamma, zeta):
    """pi_j = P(z_j > 0) = sigmoid(alpha_j - beta log(-gamma/zeta))   (Eq. 3).

    The paper prints the beta = 1 case, sigmoid(alpha - log(-l/r)).
    """
    return sigmoid(np.asarray(log_alpha, dtype=np.float64) - beta * np.log(-gamma / zeta))


# ----------------------------------------------------------------------------
# The gated factorized layer W = P diag(z) Q (Section 4.1)
# ----------------------------------------------------------------------------
def gated_lowrank_fwd(X, Q, P, z):
    """y = P G Q x for every token row of X.

    H = X Q^T, H' = H * z (column k times z_k), Y = H' P^T.
    Returns (H, H', Y).
    """
    X = np.asarray(X, dtype=np.float64)
    Q = np.asarray(Q, dtype=np.float64)
    P = np.asarray(P, dtype=np.float64)
    z = np.asarray(z, dtype=np.float64)
    H = X @ Q.T
    Hp = H * z[None, :]
    Y = Hp @ P.T
    return H, Hp, Y


def gated_lowrank_bwd(dY, X, Q, P, z, dz_dla):
    """Chain rule through Y = ((X Q^T) * z) P^T  (Section 3: gradient updates
    for theta and alpha; Section 4.1 for the product).

        dH' = dY P          dP = dY^T H'        dz_k = sum_t H[t,k] dH'[t,k]
        dH  = dH' * z       dQ = dH^T X         dX   = dH Q
        dalpha = dz * dz/dalpha
    Returns dict(dX, dP, dQ, dz, dlog_alpha).
    """
    dY = np.asarray(dY, dtype=np.float64)
    X = np.asarray(X, dtype=np.float64)
    Q = np.asarray(Q, dtype=np.float64)
    P = np.asarray(P, dtype=np.float64)
    z = np.asarray(z, dtype=np.float64)
    H = X @ Q.T
    Hp = H * z[None, :]
    dHp = dY @ P
    dP = dY.T @ Hp
    dz = np.sum(H * dHp, axis=0)
    dH = dHp * z[None, :]
    dQ = dH.T @ X
    dX = dH @ Q
    return dict(dX=dX, dP=dP, dQ=dQ, dz=dz,
                dlog_alpha=dz * np.asarray(dz_dla, dtype=np.float64))


# ----------------------------------------------------------------------------
# Expected size and augmented-Lagrangian penalty (Eq. 3, Section 4.3)
# ----------------------------------------------------------------------------
def expected_l0_lagrangian(log_alpha, seg_off, seg_size, beta, gamma, zeta,
                           target, lambda1, lambda2):
    """s(alpha), g(lambda, alpha) and their derivatives over all gates at once.

    Segment i (one weight matrix) owns gates seg_off[i]..seg_off[i+1]-1; each
    of its gates stands for a parameter block of seg_size[i] = d + d'
    parameters (one column of P plus one row of Q).

        pi_j = P(z_j > 0)                                         (Eq. 3)
        s    = sum_j pi_j size_j / sum_j size_j   (fraction of the prunable
               parameters expected to remain; Section 4.3 multiplies Eq. 3 by
               the block size, the division makes s and t fractions)
        g    = lambda1 (s - t) + lambda2 (s - t)^2                (Section 4.3)
        dg/dlambda1 = s - t,  dg/dlambda2 = (s - t)^2
        dg/dalpha_j = (lambda1 + 2 lambda2 (s - t)) (size_j / S) pi_j (1 - pi_j)
        seg_expected[i] = sum of pi_j over segment i (expected surviving rank)
    """
    a = np.asarray(log_alpha, dtype=np.float64)
    seg_off = np.asarray(seg_off, dtype=np.int64)
    seg_size = np.asarray(seg_size, dtype=np.float64)
    n_seg = len(seg_size)
    pi = prob_nonzero(a, beta, gamma, zeta)
    size_j = np.zeros_like(a)
    seg_expected = np.zeros(n_seg)
    for i in range(n_seg):
        lo, hi = int(seg_off[i]), int(seg_off[i + 1])
        size_j[lo:hi] = seg_size[i]
        seg_expected[i] = np.sum(pi[lo:hi])
    S = np.sum(size_j)
    s = np.sum(pi * size_j) / S if S > 0 else 0.0
    diff = s - target
    g = lambda1 * diff + lambda2 * diff * diff
    dalpha = (lambda1 + 2.0 * lambda2 * diff) * (size_j / S) * pi * (1.0 - pi) if S > 0 else np.zeros_like(a)
    return dict(s=s, g=g, dg_dlambda1=diff, dg_dlambda2=diff * diff,
                seg_expected=seg_expected, dlog_alpha=dalpha)


# ----------------------------------------------------------------------------
# Inference: deterministic mask and compaction (Sections 4.4 and 4.1)
# ----------------------------------------------------------------------------
def deterministic_mask(log_alpha, beta, gamma, zeta):
    """Fixed inference mask of one weight matrix (Section 4.4).

    Each gate's value is its Eq. 3 probability pi_j; the number kept matches
    the expected L0 norm, k = floor(sum_j pi_j + 1/2); the k largest are kept
    (ranked by alpha, which orders exactly as pi does but cannot saturate;
    ties go to the lower index), the rest are clipped to 0.
    Returns (k, idx ascending int32[k], z_det[r]).
    """
    a = np.asarray(log_alpha, dtype=np.float64)
    r = len(a)
    pi = prob_nonzero(a, beta, gamma, zeta)
    k = int(np.floor(np.sum(pi) + 0.5))
    k = max(0, min(r, k))
    order = sorted(range(r), key=lambda j: (-a[j], j))     # descending alpha, then index
    keep = np.zeros(r, dtype=bool)
    keep[order[:k]] = True
    z_det = np.where(keep, pi, 0.0)
    idx = np.nonzero(keep)[0].astype(np.int32)
    return k, idx, z_det


def active_ranks(z):
    """Mode-1 compaction rule: keep component k iff z_k > 0 (Section 4.4)."""
    z = np.asarray(z, dtype=np.float64)
    idx = np.nonzero(z > 0.0)[0].astype(np.int32)
    return len(idx), idx


def compact_ranks(P, Q, idx, z):
    """Keep only the surviving columns of P and rows of Q; the gate values are
    absorbed into Q (Section 4.1: "absorbed into either P or Q").

        P_c = P[:, idx]            Q_c = diag(z[idx]) Q[idx, :]
    """
    P = np.asarray(P, dtype=np.float64)
    Q = np.asarray(Q, dtype=np.float64)
    z = np.asarray(z, dtype=np.float64)
    idx = np.asarray(idx, dtype=np.int64)
    return P[:, idx].copy(), z[idx][:, None] * Q[idx, :]


def compact_fwd(X, Qc, Pc):
    """Inference forward on the compact factors: Y = (X Q_c^T) P_c^T (Section 4.1)."""
    X = np.asarray(X, dtype=np.float64)
    return (X @ np.asarray(Qc, dtype=np.float64).T) @ np.asarray(Pc, dtype=np.float64).T


# ----------------------------------------------------------------------------
# FLOP-AGP variant (Section 5, baselines): magnitude pruning of the diagonal mask
# ----------------------------------------------------------------------------
def agp_gates(g, seg_off, sparsity, l1):
    """Magnitude-based pruning of the learnable diagonal G = diag(g) of every matrix.

    Per segment (weight matrix) with r_i components, the round(sparsity * r_i)
    entries of smallest |g_k| are pruned (ties: the higher index goes first), the
    others keep their value:  z_k = g_k if kept else 0,  dz_k/dg_k = [kept].
    The L1 term on the masks is l1 * sum_k |g_k| with gradient l1 * sign(g_k)
    (the paper: "l1 regularization on the masks to encourage sparsity").
    Returns dict(z, mask, dz_dg, seg_l1 (sum |g| per segment), l1_grad).
    """
    g = np.asarray(g, dtype=np.float64)
    seg_off = np.asarray(seg_off, dtype=np.int64)
    z = np.zeros_like(g)
    mask = np.zeros(len(g), dtype=np.uint8)
    seg_l1 = np.zeros(len(seg_off) - 1)
    for i in range(len(seg_off) - 1):
        lo, hi = int(seg_off[i]), int(seg_off[i + 1])
        r = hi - lo
        n_pruned = int(np.floor(float(sparsity) * r + 0.5))
        keep = max(0, min(r, r - n_pruned))
        order = sorted(range(r), key=lambda k: (-abs(g[lo + k]), k))     # largest magnitude first, then lower index
        for k in order[:keep]:
            mask[lo + k] = 1
            z[lo + k] = g[lo + k]
        seg_l1[i] = np.sum(np.abs(g[lo:hi]))
    return dict(z=z, mask=mask, dz_dg=mask.astype(np.float64), seg_l1=seg_l1, l1_grad=float(l1) * np.sign(g))


# ----------------------------------------------------------------------------
# Gated adaptive embedding of one word cluster (Section 4.2): E~ = E G O
# ----------------------------------------------------------------------------
def gated_embedding_fwd(ids, E, O, z):
    """Embedding lookup through the gated factorization of one word cluster.

    E [n, d_i] holds the reduced-dimension embeddings of the cluster's n words,
    O [d_i, d] projects them back to the model dimension, G = diag(z) prunes
    the d_i reduced dimensions:  row t of Y is (E[ids[t], :] * z) O.
    Returns (H = E[ids], H' = H * z, Y).
    """
    E = np.asarray(E, dtype=np.float64)
    O = np.asarray(O, dtype=np.float64)
    z = np.asarray(z, dtype=np.float64)
    H = E[np.asarray(ids, dtype=np.int64)]
    Hp = H * z[None, :]
    return H, Hp, Hp @ O


def gated_embedding_bwd(dY, ids, E, O, z, dz_dla):
    """Chain rule through gated_embedding_fwd:
        dH' = dY O^T      dO = H'^T dY      dz_k = sum_t H[t,k] dH'[t,k]
        dE[w, :] = sum over the tokens t with ids[t] = w of dH'[t, :] * z
        dalpha = dz * dz/dalpha
    """
    dY = np.asarray(dY, dtype=np.float64)
    E = np.asarray(E, dtype=np.float64)
    O = np.asarray(O, dtype=np.float64)
    z = np.asarray(z, dtype=np.float64)
    ids = np.asarray(ids, dtype=np.int64)
    H = E[ids]
    Hp = H * z[None, :]
    dHp = dY @ O.T
    dO = Hp.T @ dY
    dz = np.sum(H * dHp, axis=0)
    dE = np.zeros_like(E)
    for t in range(len(ids)):
        dE[ids[t]] += dHp[t] * z
    return dict(dE=dE, dO=dO, dz=dz, dlog_alpha=dz * np.asarray(dz_dla, dtype=np.float64))
