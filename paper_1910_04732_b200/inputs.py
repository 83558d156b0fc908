"""Seeded synthetic inputs for the FLOP gated low-rank layer.

This module only *generates numbers* (numpy's seeded generators, a bf16
rounding of the generated values, an SVD used to initialise factors).  It
holds none of the method's arithmetic and is the one module that both the CPU
oracle's tests and the CUDA path's tests/benchmark read, so that both sides
see the same arrays.

The workloads mirror the layer shapes, token counts and gate statistics of the
models the paper prunes (SRU language models, Transformer-XL, BERT/RoBERTa
base); no dataset item is reproduced.  "N(a, b)" means mean a, standard
deviation b for log_alpha; factor matrices are scaled so that H = X Q^T and
Y = H' P^T keep roughly unit scale.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np

# Hard-concrete constants used by every workload: temperature and stretch.
BETA = 2.0 / 3.0
GAMMA = -0.1
ZETA = 1.1


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result stays fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32).astype(np.uint64)
    rounded = ((bits + np.uint64(0x7FFF) + ((bits >> np.uint64(16)) & np.uint64(1)))
               & np.uint64(0xFFFF0000)).astype(np.uint32)
    return rounded.view(np.float32).reshape(a.shape)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of values that are already bf16-representable."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> np.uint32(16)).astype(np.uint16).reshape(a.shape)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).reshape(b.shape)


@dataclass(frozen=True)
class Matrix:
    """One factorized weight matrix W[d_out, d_in] = P[d_out, r] diag(z) Q[r, d_in]."""
    name: str
    d_in: int
    d_out: int
    r: int


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str                      # "f32" or "bf16": storage type of X, P, Q, Y, H'
    T: int                          # tokens = batch x sequence
    layers: int
    matrices: Tuple[Matrix, ...]    # the matrices of ONE layer
    alpha: Tuple                    # ("normal", mean, std) | ("bimodal", m, s) | ("subset", frac, hi, lo, jitter)
    target: float                   # t: target fraction of prunable parameters remaining
    note: str = ""

    def all_matrices(self) -> List[Tuple[int, int, Matrix]]:
        return [(l, i, m) for l in range(self.layers) for i, m in enumerate(self.matrices)]

    def n_gates(self) -> int:
        return self.layers * sum(m.r for m in self.matrices)

    def flops_per_step(self) -> float:
        """6 T r (d + d') per matrix: 2 forward GEMMs + 4 backward GEMMs."""
        return float(self.layers) * sum(6.0 * self.T * m.r * (m.d_in + m.d_out) for m in self.matrices)


def _txl_layer(d, ff, r):
    return (Matrix("q", d, d, r), Matrix("k", d, d, r), Matrix("v", d, d, r), Matrix("o", d, d, r),
            Matrix("ffn1", d, ff, r), Matrix("ffn2", ff, d, r))


WORKLOADS = {
    # single layer, fp32, full rank, factors from the SVD of a dense W
    "single_f32": Workload("single_f32", "f32", 512, 1, (Matrix("w", 256, 256, 256),),
                           ("normal", 2.0, 1.0), 0.5, "correctness case, SVD-initialised factors"),
    # SRU-style recurrent LM projection: one 2048 -> 3x2048 matrix per layer, batch 64 x unroll 256
    "sru": Workload("sru", "bf16", 64 * 256, 6, (Matrix("proj", 2048, 3 * 2048, 2048),),
                    ("normal", 1.0, 1.5), 0.30),
    # Transformer-XL-base-shaped block
    "txl": Workload("txl", "bf16", 60 * 150, 16, _txl_layer(410, 2100, 410),
                    ("normal", 0.5, 1.0), 0.35),
    # BERT-base-shaped encoder linears
    "bert": Workload("bert", "bf16", 32 * 128, 12, _txl_layer(768, 3072, 768),
                     ("bimodal", 3.0, 0.5), 0.5),
    # pruned inference: ~35 % of the rank components survive
    "infer": Workload("infer", "bf16", 4096, 1, (Matrix("w", 1024, 4096, 1024),),
                      ("subset", 0.35, 4.0, -4.0, 0.1), 0.35),
}


def _rng(seed: int, *stream) -> np.random.Generator:
    return np.random.default_rng([int(seed)] + [int(s) for s in stream])


def log_alpha(kind: Tuple, n: int, seed: int, *stream) -> np.ndarray:
    g = _rng(seed, 4, *stream)
    if kind[0] == "normal":
        a = g.normal(kind[1], kind[2], size=n)
    elif kind[0] == "bimodal":          # a random half near +m, the other half near -m
        sign = np.where(g.permutation(n) < n // 2, 1.0, -1.0)
        a = sign * kind[1] + g.normal(0.0, kind[2], size=n)
    elif kind[0] == "subset":           # a random subset of the given fraction near hi, the rest near lo
        keep = g.permutation(n) < int(round(kind[1] * n))
        a = np.where(keep, kind[2], kind[3]) + g.normal(0.0, kind[4], size=n)
    else:
        raise ValueError(kind)
    return a.astype(np.float32)


def _cast(a: np.ndarray, dtype: str) -> np.ndarray:
    a = a.astype(np.float32)
    return round_to_bf16(a) if dtype == "bf16" else a


def activations(T: int, d: int, dtype: str, seed: int, *stream) -> np.ndarray:
    """X or dY ~ N(0,1), returned as fp32 holding values representable in `dtype`."""
    return _cast(_rng(seed, *stream).standard_normal((T, d)), dtype)


def factors(m: Matrix, dtype: str, seed: int, *stream, svd: bool = False):
    """(P[d_out, r], Q[r, d_in]).

    svd=True: W ~ N(0, variance 1/d_in), W = U S V^T, P = U sqrt(S), Q = sqrt(S) V^T
    (full rank r = min(d_in, d_out) required), the way a pretrained dense matrix
    is factorized before the gates are inserted.  Otherwise independent Gaussian
    factors with std 1/sqrt(d_in) for Q and 1/sqrt(r) for P.
    """
    g = _rng(seed, 3, *stream)
    if svd:
        assert m.r == min(m.d_in, m.d_out)
        W = g.normal(0.0, 1.0 / np.sqrt(m.d_in), size=(m.d_out, m.d_in))
        U, S, Vt = np.linalg.svd(W, full_matrices=False)
        P, Q = U * np.sqrt(S)[None, :], np.sqrt(S)[:, None] * Vt
    else:
        Q = g.normal(0.0, 1.0 / np.sqrt(m.d_in), size=(m.r, m.d_in))
        P = g.normal(0.0, 1.0 / np.sqrt(m.r), size=(m.d_out, m.r))
    return _cast(P, dtype), _cast(Q, dtype)


def gate_offset(layer: int, matrix: int) -> int:
    """Philox counter offset of the first gate of a matrix, so that every
    matrix of every layer draws from its own stretch of the stream."""
    return layer * (1 << 20) + matrix * (1 << 16)


def layer_problem(w: Workload, layer: int, matrix: int, seed: int = 0, T: int | None = None):
    """All inputs of one matrix of one layer: dict(X, dY, P, Q, log_alpha, m, T)."""
    m = w.matrices[matrix]
    T = w.T if T is None else T
    P, Q = factors(m, w.dtype, seed, layer, matrix, svd=(w.name == "single_f32"))
    return dict(m=m, T=T,
                X=activations(T, m.d_in, w.dtype, seed, 1, layer, matrix),
                dY=activations(T, m.d_out, w.dtype, seed, 2, layer, matrix),
                P=P, Q=Q,
                log_alpha=log_alpha(w.alpha, m.r, seed, layer, matrix))
