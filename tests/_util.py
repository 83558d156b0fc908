"""Helpers shared by the GPU parity tests: host arrays -> device tensors and error norms."""
import numpy as np
import torch

from paper_1910_04732_b200 import inputs as I

# the C ABI takes the hard-concrete constants as fp32; the oracle gets the same values
HC = tuple(float(np.float32(v)) for v in (I.BETA, I.GAMMA, I.ZETA))


def to_dev(a: np.ndarray, dtype: str) -> torch.Tensor:
    """Row-major device copy whose leading dimension is padded to 8 elements."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    rows, cols = a.shape
    ld = max((cols + 7) // 8 * 8, 8)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    buf = torch.zeros(rows, ld, dtype=tdt, device="cuda")
    view = buf[:, :cols]
    view.copy_(torch.from_numpy(a).to(tdt))
    return view


def empty_dev(rows: int, cols: int, dtype, fill=float("nan")) -> torch.Tensor:
    """Output buffer, poisoned so that an unwritten element shows up."""
    ld = max((cols + 7) // 8 * 8, 8)
    buf = torch.full((rows, ld), fill, dtype=dtype, device="cuda")
    return buf[:, :cols]


def host(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def rel_fro(got: np.ndarray, want: np.ndarray) -> float:
    denom = np.linalg.norm(want)
    return float(np.linalg.norm(got - want) / denom) if denom > 0 else float(np.linalg.norm(got))


# Element-wise parity bounds.  A global relative Frobenius norm cannot see a wrong row or a mis-scaled
# 32 x 64 epilogue block of a large output, so every output is also held to
#     |got - want| <= REL * |want| + ABS * rms(row of want)           (each element)
#     ||got - want||_F <= BLOCK * ||want||_F                          (each 128 x 64 block)
# "bf16": the output is stored in bf16 (half an ulp = 2^-9 relative... allow a full ulp 2^-8 plus headroom: 2^-7)
# and was accumulated in fp32 from bf16-rounded intermediates (H', dH', diag(z) Q: 2^-9 relative each, summed as
# a random walk over the contraction, which stays below 1 % of the row's rms).  "f32": fp32 storage and fp32
# accumulation in another order than the oracle's.
ELEMENT_BOUNDS = {
    "bf16": dict(rel=2.0 ** -7, abs_rms=2.0e-2, block=2.0e-2, fro=2.0e-2),
    "f32": dict(rel=1.0e-5, abs_rms=2.0e-5, block=1.0e-5, fro=1.0e-5),
}


def closeness(got: np.ndarray, want: np.ndarray, kind: str = "bf16") -> dict:
    """The three error measures of `got` against `want`, each as a fraction of its bound (<= 1 passes)."""
    bd = ELEMENT_BOUNDS[kind]
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    if got.ndim == 1:
        got, want = got[None, :], want[None, :]
    err = np.abs(got - want)
    rms = np.sqrt(np.mean(want * want, axis=1, keepdims=True))
    allowed = bd["rel"] * np.abs(want) + bd["abs_rms"] * rms
    with np.errstate(divide="ignore", invalid="ignore"):
        ratio = np.where(allowed > 0, err / allowed, np.where(err > 0, np.inf, 0.0))
    worst_elem = float(ratio.max()) if ratio.size else 0.0
    worst_block = 0.0
    rows, cols = want.shape
    for r0 in range(0, rows, 128):
        for c0 in range(0, cols, 64):
            w = want[r0:r0 + 128, c0:c0 + 64]
            e = np.linalg.norm(got[r0:r0 + 128, c0:c0 + 64] - w)
            n = np.linalg.norm(w)
            frac = e / (bd["block"] * n) if n > 0 else (np.inf if e > 0 else 0.0)
            worst_block = max(worst_block, float(frac))
    return {"fro": rel_fro(got, want) / bd["fro"], "element": worst_elem, "block": worst_block}


def assert_close(got, want, kind: str = "bf16", name: str = "") -> dict:
    """Global, per-block and per-element parity of one output (see ELEMENT_BOUNDS)."""
    g = host(got) if isinstance(got, torch.Tensor) else np.asarray(got, dtype=np.float64)
    assert np.all(np.isfinite(g)), f"{name}: non-finite values"
    c = closeness(g, want, kind)
    assert c["fro"] <= 1.0, (name, "relative Frobenius error over its bound", c)
    assert c["block"] <= 1.0, (name, "a 128 x 64 block over its bound", c)
    assert c["element"] <= 1.0, (name, "an element over its bound", c)
    return c
