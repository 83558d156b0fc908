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
