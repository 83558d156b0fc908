"""GPU parity of the tensor-core GEMM building block against a plain fp64 matrix product,
over operand majors, tile shapes (one CTA / CTA pair, N tile, split-K) and ragged sizes."""
import numpy as np
import pytest
import torch

from paper_1910_04732_b200 import inputs as I
from tests._util import assert_close, empty_dev, host, rel_fro, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_1910_04732_b200 import build, binding
    build.build()
    binding.load_library()
    return binding


def _operands(M, N, K, seed):
    g = np.random.default_rng(seed)
    A = I.round_to_bf16(g.standard_normal((M, K)).astype(np.float32))
    B = I.round_to_bf16(g.standard_normal((N, K)).astype(np.float32) / np.sqrt(K))
    return A, B, A.astype(np.float64) @ B.astype(np.float64).T


SHAPES = [(128, 64, 64), (256, 256, 128), (300, 200, 136), (1000, 410, 410), (520, 72, 900), (77, 768, 520),
          (2048, 768, 768)]
TILES = [(0, -1), (64, 0), (128, 0), (192, 0), (256, 0), (64, 1), (128, 1), (192, 1), (208, 1), (256, 1)]


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("bn,cta2", TILES)
def test_k_major_operands(b, M, N, K, bn, cta2):
    A, B, want = _operands(M, N, K, M + N + K)
    D = empty_dev(M, N, torch.bfloat16)
    scale = np.linspace(0.0, 2.0, N).astype(np.float32)
    b.tc_gemm(to_dev(A, "bf16"), False, to_dev(B, "bf16"), False, M, N, K, D=D, bn=bn, cta2=cta2)
    assert rel_fro(host(D), want) < 4e-3            # one bf16 rounding of the output
    assert_close(D, want, "bf16", "D")              # and no element or block off (tile seams, ragged tails)
    D.fill_(float("nan"))
    b.tc_gemm(to_dev(A, "bf16"), False, to_dev(B, "bf16"), False, M, N, K, D=D,
              col_scale=torch.from_numpy(scale).cuda(), bn=bn, cta2=cta2)
    assert rel_fro(host(D), want * scale[None, :]) < 4e-3
    assert_close(D, want * scale[None, :], "bf16", "D scaled")
    assert np.all(host(D)[:, 0] == 0)               # a closed gate zeroes its column exactly
    assert b.device_status() == b.OK


@pytest.mark.parametrize("M,N,K", SHAPES)
@pytest.mark.parametrize("bn,cta2", [(0, -1), (64, 0), (192, 0), (256, 0), (128, 1), (256, 1)])
def test_b_read_transposed(b, M, N, K, bn, cta2):
    """B given as a row-major [K, N] matrix (the dH' = dY P and dX = dH' Qz products)."""
    A, B, want = _operands(M, N, K, 7 + M + N + K)
    D = empty_dev(M, N, torch.bfloat16)
    b.tc_gemm(to_dev(A, "bf16"), False, to_dev(np.ascontiguousarray(B.T), "bf16"), True, M, N, K, D=D, bn=bn, cta2=cta2)
    assert rel_fro(host(D), want) < 4e-3
    assert b.device_status() == b.OK


@pytest.mark.parametrize("M,N,K", [(128, 64, 64), (256, 128, 512), (300, 200, 1000), (410, 410, 2200), (768, 768, 4096),
                                   (2100, 410, 1300), (72, 136, 9000)])
@pytest.mark.parametrize("bn,cta2,splits", [(0, -1, 0), (64, 0, 1), (128, 0, 4), (192, 0, 3), (256, 0, 16),
                                            (128, 1, 1), (128, 1, 5), (256, 1, 2), (256, 1, 32)])
def test_token_contraction_split_k(b, M, N, K, bn, cta2, splits):
    """Both operands row-major [K, *] (the weight-gradient products contract over tokens):
    fp32 slices whose ordered sum is the product; fp32 accuracy, no output rounding."""
    A, B, want = _operands(M, N, K, 13 + M + N + K)
    ldn = (N + 3) // 4 * 4
    slices = torch.full((32 * M * ldn,), float("nan"), device="cuda")
    n = b.tc_gemm(to_dev(np.ascontiguousarray(A.T), "bf16"), True, to_dev(np.ascontiguousarray(B.T), "bf16"), True,
                  M, N, K, slices=slices, bn=bn, cta2=cta2, splits=splits)
    assert 1 <= n <= 32 and (splits == 0 or n <= splits)
    got = slices[: n * M * ldn].view(n, M, ldn)[:, :, :N].double().sum(0).cpu().numpy()
    assert rel_fro(got, want) < 5e-5          # fp32 accumulation over up to 9000 terms, no output rounding
    assert b.device_status() == b.OK
