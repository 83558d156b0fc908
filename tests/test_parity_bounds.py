"""The parity checks themselves, on the CPU: the per-element and per-block bounds that every GPU parity test
applies (tests/_util.py) must reject the mistakes a global norm lets through, and accept honest bf16 rounding."""
import numpy as np
import pytest

from oracle import flop_oracle as O
from paper_1910_04732_b200 import inputs as I
from tests._util import assert_close, closeness, rel_fro


def _bf16_round(a):
    """Round-to-nearest-even to bf16 precision, in numpy."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


@pytest.fixture(scope="module")
def layer():
    w = I.Workload("p", "bf16", 4096, 1, (I.Matrix("w", 256, 768, 128),), ("normal", 0.5, 1.0), 0.5)
    p = I.layer_problem(w, 0, 0, seed=3)
    z = np.linspace(0.0, 1.0, 128)
    _, Hp, Y = O.gated_lowrank_fwd(p["X"], p["Q"], p["P"], z)
    return Y


def test_honest_bf16_output_passes(layer):
    c = assert_close(_bf16_round(layer), layer, "bf16", "Y")
    assert c["element"] < 0.6 and c["block"] < 0.3


def test_one_shifted_row_is_caught_although_the_global_norm_passes(layer):
    bad = _bf16_round(layer)
    bad[1000] = bad[999]
    assert rel_fro(bad, layer) < 2e-2 * 1.2            # about sqrt(2 / 4096) = 2.2e-2: at the edge of the global bound
    c = closeness(bad, layer, "bf16")
    assert c["element"] > 10 and c["block"] > 5
    with pytest.raises(AssertionError):
        assert_close(bad, layer, "bf16", "Y")


def test_mis_scaled_or_ungated_epilogue_block_is_caught(layer):
    for factor in (0.5, 1.5, 1.05):
        bad = _bf16_round(layer)
        bad[256:288, 128:192] *= factor                # one 32 x 64 epilogue block
        assert rel_fro(bad, layer) < 2e-2              # invisible to the global norm
        with pytest.raises(AssertionError):
            assert_close(bad, layer, "bf16", "Y")


def test_whole_output_shifted_by_one_row_is_caught(layer):
    bad = np.roll(_bf16_round(layer), 1, axis=0)
    with pytest.raises(AssertionError):
        assert_close(bad, layer, "bf16", "Y")


def test_exact_zero_rows_demand_exact_zeros():
    want = np.zeros((4, 8)); want[1] = 1.0
    got = want.copy(); got[0, 3] = 1e-30
    with pytest.raises(AssertionError):
        assert_close(got, want, "bf16", "dQ")
    assert_close(want, want, "f32", "dQ")
