"""GPU parity: deterministic mask, rank compaction and the compact inference forward."""
import numpy as np
import pytest
import torch

from oracle import flop_oracle as O
from paper_1910_04732_b200 import inputs as I
from tests._util import HC, empty_dev, host, rel_fro, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_1910_04732_b200 import build, binding
    build.build()
    binding.load_library()
    return binding


def _select(b, vec, mode):
    r = len(vec)
    v = torch.from_numpy(np.asarray(vec, np.float32)).cuda()
    idx = torch.full((max(r, 1),), -1, dtype=torch.int32, device="cuda")
    k = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    zd = torch.full((max(r, 1),), float("nan"), device="cuda")
    b.compact_ranks(v[:r], mode, HC, idx, k, zd)
    return int(k.item()), idx.cpu().numpy(), zd.cpu().numpy()[:r]


@pytest.mark.parametrize("r,kind", [(1, ("normal", 0.0, 1.0)), (33, ("normal", 0.5, 1.0)), (1024, I.WORKLOADS["infer"].alpha),
                                    (768, ("bimodal", 3.0, 0.5)), (4099, ("normal", -1.0, 2.0)), (65536, ("normal", 1.0, 1.5))])
def test_deterministic_mask_is_bit_exact(b, r, kind):
    a = I.log_alpha(kind, r, 0, 9)
    k, idx, zd = _select(b, a, 0)
    ko, idxo, zo = O.deterministic_mask(a, *HC)
    assert k == ko
    assert np.array_equal(idx[:k], idxo)
    assert np.array_equal(zd > 0, zo > 0) and np.max(np.abs(zd - zo)) < 1e-7


def test_topk_ties_edges_and_mode1(b):
    # heavy ties: only 5 distinct values, the cut falls inside a tie class
    g = np.random.default_rng(0)
    a = g.choice(np.array([-2.0, -0.5, 0.0, 0.5, 2.0], np.float32), size=3000)
    a[::7] = -0.0
    k, idx, zd = _select(b, a, 0)
    ko, idxo, zo = O.deterministic_mask(a, *HC)
    assert k == ko and np.array_equal(idx[:k], idxo)
    for val, want in ((-30.0, 0), (30.0, 500)):
        k, idx, zd = _select(b, np.full(500, val, np.float32), 0)
        assert k == want and np.array_equal(idx[:k], np.arange(want))
    # mode 1: keep z > 0 of a sampled mask
    alpha = I.log_alpha(("normal", -0.5, 2.0), 5000, 0, 3)
    z, mask, _ = O.gate_sample(alpha, *HC, 0, 0)
    k, idx, zd = _select(b, z.astype(np.float32), 1)
    ko, idxo = O.active_ranks(z.astype(np.float32))
    assert k == ko == int(mask.sum()) and np.array_equal(idx[:k], idxo)
    assert np.array_equal(zd, z.astype(np.float32))
    k, idx, zd = _select(b, np.zeros(0, np.float32), 0)
    assert k == 0


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_pruned_inference_config(b, dtype):
    """d_in = 1024, d_out = 4096, r = 1024, about 35 % of the components survive;
    compact path against the oracle and against the uncompacted gated path."""
    w = I.WORKLOADS["infer"]
    m = w.matrices[0]
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    prob = I.layer_problem(I.Workload("i", dtype, 4096, 1, w.matrices, w.alpha, w.target), 0, 0)
    P, Q = to_dev(prob["P"], dtype), to_dev(prob["Q"], dtype)
    la = torch.from_numpy(prob["log_alpha"]).cuda()
    idx = torch.full((m.r,), -1, dtype=torch.int32, device="cuda")
    kd = torch.zeros(1, dtype=torch.int32, device="cuda")
    zd = torch.empty(m.r, device="cuda")
    Pc, Qc = empty_dev(m.d_out, m.r, tdt), empty_dev(m.r, m.d_in, tdt)
    b.compact_ranks(la, 0, HC, idx, kd, zd, P, Q, Pc, Qc)
    k = int(kd.item())
    ko, idxo, zo = O.deterministic_mask(prob["log_alpha"], *HC)
    assert k == ko and 300 < k < 420
    assert np.array_equal(idx.cpu().numpy()[:k], idxo)
    Pco, Qco = O.compact_ranks(prob["P"], prob["Q"], idxo, zo)
    assert np.array_equal(host(Pc)[:, :k], Pco)                    # a pure gather: exact
    assert np.all(np.isnan(host(Pc)[:, k:])) and np.all(np.isnan(host(Qc)[k:]))     # the rest is untouched
    assert rel_fro(host(Qc)[:k], Qco) < (4e-3 if dtype == "bf16" else 1e-6)
    tol = 2e-2 if dtype == "bf16" else 1e-5
    for T in (1, 3, 4, 5, 9, 16, 17, 64, 256, 4096):   # 1..4: CUDA-core streaming, 5..16: warp-level MMA, above: tcgen05
        X = to_dev(prob["X"][:T], dtype)
        Y = empty_dev(T, m.d_out, tdt)
        ws = b.alloc_workspace(b.workspace_bytes(b.OP_COMPACT_FWD, T, m.d_in, m.d_out, k, b.BF16 if dtype == "bf16" else b.F32))
        b.compact_fwd(X, Qc[:k], Pc[:, :k], Y, k, ws)
        Yo = O.compact_fwd(prob["X"][:T], Qco, Pco)
        assert rel_fro(host(Y), Yo) < tol, T
        # against the uncompacted gated path with the same deterministic gates
        Yg, H = empty_dev(T, m.d_out, tdt), empty_dev(T, m.r, tdt)
        b.gated_lowrank_fwd(X, Q, P, zd, Yg, H, None)
        assert rel_fro(host(Y), host(Yg)) < tol, T
    assert b.device_status() == b.OK


def test_compact_fwd_with_no_survivors(b):
    X = torch.ones(5, 16, dtype=torch.bfloat16, device="cuda")
    Y = torch.full((5, 24), float("nan"), dtype=torch.bfloat16, device="cuda")
    b.compact_fwd(X, X[:0], torch.zeros(24, 8, dtype=torch.bfloat16, device="cuda")[:, :0], Y, 0, None)
    assert torch.count_nonzero(Y) == 0


@pytest.mark.parametrize("r,d_out,d_in,keep", [
    (1024, 40003, 16, 0.35),    # 8 rows per stage, more groups than buffers per block (buffers reused, parity flips), ragged last group
    (16384, 1003, 8, 0.40),     # one 32 KB row per stage, two buffers
    (64, 777, 24, 0.5),         # 16 rows per stage, tiny rows
    (1024, 517, 8, 0.001),      # one or two survivors: the scalar tail of a row
    (1032, 300, 8, 1.0),        # every component survives
    (1020, 300, 8, 0.35),       # rows that are not 16-byte multiples: the plain kernel
])
def test_gather_of_survivors_is_exact(b, r, d_out, d_in, keep):
    """P_c = P[:, idx] and Q_c = diag(z) Q[idx, :] for a supplied gate vector (mode 1): a pure gather on the P side,
    compared element by element with the oracle's indexing; columns from k on stay untouched."""
    g = np.random.default_rng(r + d_out)
    z = np.where(g.random(r) < keep, g.uniform(0.05, 1.0, r), 0.0).astype(np.float32)
    if keep < 0.01:
        z[:] = 0.0
        z[[5, r - 3]] = (0.25, 0.75)
    P = g.standard_normal((d_out, r)).astype(np.float32)
    Q = g.standard_normal((r, d_in)).astype(np.float32)
    Pd, Qd = to_dev(P, "bf16"), to_dev(Q, "bf16")
    Pb, Qb = host(Pd), host(Qd)                      # the bf16-rounded values both sides use
    zt = torch.from_numpy(z).cuda()
    idx = torch.full((r,), -1, dtype=torch.int32, device="cuda")
    kd = torch.zeros(1, dtype=torch.int32, device="cuda")
    Pc, Qc = empty_dev(d_out, r, torch.bfloat16), empty_dev(r, d_in, torch.bfloat16)
    b.compact_ranks(zt, 1, HC, idx, kd, None, Pd, Qd, Pc, Qc)
    k = int(kd.item())
    ko, idxo = O.active_ranks(z)
    assert k == ko and np.array_equal(idx.cpu().numpy()[:k], idxo)
    Pco, Qco = O.compact_ranks(Pb, Qb, idxo, z.astype(np.float64))
    got = host(Pc)
    assert np.array_equal(got[:, :k], Pco)
    assert np.all(np.isnan(got[:, k:]))
    assert rel_fro(host(Qc)[:k], Qco) < 4e-3
    assert b.device_status() == b.OK
