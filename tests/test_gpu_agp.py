"""GPU parity of the FLOP-AGP gate rule (magnitude pruning of the diagonal mask) and of a layer
step driven by those gates."""
import numpy as np
import pytest
import torch

from oracle import flop_oracle as O
from paper_1910_04732_b200 import inputs as I
from tests._util import empty_dev, host, rel_fro, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_1910_04732_b200 import build, binding
    build.build()
    binding.load_library()
    return binding


def _run(b, g_np, off, sparsity, l1, dg0=None):
    n, n_seg = len(g_np), len(off) - 1
    g = torch.from_numpy(g_np).cuda()
    so = torch.tensor(off, dtype=torch.int64, device="cuda")
    sp = torch.tensor([sparsity], dtype=torch.float32, device="cuda")
    z = torch.full((n,), float("nan"), device="cuda")
    m = torch.full((n,), 7, dtype=torch.uint8, device="cuda")
    d = torch.full((n,), float("nan"), device="cuda")
    l1s = torch.full((n_seg,), float("nan"), device="cuda")
    dg = torch.from_numpy(dg0).cuda() if dg0 is not None else None
    b.agp_gates(g, so, sp, l1, z, m, d, l1s, dg)
    torch.cuda.synchronize()
    return z.cpu().numpy(), m.cpu().numpy(), d.cpu().numpy(), l1s.cpu().numpy(), None if dg is None else dg.cpu().numpy()


@pytest.mark.parametrize("sparsity", [0.0, 0.3, 0.5, 0.9, 1.0])
def test_agp_gates_bit_exact(b, sparsity):
    rng = np.random.default_rng(3)
    counts = [1, 5, 768, 410, 2100, 4099]
    off = np.concatenate([[0], np.cumsum(counts)])
    g_np = rng.standard_normal(off[-1]).astype(np.float32)
    g_np[800:900] = np.float32(0.25) * np.sign(g_np[800:900])       # a block of tied magnitudes
    g_np[10] = 0.0
    dg0 = rng.standard_normal(off[-1]).astype(np.float32)
    s32 = float(np.float32(sparsity))
    z, m, d, l1s, dg = _run(b, g_np, off, s32, 0.05, dg0)
    ref = O.agp_gates(g_np, off, s32, float(np.float32(0.05)))
    assert np.array_equal(m, ref["mask"])
    assert np.array_equal(z, ref["z"].astype(np.float32)) and np.array_equal(d, ref["dz_dg"].astype(np.float32))
    assert np.allclose(l1s, ref["seg_l1"], rtol=2e-6)
    assert np.allclose(dg - dg0, ref["l1_grad"], rtol=1e-6, atol=1e-7)


def test_layer_step_with_agp_gates(b):
    """z = pruned diagonal, dz/dg = mask: the layer's dlog_alpha output is then the gradient w.r.t. g."""
    w = I.Workload("a", "bf16", 300, 1, (I.Matrix("w", 200, 136, 72),), ("normal", 0.0, 1.0), 0.5)
    prob = I.layer_problem(w, 0, 0, seed=4)
    m, T = prob["m"], prob["T"]
    g_np = np.random.default_rng(1).normal(1.0, 0.5, m.r).astype(np.float32)
    z, mask, dzdg, _, _ = _run(b, g_np, [0, m.r], 0.4, 0.0)
    bf = torch.bfloat16
    X, dY, P, Q = (to_dev(prob[k], "bf16") for k in ("X", "dY", "P", "Q"))
    zt, dt = torch.from_numpy(z).cuda(), torch.from_numpy(dzdg).cuda()
    Y, H, dX = empty_dev(T, m.d_out, bf), empty_dev(T, m.r, bf), empty_dev(T, m.d_in, bf)
    dP, dQ = empty_dev(m.d_out, m.r, bf), empty_dev(m.r, m.d_in, bf)
    dgr = torch.full((m.r,), float("nan"), device="cuda")
    b.gated_lowrank_fwd(X, Q, P, zt, Y, H, None)
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_BWD, T, m.d_in, m.d_out, m.r, b.BF16))
    b.gated_lowrank_bwd(dY, X, Q, P, zt, dt, H, dX, dP, dQ, dgr, ws)
    ref = O.agp_gates(g_np, [0, m.r], float(np.float32(0.4)), 0.0)
    G = O.gated_lowrank_bwd(prob["dY"], prob["X"], prob["Q"], prob["P"], ref["z"], ref["dz_dg"])
    assert rel_fro(host(Y), O.gated_lowrank_fwd(prob["X"], prob["Q"], prob["P"], ref["z"])[2]) < 2e-2
    assert rel_fro(host(dgr), G["dlog_alpha"]) < 2e-2 and np.all(host(dgr)[ref["mask"] == 0] == 0)
    assert b.device_status() == b.OK
