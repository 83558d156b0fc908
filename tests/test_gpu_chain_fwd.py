"""GPU parity of the on-chip forward chain: Y = ((X Q^T) * z) P^T in one launch with the intermediate kept in
tensor memory and shared memory, against the oracle's two plain products."""
import numpy as np
import pytest
import torch

from oracle import flop_oracle as O
from paper_1910_04732_b200 import inputs as I
from tests._util import HC, assert_close, empty_dev, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_1910_04732_b200 import build, binding
    build.build()
    binding.load_library()
    return binding


@pytest.mark.parametrize("T,d_in,d_out,r", [
    (128, 64, 128, 64),          # one row block, one k-block, one N tile
    (17, 1024, 4096, 358),       # pruned-inference shapes: ragged k (pads to 384: two MMAs per k-step), few tokens
    (64, 1024, 4096, 358), (256, 1024, 4096, 358),
    (300, 200, 136, 72),         # ragged everywhere
    (1000, 410, 2100, 256),      # k = 256 exactly, ragged d_in / d_out tails
    (640, 2100, 410, 384),       # d_out tail of 26 columns
    (700, 520, 1000, 448), (333, 264, 520, 512), (200, 136, 264, 200),   # 3-stage and 2-stage second ring; k_pad = 256
    (4096, 1024, 4096, 358)])    # 32 row blocks x 4 slices of 8 N tiles
def test_chain_fwd_matches_oracle(b, T, d_in, d_out, r):
    w = I.Workload("c", "bf16", T, 1, (I.Matrix("w", d_in, d_out, r),), ("normal", 0.5, 1.5), 0.5)
    prob = I.layer_problem(w, 0, 0, seed=T + r)
    X, P, Q = (to_dev(prob[k], "bf16") for k in ("X", "P", "Q"))
    z_np, _, _ = O.gate_sample(prob["log_alpha"], *HC, seed=3, offset=11)
    z_np = z_np.astype(np.float32)
    z = torch.from_numpy(z_np).cuda()
    Y = empty_dev(T, d_out, torch.bfloat16)
    n0 = b.launch_count()
    b.chain_fwd(X, Q, P, z, Y)
    assert b.launch_count() - n0 == 1
    assert b.device_status() == b.OK
    _, _, want = O.gated_lowrank_fwd(prob["X"], prob["Q"], prob["P"], z_np)
    assert_close(Y, want, "bf16", "Y")
    # without a gate vector (compact factors carry the gate): plain (X Q^T) P^T
    Y2 = empty_dev(T, d_out, torch.bfloat16)
    b.chain_fwd(X, Q, P, None, Y2)
    _, _, want2 = O.gated_lowrank_fwd(prob["X"], prob["Q"], prob["P"], np.ones(r))
    assert_close(Y2, want2, "bf16", "Y ungated")
    assert b.device_status() == b.OK


def test_chain_fwd_on_compact_factors_equals_the_uncompacted_gated_layer(b):
    """The inference workload: deterministic gates, compaction, then the chain on (Qc, Pc, k)."""
    w = I.WORKLOADS["infer"]
    m = w.matrices[0]
    prob = I.layer_problem(w, 0, 0, T=256)
    X, P, Q = (to_dev(prob[k], "bf16") for k in ("X", "P", "Q"))
    la = torch.from_numpy(prob["log_alpha"]).cuda()
    idx, kd, zd = torch.empty(m.r, dtype=torch.int32, device="cuda"), torch.zeros(1, dtype=torch.int32, device="cuda"), torch.empty(m.r, device="cuda")
    Pc, Qc = empty_dev(m.d_out, m.r, torch.bfloat16), empty_dev(m.r, m.d_in, torch.bfloat16)
    b.compact_ranks(la, 0, HC, idx, kd, zd, P, Q, Pc, Qc)
    k = int(kd.item())
    assert 0 < k <= 512
    Y = empty_dev(256, m.d_out, torch.bfloat16)
    b.chain_fwd(X, Qc[:k], Pc[:, :k], None, Y)
    k_o, idx_o, z_det = O.deterministic_mask(prob["log_alpha"], *HC)
    assert k_o == k
    _, _, want = O.gated_lowrank_fwd(prob["X"], prob["Q"], prob["P"], z_det)
    assert_close(Y, want, "bf16", "Y")
    assert b.device_status() == b.OK


def test_chain_fwd_refuses_what_it_cannot_hold(b):
    X, Q, P = (torch.zeros(s, dtype=torch.bfloat16, device="cuda") for s in ((64, 64), (520, 64), (64, 520)))
    Y = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(b.FlopError) as ei:
        b.chain_fwd(X, Q, P, None, Y)
    assert ei.value.code == b.ERR_UNSUPPORTED          # r = 520 > 512
    Xf = torch.zeros(64, 64, device="cuda")
    with pytest.raises(b.FlopError) as ei:
        b.chain_fwd(Xf, Xf, Xf, None, Xf, dt=b.F32)
    assert ei.value.code == b.ERR_UNSUPPORTED
