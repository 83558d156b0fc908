"""GPU parity of the per-step launches that replace per-call small kernels: diag(z) Q formed for all matrices at
once (flop_scale_rows_grouped) and the second stage of dlog_alpha left to one launch at the end
(defer_dlog_alpha + flop_dlog_alpha_finish_grouped).  Results must equal, bit for bit, those of backward calls
that do both themselves, and match the oracle."""
import numpy as np
import pytest
import torch

from oracle import flop_oracle as O
from paper_1910_04732_b200 import inputs as I
from tests._util import HC, assert_close, empty_dev, host, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_1910_04732_b200 import build, binding
    build.build()
    binding.load_library()
    return binding


def _layer(b, w, layer, seed, init=float("nan")):
    bf = torch.bfloat16
    es = []
    for i, m in enumerate(w.matrices):
        prob = I.layer_problem(w, layer, i, seed=seed)
        e = dict(prob=prob, m=m)
        for k in ("X", "dY", "P", "Q"):
            e[k] = to_dev(prob[k], "bf16")
        z, mask, dzd = O.gate_sample(prob["log_alpha"], *HC, seed=seed, offset=I.gate_offset(layer, i))
        e["z_np"], e["dzd_np"] = z.astype(np.float32), dzd.astype(np.float32)
        e["z"], e["dzd"] = torch.from_numpy(e["z_np"]).cuda(), torch.from_numpy(e["dzd_np"]).cuda()
        T = prob["T"]
        e["Y"], e["H"] = empty_dev(T, m.d_out, bf), empty_dev(T, m.r, bf)
        e["Qz"] = empty_dev(m.r, m.d_in, bf)
        for tag in ("a", "b"):
            e["dX" + tag] = empty_dev(T, m.d_in, bf)
            e["dP" + tag], e["dQ" + tag] = empty_dev(m.d_out, m.r, bf, init), empty_dev(m.r, m.d_in, bf, init)
            e["dla" + tag] = torch.full((m.r,), init, device="cuda")
            e["ws" + tag] = b.alloc_workspace(b.workspace_bytes(b.OP_BWD, T, m.d_in, m.d_out, m.r, b.BF16))
            e["ws" + tag].fill_(0xFF)
        es.append(e)
    return es


def _bwd(b, es, tag, **kw):
    return [b.bwd_problem(e["dY"], e["X"], e["Q"], e["P"], e["z"], e["dzd"], e["H"], e["dX" + tag], e["dP" + tag], e["dQ" + tag],
                          e["dla" + tag], e["ws" + tag], Qz=e["Qz"] if kw.get("qz") else None,
                          defer_dlog_alpha=kw.get("defer", False)) for e in es]


@pytest.mark.parametrize("accumulate", [False, True])
def test_two_layers_with_one_scale_launch_and_one_dlog_alpha_launch(b, accumulate):
    """Two Transformer-XL-shaped layers (ragged widths) at T = 700: the backward calls of both layers defer
    dlog_alpha; one finishing launch serves all twelve matrices."""
    w = I.Workload("s", "bf16", 700, 2, I.WORKLOADS["txl"].matrices, ("normal", 0.5, 1.0), 0.35)
    init = 0.25 if accumulate else float("nan")
    layers = [_layer(b, w, l, 5 + l, init) for l in range(2)]
    every = [e for es in layers for e in es]
    n0 = b.launch_count()
    b.scale_rows_grouped([b.scale_rows_problem(e["Q"], e["z"], e["Qz"]) for e in every])
    assert b.launch_count() - n0 == 1
    for e in every:
        want = (e["Q"].float() * e["z"][:, None]).to(torch.bfloat16)
        assert torch.equal(e["Qz"].view(torch.int16), want.view(torch.int16))          # one rounding, exact
    for es in layers:
        b.gated_lowrank_fwd_grouped([b.fwd_problem(e["X"], e["Q"], e["P"], e["z"], e["Y"], e["H"]) for e in es])
        n0 = b.launch_count()
        b.gated_lowrank_bwd_grouped(_bwd(b, es, "a", qz=True, defer=True), accumulate=accumulate)
        assert b.launch_count() - n0 == 2                                               # the two GEMM launches only
        b.gated_lowrank_bwd_grouped(_bwd(b, es, "b"), accumulate=accumulate)            # does both by itself
    n0 = b.launch_count()
    b.dlog_alpha_finish_grouped(_bwd(b, every, "a", qz=True, defer=True), accumulate=accumulate)
    assert b.launch_count() - n0 == 1
    assert b.device_status() == b.OK
    off = 0.25 if accumulate else 0.0
    for e in every:
        p = e["prob"]
        G = O.gated_lowrank_bwd(p["dY"], p["X"], p["Q"], p["P"], e["z_np"], e["dzd_np"])
        for k, want in (("dX", G["dX"]), ("dP", G["dP"] + off), ("dQ", G["dQ"] + off), ("dla", G["dlog_alpha"] + off)):
            assert_close(e[k + "a"], want, "bf16", f"{e['m'].name}.{k}")
            x, y = e[k + "a"], e[k + "b"]
            same = torch.equal(x.view(torch.int16), y.view(torch.int16)) if x.dtype == torch.bfloat16 else torch.equal(x, y)
            assert same, (e["m"].name, k)


def test_deferred_dlog_alpha_needs_the_grouped_bf16_path(b):
    w = I.Workload("s", "f32", 50, 1, (I.Matrix("a", 24, 40, 16),), ("normal", 0.5, 1.0), 0.5)
    prob = I.layer_problem(w, 0, 0, seed=1)
    X, dY, P, Q = (to_dev(prob[k], "f32") for k in ("X", "dY", "P", "Q"))
    z, dzd = torch.ones(16, device="cuda"), torch.ones(16, device="cuda")
    H, dX = empty_dev(50, 16, torch.float32), empty_dev(50, 24, torch.float32)
    dP, dQ, dla = empty_dev(40, 16, torch.float32), empty_dev(16, 24, torch.float32), torch.zeros(16, device="cuda")
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_BWD, 50, 24, 40, 16, b.F32))
    pr = [b.bwd_problem(dY, X, Q, P, z, dzd, H, dX, dP, dQ, dla, ws, defer_dlog_alpha=True)]
    with pytest.raises(b.FlopError) as ei:
        b.gated_lowrank_bwd_grouped(pr, dt=b.F32, wgrad_dt=b.F32)
    assert ei.value.code == b.ERR_UNSUPPORTED
