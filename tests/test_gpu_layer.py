"""GPU parity: gated low-rank forward/backward through the C ABI against the fp64 oracle.

Tolerances (relative Frobenius error): 1e-5 for fp32 storage, 2e-2 for bf16
storage with fp32 accumulation.  For bf16 the oracle consumes the bf16-rounded
inputs exactly, so the tolerance covers only the kernels' own roundings of the
intermediates (H', dH', diag(z)Q) and the fp32 summation order."""
import numpy as np
import pytest
import torch

from oracle import flop_oracle as O
from paper_1910_04732_b200 import inputs as I
from tests._util import HC, assert_close, empty_dev, host, rel_fro, to_dev

pytestmark = pytest.mark.gpu
TOL = {"f32": 1e-5, "bf16": 2e-2}


@pytest.fixture(scope="module")
def b():
    from paper_1910_04732_b200 import build, binding
    build.build()
    binding.load_library()
    return binding


def run_layer(b, prob, dtype, seed=0, offset=0, wgrad_dtype=None, accumulate=False, check=True):
    """Sample gates, run fwd + bwd on the GPU and on the oracle; returns (gpu, ref) dicts."""
    m, T = prob["m"], prob["T"]
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    wdt = tdt if wgrad_dtype is None else wgrad_dtype
    X, dY, P, Q = (to_dev(prob[k], dtype) for k in ("X", "dY", "P", "Q"))
    la = torch.from_numpy(prob["log_alpha"]).cuda()
    z = torch.empty(m.r, device="cuda"); dzd = torch.empty(m.r, device="cuda")
    mask = torch.empty(m.r, dtype=torch.uint8, device="cuda")
    b.gate_sample(la, HC, seed, offset, z, mask, dzd)
    Y, H = empty_dev(T, m.d_out, tdt), empty_dev(T, m.r, tdt)
    b.gated_lowrank_fwd(X, Q, P, z, Y, H, None)
    init = 0.5 if accumulate else float("nan")
    dX = empty_dev(T, m.d_in, tdt)
    dP, dQ = empty_dev(m.d_out, m.r, wdt, init), empty_dev(m.r, m.d_in, wdt, init)
    dla = torch.full((m.r,), init, device="cuda")
    dti = b.BF16 if dtype == "bf16" else b.F32
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_BWD, T, m.d_in, m.d_out, m.r, dti))
    ws.fill_(0xFF)                                       # NaN poison
    b.gated_lowrank_bwd(dY, X, Q, P, z, dzd, H, dX, dP, dQ, dla, ws, accumulate)
    assert b.device_status() == b.OK
    gpu = dict(z=host(z), mask=mask.cpu().numpy(), Y=host(Y), Hp=host(H), dX=host(dX), dP=host(dP), dQ=host(dQ),
               dlog_alpha=host(dla))
    zo, mo, dzo = O.gate_sample(prob["log_alpha"], *HC, seed=seed, offset=offset)
    # the oracle takes the gates the kernels consumed (fp32 values of z), so GEMM parity is
    # not polluted by the sampler's 1e-7 differences; the sampler has its own test
    zg, dzg = gpu["z"], host(dzd)
    assert np.array_equal(gpu["mask"], mo) and np.max(np.abs(zg - zo)) < 2e-6
    _, Hp, Yo = O.gated_lowrank_fwd(prob["X"], prob["Q"], prob["P"], zg)
    G = O.gated_lowrank_bwd(prob["dY"], prob["X"], prob["Q"], prob["P"], zg, dzg)
    ref = dict(Y=Yo, Hp=Hp, dX=G["dX"], dP=G["dP"], dQ=G["dQ"], dlog_alpha=G["dlog_alpha"])
    if accumulate:
        for k in ("dP", "dQ", "dlog_alpha"):
            ref[k] = ref[k] + 0.5
    if check:
        # global relative Frobenius error (1e-5 / 2e-2) plus per-block and per-element bounds
        for k in ("Hp", "Y", "dX", "dP", "dQ", "dlog_alpha"):
            assert_close(gpu[k], ref[k], dtype, k)
    return gpu, ref


def test_single_layer_f32_full_config(b):
    """fp32, d_in = d_out = r = 256, T = 512, SVD factors, Philox seed 0."""
    w = I.WORKLOADS["single_f32"]
    gpu, ref = run_layer(b, I.layer_problem(w, 0, 0), "f32")
    assert 0 < gpu["mask"].sum() <= 256
    # closed gates kill their column of dP and row of dQ exactly
    dead = gpu["z"] == 0
    assert np.all(gpu["dQ"][dead] == 0) and np.all(gpu["dP"][:, dead] == 0)


@pytest.mark.parametrize("T,d_in,d_out,r", [(1, 8, 8, 8), (5, 4, 3, 6), (77, 130, 67, 45), (300, 200, 136, 72),
                                            (129, 64, 256, 64), (512, 256, 256, 256)])
def test_f32_ragged_shapes(b, T, d_in, d_out, r):
    w = I.Workload("t", "f32", T, 1, (I.Matrix("w", d_in, d_out, r),), ("normal", 0.5, 1.5), 0.5)
    run_layer(b, I.layer_problem(w, 0, 0, seed=T), "f32", seed=3, offset=17)


@pytest.mark.parametrize("T,d_in,d_out,r", [
    (128, 64, 128, 64),        # single tile, single k-block
    (256, 128, 256, 128),      # two k-blocks
    (300, 200, 136, 72),       # ragged everywhere, r not a multiple of 16
    (1000, 410, 410, 410),     # Transformer-XL attention shape, K tail of 26
    (640, 410, 2100, 410),     # FFN1 shape
    (640, 2100, 410, 410),     # FFN2 shape
    (1, 64, 64, 64), (16, 1024, 4096, 358), (40, 200, 136, 72), (64, 410, 2100, 410),
    (2048, 768, 768, 768)])
def test_bf16_shapes(b, T, d_in, d_out, r):
    w = I.Workload("t", "bf16", T, 1, (I.Matrix("w", d_in, d_out, r),), ("normal", 0.5, 1.5), 0.5)
    run_layer(b, I.layer_problem(w, 0, 0, seed=T + r), "bf16", seed=1, offset=5)


@pytest.mark.parametrize("name,matrix", [("txl", 0), ("txl", 4), ("txl", 5), ("bert", 0), ("bert", 4), ("bert", 5),
                                         ("sru", 0)])
def test_bf16_full_size_layers(b, name, matrix):
    """One matrix of each distinct shape of the benchmark workloads, at full token count."""
    w = I.WORKLOADS[name]
    gpu, ref = run_layer(b, I.layer_problem(w, 1, matrix), "bf16", seed=0, offset=I.gate_offset(1, matrix))
    assert gpu["mask"].sum() > 0


def test_bf16_fp32_weight_gradients_and_accumulate(b):
    w = I.Workload("t", "bf16", 900, 1, (I.Matrix("w", 264, 520, 200),), ("bimodal", 3.0, 0.5), 0.5)
    prob = I.layer_problem(w, 0, 0, seed=5)
    g1, r1 = run_layer(b, prob, "bf16", wgrad_dtype=torch.float32)
    g2, r2 = run_layer(b, prob, "bf16", wgrad_dtype=torch.float32, accumulate=True)
    assert np.allclose(g2["dP"] - 0.5, g1["dP"], atol=1e-4) and np.allclose(g2["dQ"] - 0.5, g1["dQ"], atol=1e-4)
    # fp32 weight gradients keep fp32 accumulation accuracy given the bf16 intermediates
    assert rel_fro(g1["dP"], r1["dP"]) < 5e-3
    run_layer(b, prob, "bf16", accumulate=True)


def test_bwd_is_bit_reproducible(b):
    w = I.Workload("t", "bf16", 1500, 1, (I.Matrix("w", 384, 640, 256),), ("normal", 0.5, 1.5), 0.5)
    prob = I.layer_problem(w, 0, 0, seed=6)
    g1, _ = run_layer(b, prob, "bf16", wgrad_dtype=torch.float32)
    g2, _ = run_layer(b, prob, "bf16", wgrad_dtype=torch.float32)
    for k in ("Y", "dX", "dP", "dQ", "dlog_alpha"):
        assert np.array_equal(g1[k], g2[k]), k


def test_optional_outputs_and_inference_forward(b):
    w = I.Workload("t", "bf16", 200, 1, (I.Matrix("w", 128, 192, 96),), ("normal", 0.5, 1.5), 0.5)
    prob = I.layer_problem(w, 0, 0, seed=7)
    m, T = prob["m"], prob["T"]
    X, dY, P, Q = (to_dev(prob[k], "bf16") for k in ("X", "dY", "P", "Q"))
    z = torch.from_numpy(O.gate_sample(prob["log_alpha"], *HC, 0, 0)[0].astype(np.float32)).cuda()
    dzd = torch.ones(m.r, device="cuda")
    Y1, Y2, H = (empty_dev(T, m.d_out, torch.bfloat16), empty_dev(T, m.d_out, torch.bfloat16),
                 empty_dev(T, m.r, torch.bfloat16))
    b.gated_lowrank_fwd(X, Q, P, z, Y1, H, None)
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_FWD, T, m.d_in, m.d_out, m.r, b.BF16))
    b.gated_lowrank_fwd(X, Q, P, z, Y2, None, ws)          # inference: H' lives in the workspace
    assert torch.equal(Y1, Y2)
    with pytest.raises(b.FlopError) as e:
        b.gated_lowrank_fwd(X, Q, P, z, Y2, None, None)
    assert e.value.code == b.ERR_WORKSPACE
    wsb = b.alloc_workspace(b.workspace_bytes(b.OP_BWD, T, m.d_in, m.d_out, m.r, b.BF16))
    dX = empty_dev(T, m.d_in, torch.bfloat16)
    b.gated_lowrank_bwd(dY, X, Q, P, z, dzd, H, dX, None, None, None, wsb)        # only dX
    G = O.gated_lowrank_bwd(prob["dY"], prob["X"], prob["Q"], prob["P"], host(z), np.ones(m.r))
    assert rel_fro(host(dX), G["dX"]) < 2e-2
    dla = torch.full((m.r,), float("nan"), device="cuda")
    b.gated_lowrank_bwd(dY, X, Q, P, z, dzd, H, None, None, None, dla, wsb)       # only dlog_alpha
    assert rel_fro(host(dla), G["dz"]) < 2e-2
    with pytest.raises(b.FlopError) as e:
        b.gated_lowrank_bwd(dY, X, Q, P, z, dzd, H, dX, None, None, None, wsb[:1024])
    assert e.value.code == b.ERR_WORKSPACE
    # rows that are not 16-byte aligned are refused, not mis-read
    Xbad = torch.zeros(T, 129, dtype=torch.bfloat16, device="cuda")[:, :128]
    with pytest.raises(b.FlopError) as e:
        b.gated_lowrank_fwd(Xbad, Q, P, z, Y2, H, None)
    assert e.value.code == b.ERR_UNSUPPORTED
    assert b.device_status() == b.OK


def test_degenerate_sizes(b):
    z = torch.ones(8, device="cuda")
    for tdt in (torch.float32, torch.bfloat16):
        X = torch.zeros(0, 16, dtype=tdt, device="cuda"); Q = torch.ones(8, 16, dtype=tdt, device="cuda")
        P = torch.ones(24, 8, dtype=tdt, device="cuda"); Y = torch.zeros(0, 24, dtype=tdt, device="cuda")
        b.gated_lowrank_fwd(X, Q, P, z, Y, None, None)                     # T = 0: nothing runs
        dP = torch.full((24, 8), float("nan"), dtype=tdt, device="cuda")
        dQ = torch.full((8, 16), float("nan"), dtype=tdt, device="cuda")
        dla = torch.full((8,), float("nan"), device="cuda")
        dY = torch.zeros(0, 24, dtype=tdt, device="cuda"); H = torch.zeros(0, 8, dtype=tdt, device="cuda")
        b.gated_lowrank_bwd(dY, X, Q, P, z, z, H, None, dP, dQ, dla, None)  # empty batch: zero gradients
        assert torch.count_nonzero(dP) == 0 and torch.count_nonzero(dQ) == 0 and torch.count_nonzero(dla) == 0
    assert b.device_status() == b.OK


def test_bounded_wait_gives_up_and_reports_timeout(b):
    """A device-side wait that nothing will ever satisfy: the kernel must return on its own, the status
    word must say FLOP_ERR_TIMEOUT once, and the library must keep working afterwards."""
    assert b.device_status() == b.OK
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.selftest_wait_timeout(2_000_000, flag)            # about a millisecond
    assert b.device_status() == b.ERR_TIMEOUT
    assert int(flag.item()) == 1
    assert b.device_status() == b.OK                    # reading the status clears it
    w = I.Workload("t", "bf16", 256, 1, (I.Matrix("w", 128, 128, 64),), ("normal", 0.5, 1.5), 0.5)
    run_layer(b, I.layer_problem(w, 0, 0, seed=9), "bf16")
