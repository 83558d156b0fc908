"""GPU parity of the grouped forward/backward calls: several independent matrices per launch
must give what the single calls (and the oracle) give."""
import numpy as np
import pytest
import torch

from oracle import flop_oracle as O
from paper_1910_04732_b200 import inputs as I
from tests._util import HC, assert_close, empty_dev, host, rel_fro, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_1910_04732_b200 import build, binding
    build.build()
    binding.load_library()
    return binding


def _setup(b, w: I.Workload, layer, seed, wdt=torch.bfloat16):
    bf = torch.bfloat16
    out = []
    for i, m in enumerate(w.matrices):
        prob = I.layer_problem(w, layer, i, seed=seed)
        e = dict(prob=prob, m=m)
        for k in ("X", "dY", "P", "Q"):
            e[k] = to_dev(prob[k], "bf16")
        z, mask, dzd = O.gate_sample(prob["log_alpha"], *HC, seed=seed, offset=I.gate_offset(layer, i))
        e["z_np"], e["dzd_np"] = z.astype(np.float32), dzd.astype(np.float32)
        e["z"], e["dzd"] = torch.from_numpy(e["z_np"]).cuda(), torch.from_numpy(e["dzd_np"]).cuda()
        T = prob["T"]
        for tag in ("g", "s"):     # grouped and single outputs
            e["Y" + tag], e["H" + tag], e["dX" + tag] = (empty_dev(T, c, bf) for c in (m.d_out, m.r, m.d_in))
            e["dP" + tag], e["dQ" + tag] = empty_dev(m.d_out, m.r, wdt), empty_dev(m.r, m.d_in, wdt)
            e["dla" + tag] = torch.full((m.r,), float("nan"), device="cuda")
            e["ws" + tag] = b.alloc_workspace(b.workspace_bytes(b.OP_BWD, T, m.d_in, m.d_out, m.r, b.BF16))
            e["ws" + tag].fill_(0xFF)
        out.append(e)
    return out


def _check_against_oracle(e, tag):
    p = e["prob"]
    _, Hp, Y = O.gated_lowrank_fwd(p["X"], p["Q"], p["P"], e["z_np"])
    G = O.gated_lowrank_bwd(p["dY"], p["X"], p["Q"], p["P"], e["z_np"], e["dzd_np"])
    for name, got, want in (("H", e["H" + tag], Hp), ("Y", e["Y" + tag], Y), ("dX", e["dX" + tag], G["dX"]),
                            ("dP", e["dP" + tag], G["dP"]), ("dQ", e["dQ" + tag], G["dQ"]),
                            ("dla", e["dla" + tag], G["dlog_alpha"])):
        assert_close(got, want, "bf16", f"{e['m'].name}.{name}")


@pytest.mark.parametrize("wgrad", [torch.bfloat16, torch.float32])
def test_grouped_layer_matches_single_calls_and_oracle(b, wgrad):
    """The six matrices of a Transformer-XL-shaped layer (ragged 410 / 2100 widths), T = 700."""
    w = I.Workload("g", "bf16", 700, 1, I.WORKLOADS["txl"].matrices, ("normal", 0.5, 1.0), 0.35)
    es = _setup(b, w, 0, 3, wgrad)
    b.gated_lowrank_fwd_grouped([b.fwd_problem(e["X"], e["Q"], e["P"], e["z"], e["Yg"], e["Hg"]) for e in es])
    b.gated_lowrank_bwd_grouped([b.bwd_problem(e["dY"], e["X"], e["Q"], e["P"], e["z"], e["dzd"], e["Hg"], e["dXg"],
                                               e["dPg"], e["dQg"], e["dlag"], e["wsg"]) for e in es],
                                wgrad_dt=b.BF16 if wgrad == torch.bfloat16 else b.F32)
    assert b.device_status() == b.OK
    for e in es:
        b.gated_lowrank_fwd(e["X"], e["Q"], e["P"], e["z"], e["Ys"], e["Hs"], None)
        b.gated_lowrank_bwd(e["dY"], e["X"], e["Q"], e["P"], e["z"], e["dzd"], e["Hs"], e["dXs"], e["dPs"], e["dQs"],
                            e["dlas"], e["wss"])
        _check_against_oracle(e, "g")
        assert torch.equal(e["Hg"], e["Hs"]) and torch.equal(e["Yg"], e["Ys"])      # same K order: identical bits
        for k in ("dX", "dP", "dQ", "dla"):
            assert rel_fro(host(e[k + "g"]), host(e[k + "s"])) < 4e-3, k
    assert b.device_status() == b.OK


def test_more_problems_than_one_launch_holds_and_optional_outputs(b):
    """11 problems (two launches per stage), mixed sizes; some outputs skipped; accumulate."""
    mats = tuple(I.Matrix(f"m{i}", d_in, d_out, r) for i, (d_in, d_out, r) in enumerate(
        [(64, 64, 64), (128, 256, 72), (200, 136, 72), (256, 128, 128), (72, 520, 200), (384, 64, 192),
         (64, 384, 64), (136, 136, 136), (512, 256, 256), (96, 96, 40), (264, 520, 200)]))
    w = I.Workload("g", "bf16", 333, 1, mats, ("bimodal", 3.0, 0.5), 0.5)
    es = _setup(b, w, 0, 5)
    b.gated_lowrank_fwd_grouped([b.fwd_problem(e["X"], e["Q"], e["P"], e["z"], e["Yg"], e["Hg"]) for e in es])
    for e in es:
        for k in ("dPg", "dQg"):
            e[k].fill_(0.25)
        e["dlag"].fill_(0.25)
    probs = []
    for i, e in enumerate(es):
        dX = None if i % 3 == 0 else e["dXg"]
        dP = None if i % 4 == 1 else e["dPg"]
        probs.append(b.bwd_problem(e["dY"], e["X"], e["Q"], e["P"], e["z"], e["dzd"], e["Hg"], dX, dP, e["dQg"],
                                   e["dlag"], e["wsg"]))
    b.gated_lowrank_bwd_grouped(probs, accumulate=True)
    assert b.device_status() == b.OK
    for i, e in enumerate(es):
        p = e["prob"]
        G = O.gated_lowrank_bwd(p["dY"], p["X"], p["Q"], p["P"], e["z_np"], e["dzd_np"])
        # accumulating outputs hold bf16(0.25 + g): they are compared as stored, against 0.25 + the oracle's g
        if i % 3 != 0:
            assert_close(e["dXg"], G["dX"], "bf16", "dX")
        else:
            assert torch.isnan(e["dXg"]).all()                      # untouched
        if i % 4 != 1:
            assert_close(e["dPg"], G["dP"] + 0.25, "bf16", "dP")
        else:
            assert torch.all(e["dPg"] == 0.25)
        assert_close(e["dQg"], G["dQ"] + 0.25, "bf16", "dQ")
        assert_close(e["dlag"], G["dlog_alpha"] + 0.25, "bf16", "dla")


def test_grouped_falls_back_per_problem_for_fp32_and_empty_problems(b):
    w = I.Workload("g", "f32", 50, 1, (I.Matrix("a", 24, 40, 16), I.Matrix("b", 16, 8, 8)), ("normal", 0.5, 1.0), 0.5)
    fps, es = [], []
    for i, m in enumerate(w.matrices):
        prob = I.layer_problem(w, 0, i, seed=1)
        X, P, Q = (to_dev(prob[k], "f32") for k in ("X", "P", "Q"))
        z = torch.ones(m.r, device="cuda")
        Y, H = empty_dev(50, m.d_out, torch.float32), empty_dev(50, m.r, torch.float32)
        fps.append(b.fwd_problem(X, Q, P, z, Y, H)); es.append((prob, Y, X, P, Q, z, H))
    b.gated_lowrank_fwd_grouped(fps, dt=b.F32)
    for prob, Y, *_ in es:
        assert rel_fro(host(Y), O.gated_lowrank_fwd(prob["X"], prob["Q"], prob["P"], np.ones(prob["m"].r))[2]) < 1e-5
    assert b.device_status() == b.OK


@pytest.mark.parametrize("name", ["bert", "txl"])
def test_grouped_full_size_layer_as_the_benchmark_issues_it(b, name):
    """All matrices of one layer of the benchmark workload at the full token count, in ONE grouped
    forward and ONE grouped backward call (the launch configuration bench.py times), every output
    against the oracle."""
    w = I.WORKLOADS[name]
    es = _setup(b, w, 2, 0)
    b.gated_lowrank_fwd_grouped([b.fwd_problem(e["X"], e["Q"], e["P"], e["z"], e["Yg"], e["Hg"]) for e in es])
    b.gated_lowrank_bwd_grouped([b.bwd_problem(e["dY"], e["X"], e["Q"], e["P"], e["z"], e["dzd"], e["Hg"], e["dXg"],
                                               e["dPg"], e["dQg"], e["dlag"], e["wsg"]) for e in es])
    assert b.device_status() == b.OK
    for e in es:
        _check_against_oracle(e, "g")
        dead = e["z_np"] == 0
        assert dead.any() and np.all(host(e["dQg"])[dead] == 0)          # closed gates: exact zeros in dQ


def test_two_launch_backward_with_optional_outputs(b):
    """Eight 768-wide matrices at T = 512: the weight gradients fill the machine, so the backward call runs as the
    two shared launches (dH' with dP, then dX with dQ) plus the two small ones; some problems leave out dX, dP or
    dlog_alpha, one launch list or the other may then hold fewer problems."""
    mats = tuple(I.Matrix(f"m{i}", 768, 768, 768) for i in range(8))
    w = I.Workload("g", "bf16", 512, 1, mats, ("bimodal", 3.0, 0.5), 0.5)
    es = _setup(b, w, 0, 11)
    b.gated_lowrank_fwd_grouped([b.fwd_problem(e["X"], e["Q"], e["P"], e["z"], e["Yg"], e["Hg"]) for e in es])
    probs = []
    for i, e in enumerate(es):
        dX = None if i in (1, 5) else e["dXg"]
        dP = None if i in (2, 5) else e["dPg"]
        dla = None if i == 3 else e["dlag"]
        probs.append(b.bwd_problem(e["dY"], e["X"], e["Q"], e["P"], e["z"], e["dzd"], e["Hg"], dX, dP, e["dQg"], dla, e["wsg"]))
    n0 = b.launch_count()
    b.gated_lowrank_bwd_grouped(probs)
    assert b.launch_count() - n0 == 4          # diag(z) Q, two GEMM launches, dlog_alpha
    assert b.device_status() == b.OK
    for i, e in enumerate(es):
        p = e["prob"]
        G = O.gated_lowrank_bwd(p["dY"], p["X"], p["Q"], p["P"], e["z_np"], e["dzd_np"])
        if i in (1, 5):
            assert torch.isnan(e["dXg"]).all()
        else:
            assert_close(e["dXg"], G["dX"], "bf16", "dX")
        if i in (2, 5):
            assert torch.isnan(e["dPg"]).all()
        else:
            assert_close(e["dPg"], G["dP"], "bf16", "dP")
        assert_close(e["dQg"], G["dQ"], "bf16", "dQ")
        if i == 3:
            assert torch.isnan(e["dlag"]).all()
        else:
            assert_close(e["dlag"], G["dlog_alpha"], "bf16", "dla")
