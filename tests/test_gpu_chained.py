"""GPU parity of the chained calls: both forward products in one launch and all four backward products
(plus diag(z) Q and the second stage of dlog_alpha) in one launch, ordered on the device by counters.
They must give, bit for bit, what the grouped sequence of launches gives (same tiles, same summation
order), match the oracle, leave the sync area zero-filled, and do so again when called again."""
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


def _setup(b, w: I.Workload, layer, seed, wdt=torch.bfloat16, init=float("nan")):
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
        for tag in ("c", "g"):     # chained and grouped outputs
            e["Y" + tag], e["H" + tag], e["dX" + tag] = (empty_dev(T, c, bf) for c in (m.d_out, m.r, m.d_in))
            e["dP" + tag], e["dQ" + tag] = empty_dev(m.d_out, m.r, wdt, init), empty_dev(m.r, m.d_in, wdt, init)
            e["dla" + tag] = torch.full((m.r,), init, device="cuda")
            e["ws" + tag] = b.alloc_workspace(b.workspace_bytes(b.OP_BWD, T, m.d_in, m.d_out, m.r, b.BF16))
            e["ws" + tag].fill_(0xFF)
        out.append(e)
    return out


def _fwd(b, es, tag):
    return [b.fwd_problem(e["X"], e["Q"], e["P"], e["z"], e["Y" + tag], e["H" + tag]) for e in es]


def _bwd(b, es, tag, skip=lambda i, name: False, qz=False):
    pick = lambda i, e, name: None if skip(i, name) else e[name + tag]
    return [b.bwd_problem(e["dY"], e["X"], e["Q"], e["P"], e["z"], e["dzd"], e["H" + tag], pick(i, e, "dX"), pick(i, e, "dP"),
                          pick(i, e, "dQ"), pick(i, e, "dla"), e["ws" + tag], Qz=e["Qz"] if qz else None)
            for i, e in enumerate(es)]


def _form_qz(b, es):
    """diag(z) Q of every problem in one launch, checked bit for bit against bf16(z * Q) (one rounding)."""
    for e in es:
        e["Qz"] = empty_dev(e["m"].r, e["m"].d_in, torch.bfloat16)
    n0 = b.launch_count()
    b.scale_rows_grouped([b.scale_rows_problem(e["Q"], e["z"], e["Qz"]) for e in es])
    assert b.launch_count() - n0 == 1
    for e in es:
        want = (e["Q"].float() * e["z"][:, None]).to(torch.bfloat16)
        assert torch.equal(e["Qz"].view(torch.int16), want.view(torch.int16))


def _oracle(e):
    p = e["prob"]
    _, Hp, Y = O.gated_lowrank_fwd(p["X"], p["Q"], p["P"], e["z_np"])
    G = O.gated_lowrank_bwd(p["dY"], p["X"], p["Q"], p["P"], e["z_np"], e["dzd_np"])
    return dict(H=Hp, Y=Y, dX=G["dX"], dP=G["dP"], dQ=G["dQ"], dla=G["dlog_alpha"])


def _same_bits(x, y):
    return torch.equal(x.view(torch.int16) if x.dtype == torch.bfloat16 else x.view(torch.int32),
                       y.view(torch.int16) if y.dtype == torch.bfloat16 else y.view(torch.int32))


@pytest.mark.parametrize("name,T", [("bert", 1024), ("txl", 700)])
@pytest.mark.parametrize("wgrad", [torch.bfloat16, torch.float32])
def test_chained_layer_is_one_launch_each_way_and_matches_grouped_and_oracle(b, name, T, wgrad):
    base = I.WORKLOADS[name]
    w = I.Workload("c", "bf16", T, 1, base.matrices, base.alpha, base.target)
    es = _setup(b, w, 0, 7, wgrad)
    wd = b.BF16 if wgrad == torch.bfloat16 else b.F32
    sync = b.alloc_sync()
    for rep in range(2):            # the second call finds the area as the first left it
        n0 = b.launch_count()
        b.gated_lowrank_fwd_chained(_fwd(b, es, "c"), sync)
        assert b.launch_count() - n0 == 2                  # one launch per product, no small kernels
        b.gated_lowrank_bwd_chained(_bwd(b, es, "c"), sync, wgrad_dt=wd)
        assert b.launch_count() - n0 == 5                  # diag(z) Q, then {dH', dP} and {dQ, dX}; dlog_alpha inside
        assert b.device_status() == b.OK
        assert int(sync.view(torch.int32).abs().sum().item()) == 0       # left zero-filled
        if rep == 0:
            b.gated_lowrank_fwd_grouped(_fwd(b, es, "g"))
            b.gated_lowrank_bwd_grouped(_bwd(b, es, "g"), wgrad_dt=wd)
            assert b.device_status() == b.OK
        for e in es:
            want = _oracle(e) if rep == 0 else e["want"]
            e["want"] = want
            for k in ("H", "Y", "dX", "dP", "dQ", "dla"):
                assert_close(e[k + "c"], want[k], "bf16", f"{e['m'].name}.{k}")
                assert _same_bits(e[k + "c"], e[k + "g"]), (e["m"].name, k)
            dead = e["z_np"] == 0
            assert np.all(host(e["dQc"])[dead] == 0)
        if rep == 0:                # poison the chained outputs again before the second call
            for e in es:
                for k in ("H", "Y", "dX", "dP", "dQ"):
                    e[k + "c"].fill_(float("nan"))
                e["dlac"].fill_(float("nan"))
                e["wsc"].fill_(0xFF)


def test_chained_optional_outputs_and_accumulate(b):
    """Six 768-wide matrices at T = 512; some problems leave out dX, dP, dQ or dlog_alpha; accumulate adds."""
    mats = tuple(I.Matrix(f"m{i}", 768, 768, 768) for i in range(6))
    w = I.Workload("c", "bf16", 512, 1, mats, ("bimodal", 3.0, 0.5), 0.5)
    es = _setup(b, w, 0, 11, init=0.25)
    sync = b.alloc_sync()
    skip = lambda i, name: (name == "dX" and i in (1, 5)) or (name == "dP" and i in (2, 5)) or (name == "dla" and i == 3) or \
        (name == "dQ" and i == 4)
    b.gated_lowrank_fwd_chained(_fwd(b, es, "c"), sync)
    n0 = b.launch_count()
    b.gated_lowrank_bwd_chained(_bwd(b, es, "c", skip), sync, accumulate=True)
    assert b.launch_count() - n0 == 3
    assert b.device_status() == b.OK
    assert int(sync.view(torch.int32).abs().sum().item()) == 0
    for i, e in enumerate(es):
        want = _oracle(e)
        assert_close(e["Yc"], want["Y"], "bf16", "Y")
        if skip(i, "dX"):
            assert torch.isnan(e["dXc"]).all()
        else:
            assert_close(e["dXc"], want["dX"], "bf16", "dX")
        for k in ("dP", "dQ", "dla"):
            if skip(i, k):
                assert torch.all(e[k + "c"] == 0.25), k             # untouched
            else:
                assert_close(e[k + "c"], want[k] + 0.25, "bf16", k)  # stored as bf16(0.25 + g)


@pytest.mark.parametrize("name", ["bert", "txl"])
def test_chained_full_size_layer_as_the_benchmark_issues_it(b, name):
    """All matrices of one layer of the benchmark workload at the full token count, as bench.py issues them
    (diag(z) Q formed beforehand, one launch for all matrices)."""
    w = I.WORKLOADS[name]
    es = _setup(b, w, 2, 0)
    sync = b.alloc_sync()
    _form_qz(b, es)
    n0 = b.launch_count()
    b.gated_lowrank_fwd_chained(_fwd(b, es, "c"), sync)
    b.gated_lowrank_bwd_chained(_bwd(b, es, "c", qz=True), sync)
    assert b.launch_count() - n0 == 4
    assert b.device_status() == b.OK
    assert int(sync.view(torch.int32).abs().sum().item()) == 0
    for e in es:
        want = _oracle(e)
        for k in ("H", "Y", "dX", "dP", "dQ", "dla"):
            assert_close(e[k + "c"], want[k], "bf16", f"{e['m'].name}.{k}")


def test_chained_sru_layer_with_more_tiles_than_the_schedule_table(b):
    """One SRU-shaped matrix at T = 4096 and at T = 16 640 (2080 forward tiles, more than the schedule table
    holds: the launch then walks the stage-ordered list round-robin)."""
    base = I.WORKLOADS["sru"]
    for T in (4096, base.T + 256):
        w = I.Workload("c", "bf16", T, 1, base.matrices, base.alpha, base.target)
        es = _setup(b, w, 0, 2)
        sync = b.alloc_sync()
        n0 = b.launch_count()
        b.gated_lowrank_fwd_chained(_fwd(b, es, "c"), sync)
        b.gated_lowrank_bwd_chained(_bwd(b, es, "c"), sync)
        assert b.launch_count() - n0 == 5
        assert b.device_status() == b.OK
        assert int(sync.view(torch.int32).abs().sum().item()) == 0
        for e in es:
            want = _oracle(e)
            for k in ("H", "Y", "dX", "dP", "dQ", "dla"):
                assert_close(e[k + "c"], want[k], "bf16", f"T={T}.{k}")
        del es
        torch.cuda.empty_cache()


def test_chained_falls_back_to_the_grouped_launches(b):
    """Small ragged problems pick one-CTA tiles or split-K: the chained call then runs the grouped sequence."""
    mats = tuple(I.Matrix(f"m{i}", d_in, d_out, r) for i, (d_in, d_out, r) in enumerate(
        [(64, 64, 64), (200, 136, 72), (72, 520, 200)]))
    w = I.Workload("c", "bf16", 333, 1, mats, ("bimodal", 3.0, 0.5), 0.5)
    es = _setup(b, w, 0, 5)
    sync = b.alloc_sync()
    b.gated_lowrank_fwd_chained(_fwd(b, es, "c"), sync)
    b.gated_lowrank_bwd_chained(_bwd(b, es, "c"), sync)
    assert b.device_status() == b.OK
    assert int(sync.view(torch.int32).abs().sum().item()) == 0
    for e in es:
        want = _oracle(e)
        for k in ("H", "Y", "dX", "dP", "dQ", "dla"):
            assert_close(e[k + "c"], want[k], "bf16", f"{e['m'].name}.{k}")


def test_chained_argument_checks(b):
    w = I.Workload("c", "bf16", 256, 1, (I.Matrix("a", 128, 128, 128),), ("normal", 0.5, 1.0), 0.5)
    es = _setup(b, w, 0, 1)
    small = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(b.FlopError) as ei:
        b.gated_lowrank_fwd_chained(_fwd(b, es, "c"), small)
    assert ei.value.code == b.ERR_WORKSPACE
    with pytest.raises(b.FlopError) as ei:
        b.gated_lowrank_bwd_chained(_bwd(b, es, "c"), small)
    assert ei.value.code == b.ERR_WORKSPACE
    assert b.sync_bytes() >= 4096


def test_chained_step_replays_in_a_cuda_graph(b):
    """A captured forward + backward replays correctly: every replay finds the sync area zero-filled."""
    mats = tuple(I.Matrix(f"m{i}", 768, 768, 768) for i in range(6))
    w = I.Workload("c", "bf16", 1024, 1, mats, ("bimodal", 3.0, 0.5), 0.5)
    es = _setup(b, w, 0, 4)
    sync = b.alloc_sync()
    fwd, bwd = b.problem_array(_fwd(b, es, "c")), b.problem_array(_bwd(b, es, "c"))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        b.gated_lowrank_fwd_chained(fwd, sync)
        b.gated_lowrank_bwd_chained(bwd, sync)
        torch.cuda.synchronize()
        with torch.cuda.graph(g, stream=side):
            b.gated_lowrank_fwd_chained(fwd, sync)
            b.gated_lowrank_bwd_chained(bwd, sync)
    torch.cuda.current_stream().wait_stream(side)
    want = [_oracle(e) for e in es]
    for rep in range(3):
        for e in es:
            for k in ("H", "Y", "dX", "dP", "dQ"):
                e[k + "c"].fill_(float("nan"))
            e["dlac"].fill_(float("nan"))
        n0 = b.launch_count()
        g.replay()
        torch.cuda.synchronize()
        assert b.launch_count() == n0 and b.device_status() == b.OK
        assert int(sync.view(torch.int32).abs().sum().item()) == 0
        for e, wnt in zip(es, want):
            for k in ("H", "Y", "dX", "dP", "dQ", "dla"):
                assert_close(e[k + "c"], wnt[k], "bf16", f"replay {rep} {e['m'].name}.{k}")
