"""GPU parity of training on the active rank components: gather the components with z_k > 0, run the
grouped forward/backward with the rank read from device memory, scatter the gradients back.  Results
must equal the oracle's full (uncompacted) layer, with exact zeros for the closed components."""
import numpy as np
import pytest
import torch

from oracle import flop_oracle as O
from paper_1910_04732_b200 import inputs as I
from tests._util import HC, empty_dev, host, rel_fro, to_dev, assert_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_1910_04732_b200 import build, binding
    build.build()
    binding.load_library()
    return binding


def _run(b, w: I.Workload, seed, alpha_shift=0.0, wdt=torch.bfloat16, accumulate=False, chained=False, per_step=False):
    bf = torch.bfloat16
    es, gat, fwd, bwd, sca = [], [], [], [], []
    for i, m in enumerate(w.matrices):
        prob = I.layer_problem(w, 0, i, seed=seed)
        la = prob["log_alpha"] + np.float32(alpha_shift)
        z, mask, dzd = O.gate_sample(la, *HC, seed=seed, offset=I.gate_offset(0, i))
        e = dict(prob=prob, m=m, z_np=z.astype(np.float32), dzd_np=dzd.astype(np.float32), mask=mask)
        T = prob["T"]
        for k in ("X", "dY", "P", "Q"):
            e[k] = to_dev(prob[k], "bf16")
        e["z"], e["dzd"] = torch.from_numpy(e["z_np"]).cuda(), torch.from_numpy(e["dzd_np"]).cuda()
        e["idx"] = torch.full((m.r,), -7, dtype=torch.int32, device="cuda")
        e["pos"] = torch.full((m.r,), -7, dtype=torch.int32, device="cuda")
        e["k"] = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        e["zc"], e["dzc"] = torch.full((m.r,), float("nan"), device="cuda"), torch.full((m.r,), float("nan"), device="cuda")
        e["Pc"], e["Qc"] = empty_dev(m.d_out, m.r, bf), empty_dev(m.r, m.d_in, bf)       # NaN-poisoned capacity buffers
        e["Hc"], e["Y"], e["dX"] = empty_dev(T, m.r, bf), empty_dev(T, m.d_out, bf), empty_dev(T, m.d_in, bf)
        e["dPc"], e["dQc"] = empty_dev(m.d_out, m.r, wdt), empty_dev(m.r, m.d_in, wdt)
        e["dlac"] = torch.full((m.r,), float("nan"), device="cuda")
        init = 0.5 if accumulate else float("nan")
        e["dP"], e["dQ"] = empty_dev(m.d_out, m.r, wdt, init), empty_dev(m.r, m.d_in, wdt, init)
        e["dla"] = torch.full((m.r,), init, device="cuda")
        e["ws"] = b.alloc_workspace(b.workspace_bytes(b.OP_BWD, T, m.d_in, m.d_out, m.r, b.BF16))
        e["ws"].fill_(0xFF)
        e["Qzc"] = empty_dev(m.r, m.d_in, bf) if per_step else None
        gat.append(b.active_gather_problem(e["z"], e["dzd"], e["P"], e["Q"], e["idx"], e["pos"], e["k"], e["zc"], e["dzc"],
                                           e["Pc"], e["Qc"], Qz_c=e["Qzc"] if per_step == "gather" else None))
        fwd.append(b.fwd_problem(e["X"], e["Qc"], e["Pc"], e["zc"], e["Y"], e["Hc"], r_dev=e["k"]))
        bwd.append(b.bwd_problem(e["dY"], e["X"], e["Qc"], e["Pc"], e["zc"], e["dzc"], e["Hc"], e["dX"], e["dPc"], e["dQc"],
                                 e["dlac"], e["ws"], r_dev=e["k"], Qz=e["Qzc"], defer_dlog_alpha=bool(per_step)))
        sca.append(b.active_scatter_problem(e["idx"], e["pos"], e["k"], m.d_in, m.d_out, m.r, e["dPc"], e["dQc"], e["dlac"],
                                            e["dP"], e["dQ"], e["dla"]))
        es.append(e)
    wd = b.BF16 if wdt == torch.bfloat16 else b.F32
    b.active_ranks_gather(gat)
    if chained:
        sync = b.alloc_sync()
        b.gated_lowrank_fwd_chained(fwd, sync)
        b.gated_lowrank_bwd_chained(bwd, sync, wgrad_dt=wd)
        assert int(sync.view(torch.int32).abs().sum().item()) == 0
    elif per_step:
        # the per-step form: diag(z_c) Q_c formed once for all matrices, dlog_alpha_c finished once after all backward calls
        if per_step == "gather":     # diag(z_c) Q_c came out of the gather launch
            for e in es:
                k = int(e["k"].item())
                sel = np.nonzero(e["mask"])[0]
                want = I.round_to_bf16(e["prob"]["Q"][sel].astype(np.float32) * e["z_np"][sel, None])
                assert np.array_equal(host(e["Qzc"])[:k], want.astype(np.float64))
        else:
            b.scale_rows_grouped([b.scale_rows_problem(e["Qc"], e["zc"], e["Qzc"]) for e in es])
        b.gated_lowrank_fwd_grouped(fwd)
        b.gated_lowrank_bwd_grouped(bwd, wgrad_dt=wd)
        b.dlog_alpha_finish_grouped(bwd)
    else:
        b.gated_lowrank_fwd_grouped(fwd)
        b.gated_lowrank_bwd_grouped(bwd, wgrad_dt=wd)
    b.active_ranks_scatter(sca, accumulate=accumulate, wgrad_dt=wd)
    assert b.device_status() == b.OK
    for e in es:
        m, p = e["m"], e["prob"]
        k = int(e["k"].item())
        want_idx = np.nonzero(e["mask"])[0]
        assert k == len(want_idx) and np.array_equal(e["idx"].cpu().numpy()[:k], want_idx)      # bit-exact index list
        pos = e["pos"].cpu().numpy()
        assert np.array_equal(np.nonzero(pos >= 0)[0], want_idx) and np.array_equal(pos[want_idx], np.arange(k))
        assert np.array_equal(host(e["Qc"])[:k], p["Q"][want_idx].astype(np.float64))             # pure gathers: exact
        assert np.array_equal(host(e["Pc"])[:, :k], p["P"][:, want_idx].astype(np.float64))
        _, _, Y = O.gated_lowrank_fwd(p["X"], p["Q"], p["P"], e["z_np"])
        G = O.gated_lowrank_bwd(p["dY"], p["X"], p["Q"], p["P"], e["z_np"], e["dzd_np"])
        off = 0.5 if accumulate else 0.0
        for name, got, want in (("Y", e["Y"], Y), ("dX", e["dX"], G["dX"]), ("dP", e["dP"], G["dP"] + off),
                                ("dQ", e["dQ"], G["dQ"] + off), ("dla", e["dla"], G["dlog_alpha"] + off)):
            assert_close(got, want, "bf16", f"{m.name}.{name}")     # a zero `want` demands exact zeros
        if not accumulate:
            dead = ~e["mask"].astype(bool)
            assert np.all(host(e["dQ"])[dead] == 0) and np.all(host(e["dP"])[:, dead] == 0) and np.all(host(e["dla"])[dead] == 0)
    return es


def test_active_ranks_layer_matches_full_oracle(b):
    """Six ragged Transformer-XL-shaped matrices, about 60 % of the gates open."""
    w = I.Workload("a", "bf16", 700, 1, I.WORKLOADS["txl"].matrices, ("normal", 0.5, 1.0), 0.35)
    es = _run(b, w, 3)
    assert all(0 < int(e["k"].item()) < e["m"].r for e in es)


def test_active_ranks_bimodal_full_size_bert_layer(b):
    w = I.WORKLOADS["bert"]
    es = _run(b, I.Workload("a", "bf16", w.T, 1, w.matrices, w.alpha, w.target), 0)
    ks = [int(e["k"].item()) for e in es]
    assert all(300 < k < 470 for k in ks), ks


@pytest.mark.parametrize("shift,expect", [(-30.0, "none"), (30.0, "all")])
def test_active_ranks_edges_no_or_all_components(b, shift, expect):
    w = I.Workload("a", "bf16", 300, 1, (I.Matrix("x", 200, 136, 72), I.Matrix("y", 128, 256, 128)), ("normal", 0.0, 1.0), 0.5)
    es = _run(b, w, 1, alpha_shift=shift)
    for e in es:
        assert int(e["k"].item()) == (0 if expect == "none" else e["m"].r)


def test_active_ranks_fp32_weight_gradients_and_accumulate(b):
    w = I.Workload("a", "bf16", 500, 1, (I.Matrix("x", 264, 520, 200), I.Matrix("y", 384, 64, 192)), ("bimodal", 3.0, 0.5), 0.5)
    _run(b, w, 2, wdt=torch.float32)
    _run(b, w, 2, accumulate=True)


def test_active_ranks_through_the_chained_calls(b):
    """The device-side rank with the queue-drawn launches (dlog_alpha finished inside the second backward launch)."""
    w = I.WORKLOADS["bert"]
    es = _run(b, I.Workload("a", "bf16", 1024, 1, w.matrices, w.alpha, w.target), 4, chained=True)
    assert all(0 < int(e["k"].item()) < e["m"].r for e in es)


@pytest.mark.parametrize("wdt", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("qz_from", ["gather", "scale_rows"])
def test_active_ranks_per_step_side_work(b, wdt, qz_from):
    """diag(z_c) Q_c from the gather launch (or one grouped scaling launch) and dlog_alpha_c from one deferred finish,
    with the rank read on the device."""
    w = I.WORKLOADS["bert"]
    es = _run(b, I.Workload("a", "bf16", 1024, 1, w.matrices, w.alpha, w.target), 5, wdt=wdt, per_step=qz_from)
    assert all(0 < int(e["k"].item()) < e["m"].r for e in es)
    w2 = I.Workload("a", "bf16", 700, 1, I.WORKLOADS["txl"].matrices, ("normal", 0.5, 1.0), 0.35)
    _run(b, w2, 6, wdt=wdt, per_step=qz_from)
