"""GPU parity: gate sampler and expected-L0 / Lagrangian kernels against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import flop_oracle as O
from paper_1910_04732_b200 import inputs as I
from tests._util import HC

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_1910_04732_b200 import build, binding
    build.build()
    binding.load_library()
    return binding


def _run_sampler(b, alpha_np, seed, offset, misalign=0):
    n = len(alpha_np)
    buf = torch.zeros(n + 8, dtype=torch.float32, device="cuda")
    a = buf[misalign:misalign + n]
    a.copy_(torch.from_numpy(alpha_np))
    z = torch.full((n + 8,), float("nan"), device="cuda")[misalign:misalign + n]
    m = torch.full((n + 8,), 7, dtype=torch.uint8, device="cuda")[misalign:misalign + n]
    d = torch.full((n + 8,), float("nan"), device="cuda")[misalign:misalign + n]
    b.gate_sample(a, HC, seed, offset, z, m, d)
    torch.cuda.synchronize()
    return z.cpu().numpy(), m.cpu().numpy(), d.cpu().numpy()


@pytest.mark.parametrize("n,seed,offset,misalign", [
    (1, 0, 0, 0), (3, 0, 5, 0), (4, 1, 0, 0), (5, 2, 7, 1), (255, 3, 1 << 20, 0), (1027, 0, (1 << 32) - 3, 0),
    (55296, 0, 0, 0), (1 << 22, 0xDEADBEEF12345678, 1 << 40, 0), ((1 << 20) + 3, 9, 11, 3)])
def test_gate_sample_matches_oracle(b, n, seed, offset, misalign):
    alpha = I.log_alpha(("normal", 1.0, 1.5), n, seed % 1000, 77)
    z, m, d = _run_sampler(b, alpha, seed, offset, misalign)
    zo, mo, do = O.gate_sample(alpha, *HC, seed=seed, offset=offset)
    assert np.array_equal(m, mo), f"mask mismatch at {np.nonzero(m != mo)[0][:10]}"
    assert np.array_equal(z > 0, mo.astype(bool))
    assert np.all(z[zo == 1.0] == 1.0) and np.all(z[zo < 1.0 - 1e-6] < 1.0)
    assert np.max(np.abs(z - zo)) < 2e-6
    assert np.max(np.abs(d - do)) < 2e-6
    assert np.array_equal(d == 0, do == 0)              # the same gates sit on a clamp


def test_gate_sample_distributions_of_all_workloads(b):
    for name, w in I.WORKLOADS.items():
        n = w.n_gates()
        alpha = I.log_alpha(w.alpha, n, 0, 1)
        z, m, d = _run_sampler(b, alpha, 0, 0)
        zo, mo, do = O.gate_sample(alpha, *HC, seed=0, offset=0)
        assert np.array_equal(m, mo), name
        assert np.max(np.abs(z - zo)) < 2e-6 and np.max(np.abs(d - do)) < 2e-6


def test_gate_sample_near_clamp_decisions_use_fp64(b):
    """Gates placed within 1e-6 of either clamp threshold in logit space: the fp32 value of
    t cannot decide them, the fp64 re-evaluation must."""
    n = 1 << 16
    u = O.gate_uniforms(n, 4, 0)
    logit = np.log(u) - np.log1p(-u)
    c0 = HC[0] * np.log(-HC[1] / HC[2])
    c1 = HC[0] * np.log((1 - HC[1]) / (HC[2] - 1))
    g = np.random.default_rng(0)
    target = np.where(g.random(n) < 0.5, c0, c1) + g.normal(0, 1e-6, n)
    alpha = (target - logit).astype(np.float32)
    z, m, d = _run_sampler(b, alpha, 4, 0)
    zo, mo, do = O.gate_sample(alpha, *HC, seed=4, offset=0)
    assert 0.2 < mo.mean() < 0.99 and 0.1 < (zo == 1).mean() < 0.9       # decisions really are mixed
    assert np.array_equal(m, mo)
    assert np.array_equal(d == 0, do == 0)              # both clamp decisions, bit for bit
    assert np.all(z[zo == 1.0] == 1.0)
    assert np.max(np.abs(z - zo)) < 2e-6 and np.max(np.abs(d - do)) < 2e-6


def test_gate_sample_is_reproducible_and_nullable_outputs(b):
    alpha = torch.from_numpy(I.log_alpha(("normal", 0.5, 1.0), 5000, 0, 2)).cuda()
    z1 = torch.empty(5000, device="cuda"); z2 = torch.empty(5000, device="cuda")
    b.gate_sample(alpha, HC, 1, 2, z1)
    b.gate_sample(alpha, HC, 1, 2, z2, None, None)
    assert torch.equal(z1, z2)
    b.gate_sample(alpha[:0], HC, 1, 2, z1[:0])           # n = 0
    assert b.device_status() == b.OK


def _l0_case(b, w: I.Workload, lam, target, with_grad=True, accumulate_into=None):
    offs, sizes, alphas = [0], [], []
    for l, i, m in w.all_matrices():
        alphas.append(I.log_alpha(w.alpha, m.r, 0, l, i))
        offs.append(offs[-1] + m.r)
        sizes.append(float(m.d_in + m.d_out))
    alpha = np.concatenate(alphas)
    n, n_seg = len(alpha), len(sizes)
    dev = lambda a, dt: torch.from_numpy(np.asarray(a, dtype=dt)).cuda()
    la, so, ss = dev(alpha, np.float32), dev(offs, np.int64), dev(sizes, np.float32)
    tg, lm = dev([target], np.float32), dev(lam, np.float32)
    out4 = torch.full((4,), float("nan"), device="cuda")
    seg = torch.full((n_seg,), float("nan"), device="cuda")
    base = np.zeros(n, np.float32) if accumulate_into is None else accumulate_into
    dla = dev(base, np.float32) if with_grad else None
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_L0, n, 0, 0, n_seg, b.F32))
    b.expected_l0_lagrangian(la, so, ss, HC, tg, lm, out4, seg, dla, ws)
    torch.cuda.synchronize()
    ref = O.expected_l0_lagrangian(alpha, offs, sizes, *HC, float(np.float32(target)),
                                   float(np.float32(lam[0])), float(np.float32(lam[1])))
    return out4.cpu().numpy(), seg.cpu().numpy(), None if dla is None else dla.cpu().numpy(), ref, base


@pytest.mark.parametrize("name", ["single_f32", "sru", "txl", "bert"])
@pytest.mark.parametrize("lam", [(0.0, 0.0), (0.3, 1.7)])
def test_expected_l0_lagrangian_matches_oracle(b, name, lam):
    w = I.WORKLOADS[name]
    out4, seg, dla, ref, _ = _l0_case(b, w, lam, w.target)
    want = np.array([ref["s"], ref["g"], ref["dg_dlambda1"], ref["dg_dlambda2"]])
    assert np.allclose(out4, want, rtol=2e-6, atol=1e-7)
    assert np.allclose(seg, ref["seg_expected"], rtol=2e-6)
    assert np.allclose(dla, ref["dlog_alpha"], rtol=2e-5, atol=1e-12)
    if lam == (0.0, 0.0):
        assert out4[1] == 0 and np.all(dla == 0)


def test_expected_l0_accumulates_and_is_bit_reproducible(b):
    w = I.WORKLOADS["txl"]
    base = np.random.default_rng(0).standard_normal(w.n_gates()).astype(np.float32)
    o1, s1, d1, ref, _ = _l0_case(b, w, (0.3, 1.7), 0.35, accumulate_into=base)
    o2, s2, d2, _, _ = _l0_case(b, w, (0.3, 1.7), 0.35, accumulate_into=base)
    assert np.array_equal(o1, o2) and np.array_equal(s1, s2) and np.array_equal(d1, d2)
    assert np.allclose(d1 - base, ref["dlog_alpha"], rtol=1e-3, atol=5e-7)     # fp32 += onto values of order 1
    o3, s3, d3, _, _ = _l0_case(b, w, (0.3, 1.7), 0.35, with_grad=False)
    assert np.array_equal(o1, o3) and d3 is None


def test_expected_l0_ragged_segments_and_large_single_segment(b):
    # segments with 0, 1, chunk-1, chunk, chunk+1 gates, and one segment spanning many chunks
    counts = [0, 1, 1023, 4095, 4096, 4097, 0, 300000, 7]
    sizes = [10.0, 820.0, 2510.0, 1.0, 4096.0, 77.0, 5.0, 1536.0, 64.0]
    w_alpha = np.random.default_rng(1).normal(0.5, 2.0, sum(counts)).astype(np.float32)
    offs = np.concatenate([[0], np.cumsum(counts)])
    dev = lambda a, dt: torch.from_numpy(np.asarray(a, dtype=dt)).cuda()
    la, so, ss = dev(w_alpha, np.float32), dev(offs, np.int64), dev(sizes, np.float32)
    tg, lm = dev([0.4], np.float32), dev([-0.7, 2.5], np.float32)
    out4 = torch.empty(4, device="cuda"); seg = torch.empty(len(sizes), device="cuda")
    dla = torch.zeros(len(w_alpha), device="cuda")
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_L0, len(w_alpha), 0, 0, len(sizes), b.F32))
    b.expected_l0_lagrangian(la, so, ss, HC, tg, lm, out4, seg, dla, ws)
    ref = O.expected_l0_lagrangian(w_alpha, offs, sizes, *HC, float(np.float32(0.4)), float(np.float32(-0.7)), 2.5)
    assert np.allclose(out4.cpu().numpy(), [ref["s"], ref["g"], ref["dg_dlambda1"], ref["dg_dlambda2"]], rtol=2e-6, atol=1e-7)
    assert np.allclose(seg.cpu().numpy(), ref["seg_expected"], rtol=2e-6)
    assert np.allclose(dla.cpu().numpy(), ref["dlog_alpha"], rtol=2e-5, atol=1e-13)
    # no segments at all: s = 0, g = lambda1 (0 - t) + lambda2 t^2
    b.expected_l0_lagrangian(la[:0], so[:1], ss[:0], HC, tg, lm, out4, None, None, ws)
    t = float(np.float32(0.4))
    assert np.allclose(out4.cpu().numpy(), [0.0, -0.7 * (-t) + 2.5 * t * t, -t, t * t], rtol=1e-6)
    assert b.device_status() == b.OK


def test_gate_sample_with_device_side_offset(b):
    """The counter offset read from device memory: base + *offset_dev, advanced between calls."""
    n = 10007
    alpha = I.log_alpha(("normal", 0.5, 1.5), n, 0, 21)
    a = torch.from_numpy(alpha).cuda()
    off = torch.tensor([(1 << 33) + 5], dtype=torch.int64, device="cuda")
    z = torch.empty(n, device="cuda"); m = torch.empty(n, dtype=torch.uint8, device="cuda"); d = torch.empty(n, device="cuda")
    for step in range(3):
        b.gate_sample_devoff(a, HC, 7, 1000, off, z, m, d)
        zo, mo, do = O.gate_sample(alpha, *HC, seed=7, offset=1000 + (1 << 33) + 5 + step * (1 << 24))
        assert np.array_equal(m.cpu().numpy(), mo)
        assert np.max(np.abs(z.cpu().numpy() - zo)) < 2e-6 and np.max(np.abs(d.cpu().numpy() - do)) < 2e-6
        off.add_(1 << 24)
    with pytest.raises(b.FlopError):
        b.load_library()  # keep the import used
        b._check(b.load_library().flop_gate_sample_devoff(None, 4, b.HcParams(*HC), 0, 0, None, None, None, None, None),
                 "flop_gate_sample_devoff")
