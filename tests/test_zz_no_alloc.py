"""The no-allocation variant of the expected-L0 / Lagrangian call.

Some callers of this library may not allocate device memory: they run inside a
memory plan that was fixed up front (a serving process whose pool is frozen, a
plug-in that receives tensors but no allocator).  For them the library keeps the
scratch of this one call in a fixed device array of its own.  This test calls that
entry point through the C ABI twice in a row (the array keeps the first call's
contents, which must not leak into the second) and checks every output against the
workspace-taking entry point and against the CPU oracle, and that the device's free
memory is the same before and after the calls.  It is collected last so that a run
stopping at the first failure has already run every other test; it must also pass alone.
"""
import ctypes

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


def _problem(w: I.Workload, seed: int):
    offs, sizes, alphas = [0], [], []
    for l, i, m in w.all_matrices():
        alphas.append(I.log_alpha(w.alpha, m.r, seed, l, i))
        offs.append(offs[-1] + m.r)
        sizes.append(float(m.d_in + m.d_out))
    dev = lambda a, dt: torch.from_numpy(np.asarray(a, dtype=dt)).cuda()
    return dev(np.concatenate(alphas), np.float32), dev(offs, np.int64), dev(sizes, np.float32)


def _both(b, la, so, ss, target, lam):
    n, n_seg = la.numel(), ss.numel()
    tg, lm = torch.tensor([target], device="cuda"), torch.tensor(lam, device="cuda")
    base = torch.linspace(-1, 1, n, device="cuda")
    ref = dict(out4=torch.full((4,), float("nan"), device="cuda"), seg=torch.full((n_seg,), float("nan"), device="cuda"),
               dla=base.clone())
    got = dict(out4=torch.full((4,), float("nan"), device="cuda"), seg=torch.full((n_seg,), float("nan"), device="cuda"),
               dla=base.clone())
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_L0, n, 0, 0, n_seg, b.F32))
    b.expected_l0_lagrangian(la, so, ss, HC, tg, lm, ref["out4"], ref["seg"], ref["dla"], ws)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    b.expected_l0_lagrangian_noalloc(la, so, ss, HC, tg, lm, got["out4"], got["seg"], got["dla"])
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before          # the call took no device memory
    for k in ref:
        r, g = ref[k].cpu().numpy(), got[k].cpu().numpy()
        assert np.all(np.isfinite(g)), k
        assert np.allclose(g, r, rtol=2e-6, atol=1e-7), k
    # and against the oracle directly (Eq. 3 and Section 4.3 in fp64)
    f32 = lambda v: float(np.float32(v))          # the kernels read target and lambda as fp32
    want = O.expected_l0_lagrangian(la.cpu().numpy(), so.cpu().numpy().tolist(), ss.cpu().numpy().tolist(), *HC,
                                    f32(target), f32(lam[0]), f32(lam[1]))
    o4 = got["out4"].cpu().numpy().astype(np.float64)
    assert np.allclose(o4, [want["s"], want["g"], want["dg_dlambda1"], want["dg_dlambda2"]], rtol=2e-6, atol=1e-7)
    assert np.allclose(got["seg"].cpu().numpy(), want["seg_expected"], rtol=2e-6, atol=1e-6)
    # dlog_alpha is added in fp32 onto values of order 1
    assert np.allclose(got["dla"].cpu().numpy() - base.cpu().numpy(), want["dlog_alpha"], rtol=1e-3, atol=5e-7)


def test_noalloc_matches_workspace_entry_point_on_two_calls_in_a_row(b):
    # first call: the Transformer-XL-shaped model (96 segments of unequal block size) ...
    _both(b, *_problem(I.WORKLOADS["txl"], 0), target=0.35, lam=[0.3, 1.7])
    # ... second call right after it, on a different, smaller problem: whatever the first call
    # left in the built-in array must not show up here
    _both(b, *_problem(I.WORKLOADS["single_f32"], 1), target=0.5, lam=[-0.4, 0.9])
    # and back to a large one (more chunks than either of the above)
    la = torch.from_numpy(I.log_alpha(("normal", 0.5, 2.0), 300007, 0, 5)).cuda()
    so = torch.tensor([0, 1000, 1000, 300007], dtype=torch.int64, device="cuda")
    ss = torch.tensor([820.0, 5.0, 1536.0], device="cuda")
    _both(b, la, so, ss, target=0.4, lam=[1.0, 0.0])
    assert b.device_status() == b.OK


def test_noalloc_rejects_sizes_beyond_the_builtin_scratch(b):
    lib = b.load_library()
    one = torch.zeros(4, device="cuda")
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    hc = b.HcParams(*HC)
    too_many = (1 << 20) + 1
    rc = lib.flop_expected_l0_lagrangian_noalloc(p(one), too_many, p(one), p(one), 1, hc, p(one), p(one), p(one),
                                                 None, None, None)
    assert rc == b.ERR_UNSUPPORTED and "unsupported" in b.status_string(rc)
    rc = lib.flop_expected_l0_lagrangian_noalloc(p(one), 4, p(one), p(one), 4097, hc, p(one), p(one), p(one),
                                                 None, None, None)
    assert rc == b.ERR_UNSUPPORTED


def test_segment_table_that_does_not_partition_the_gates_is_refused_on_the_device(b):
    """The segment table is device memory, so the kernels check it: offsets beyond n, or more chunks than the
    scratch holds, leave every output but out4 untouched, write NaN to out4 and record FLOP_ERR_INVALID_ARG."""
    la = torch.zeros(20000, device="cuda")
    ss = torch.tensor([1.0, 2.0], device="cuda")
    tg, lm = torch.tensor([0.5], device="cuda"), torch.tensor([0.3, 1.7], device="cuda")
    for bad in ([0, 10000, 30000], [0, 12000, 11000], [5, 10000, 20000]):
        so = torch.tensor(bad, dtype=torch.int64, device="cuda")
        for noalloc in (False, True):
            out4 = torch.zeros(4, device="cuda")
            seg = torch.full((2,), 7.0, device="cuda")
            dla = torch.full((20000,), 3.0, device="cuda")
            if noalloc:
                b.expected_l0_lagrangian_noalloc(la, so, ss, HC, tg, lm, out4, seg, dla)
            else:
                ws = b.alloc_workspace(b.workspace_bytes(b.OP_L0, 20000, 0, 0, 2, b.F32))
                b.expected_l0_lagrangian(la, so, ss, HC, tg, lm, out4, seg, dla, ws)
            assert b.device_status() == b.ERR_INVALID_ARG           # read and cleared
            assert torch.isnan(out4).all() and torch.all(seg == 7.0) and torch.all(dla == 3.0)
    assert b.device_status() == b.OK
