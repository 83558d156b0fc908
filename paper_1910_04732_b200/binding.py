"""Thin ctypes binding over the C ABI in include/flop.h.

Argument marshalling only: torch tensors provide device memory and the
current CUDA stream; every step of the path runs in the library's kernels.
If the library is missing or a call fails this module raises -- there is no
CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libflop_b200.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)
F32, BF16 = 0, 1
OP_FWD, OP_BWD, OP_L0, OP_COMPACT, OP_COMPACT_FWD, OP_EMBEDDING_BWD = range(6)

EXPORTS = ("flop_status_string", "flop_last_async_status", "flop_device_status", "flop_sync_bytes",
           "flop_gated_lowrank_fwd_chained", "flop_gated_lowrank_bwd_chained", "flop_selftest_wait_timeout", "flop_launch_count", "flop_plan_tile_schedule", "flop_plan_chain_queue", "flop_scale_rows_grouped", "flop_dlog_alpha_finish_grouped", "flop_gemm_timing_begin",
           "flop_gemm_timing_end", "flop_gemm_stamps_begin", "flop_gemm_stamps_end", "flop_gemm_stamps_accumulate", "flop_workspace_bytes", "flop_tc_gemm", "flop_gate_sample", "flop_gate_sample_devoff",
           "flop_gated_lowrank_fwd", "flop_gated_lowrank_bwd", "flop_gated_lowrank_fwd_grouped",
           "flop_gated_lowrank_bwd_grouped", "flop_active_ranks_gather", "flop_active_ranks_scatter",
           "flop_expected_l0_lagrangian",
           "flop_expected_l0_lagrangian_noalloc", "flop_agp_gates", "flop_gated_embedding_fwd",
           "flop_gated_embedding_bwd",
           "flop_compact_ranks", "flop_compact_fwd", "flop_chain_fwd")


class HcParams(ctypes.Structure):
    _fields_ = [("beta", ctypes.c_float), ("gamma", ctypes.c_float), ("zeta", ctypes.c_float)]


class FwdProblem(ctypes.Structure):
    _fields_ = [("X", ctypes.c_void_p), ("ldx", ctypes.c_int64), ("Q", ctypes.c_void_p), ("ldq", ctypes.c_int64),
                ("P", ctypes.c_void_p), ("ldp", ctypes.c_int64), ("z", ctypes.c_void_p), ("Y", ctypes.c_void_p),
                ("ldy", ctypes.c_int64), ("H_save", ctypes.c_void_p), ("ldh", ctypes.c_int64),
                ("T", ctypes.c_int64), ("d_in", ctypes.c_int64), ("d_out", ctypes.c_int64), ("r", ctypes.c_int64),
                ("r_dev", ctypes.c_void_p)]


class BwdProblem(ctypes.Structure):
    _fields_ = [("dY", ctypes.c_void_p), ("lddy", ctypes.c_int64), ("X", ctypes.c_void_p), ("ldx", ctypes.c_int64),
                ("Q", ctypes.c_void_p), ("ldq", ctypes.c_int64), ("P", ctypes.c_void_p), ("ldp", ctypes.c_int64),
                ("z", ctypes.c_void_p), ("dz_dla", ctypes.c_void_p), ("H_save", ctypes.c_void_p), ("ldh", ctypes.c_int64),
                ("dX", ctypes.c_void_p), ("lddx", ctypes.c_int64), ("dP", ctypes.c_void_p), ("lddp", ctypes.c_int64),
                ("dQ", ctypes.c_void_p), ("lddq", ctypes.c_int64), ("dlog_alpha", ctypes.c_void_p),
                ("T", ctypes.c_int64), ("d_in", ctypes.c_int64), ("d_out", ctypes.c_int64), ("r", ctypes.c_int64),
                ("ws", ctypes.c_void_p), ("ws_bytes", ctypes.c_size_t), ("r_dev", ctypes.c_void_p),
                ("Qz", ctypes.c_void_p), ("ldqz", ctypes.c_int64), ("defer_dlog_alpha", ctypes.c_int32)]


class ScaleRows(ctypes.Structure):
    _fields_ = [("Q", ctypes.c_void_p), ("ldq", ctypes.c_int64), ("z", ctypes.c_void_p), ("Qz", ctypes.c_void_p),
                ("ldqz", ctypes.c_int64), ("r", ctypes.c_int64), ("d_in", ctypes.c_int64)]


class ActiveGather(ctypes.Structure):
    _fields_ = [("z", ctypes.c_void_p), ("dz_dla", ctypes.c_void_p), ("P", ctypes.c_void_p), ("ldp", ctypes.c_int64),
                ("Q", ctypes.c_void_p), ("ldq", ctypes.c_int64),
                ("d_in", ctypes.c_int64), ("d_out", ctypes.c_int64), ("r", ctypes.c_int64),
                ("idx", ctypes.c_void_p), ("pos", ctypes.c_void_p), ("k_dev", ctypes.c_void_p),
                ("z_c", ctypes.c_void_p), ("dz_dla_c", ctypes.c_void_p),
                ("P_c", ctypes.c_void_p), ("ldpc", ctypes.c_int64), ("Q_c", ctypes.c_void_p), ("ldqc", ctypes.c_int64),
                ("Qz_c", ctypes.c_void_p), ("ldqzc", ctypes.c_int64)]


class ActiveScatter(ctypes.Structure):
    _fields_ = [("idx", ctypes.c_void_p), ("pos", ctypes.c_void_p), ("k_dev", ctypes.c_void_p),
                ("d_in", ctypes.c_int64), ("d_out", ctypes.c_int64), ("r", ctypes.c_int64),
                ("dP_c", ctypes.c_void_p), ("lddpc", ctypes.c_int64), ("dQ_c", ctypes.c_void_p), ("lddqc", ctypes.c_int64),
                ("dlog_alpha_c", ctypes.c_void_p),
                ("dP", ctypes.c_void_p), ("lddp", ctypes.c_int64), ("dQ", ctypes.c_void_p), ("lddq", ctypes.c_int64),
                ("dlog_alpha", ctypes.c_void_p)]


class FlopError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


_lib = None


def load_library() -> ctypes.CDLL:
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_1910_04732_b200.build` "
                           "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    i64, vp, sz, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
    lib.flop_status_string.restype = ctypes.c_char_p
    lib.flop_status_string.argtypes = [ci]
    lib.flop_device_status.argtypes = [vp]
    lib.flop_last_async_status.argtypes = [vp]
    lib.flop_sync_bytes.argtypes = [ctypes.POINTER(sz)]
    lib.flop_gated_lowrank_fwd_chained.argtypes = [ctypes.POINTER(FwdProblem), ci, ci, vp, sz, vp]
    lib.flop_gated_lowrank_bwd_chained.argtypes = [ctypes.POINTER(BwdProblem), ci, ci, ci, ci, vp, sz, vp]
    lib.flop_workspace_bytes.argtypes = [ci, i64, i64, i64, i64, ci, ctypes.POINTER(sz)]
    lib.flop_launch_count.argtypes = []
    lib.flop_plan_tile_schedule.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.c_int32, ctypes.c_int32,
                                            ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_double),
                                            ctypes.POINTER(ctypes.c_double)]
    lib.flop_plan_chain_queue.argtypes = [ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int64), ctypes.c_int32,
                                          ctypes.POINTER(ctypes.c_int32)]
    lib.flop_scale_rows_grouped.argtypes = [ctypes.POINTER(ScaleRows), ci, ci, vp]
    lib.flop_dlog_alpha_finish_grouped.argtypes = [ctypes.POINTER(BwdProblem), ci, ci, ci, vp]
    lib.flop_selftest_wait_timeout.argtypes = [i64, vp, vp]
    lib.flop_gemm_timing_begin.argtypes = []
    lib.flop_gemm_timing_end.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double),
                                         ctypes.POINTER(ctypes.c_int64)]
    lib.flop_tc_gemm.argtypes = [vp, i64, ci, vp, i64, ci, vp, i64, vp, vp, i64, i64, i64, ci, ci, ci,
                                 ctypes.POINTER(ctypes.c_int), vp]
    lib.flop_gemm_stamps_begin.argtypes = [vp, ci]
    lib.flop_gemm_stamps_end.argtypes = [ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_double)]
    lib.flop_gemm_stamps_accumulate.argtypes = [vp, ci, vp, vp]
    lib.flop_gate_sample.argtypes = [vp, i64, HcParams, ctypes.c_uint64, ctypes.c_uint64, vp, vp, vp, vp]
    lib.flop_gate_sample_devoff.argtypes = [vp, i64, HcParams, ctypes.c_uint64, ctypes.c_uint64, vp, vp, vp, vp, vp]
    lib.flop_gated_lowrank_fwd.argtypes = [vp, i64, vp, i64, vp, i64, vp, vp, i64, vp, i64,
                                           i64, i64, i64, i64, ci, vp, sz, vp]
    lib.flop_gated_lowrank_bwd.argtypes = [vp, i64, vp, i64, vp, i64, vp, i64, vp, vp, vp, i64,
                                           vp, i64, vp, i64, vp, i64, vp, ci,
                                           i64, i64, i64, i64, ci, ci, vp, sz, vp]
    lib.flop_chain_fwd.argtypes = [vp, i64, vp, i64, vp, i64, vp, vp, i64, i64, i64, i64, i64, ci, vp]
    lib.flop_gated_lowrank_fwd_grouped.argtypes = [ctypes.POINTER(FwdProblem), ci, ci, vp]
    lib.flop_gated_lowrank_bwd_grouped.argtypes = [ctypes.POINTER(BwdProblem), ci, ci, ci, ci, vp]
    lib.flop_active_ranks_gather.argtypes = [ctypes.POINTER(ActiveGather), ci, ci, vp]
    lib.flop_active_ranks_scatter.argtypes = [ctypes.POINTER(ActiveScatter), ci, ci, ci, vp]
    lib.flop_expected_l0_lagrangian.argtypes = [vp, i64, vp, vp, ctypes.c_int32, HcParams, vp, vp, vp, vp, vp,
                                                vp, sz, vp]
    lib.flop_expected_l0_lagrangian_noalloc.argtypes = [vp, i64, vp, vp, ctypes.c_int32, HcParams, vp, vp, vp, vp, vp, vp]
    lib.flop_gated_embedding_fwd.argtypes = [vp, i64, vp, i64, i64, vp, i64, vp, vp, i64, vp, i64, i64, i64, ci, vp]
    lib.flop_gated_embedding_bwd.argtypes = [vp, i64, vp, i64, vp, i64, i64, vp, i64, vp, vp, vp, i64, vp, i64, vp, i64,
                                             vp, ci, i64, i64, ci, ci, vp, sz, vp]
    lib.flop_agp_gates.argtypes = [vp, i64, vp, ctypes.c_int32, vp, ctypes.c_float, vp, vp, vp, vp, vp, vp]
    lib.flop_compact_ranks.argtypes = [vp, ci, HcParams, i64, vp, i64, vp, i64, i64, i64, ci,
                                       vp, vp, vp, vp, i64, vp, i64, vp, sz, vp]
    lib.flop_compact_fwd.argtypes = [vp, i64, vp, i64, vp, i64, vp, i64, i64, i64, i64, i64, ci, vp, sz, vp]
    for name in EXPORTS[1:]:
        getattr(lib, name).restype = ci
    lib.flop_launch_count.restype = ctypes.c_ulonglong
    _lib = lib
    return lib


def plan_tile_schedule(cost, units: int):
    """Host-only: (unit of every work item, largest unit load, largest load of the round-robin deal)."""
    n = len(cost)
    c = (ctypes.c_double * max(n, 1))(*[float(v) for v in cost])
    out = (ctypes.c_int32 * max(n, 1))()
    ms, rr = ctypes.c_double(0.0), ctypes.c_double(0.0)
    _check(load_library().flop_plan_tile_schedule(c, n, int(units), out, ctypes.byref(ms), ctypes.byref(rr)),
           "flop_plan_tile_schedule")
    return list(out)[:n], ms.value, rr.value


def plan_chain_queue(stage, key):
    """Host-only: the position of every work item in the queue of a chained launch."""
    n = len(stage)
    st = (ctypes.c_int32 * max(n, 1))(*[int(v) for v in stage])
    k = (ctypes.c_int64 * max(n, 1))(*[int(v) for v in key])
    pos = (ctypes.c_int32 * max(n, 1))()
    _check(load_library().flop_plan_chain_queue(st, k, n, pos), "flop_plan_chain_queue")
    return list(pos)[:n]


def status_string(code: int) -> str:
    return load_library().flop_status_string(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != OK:
        raise FlopError(code, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ld(t: torch.Tensor) -> int:
    assert t.dim() == 2 and t.stride(1) == 1, "matrices must be row-major with unit column stride"
    return t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])


def _hc(hc) -> HcParams:
    return HcParams(float(hc[0]), float(hc[1]), float(hc[2]))


def workspace_bytes(op: int, T: int, d_in: int, d_out: int, r: int, dt: int) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().flop_workspace_bytes(op, T, d_in, d_out, r, dt, ctypes.byref(out)), "flop_workspace_bytes")
    return int(out.value)


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A 256-byte aligned scratch buffer (torch's caching allocator aligns to 512)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def selftest_wait_timeout(limit_cycles: int, gave_up: torch.Tensor) -> None:
    """Launch the bounded-wait self-test: a wait that can never complete must give up after limit_cycles."""
    _check(load_library().flop_selftest_wait_timeout(int(limit_cycles), _ptr(gave_up), _stream()),
           "flop_selftest_wait_timeout")


def launch_count() -> int:
    return int(load_library().flop_launch_count())


def gemm_timing_begin() -> None:
    _check(load_library().flop_gemm_timing_begin(), "flop_gemm_timing_begin")


def gemm_timing_end():
    """(total kernel ms, total algorithmic flops, launches) of the GEMMs since gemm_timing_begin()."""
    ms, fl, n = ctypes.c_double(0), ctypes.c_double(0), ctypes.c_int64(0)
    _check(load_library().flop_gemm_timing_end(ctypes.byref(ms), ctypes.byref(fl), ctypes.byref(n)),
           "flop_gemm_timing_end")
    return ms.value, fl.value, int(n.value)


def gemm_stamps_begin(stamps: torch.Tensor) -> None:
    """stamps: zeroed int64 device tensor of 2 * capacity elements (start, end ns per GEMM launch)."""
    assert stamps.element_size() == 8
    _check(load_library().flop_gemm_stamps_begin(_ptr(stamps), stamps.numel() // 2), "flop_gemm_stamps_begin")


def gemm_stamps_end():
    """(stamped launches, sum of their algorithmic flops)."""
    n, fl = ctypes.c_int(0), ctypes.c_double(0)
    _check(load_library().flop_gemm_stamps_end(ctypes.byref(n), ctypes.byref(fl)), "flop_gemm_stamps_end")
    return int(n.value), fl.value


def gemm_stamps_accumulate(stamps: torch.Tensor, acc: torch.Tensor) -> None:
    """acc (zeroed int64[2] device tensor): [0] += stamped GEMM kernel time (ns) of the step just issued, [1] += 1."""
    assert stamps.element_size() == 8 and acc.element_size() == 8 and acc.numel() >= 2
    _check(load_library().flop_gemm_stamps_accumulate(_ptr(stamps), stamps.numel() // 2, _ptr(acc), _stream()),
           "flop_gemm_stamps_accumulate")


def device_status() -> int:
    return int(load_library().flop_device_status(_stream()))


def padded(rows: int, cols: int, dtype, device="cuda", multiple: int = 8) -> torch.Tensor:
    """A [rows, cols] view whose leading dimension is rounded up to `multiple`
    elements (bf16 operands need 16-byte aligned rows)."""
    ld = (cols + multiple - 1) // multiple * multiple
    return torch.zeros(rows, max(ld, multiple), dtype=dtype, device=device)[:, :cols]


def tc_gemm(A, a_mn_major: bool, B, b_mn_major: bool, M: int, N: int, K: int, D=None, col_scale=None, slices=None,
            bn: int = 0, cta2: int = -1, splits: int = 0) -> int:
    """flop_tc_gemm: D[M,N] = sum_k A(m,k) B(n,k).  Returns the number of fp32 slices written (1 for a bf16 D)."""
    n = ctypes.c_int(0)
    _check(load_library().flop_tc_gemm(_ptr(A), _ld(A), int(a_mn_major), _ptr(B), _ld(B), int(b_mn_major),
                                       _ptr(D), _ld(D) if D is not None else 0, _ptr(col_scale), _ptr(slices),
                                       M, N, K, bn, cta2, splits, ctypes.byref(n), _stream()), "flop_tc_gemm")
    return int(n.value)


def gate_sample(log_alpha: torch.Tensor, hc, seed: int, offset: int, z: torch.Tensor,
                mask: Optional[torch.Tensor] = None, dz_dla: Optional[torch.Tensor] = None) -> None:
    n = log_alpha.numel()
    _check(load_library().flop_gate_sample(_ptr(log_alpha), n, _hc(hc), seed, offset, _ptr(z), _ptr(mask),
                                           _ptr(dz_dla), _stream()), "flop_gate_sample")


def gate_sample_devoff(log_alpha: torch.Tensor, hc, seed: int, offset: int, offset_dev: torch.Tensor, z: torch.Tensor,
                       mask: Optional[torch.Tensor] = None, dz_dla: Optional[torch.Tensor] = None) -> None:
    """Gate sampling with counter offset `offset + offset_dev[0]` (offset_dev: one 64-bit integer on the device)."""
    assert offset_dev.element_size() == 8 and offset_dev.numel() >= 1
    _check(load_library().flop_gate_sample_devoff(_ptr(log_alpha), log_alpha.numel(), _hc(hc), seed, offset,
                                                  _ptr(offset_dev), _ptr(z), _ptr(mask), _ptr(dz_dla), _stream()),
           "flop_gate_sample_devoff")


def gated_lowrank_fwd(X, Q, P, z, Y, H_save=None, ws=None) -> None:
    T, d_in = X.shape
    d_out, r = P.shape
    _check(load_library().flop_gated_lowrank_fwd(
        _ptr(X), _ld(X), _ptr(Q), _ld(Q), _ptr(P), _ld(P), _ptr(z), _ptr(Y), _ld(Y),
        _ptr(H_save), _ld(H_save) if H_save is not None else 0, T, d_in, d_out, r, _dt(X),
        _ptr(ws), ws.numel() if ws is not None else 0, _stream()), "flop_gated_lowrank_fwd")


def gated_lowrank_bwd(dY, X, Q, P, z, dz_dla, H_save, dX, dP, dQ, dlog_alpha, ws, accumulate: bool = False) -> None:
    T, d_in = X.shape
    d_out, r = P.shape
    wdt = _dt(dP) if dP is not None else (_dt(dQ) if dQ is not None else _dt(X))
    _check(load_library().flop_gated_lowrank_bwd(
        _ptr(dY), _ld(dY), _ptr(X), _ld(X), _ptr(Q), _ld(Q), _ptr(P), _ld(P), _ptr(z), _ptr(dz_dla),
        _ptr(H_save), _ld(H_save),
        _ptr(dX), _ld(dX) if dX is not None else 0, _ptr(dP), _ld(dP) if dP is not None else 0,
        _ptr(dQ), _ld(dQ) if dQ is not None else 0, _ptr(dlog_alpha), int(accumulate),
        T, d_in, d_out, r, _dt(X), wdt, _ptr(ws), ws.numel() if ws is not None else 0, _stream()),
        "flop_gated_lowrank_bwd")


def _p(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def fwd_problem(X, Q, P, z, Y, H_save, r_dev=None) -> FwdProblem:
    T, d_in = X.shape
    d_out, r = P.shape
    return FwdProblem(_p(X), _ld(X), _p(Q), _ld(Q), _p(P), _ld(P), _p(z), _p(Y), _ld(Y), _p(H_save), _ld(H_save),
                      T, d_in, d_out, r, _p(r_dev))


def bwd_problem(dY, X, Q, P, z, dz_dla, H_save, dX, dP, dQ, dlog_alpha, ws, r_dev=None, Qz=None,
                defer_dlog_alpha: bool = False) -> BwdProblem:
    T, d_in = X.shape
    d_out, r = P.shape
    ld = lambda t: _ld(t) if t is not None else 0
    return BwdProblem(_p(dY), _ld(dY), _p(X), _ld(X), _p(Q), _ld(Q), _p(P), _ld(P), _p(z), _p(dz_dla), _p(H_save),
                      _ld(H_save), _p(dX), ld(dX), _p(dP), ld(dP), _p(dQ), ld(dQ), _p(dlog_alpha), T, d_in, d_out, r,
                      _p(ws), ws.numel() if ws is not None else 0, _p(r_dev), _p(Qz), ld(Qz), int(defer_dlog_alpha))


def dlog_alpha_finish_grouped(problems, accumulate: bool = False, dt: int = BF16) -> None:
    arr = problems if isinstance(problems, ctypes.Array) else problem_array(problems)
    _check(load_library().flop_dlog_alpha_finish_grouped(arr, len(arr), int(accumulate), dt, _stream()),
           "flop_dlog_alpha_finish_grouped")


def scale_rows_problem(Q, z, Qz) -> ScaleRows:
    r, d_in = Q.shape
    return ScaleRows(_p(Q), _ld(Q), _p(z), _p(Qz), _ld(Qz), r, d_in)


def scale_rows_grouped(problems, dt: int = BF16) -> None:
    """Qz = diag(z) Q for every problem, one launch (per 96 matrices)."""
    arr = problems if isinstance(problems, ctypes.Array) else problem_array(problems)
    _check(load_library().flop_scale_rows_grouped(arr, len(arr), dt, _stream()), "flop_scale_rows_grouped")


def active_gather_problem(z, dz_dla, P, Q, idx, pos, k_dev, z_c, dz_dla_c, P_c, Q_c, Qz_c=None) -> ActiveGather:
    d_out, r = P.shape
    d_in = Q.shape[1]
    return ActiveGather(_p(z), _p(dz_dla), _p(P), _ld(P), _p(Q), _ld(Q), d_in, d_out, r, _p(idx), _p(pos), _p(k_dev),
                        _p(z_c), _p(dz_dla_c), _p(P_c), _ld(P_c), _p(Q_c), _ld(Q_c), _p(Qz_c),
                        _ld(Qz_c) if Qz_c is not None else 0)


def active_scatter_problem(idx, pos, k_dev, d_in, d_out, r, dP_c, dQ_c, dla_c, dP, dQ, dla) -> ActiveScatter:
    ld = lambda t: _ld(t) if t is not None else 0
    return ActiveScatter(_p(idx), _p(pos), _p(k_dev), d_in, d_out, r, _p(dP_c), ld(dP_c), _p(dQ_c), ld(dQ_c), _p(dla_c),
                         _p(dP), ld(dP), _p(dQ), ld(dQ), _p(dla))


def active_ranks_gather(problems, dt: int = BF16) -> None:
    arr = problems if isinstance(problems, ctypes.Array) else problem_array(problems)
    _check(load_library().flop_active_ranks_gather(arr, len(arr), dt, _stream()), "flop_active_ranks_gather")


def active_ranks_scatter(problems, accumulate: bool = False, wgrad_dt: int = BF16) -> None:
    arr = problems if isinstance(problems, ctypes.Array) else problem_array(problems)
    _check(load_library().flop_active_ranks_scatter(arr, len(arr), int(accumulate), wgrad_dt, _stream()),
           "flop_active_ranks_scatter")


def problem_array(problems):
    """ctypes array of FwdProblem / BwdProblem; build it once and reuse it when the pointers do not change."""
    return (type(problems[0]) * len(problems))(*problems)


def gated_lowrank_fwd_grouped(problems, dt: int = BF16) -> None:
    arr = problems if isinstance(problems, ctypes.Array) else problem_array(problems)
    _check(load_library().flop_gated_lowrank_fwd_grouped(arr, len(arr), dt, _stream()), "flop_gated_lowrank_fwd_grouped")


def gated_lowrank_bwd_grouped(problems, accumulate: bool = False, dt: int = BF16, wgrad_dt: int = BF16) -> None:
    arr = problems if isinstance(problems, ctypes.Array) else problem_array(problems)
    _check(load_library().flop_gated_lowrank_bwd_grouped(arr, len(arr), int(accumulate), dt, wgrad_dt, _stream()),
           "flop_gated_lowrank_bwd_grouped")


def chain_fwd(X, Q, P, z, Y, dt: int = BF16) -> None:
    """flop_chain_fwd: Y = ((X Q^T) * z) P^T in one launch (z may be None)."""
    T, d_in = X.shape
    d_out, r = P.shape
    _check(load_library().flop_chain_fwd(_ptr(X), _ld(X), _ptr(Q), _ld(Q), _ptr(P), _ld(P), _ptr(z), _ptr(Y), _ld(Y),
                                         T, d_in, d_out, r, dt, _stream()), "flop_chain_fwd")


def sync_bytes() -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().flop_sync_bytes(ctypes.byref(out)), "flop_sync_bytes")
    return int(out.value)


def alloc_sync(device="cuda") -> torch.Tensor:
    """A zero-filled sync area for the chained calls (they leave it zero-filled)."""
    return torch.zeros(sync_bytes(), dtype=torch.uint8, device=device)


def gated_lowrank_fwd_chained(problems, sync: torch.Tensor, dt: int = BF16) -> None:
    arr = problems if isinstance(problems, ctypes.Array) else problem_array(problems)
    _check(load_library().flop_gated_lowrank_fwd_chained(arr, len(arr), dt, _ptr(sync), sync.numel(), _stream()),
           "flop_gated_lowrank_fwd_chained")


def gated_lowrank_bwd_chained(problems, sync: torch.Tensor, accumulate: bool = False, dt: int = BF16,
                              wgrad_dt: int = BF16) -> None:
    arr = problems if isinstance(problems, ctypes.Array) else problem_array(problems)
    _check(load_library().flop_gated_lowrank_bwd_chained(arr, len(arr), int(accumulate), dt, wgrad_dt, _ptr(sync),
                                                         sync.numel(), _stream()), "flop_gated_lowrank_bwd_chained")


def expected_l0_lagrangian(log_alpha, seg_off, seg_size, hc, target, lam, out4, seg_expected=None,
                           dlog_alpha=None, ws=None) -> None:
    _check(load_library().flop_expected_l0_lagrangian(
        _ptr(log_alpha), log_alpha.numel(), _ptr(seg_off), _ptr(seg_size), seg_size.numel(), _hc(hc),
        _ptr(target), _ptr(lam), _ptr(out4), _ptr(seg_expected), _ptr(dlog_alpha),
        _ptr(ws), ws.numel() if ws is not None else 0, _stream()), "flop_expected_l0_lagrangian")


def expected_l0_lagrangian_noalloc(log_alpha, seg_off, seg_size, hc, target, lam, out4, seg_expected=None,
                                   dlog_alpha=None) -> None:
    """flop_expected_l0_lagrangian_noalloc: same outputs, no workspace argument.  For callers that
    may not allocate device memory (a frozen memory pool, a plug-in without an allocator): the
    scratch is a fixed array inside the library, limited to 1,048,576 gates in 4096 segments and
    shared by all calls on a device, so calls must not overlap on the GPU."""
    _check(load_library().flop_expected_l0_lagrangian_noalloc(
        _ptr(log_alpha), log_alpha.numel(), _ptr(seg_off), _ptr(seg_size), seg_size.numel(), _hc(hc),
        _ptr(target), _ptr(lam), _ptr(out4), _ptr(seg_expected), _ptr(dlog_alpha), _stream()),
        "flop_expected_l0_lagrangian_noalloc")


def gated_embedding_fwd(ids, E, O, z, Y, H_save) -> None:
    T, (n_rows, d_i), d = ids.numel(), E.shape, O.shape[1]
    _check(load_library().flop_gated_embedding_fwd(_ptr(ids), T, _ptr(E), _ld(E), n_rows, _ptr(O), _ld(O), _ptr(z), _ptr(Y),
                                                   _ld(Y), _ptr(H_save), _ld(H_save), d_i, d, _dt(E), _stream()),
           "flop_gated_embedding_fwd")


def gated_embedding_bwd(dY, ids, E, O, z, dz_dla, H_save, dE, dO, dlog_alpha, ws, accumulate: bool = False) -> None:
    T, (n_rows, d_i), d = ids.numel(), E.shape, O.shape[1]
    wdt = _dt(dO) if dO is not None else BF16
    _check(load_library().flop_gated_embedding_bwd(
        _ptr(dY), _ld(dY), _ptr(ids), T, _ptr(E), _ld(E), n_rows, _ptr(O), _ld(O), _ptr(z), _ptr(dz_dla), _ptr(H_save),
        _ld(H_save), _ptr(dE), _ld(dE) if dE is not None else 0, _ptr(dO), _ld(dO) if dO is not None else 0,
        _ptr(dlog_alpha), int(accumulate), d_i, d, _dt(E), wdt, _ptr(ws), ws.numel() if ws is not None else 0, _stream()),
        "flop_gated_embedding_bwd")


def agp_gates(g, seg_off, sparsity, l1: float, z, mask=None, dz_dg=None, seg_l1=None, dg=None) -> None:
    """flop_agp_gates: magnitude pruning of the diagonal mask per segment (sparsity: 1-element device tensor)."""
    _check(load_library().flop_agp_gates(_ptr(g), g.numel(), _ptr(seg_off), seg_off.numel() - 1, _ptr(sparsity), float(l1),
                                         _ptr(z), _ptr(mask), _ptr(dz_dg), _ptr(seg_l1), _ptr(dg), _stream()),
           "flop_agp_gates")


def compact_ranks(log_alpha_or_z, mode: int, hc, idx, k_dev, z_det=None, P=None, Q=None, Pc=None, Qc=None) -> None:
    r = log_alpha_or_z.numel()
    d_in = Q.shape[1] if Q is not None else 0
    d_out = P.shape[0] if P is not None else 0
    dt = _dt(P) if P is not None else F32
    _check(load_library().flop_compact_ranks(
        _ptr(log_alpha_or_z), mode, _hc(hc), r, _ptr(P), _ld(P) if P is not None else 0,
        _ptr(Q), _ld(Q) if Q is not None else 0, d_in, d_out, dt, _ptr(idx), _ptr(k_dev), _ptr(z_det),
        _ptr(Pc), _ld(Pc) if Pc is not None else 0, _ptr(Qc), _ld(Qc) if Qc is not None else 0,
        None, 0, _stream()), "flop_compact_ranks")


def compact_fwd(X, Qc, Pc, Y, k: int, ws) -> None:
    T, d_in = X.shape
    d_out = Pc.shape[0]
    _check(load_library().flop_compact_fwd(
        _ptr(X), _ld(X), _ptr(Qc), _ld(Qc), _ptr(Pc), _ld(Pc), _ptr(Y), _ld(Y), T, d_in, d_out, k, _dt(X),
        _ptr(ws), ws.numel() if ws is not None else 0, _stream()), "flop_compact_fwd")
