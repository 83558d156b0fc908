#!/usr/bin/env python
"""Benchmark of the FLOP gated low-rank hot path on B200.

One step = one pass of the whole hot path over one batch of synthetic input:
sample every gate of every layer (one launch), form diag(z)Q of every matrix
(one launch), then for every factorized matrix of every layer the gated forward
(2 GEMMs) and backward (4 GEMMs + the fused dlog_alpha row dots; grouped per
layer into two forward and two backward launches), the second stage of
dlog_alpha for every matrix (one launch), then the expected-L0 / Lagrangian term
over all gates.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload bert|sru|txl] [--impl ours|reference]

Prints ONE JSON line.  `value` is tokens/s with inputs resident in HBM; `e2e`
is the same step through the same calls with every X and dY copied from pinned
host memory and Y, dX, all weight gradients, dlog_alpha and the Lagrangian
scalars copied back inside the timed region; `roofline` times the tensor-core
GEMM launches with device-side stamps inside the replayed CUDA graph (and, for
comparison, with CUDA events in an eager pass); `cpu_baseline` is the fp64
oracle timed on the host cores on a bounded sample.  `--impl reference` times
the oracle alone.  Under torchrun every rank processes its own token batch
with the same gate sample and the weight gradients are all-reduced (NCCL).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1910_04732_b200 import inputs as I  # noqa: E402

METRIC = "gated low-rank fwd+bwd tokens/s and TFLOP/s, % of B200 bf16 tensor peak"
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
HC = tuple(float(np.float32(v)) for v in (I.BETA, I.GAMMA, I.ZETA))


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


def roofline_traffic(workload: str, group: int):
    """DRAM bytes per GEMM launch from the ncu capture summarised in profiles/gemm_traffic.txt, valid only while the
    GEMM kernel sources are the ones the capture was taken with (the file records their hash)."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "gemm_traffic.txt")
    try:
        fields = {}
        for ln in open(path):
            if "=" in ln and not ln.startswith("#"):
                k, v = ln.strip().split("=", 1)
                fields[k.strip()] = v.strip()
        h = hashlib.sha1()
        d = os.path.join(ROOT, "paper_1910_04732_b200", "csrc")
        for f in ("gemm_tc.cuh", "gemm_tc2.cuh", "gemm_tc_group.cuh", "gemm_tc2_group.cuh", "gemm_tc2_dual.cuh", "schedule.cuh"):
            h.update(open(os.path.join(d, f), "rb").read())
        if fields.get("workload") != workload or int(fields.get("matrices_per_call", -1)) != group:
            return None, "no capture for this workload"
        if fields.get("kernel_sources_sha1") != h.hexdigest():
            return None, "the GEMM kernels have changed since the capture in profiles/gemm_traffic.txt"
        return float(fields["dram_bytes_per_launch"]), fields.get("note", "")
    except Exception:
        return None, "profiles/gemm_traffic.txt not found"


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, mx, pw, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            try:
                pw.append(float(parts[2]))
            except ValueError:
                pass
            for n, v in zip(names, parts[3:7]):
                if v.lower() == "active":
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "sm_mhz_min": min(sm) if sm else None, "power_w": float(np.median(pw)) if pw else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- our arm
class Job:
    """Device state of one workload: inputs, outputs and scratch of every matrix."""

    def __init__(self, w: I.Workload, device, seed: int, n_streams: int = 1, group: int = 0):
        import torch
        from paper_1910_04732_b200 import binding as b
        self.w, self.b, self.torch = w, b, torch
        bf = torch.bfloat16
        g = torch.Generator(device=device)
        g.manual_seed(seed)                 # activations: every rank its own batch
        gw = torch.Generator(device=device)
        gw.manual_seed(1234)                # weights: one model on every rank (their gradients are summed)
        mats = w.all_matrices()
        self.n_gates = w.n_gates()
        # gate state, concatenated over all matrices
        alphas, offs, sizes = [], [0], []
        for l, i, m in mats:
            alphas.append(I.log_alpha(w.alpha, m.r, 0, l, i))
            offs.append(offs[-1] + m.r)
            sizes.append(float(m.d_in + m.d_out))
        self.log_alpha = torch.from_numpy(np.concatenate(alphas)).to(device)
        self.seg_off = torch.tensor(offs, dtype=torch.int64, device=device)
        self.seg_size = torch.tensor(sizes, dtype=torch.float32, device=device)
        self.z = torch.empty(self.n_gates, device=device)
        self.dz_dla = torch.empty(self.n_gates, device=device)
        self.mask = torch.empty(self.n_gates, dtype=torch.uint8, device=device)
        self.dlog_alpha = torch.zeros(self.n_gates, device=device)
        self.target = torch.tensor([w.target], device=device)
        self.lam = torch.tensor([0.3, 1.7], device=device)
        self.out4 = torch.zeros(4, device=device)
        # weight gradients of all matrices in one flat buffer (one all-reduce under data parallelism)
        r8 = lambda v: (v + 7) // 8 * 8
        n_w = sum(m.d_out * r8(m.r) + m.r * r8(m.d_in) for _, _, m in mats)
        self.wgrad = torch.zeros(n_w, dtype=bf, device=device)
        self.mats, pos, ws_bytes = [], 0, 0
        randn = lambda rows, cols, scale=1.0, gen=g: (torch.randn(rows, r8(cols), generator=gen, device=device) * scale).to(bf)[:, :cols]
        for (l, i, m), lo in zip(mats, offs):
            e = dict(m=m, lo=lo, hi=lo + m.r)
            e["X"], e["dY"] = randn(w.T, m.d_in), randn(w.T, m.d_out)
            e["Q"], e["P"] = randn(m.r, m.d_in, m.d_in ** -0.5, gw), randn(m.d_out, m.r, m.r ** -0.5, gw)
            e["H"], e["Y"], e["dX"] = (b.padded(w.T, c, bf, device) for c in (m.r, m.d_out, m.d_in))
            e["dP"] = self.wgrad[pos:pos + m.d_out * r8(m.r)].view(m.d_out, r8(m.r))[:, :m.r]; pos += m.d_out * r8(m.r)
            e["dQ"] = self.wgrad[pos:pos + m.r * r8(m.d_in)].view(m.r, r8(m.d_in))[:, :m.d_in]; pos += m.r * r8(m.d_in)
            ws_bytes = max(ws_bytes, b.workspace_bytes(b.OP_BWD, w.T, m.d_in, m.d_out, m.r, b.BF16))
            self.mats.append(e)
        # independent matrices are issued round-robin on a few streams, each with its own scratch, so
        # that the tail of one matrix's kernels overlaps the head of another's
        self.n_streams = max(1, n_streams)
        self.streams = [torch.cuda.Stream(device=device) for _ in range(self.n_streams)] if self.n_streams > 1 else []
        self.wss = [b.alloc_workspace(ws_bytes, device) for _ in range(self.n_streams)]
        self.ws = self.wss[0]
        self.ev_gates = torch.cuda.Event()
        self.ev_done = [torch.cuda.Event() for _ in range(self.n_streams)]
        # grouped issue: `group` consecutive matrices (default: the matrices of one layer) per call,
        # every matrix with its own scratch; the argument arrays are built once
        self.group = group
        self.groups = []
        if group > 0:
            for e in self.mats:
                e["ws"] = b.alloc_workspace(b.workspace_bytes(b.OP_BWD, w.T, e["m"].d_in, e["m"].d_out, e["m"].r, b.BF16), device)
                e["Qz"] = b.padded(e["m"].r, e["m"].d_in, bf, device)      # diag(z) Q, formed once per step
            self.scale = b.problem_array([b.scale_rows_problem(e["Q"], self.z[e["lo"]:e["hi"]], e["Qz"]) for e in self.mats])
            for i in range(0, len(self.mats), group):
                chunk = self.mats[i:i + group]
                fwd = b.problem_array([b.fwd_problem(e["X"], e["Q"], e["P"], self.z[e["lo"]:e["hi"]], e["Y"], e["H"])
                                       for e in chunk])
                mk = lambda e, **kw: b.bwd_problem(e["dY"], e["X"], e["Q"], e["P"], self.z[e["lo"]:e["hi"]],
                                                   self.dz_dla[e["lo"]:e["hi"]], e["H"], e["dX"], e["dP"], e["dQ"],
                                                   self.dlog_alpha[e["lo"]:e["hi"]], e["ws"], **kw)
                # default: diag(z) Q comes from the one launch after sampling, the second stage of dlog_alpha is left
                # to the one launch at the end of the step; "plain": every backward call does both itself
                bwd = b.problem_array([mk(e, Qz=e["Qz"], defer_dlog_alpha=True) for e in chunk])
                bwd_chain = b.problem_array([mk(e, Qz=e["Qz"]) for e in chunk])
                bwd_plain = b.problem_array([mk(e) for e in chunk])
                self.groups.append((fwd, bwd, bwd_chain, bwd_plain))
            self.bwd_all = b.problem_array([b.bwd_problem(e["dY"], e["X"], e["Q"], e["P"], self.z[e["lo"]:e["hi"]],
                                                          self.dz_dla[e["lo"]:e["hi"]], e["H"], e["dX"], e["dP"], e["dQ"],
                                                          self.dlog_alpha[e["lo"]:e["hi"]], e["ws"], Qz=e["Qz"],
                                                          defer_dlog_alpha=True) for e in self.mats])
        # data parallelism: one gradient bucket per grouped call (a layer), reduced while later layers compute
        from paper_1910_04732_b200 import dp
        self.bucket_bounds = dp.bucket_bounds(dp.weight_gradient_sizes([e["m"] for e in self.mats]),
                                              group if group > 0 else len(self.mats))
        self.reducer = None
        self.ws_l0 = b.alloc_workspace(b.workspace_bytes(b.OP_L0, self.n_gates, 0, 0, len(sizes), b.F32), device)
        self.offset_dev = torch.zeros(1, dtype=torch.int64, device=device)
        self.graph = None
        self.world = 1
        # chained calls: one launch for the two forward products, one for the whole backward pass of a layer
        self.chain = False
        self.plain = False
        self.sync = b.alloc_sync(device)

    def enable_active_ranks(self):
        """Buffers and argument arrays for training on the active components only (z_k > 0): per step one
        select + gather (which also writes diag(z_c) Q_c), one dlog_alpha_c finish and one scatter over all matrices; per layer the
        grouped forward and backward with the rank read on the device."""
        torch, b = self.torch, self.b
        bf = torch.bfloat16
        dev = self.log_alpha.device
        self.active_groups = []
        for e in self.mats:
            m = e["m"]
            if "ws" not in e:
                e["ws"] = b.alloc_workspace(b.workspace_bytes(b.OP_BWD, self.w.T, m.d_in, m.d_out, m.r, b.BF16), dev)
            e["idx"] = torch.zeros(m.r, dtype=torch.int32, device=dev)
            e["pos"] = torch.zeros(m.r, dtype=torch.int32, device=dev)
            e["k"] = torch.zeros(1, dtype=torch.int32, device=dev)
            e["zc"], e["dzc"], e["dlac"] = (torch.zeros(m.r, device=dev) for _ in range(3))
            e["Pc"], e["Qc"] = b.padded(m.d_out, m.r, bf, dev), b.padded(m.r, m.d_in, bf, dev)
            e["dPc"], e["dQc"] = b.padded(m.d_out, m.r, bf, dev), b.padded(m.r, m.d_in, bf, dev)
            e["Qzc"] = b.padded(m.r, m.d_in, bf, dev)
        g = self.group if self.group > 0 else len(self.w.matrices)
        z = lambda e: self.z[e["lo"]:e["hi"]]
        ms = self.mats
        # once per step for the whole model: select + gather (with diag(z_c) Q_c), the dlog_alpha_c finish, the scatter
        self.active_gather = b.problem_array([b.active_gather_problem(z(e), self.dz_dla[e["lo"]:e["hi"]], e["P"], e["Q"], e["idx"], e["pos"],
                                                                      e["k"], e["zc"], e["dzc"], e["Pc"], e["Qc"], Qz_c=e["Qzc"]) for e in ms])
        self.active_scatter = b.problem_array([b.active_scatter_problem(e["idx"], e["pos"], e["k"], e["m"].d_in, e["m"].d_out, e["m"].r,
                                                                        e["dPc"], e["dQc"], e["dlac"], e["dP"], e["dQ"],
                                                                        self.dlog_alpha[e["lo"]:e["hi"]]) for e in ms])
        bwd_all = []
        for i in range(0, len(ms), g):
            ch = ms[i:i + g]
            fwd = b.problem_array([b.fwd_problem(e["X"], e["Qc"], e["Pc"], e["zc"], e["Y"], e["H"], r_dev=e["k"]) for e in ch])
            bl = [b.bwd_problem(e["dY"], e["X"], e["Qc"], e["Pc"], e["zc"], e["dzc"], e["H"], e["dX"], e["dPc"], e["dQc"], e["dlac"],
                                e["ws"], r_dev=e["k"], Qz=e["Qzc"], defer_dlog_alpha=True) for e in ch]
            bwd_all += bl
            self.active_groups.append((fwd, b.problem_array(bl)))
        self.active_finish = b.problem_array(bwd_all)

    def step_active(self):
        b = self.b
        self.sample_gates()
        b.active_ranks_gather(self.active_gather)
        for fwd, bwd in self.active_groups:
            b.gated_lowrank_fwd_grouped(fwd)
            b.gated_lowrank_bwd_grouped(bwd)
        b.dlog_alpha_finish_grouped(self.active_finish)
        b.active_ranks_scatter(self.active_scatter)
        self.finish()

    def input_bytes(self) -> int:
        return sum(e["X"].numel() * 2 + e["dY"].numel() * 2 for e in self.mats)

    def run_matrix(self, e, ws=None):
        b = self.b
        z, dzd = self.z[e["lo"]:e["hi"]], self.dz_dla[e["lo"]:e["hi"]]
        b.gated_lowrank_fwd(e["X"], e["Q"], e["P"], z, e["Y"], e["H"], None)
        b.gated_lowrank_bwd(e["dY"], e["X"], e["Q"], e["P"], z, dzd, e["H"], e["dX"], e["dP"], e["dQ"],
                            self.dlog_alpha[e["lo"]:e["hi"]], self.ws if ws is None else ws)

    def sample_gates(self):
        # one launch for all gates of all layers; every rank uses the same (seed, offset): one mask per global batch.
        # The Philox offset lives on the device and is advanced on the device, so that a step captured in a
        # CUDA graph draws a fresh mask at every replay.
        self.b.gate_sample_devoff(self.log_alpha, HC, 0, 0, self.offset_dev, self.z, self.mask, self.dz_dla)
        self.offset_dev.add_(1 << 24)

    def finish(self, deferred=False):
        if deferred:
            self.b.dlog_alpha_finish_grouped(self.bwd_all)            # second stage of dlog_alpha, all matrices, one launch
        self.b.expected_l0_lagrangian(self.log_alpha, self.seg_off, self.seg_size, HC, self.target, self.lam,
                                      self.out4, None, self.dlog_alpha, self.ws_l0)
        if self.world > 1:
            from paper_1910_04732_b200 import dp
            if self.reducer is not None and self.reducer.pending:
                dp.allreduce_gradients([self.dlog_alpha])
                self.reducer.wait()                                   # the layer buckets started during the step
            else:
                dp.allreduce_gradients([self.wgrad, self.dlog_alpha])     # the one exchange step of the path

    def step(self):
        torch = self.torch
        self.sample_gates()
        if self.group > 0:
            if self.world > 1 and self.reducer is None:
                from paper_1910_04732_b200 import dp
                self.reducer = dp.BucketedReducer(self.wgrad, self.bucket_bounds)
            if not self.plain:
                self.b.scale_rows_grouped(self.scale)                 # diag(z) Q of every matrix: one launch per step
            for i, (fwd, bwd, bwd_chain, bwd_plain) in enumerate(self.groups):
                if self.chain:
                    self.b.gated_lowrank_fwd_chained(fwd, self.sync)
                    self.b.gated_lowrank_bwd_chained(bwd_chain, self.sync)
                else:
                    self.b.gated_lowrank_fwd_grouped(fwd)
                    self.b.gated_lowrank_bwd_grouped(bwd_plain if self.plain else bwd)
                if self.reducer is not None:
                    self.reducer.launch(i)                            # this layer's dP, dQ are final
        elif self.n_streams == 1:
            for e in self.mats:
                self.run_matrix(e)
        else:
            main = torch.cuda.current_stream()
            self.ev_gates.record(main)
            for s in self.streams:
                s.wait_event(self.ev_gates)
            for i, e in enumerate(self.mats):
                k = i % self.n_streams
                with torch.cuda.stream(self.streams[k]):
                    self.run_matrix(e, self.wss[k])
            for k, s in enumerate(self.streams):
                self.ev_done[k].record(s)
                main.wait_event(self.ev_done[k])
        self.finish(deferred=self.group > 0 and not self.chain and not self.plain)


def capture_step(job: Job, fn=None, stamps=None, acc=None):
    """One whole step captured in a CUDA graph (the library's launches, programmatic dependent
    launch edges included); replays cost one host call instead of ~25."""
    import torch
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    fn = job.step if fn is None else fn
    with torch.cuda.stream(side):
        fn()                            # every kernel configured before capture
        torch.cuda.synchronize()
        if stamps is not None:          # the captured GEMM launches carry pointers into `stamps`
            job.b.gemm_stamps_begin(stamps)
        with torch.cuda.graph(g, stream=side):
            fn()
            if stamps is not None and acc is not None:      # adds this replay's GEMM kernel time up on the device
                job.b.gemm_stamps_accumulate(stamps, acc)
        if stamps is not None:
            job.stamped = job.b.gemm_stamps_end()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    job.graph = g
    return g


def time_steps(job: Job, steps: int, world: int, use_graph: bool = False):
    """K steps between two synchronisation points, timed with CUDA events on the launching stream."""
    import torch
    run = job.graph.replay if (use_graph and job.graph is not None) else job.step
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        run()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.barrier()
        ms = float(t.item())
    return ms


def time_e2e(job: Job, steps: int, world: int):
    """The same step through the same grouped calls, fed from and drained to pinned host memory inside the timed
    region: every X and dY crosses PCIe on a copy stream, layer by layer ahead of the compute; Y and dX of every
    matrix, the flat weight-gradient buffer, dlog_alpha and the Lagrangian scalars come back on a second copy
    stream as soon as the layer that produced them is done."""
    import torch
    assert job.group > 0
    pin = lambda t: torch.empty(t.shape, dtype=t.dtype).pin_memory()
    host_in = [(e["X"].cpu().pin_memory(), e["dY"].cpu().pin_memory()) for e in job.mats]
    host_out = [(pin(e["Y"]), pin(e["dX"])) for e in job.mats]
    host_wgrad, host_dla, host_out4 = pin(job.wgrad), pin(job.dlog_alpha), pin(job.out4)
    h2d, d2h = torch.cuda.Stream(), torch.cuda.Stream()
    main = torch.cuda.current_stream()
    n_groups = len(job.groups)
    per = job.group
    ev_in = [torch.cuda.Event() for _ in range(n_groups)]
    ev_done = [torch.cuda.Event() for _ in range(n_groups)]
    ev_end = torch.cuda.Event()

    def one_step():
        h2d.wait_stream(main)                  # the previous step has consumed the device input buffers
        d2h.wait_stream(main)
        with torch.cuda.stream(h2d):
            for gi in range(n_groups):
                for k in range(gi * per, min((gi + 1) * per, len(job.mats))):
                    job.mats[k]["X"].copy_(host_in[k][0], non_blocking=True)
                    job.mats[k]["dY"].copy_(host_in[k][1], non_blocking=True)
                ev_in[gi].record(h2d)
        job.sample_gates()
        job.b.scale_rows_grouped(job.scale)
        for gi, (fwd, bwd, bwd_chain, bwd_plain) in enumerate(job.groups):
            main.wait_event(ev_in[gi])
            job.b.gated_lowrank_fwd_grouped(fwd)
            job.b.gated_lowrank_bwd_grouped(bwd)
            ev_done[gi].record(main)
            with torch.cuda.stream(d2h):
                d2h.wait_event(ev_done[gi])
                for k in range(gi * per, min((gi + 1) * per, len(job.mats))):
                    host_out[k][0].copy_(job.mats[k]["Y"], non_blocking=True)
                    host_out[k][1].copy_(job.mats[k]["dX"], non_blocking=True)
        job.finish(deferred=True)
        ev_end.record(main)
        with torch.cuda.stream(d2h):
            d2h.wait_event(ev_end)
            host_wgrad.copy_(job.wgrad, non_blocking=True)
            host_dla.copy_(job.dlog_alpha, non_blocking=True)
            host_out4.copy_(job.out4, non_blocking=True)
        main.wait_stream(d2h)                  # the step ends when its results are on the host

    one_step()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        one_step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    nbytes = lambda t: t.numel() * t.element_size()
    h2d_bytes = sum(nbytes(hx) + nbytes(hdy) for hx, hdy in host_in)
    d2h_bytes = sum(nbytes(y) + nbytes(dx) for y, dx in host_out) + nbytes(host_wgrad) + nbytes(host_dla) + nbytes(host_out4)
    assert np.isfinite(host_out4.numpy()).all()
    assert torch.isfinite(host_out[-1][0].float()).all() and torch.isfinite(host_wgrad.float()).all()
    returned = "Y and dX of every matrix, all weight gradients (dP, dQ), dlog_alpha, the four Lagrangian scalars"
    return ms, h2d_bytes, d2h_bytes, returned


# ----------------------------------------------------------------------------- oracle arm
def oracle_sample(w: I.Workload):
    """The fp64 oracle on a bounded sample: the matrices of layer 0 at the full token count
    (gate sample, forward, backward) plus the Lagrangian term over all gates of the model.
    Returns (seconds for the sample, description, threads used)."""
    from oracle import flop_oracle as O
    probs = [I.layer_problem(w, 0, i) for i in range(len(w.matrices))]
    offs, sizes, alphas = [0], [], []
    for l, i, m in w.all_matrices():
        alphas.append(I.log_alpha(w.alpha, m.r, 0, l, i)); offs.append(offs[-1] + m.r); sizes.append(m.d_in + m.d_out)
    alpha_all = np.concatenate(alphas)
    t0 = time.perf_counter()
    for i, p in enumerate(probs):
        z, mask, dzd = O.gate_sample(p["log_alpha"], *HC, seed=0, offset=I.gate_offset(0, i))
        O.gated_lowrank_fwd(p["X"], p["Q"], p["P"], z)
        O.gated_lowrank_bwd(p["dY"], p["X"], p["Q"], p["P"], z, dzd)
    O.expected_l0_lagrangian(alpha_all, offs, sizes, *HC, w.target, 0.3, 1.7)
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    return dt, f"layer 0 of {w.layers} ({len(probs)} matrices) at the full T={w.T}; step time = sample x {w.layers}", threads


def run_reference(args, w: I.Workload):
    """The oracle as it stands, on the host cores.  One timed step = the bounded sample (layer 0 at the full token
    count); the throughput of a full step is extrapolated from it (every layer has the same shapes) and labelled so."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    times = []
    for i in range(args.warmup + args.steps):
        dt, sample, threads = oracle_sample(w)
        if i >= args.warmup:
            times.append(dt)
    sample_s = float(np.mean(times))
    step_s = sample_s * w.layers
    value = w.T / step_s
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sample_s * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "extrapolated_from": f"a timed step is layer 0 of {w.layers} (all layers have the same shapes); value = T / (ms_per_step x {w.layers})",
            "ms_per_full_step_extrapolated": step_s * 1e3,
            "tflops": w.flops_per_step() / step_s / 1e12,
            "config": {"workload": w.name, "T": w.T, "layers": w.layers,
                       "matrices": [[m.name, m.d_in, m.d_out, m.r] for m in w.matrices]},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default="bert", choices=["bert", "sru", "txl"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-active", action="store_true", help="skip the extra active-rank-training measurement")
    ap.add_argument("--no-graph", action="store_true", help="issue every step from the host instead of replaying a CUDA graph")
    ap.add_argument("--chain", action="store_true", help="chained calls (one launch for the forward products, one for the backward pass of a layer, "
                    "ordered on the device) instead of the grouped calls (a launch per GEMM stage); measured slower on B200")
    ap.add_argument("--no-chain", action="store_true", help="(default) grouped calls")
    ap.add_argument("--plain", action="store_true", help="every backward call forms diag(z) Q and finishes dlog_alpha itself "
                    "(two more small launches per layer) instead of one launch per step for each")
    ap.add_argument("--group", type=int, default=-1, help="matrices per grouped call (0: one call per matrix; default: one layer)")
    ap.add_argument("--streams", type=int, default=1, help="streams over which independent matrices are issued")
    args = ap.parse_args()
    w = I.WORKLOADS[args.workload]
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        run_reference(args, w)
        return
    args.steps = 100 if args.steps is None else args.steps
    args.warmup = 10 if args.warmup is None else max(args.warmup, 3)

    import torch
    from paper_1910_04732_b200 import build as _build
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if rank == 0:
        _build.build()
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    from paper_1910_04732_b200 import binding as b
    b.load_library()

    group = len(w.matrices) if args.group < 0 else args.group
    job = Job(w, torch.device("cuda", local), seed=1234 + rank, n_streams=args.streams, group=group)
    job.world = world
    job.chain = bool(args.chain) and not args.no_chain
    job.plain = bool(args.plain)
    for _ in range(args.warmup):
        job.step()
    torch.cuda.synchronize()
    assert b.device_status() == b.OK

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    n0 = b.launch_count()
    job.step()
    launches = b.launch_count() - n0            # kernels of this library per step (the same inside a graph replay)
    use_graph = not args.no_graph and world == 1   # NCCL all-reduces stay outside graphs here
    stamps = torch.zeros(2 * 4096, dtype=torch.int64, device="cuda") if use_graph else None
    acc = torch.zeros(2, dtype=torch.int64, device="cuda") if use_graph else None
    if use_graph:
        capture_step(job, stamps=stamps, acc=acc)
        launches += 1                              # the stamp-adding kernel at the end of the captured step
        for _ in range(3):
            job.graph.replay()
        torch.cuda.synchronize()
        acc.zero_()
    torch.cuda.synchronize()
    ms = time_steps(job, args.steps, world, use_graph)
    # Roofline of the dominant kernels (the tensor-core GEMM launches).  Inside the replayed graph every launch
    # stamps %globaltimer when its first CTA passes the dependency wait and when its last CTA ends, and a one-block
    # kernel at the end of the captured step adds (end - start) of all of them to a device counter: the kernel time
    # comes from the very replays whose step time is the headline, with no host work in between.
    graph_gemm = None
    if use_graph:
        n_st, fl_st = job.stamped
        tot_ns, n_rep = (int(v) for v in acc.cpu().tolist())
        if os.environ.get("FLOP_BENCH_DUMP_STAMPS"):
            st = stamps[: 2 * n_st].view(n_st, 2).cpu().numpy()
            rel = (st - st[0, 0]) / 1e3
            print("stamps_us " + " ".join(f"[{a:.1f},{b:.1f}]" for a, b in rel[:16]), file=sys.stderr)
        if n_st > 0 and n_rep == args.steps and tot_ns > 0:
            km = tot_ns / 1e6 / n_rep
            graph_gemm = {"launches": n_st, "replays": n_rep, "kernel_ms_per_step": km, "step_ms_same_replays": ms / args.steps,
                          "tflops": fl_st / (km * 1e-3) / 1e12, "flops_per_step": fl_st}
            assert km <= ms / args.steps * 1.005, f"stamped kernel time {km:.3f} ms exceeds the step it was taken in"
    # the same launches issued eagerly with CUDA events recorded around every GEMM launch (no dependent-launch overlap)
    b.gemm_timing_begin()
    ms_timed_pass = time_steps(job, args.steps, world)
    gemm_ms, gemm_flops, gemm_launches = b.gemm_timing_end()
    clocks = sampler.stop() if rank == 0 else None
    assert b.device_status() == b.OK

    # Extra (not the headline): the same step computed on the active rank components only.
    active = None
    if world == 1 and not args.no_active:
        job.enable_active_ranks()
        for _ in range(3):
            job.step_active()
        torch.cuda.synchronize()
        run = job.step_active
        if use_graph:
            g_act = capture_step(job, job.step_active)
            run = g_act.replay
            job.graph = None
        k_steps = max(3, min(args.steps, 50))
        for _ in range(3):
            run()
        torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(k_steps):
            run()
        a1.record()
        torch.cuda.synchronize()
        act_ms = a0.elapsed_time(a1) / k_steps
        frac = float(job.mask.float().mean().item())
        active = {"ms_per_step": act_ms, "value": w.T / (act_ms / 1e3), "unit": "tokens/s",
                  "active_fraction_last_step": frac,
                  "note": "select + gather of the z>0 components (writing diag(z_c)Q_c too), dlog_alpha_c finish and scatter once per step for all matrices; grouped fwd/bwd per layer with device-side rank; same outputs as the dense step"}
        assert b.device_status() == b.OK

    e2e = None
    if not args.no_e2e and group > 0:
        e2e_steps = max(3, min(args.steps, 20))
        e2e_ms, h2d, d2h, returned = time_e2e(job, e2e_steps, world)
        e2e = {"value": w.T * world / (e2e_ms / e2e_steps / 1e3), "unit": "tokens/s", "ms_per_step": e2e_ms / e2e_steps,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "returned": returned,
               "path": "the grouped calls of the headline step (eager issue: copies and compute overlap layer by layer)"}

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    peaks, peak_kind = measured_peaks()
    step_ms = ms / args.steps
    tokens_s = w.T * world / (step_ms / 1e3)
    tflops = w.flops_per_step() * world / (step_ms / 1e3) / 1e12
    event_tflops = gemm_flops / (gemm_ms / 1e3) / 1e12 if gemm_ms > 0 else 0.0
    # Which measured peak bounds this run: the burst figure (a kernel timed alone, clocks near the maximum) while the
    # timed region is short or the sampled clock is above the clock the sustained figure was taken at; the sustained
    # figure (a seconds-long loop under the power cap) otherwise.
    timed_s = ms / 1e3
    clk_sustained = None
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            clk_sustained = float(json.load(f)["clocks_under_load"]["sm_mhz_median"])
    except Exception:
        pass
    sm_mhz = clocks.get("sm_mhz") if clocks else None
    use_burst = timed_s < 1.0 or (clk_sustained is not None and sm_mhz is not None and sm_mhz > clk_sustained * 1.05)
    peak = peaks["bf16_tflops"] if use_burst else peaks["bf16_tflops_sustained"]
    achieved = graph_gemm["tflops"] if graph_gemm is not None else event_tflops
    fracs = lambda tf: {"nominal_2250": tf / NOMINAL_BF16_TFLOPS, "measured_burst": tf / peaks["bf16_tflops"],
                        "measured_sustained": tf / peaks["bf16_tflops_sustained"]}
    traffic, traffic_note = roofline_traffic(w.name, group)
    line = {
        "metric": METRIC, "value": tokens_s, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "tflops": tflops, "step_frac_of_bf16_peak": fracs(tflops / world),
        "config": {"workload": w.name, "T": w.T, "layers": w.layers,
                   "matrices": [[m.name, m.d_in, m.d_out, m.r] for m in w.matrices],
                   "gates": job.n_gates, "weight_grad_dtype": "bf16", "parallelism": f"dp{world}", "streams": args.streams,
                   "matrices_per_grouped_call": group, "cuda_graph": bool(use_graph),
                   "calls": "chained" if job.chain else ("grouped, self-contained backward" if job.plain else "grouped; diag(z)Q and dlog_alpha second stage once per step"),
                   "l2": f"inputs larger than L2: {job.input_bytes() / 1e6:.0f} MB of X and dY per step, each matrix its own buffers"},
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                     "peak_kind": f"{peak_kind} {'burst' if use_burst else 'sustained'} cuBLAS bf16 (timed region {timed_s:.2f} s, median SM clock {sm_mhz} MHz; "
                                  f"burst {peaks['bf16_tflops']}, sustained {peaks['bf16_tflops_sustained']} at {clk_sustained} MHz)",
                     "frac_of": fracs(achieved),
                     "how": "sum of 2MNK of the GEMM launches / their device-stamped time inside the replayed graph, mean over the replays of a stamped pass"
                            if graph_gemm is not None else "sum of 2MNK of the GEMM launches / their CUDA-event time, eager issue",
                     "traffic": traffic, "traffic_note": traffic_note,
                     "kernel": "tc::gemm2_group_kernel (forward) / tc::gemm2_dual_kernel (backward): every GEMM launch of the step",
                     "launches_per_step": gemm_launches // args.steps,
                     "in_graph": graph_gemm,
                     # the same launches bracketed by CUDA events in an eagerly issued pass (events break the dependent-launch overlap)
                     "event_timed": {"tflops": event_tflops, "kernel_ms_per_step": gemm_ms / args.steps,
                                     "step_ms_same_pass": ms_timed_pass / args.steps, "frac_of": fracs(event_tflops)}},
        "clocks": clocks,
    }
    if e2e is not None:
        line["e2e"] = e2e
    if active is not None:
        line["active_rank_training"] = active
    if world == 1 and not args.no_cpu_baseline:
        dt, sample, threads = oracle_sample(w)
        line["cpu_baseline"] = {"value": w.T / (dt * w.layers), "unit": "tokens/s", "cores": threads, "kind": "oracle",
                                "sample": sample, "tflops": w.flops_per_step() / (dt * w.layers) / 1e12}
    print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
