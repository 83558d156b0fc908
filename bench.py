#!/usr/bin/env python
"""Benchmark of the FLOP gated low-rank hot path on B200.

One step = one pass of the whole hot path over one batch of synthetic input:
sample every gate of every layer (one launch), then for every factorized matrix
of every layer the gated forward (2 GEMMs) and backward (4 GEMMs + the fused
dlog_alpha reduction; grouped per layer into two forward and two backward launches), then the expected-L0 / Lagrangian term over all gates.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload bert|sru|txl] [--impl ours|reference]

Prints ONE JSON line.  `value` is tokens/s with inputs resident in HBM; `e2e`
is the same step fed from pinned host memory (H2D of every X and dY inside the
timed region, D2H of dlog_alpha and the Lagrangian scalars); `roofline` times
the tensor-core GEMM launches with CUDA events; `cpu_baseline` is the fp64
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
        g.manual_seed(seed)
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
        randn = lambda rows, cols, scale=1.0: (torch.randn(rows, r8(cols), generator=g, device=device) * scale).to(bf)[:, :cols]
        for (l, i, m), lo in zip(mats, offs):
            e = dict(m=m, lo=lo, hi=lo + m.r)
            e["X"], e["dY"] = randn(w.T, m.d_in), randn(w.T, m.d_out)
            e["Q"], e["P"] = randn(m.r, m.d_in, m.d_in ** -0.5), randn(m.d_out, m.r, m.r ** -0.5)
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
        n_per = group if group > 0 else len(self.mats)
        sizes_w = [e["dP"].shape[0] * r8(e["m"].r) + e["m"].r * r8(e["m"].d_in) for e in self.mats]
        self.bucket_bounds = [0]
        for i in range(0, len(sizes_w), n_per):
            self.bucket_bounds.append(self.bucket_bounds[-1] + sum(sizes_w[i:i + n_per]))
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
        """Buffers and argument arrays for training on the active components only (z_k > 0): per layer one
        gather, the grouped forward and backward with the rank read on the device, one scatter."""
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
        g = self.group if self.group > 0 else len(self.w.matrices)
        for i in range(0, len(self.mats), g):
            ch = self.mats[i:i + g]
            z = lambda e: self.z[e["lo"]:e["hi"]]
            gat = b.problem_array([b.active_gather_problem(z(e), self.dz_dla[e["lo"]:e["hi"]], e["P"], e["Q"], e["idx"], e["pos"],
                                                           e["k"], e["zc"], e["dzc"], e["Pc"], e["Qc"]) for e in ch])
            fwd = b.problem_array([b.fwd_problem(e["X"], e["Qc"], e["Pc"], e["zc"], e["Y"], e["H"], r_dev=e["k"]) for e in ch])
            bwd = b.problem_array([b.bwd_problem(e["dY"], e["X"], e["Qc"], e["Pc"], e["zc"], e["dzc"], e["H"], e["dX"], e["dPc"],
                                                 e["dQc"], e["dlac"], e["ws"], r_dev=e["k"]) for e in ch])
            sca = b.problem_array([b.active_scatter_problem(e["idx"], e["pos"], e["k"], e["m"].d_in, e["m"].d_out, e["m"].r,
                                                            e["dPc"], e["dQc"], e["dlac"], e["dP"], e["dQ"],
                                                            self.dlog_alpha[e["lo"]:e["hi"]]) for e in ch])
            self.active_groups.append((gat, fwd, bwd, sca))

    def step_active(self):
        b = self.b
        self.sample_gates()
        for gat, fwd, bwd, sca in self.active_groups:
            b.active_ranks_gather(gat)
            b.gated_lowrank_fwd_grouped(fwd)
            b.gated_lowrank_bwd_grouped(bwd)
            b.active_ranks_scatter(sca)
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


def capture_step(job: Job, fn=None, stamps=None):
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
    """The same step fed from pinned host memory: every X and dY crosses PCIe inside the timed
    region (copy stream, overlapped with compute), dlog_alpha and the Lagrangian scalars come back."""
    import torch
    host_in = [(e["X"].cpu().pin_memory(), e["dY"].cpu().pin_memory()) for e in job.mats]
    host_dla = torch.empty(job.n_gates, dtype=torch.float32).pin_memory()
    host_out4 = torch.empty(4, dtype=torch.float32).pin_memory()
    copy_stream = torch.cuda.Stream()
    main = torch.cuda.current_stream()
    events = [torch.cuda.Event() for _ in job.mats]

    def one_step():
        copy_stream.wait_stream(main)          # the previous step has consumed the device buffers
        with torch.cuda.stream(copy_stream):
            for (hx, hdy), e, ev in zip(host_in, job.mats, events):
                e["X"].copy_(hx, non_blocking=True)
                e["dY"].copy_(hdy, non_blocking=True)
                ev.record(copy_stream)
        job.sample_gates()
        for e, ev in zip(job.mats, events):
            main.wait_event(ev)
            job.run_matrix(e)
        job.finish()
        host_dla.copy_(job.dlog_alpha, non_blocking=True)
        host_out4.copy_(job.out4, non_blocking=True)

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
    h2d = sum(hx.numel() * 2 + hdy.numel() * 2 for hx, hdy in host_in)
    d2h = host_dla.numel() * 4 + 16
    assert np.isfinite(host_out4.numpy()).all()
    return ms, h2d, d2h


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
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    times = []
    for i in range(args.warmup + args.steps):
        dt, sample, threads = oracle_sample(w)
        if i >= args.warmup:
            times.append(dt)
    step_s = float(np.mean(times)) * w.layers
    value = w.T / step_s
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
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
                    "ordered on the device) instead of the grouped calls (a launch per GEMM stage); measured slower on B200, see profiles/")
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
    if use_graph:
        capture_step(job, stamps=stamps)
        for _ in range(3):
            job.graph.replay()
    torch.cuda.synchronize()
    ms = time_steps(job, args.steps, world, use_graph)
    # the GEMM launches of the last replayed step, timed on the device (%globaltimer stamps written by the kernels)
    graph_gemm = None
    if use_graph:
        n_st, fl_st = job.stamped
        st = stamps[: 2 * n_st].view(n_st, 2).cpu().numpy()
        dur_ns = float((st[:, 1] - st[:, 0]).clip(min=0).sum())
        if n_st > 0 and dur_ns > 0:
            graph_gemm = {"launches": n_st, "kernel_ms_per_step": dur_ns / 1e6, "tflops": fl_st / dur_ns / 1e3}
            if os.environ.get("FLOP_BENCH_DUMP_STAMPS"):
                rel = (st - st[0, 0]) / 1e3
                print("stamps_us " + " ".join(f"[{a:.1f},{b:.1f}]" for a, b in rel[:16]), file=sys.stderr)
    # second pass of the same steps with CUDA events around every tensor-core GEMM launch
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
                  "note": "gather z>0 components, grouped fwd/bwd with device-side rank, scatter; same outputs as the dense step"}
        assert b.device_status() == b.OK

    e2e = None
    if not args.no_e2e:
        e2e_ms, h2d, d2h = time_e2e(job, max(3, min(args.steps, 20)), world)
        e2e_steps = max(3, min(args.steps, 20))
        e2e = {"value": w.T * world / (e2e_ms / e2e_steps / 1e3), "unit": "tokens/s", "ms_per_step": e2e_ms / e2e_steps,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h}

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    peaks, peak_kind = measured_peaks()
    step_ms = ms / args.steps
    tokens_s = w.T * world / (step_ms / 1e3)
    tflops = w.flops_per_step() * world / (step_ms / 1e3) / 1e12
    gemm_tflops = gemm_flops / (gemm_ms / 1e3) / 1e12 if gemm_ms > 0 else 0.0
    # dram__bytes_read.sum + dram__bytes_write.sum of the GEMM launches of one bert layer, from the ncu capture
    # summarised under profiles/ (grouped calls of six matrices): mean per launch
    traffic = 118.6e6 if (w.name == "bert" and group == 6) else None
    line = {
        "metric": METRIC, "value": tokens_s, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "tflops": tflops, "pct_of_bf16_peak_nominal": 100.0 * tflops / world / NOMINAL_BF16_TFLOPS,
        "pct_of_bf16_peak_measured_sustained": 100.0 * tflops / world / peaks["bf16_tflops_sustained"],
        "config": {"workload": w.name, "T": w.T, "layers": w.layers,
                   "matrices": [[m.name, m.d_in, m.d_out, m.r] for m in w.matrices],
                   "gates": job.n_gates, "weight_grad_dtype": "bf16", "parallelism": f"dp{world}", "streams": args.streams, "matrices_per_grouped_call": group, "cuda_graph": bool(use_graph),
                   "l2": f"inputs larger than L2: {job.input_bytes() / 1e6:.0f} MB of X and dY per step, each matrix its own buffers"},
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "achieved": gemm_tflops, "peak": peaks["bf16_tflops_sustained"],
                     "unit": "TFLOP/s", "frac": gemm_tflops / peaks["bf16_tflops_sustained"], "traffic": traffic,
                     "traffic_note": "DRAM read+write bytes per GEMM launch, mean of the four launches of one layer (ncu capture in profiles/)" if traffic else None,
                     "peak_kind": f"{peak_kind} (sustained; burst {peaks['bf16_tflops']})",
                     "kernel": "tc::gemm2_group_kernel (forward) / tc::gemm2_dual_kernel (backward): every GEMM launch of the step",
                     "launches_per_step": gemm_launches // args.steps,
                     "kernel_ms_per_step": gemm_ms / args.steps, "step_ms_in_timed_pass": ms_timed_pass / args.steps,
                     "frac_of_nominal": gemm_tflops / NOMINAL_BF16_TFLOPS,
                     # the same launches inside the replayed graph, timed by device-side stamps (no event gaps, PDL overlap kept)
                     "in_graph": None if graph_gemm is None else dict(graph_gemm, frac=graph_gemm["tflops"] / peaks["bf16_tflops_sustained"])},
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
