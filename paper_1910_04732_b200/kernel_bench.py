"""Timing of the memory-bound kernels and of the pruned-inference path.

    python -m paper_1910_04732_b200.kernel_bench [--small]

The per-step gate vectors of the workloads are a few tens of thousands of elements
(launch-latency bound), so the HBM figures are taken on scaled inputs that are far
larger than L2: 2^26 gates for the sampler and the expected-L0 / Lagrangian term,
and a 65536 x 16384 factor pair for the rank gather.  Bytes are the algorithmic
bytes of each call (what must be read and written once), time is the mean of CUDA
event timings after warm-up.  The second table is the inference configuration:
compaction once, then the compact forward against the uncompacted gated forward
(both replayed from CUDA graphs so that host launch cost does not hide the kernels).
The third table is one training step of a BERT-shaped layer on the active rank
components only, against the dense gated step, for several fractions of open gates.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np
import torch

from . import binding as b
from . import build, inputs as I

HC = tuple(float(np.float32(v)) for v in (I.BETA, I.GAMMA, I.ZETA))


def timed(fn, iters=10, warmup=3, graph=False):
    """Mean seconds per call.  graph=True replays a captured CUDA graph of one call, which takes
    the host's launch cost (tens of microseconds from Python) out of microsecond-sized calls."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    if graph:
        g, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                fn()
        torch.cuda.current_stream().wait_stream(side)
        fn = g.replay
        fn()
        torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters * 1e-3


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--small", action="store_true", help="sizes for a profiler capture (a few hundred MB)")
    ap.add_argument("--only-membound", action="store_true", help="stop after the table of memory-bound kernels")
    args = ap.parse_args()
    build.build()
    b.load_library()
    peak = 6650.0
    try:
        peak = float(json.load(open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))),
                                                 "MEASURED_PEAKS.json")))["hbm_gbs"])
    except Exception:
        pass
    rows = []
    g = torch.Generator(device="cuda"); g.manual_seed(0)

    # ---- gate sampler: 4 B read + 4 + 4 + 1 B written per gate
    n = 1 << (25 if args.small else 26)
    la = torch.randn(n, generator=g, device="cuda") * 1.5 + 1.0
    z, d, m = torch.empty(n, device="cuda"), torch.empty(n, device="cuda"), torch.empty(n, dtype=torch.uint8, device="cuda")
    t = timed(lambda: b.gate_sample(la, HC, 0, 0, z, m, d))
    rows.append(("gate_sample_kernel", f"n = 2^{n.bit_length() - 1} gates", 13 * n, t))

    # ---- expected L0 + Lagrangian with gradient: 4 B (pass 1) + 4 + 8 B (pass 2) per gate
    n_seg = 64
    off = torch.linspace(0, n, n_seg + 1).round().to(torch.int64).cuda()
    size = torch.rand(n_seg, generator=g, device="cuda") * 4000 + 500
    tg, lm = torch.tensor([0.3], device="cuda"), torch.tensor([0.3, 1.7], device="cuda")
    out4, dla = torch.empty(4, device="cuda"), torch.zeros(n, device="cuda")
    ws = b.alloc_workspace(b.workspace_bytes(b.OP_L0, n, 0, 0, n_seg, b.F32))
    t = timed(lambda: b.expected_l0_lagrangian(la, off, size, HC, tg, lm, out4, None, dla, ws))
    rows.append(("l0_chunk_kernel<0>+finalize+<1>", f"n = 2^{n.bit_length() - 1} gates, {n_seg} segments", 16 * n, t))
    t = timed(lambda: b.expected_l0_lagrangian(la, off, size, HC, tg, lm, out4, None, None, ws))
    rows.append(("l0_chunk_kernel<0>+finalize (no gradient)", "same", 4 * n, t))
    del z, d, m, dla

    # ---- rank compaction and gather, ~35 % of the components survive
    r, d_in, d_out = (16384, 4096, 8192) if args.small else (16384, 16384, 65536)
    a = torch.where(torch.rand(r, generator=g, device="cuda") < 0.35, 4.0, -4.0) + 0.1 * torch.randn(r, generator=g, device="cuda")
    P = torch.randn(d_out, r, generator=g, device="cuda", dtype=torch.float32).bfloat16()
    Q = torch.randn(r, d_in, generator=g, device="cuda", dtype=torch.float32).bfloat16()
    Pc, Qc = torch.empty_like(P), torch.empty_like(Q)
    idx, kd, zd = torch.empty(r, dtype=torch.int32, device="cuda"), torch.zeros(1, dtype=torch.int32, device="cuda"), torch.empty(r, device="cuda")
    t_sel = timed(lambda: b.compact_ranks(a, 0, HC, idx, kd, zd))
    t_all = timed(lambda: b.compact_ranks(a, 0, HC, idx, kd, zd, P, Q, Pc, Qc))
    k = int(kd.item())
    rows.append(("compact_select_kernel", f"r = {r}", 4 * r * 6, t_sel))
    rows.append(("gather_p_pipe_kernel + gather_q_kernel", f"r = {r}, d_in = {d_in}, d_out = {d_out}, k = {k}",
                 2 * d_out * r + 2 * k * d_out + 4 * k * d_in + 4 * r, t_all - t_sel))
    del P, Q, Pc, Qc

    # ---- diag(z) Q of every matrix of a model in one launch: 2 B read + 2 B written per element
    wl = I.WORKLOADS["bert"]
    reps = 1 if args.small else 4          # four models' worth of matrices: 255 MB read, 255 MB written (beyond L2)
    qs = []
    for _ in range(reps):
        for _, _, mm in wl.all_matrices():
            q = torch.randn(mm.r, mm.d_in, generator=g, device="cuda").bfloat16()
            qs.append((q, torch.rand(mm.r, generator=g, device="cuda"), torch.empty_like(q)))
    arr = b.problem_array([b.scale_rows_problem(q, zz, o) for q, zz, o in qs])
    t = timed(lambda: b.scale_rows_grouped(arr))
    rows.append(("scale_rows_group_kernel", f"{len(qs)} bert-shaped factors Q (r x d_in)", sum(4 * q.numel() for q, _, _ in qs), t))
    del qs

    print(f"HBM peak used: {peak:.0f} GB/s (measured copy); 'of 8 TB/s' = against the nominal figure\n")
    print(f"{'kernel(s)':44s} {'size':58s} {'MB':>9s} {'us':>9s} {'GB/s':>8s} {'of peak':>8s} {'of 8 TB/s':>10s}")
    for name, what, nbytes, t in rows:
        print(f"{name:44s} {what:58s} {nbytes / 1e6:9.1f} {t * 1e6:9.1f} {nbytes / t / 1e9:8.0f} {nbytes / t / 1e9 / peak:8.2f} {nbytes / t / 1e9 / 8000.0:10.2f}")

    if args.only_membound:
        return

    # ---- pruned inference: d_in = 1024, d_out = 4096, r = 1024, ~35 % survive
    w = I.WORKLOADS["infer"]
    mtx = w.matrices[0]
    prob = I.layer_problem(w, 0, 0, T=4096)
    bf = torch.bfloat16

    def dev(x):
        t_ = b.padded(x.shape[0], x.shape[1], bf)
        t_.copy_(torch.from_numpy(x).to(bf))
        return t_
    P, Q, X = dev(prob["P"]), dev(prob["Q"]), dev(prob["X"])
    la = torch.from_numpy(prob["log_alpha"]).cuda()
    idx, kd, zd = torch.empty(mtx.r, dtype=torch.int32, device="cuda"), torch.zeros(1, dtype=torch.int32, device="cuda"), torch.empty(mtx.r, device="cuda")
    Pc, Qc = b.padded(mtx.d_out, mtx.r, bf), b.padded(mtx.r, mtx.d_in, bf)
    t_c = timed(lambda: b.compact_ranks(la, 0, HC, idx, kd, zd, P, Q, Pc, Qc))
    k = int(kd.item())
    print(f"\npruned inference, d_in={mtx.d_in} d_out={mtx.d_out} r={mtx.r}: k = {k} survive; compaction (select + gather) {t_c * 1e6:.1f} us")
    print(f"{'T':>6s} {'compact fwd us':>15s} {'on-chip chain us':>17s} {'gated fwd us':>13s} {'speed-up':>9s} {'compact GFLOP/s':>16s} {'weight GB/s':>12s}")
    for T in (1, 4, 8, 16, 17, 64, 256, 1024, 4096, 16384):
        Xt = X[:T] if T <= X.shape[0] else torch.cat([X] * (T // X.shape[0]))
        Y, H = b.padded(T, mtx.d_out, bf), b.padded(T, mtx.r, bf)
        wsc = b.alloc_workspace(b.workspace_bytes(b.OP_COMPACT_FWD, T, mtx.d_in, mtx.d_out, k, b.BF16))
        tc_ = timed(lambda: b.compact_fwd(Xt, Qc[:k], Pc[:, :k], Y, k, wsc), iters=50, graph=True)
        # the same product through the on-chip chain (one launch, H' in shared memory), whatever compact_fwd chose
        tch = timed(lambda: b.chain_fwd(Xt, Qc[:k], Pc[:, :k], None, Y), iters=50, graph=True) if k <= 512 else float("nan")
        tg_ = timed(lambda: b.gated_lowrank_fwd(Xt, Q, P, zd, Y, H, None), iters=50, graph=True)
        flops = 2.0 * T * k * (mtx.d_in + mtx.d_out)
        wbytes = 2.0 * k * (mtx.d_in + mtx.d_out)
        print(f"{T:6d} {tc_ * 1e6:15.1f} {tch * 1e6:17.1f} {tg_ * 1e6:13.1f} {tg_ / tc_:9.2f} {flops / tc_ / 1e9:16.0f} {wbytes / tc_ / 1e9:12.0f}")
    library_table(g)
    # ---- training on the active rank components: one BERT-shaped layer (six matrices, T = 4096)
    for wl in ("bert", "sru"):
        active_table(I.WORKLOADS[wl], g)
    embedding_table(g)
    assert b.device_status() == b.OK


def library_table(g):
    """Context for the roofline denominators: the six products of every matrix of one layer issued one by one through
    the vendor library (torch.matmul on the same bf16 tensors, outputs preallocated, replayed from a CUDA graph; no
    gate, no dlog_alpha), beside this library's grouped forward + backward of the same layer.  The measured bf16 peak
    is the library's rate on an 8192^3 product; this is its rate on the products this path is made of."""
    bf = torch.bfloat16
    print("\none layer, forward + backward: this library's grouped calls against the six products per matrix through torch.matmul")
    print(f"{'workload':>9s} {'grouped us':>11s} {'TFLOP/s':>8s} {'torch.matmul us':>16s} {'TFLOP/s':>8s}")
    for name in ("bert", "txl", "sru"):
        w = I.WORKLOADS[name]
        T = w.T
        es = []
        for m in w.matrices:
            r8 = lambda v: (v + 7) // 8 * 8
            rnd = lambda a, c: torch.randn(a, r8(c), generator=g, device="cuda").to(bf)[:, :c]
            e = dict(m=m, X=rnd(T, m.d_in), dY=rnd(T, m.d_out), Q=rnd(m.r, m.d_in), P=rnd(m.d_out, m.r),
                     z=torch.rand(m.r, device="cuda"), dzd=torch.rand(m.r, device="cuda"))
            e["Y"], e["H"], e["dX"] = (b.padded(T, c, bf) for c in (m.d_out, m.r, m.d_in))
            e["dH"], e["dP"], e["dQ"] = b.padded(T, m.r, bf), b.padded(m.d_out, m.r, bf), b.padded(m.r, m.d_in, bf)
            e["dla"] = torch.zeros(m.r, device="cuda")
            e["ws"] = b.alloc_workspace(b.workspace_bytes(b.OP_BWD, T, m.d_in, m.d_out, m.r, b.BF16))
            es.append(e)
        fwd = b.problem_array([b.fwd_problem(e["X"], e["Q"], e["P"], e["z"], e["Y"], e["H"]) for e in es])
        bwd = b.problem_array([b.bwd_problem(e["dY"], e["X"], e["Q"], e["P"], e["z"], e["dzd"], e["H"], e["dX"], e["dP"], e["dQ"],
                                             e["dla"], e["ws"]) for e in es])

        def ours():
            b.gated_lowrank_fwd_grouped(fwd)
            b.gated_lowrank_bwd_grouped(bwd)

        def library():
            for e in es:
                torch.matmul(e["X"], e["Q"].t(), out=e["H"])
                torch.matmul(e["H"], e["P"].t(), out=e["Y"])
                torch.matmul(e["dY"], e["P"], out=e["dH"])
                torch.matmul(e["dY"].t(), e["H"], out=e["dP"])
                torch.matmul(e["dH"].t(), e["X"], out=e["dQ"])
                torch.matmul(e["dH"], e["Q"], out=e["dX"])
        t_o = timed(ours, iters=20, graph=True)
        t_l = timed(library, iters=20, graph=True)
        flops = sum(6.0 * T * m.r * (m.d_in + m.d_out) for m in w.matrices)
        print(f"{name:>9s} {t_o * 1e6:11.1f} {flops / t_o / 1e12:8.0f} {t_l * 1e6:16.1f} {flops / t_l / 1e12:8.0f}")
        del es
        torch.cuda.empty_cache()


def embedding_table(g):
    """Gated adaptive embedding: the three word clusters of the word-level model (reduced dimensions
    1024 / 256 / 64 for the 20K most frequent, the next 40K and the remaining words; d = 1024),
    T = 64 x 256 tokens drawn with a heavy-tailed frequency."""
    bf = torch.bfloat16
    T, d = 64 * 256, 1024
    print(f"\ngated adaptive embedding, T={T} tokens, d={d} (lookup E[ids]*z, projection O; backward dO, dE, dlog_alpha)")
    print(f"{'cluster':>22s} {'fwd us':>8s} {'bwd us':>8s} {'fwd+bwd TFLOP/s':>16s}")
    for n_rows, d_i in ((20000, 1024), (40000, 256), (200000, 64)):
        E = (torch.randn(n_rows, d_i, generator=g, device="cuda")).to(bf)
        O_ = (torch.randn(d_i, d, generator=g, device="cuda") * d_i ** -0.5).to(bf)
        dY = torch.randn(T, d, generator=g, device="cuda").to(bf)
        ids = (torch.rand(T, generator=g, device="cuda") ** 4 * n_rows).to(torch.int32).clamp_(0, n_rows - 1)
        z = (torch.rand(d_i, generator=g, device="cuda") < 0.6).float() * 0.8
        dzd = torch.ones(d_i, device="cuda")
        Y, H = b.padded(T, d, bf), b.padded(T, d_i, bf)
        dE, dO, dla = torch.zeros(n_rows, d_i, device="cuda"), b.padded(d_i, d, bf), torch.zeros(d_i, device="cuda")
        ws = b.alloc_workspace(b.workspace_bytes(b.OP_EMBEDDING_BWD, T, 0, 0, d_i, b.BF16))
        tf = timed(lambda: b.gated_embedding_fwd(ids, E, O_, z, Y, H), iters=20, graph=True)
        tb = timed(lambda: b.gated_embedding_bwd(dY, ids, E, O_, z, dzd, H, dE, dO, dla, ws), iters=20, graph=True)
        flops = 6.0 * T * d_i * d          # one forward and two backward GEMMs
        print(f"{f'n={n_rows}, d_i={d_i}':>22s} {tf * 1e6:8.1f} {tb * 1e6:8.1f} {flops / (tf + tb) / 1e12:16.0f}")


def active_table(w, g):
    bf = torch.bfloat16
    T = w.T
    es = []
    for mtx in w.matrices:
        e = dict(m=mtx)
        rn = lambda rows, cols, sc=1.0: (torch.randn(rows, cols, generator=g, device="cuda") * sc).to(bf)
        e["X"], e["dY"] = rn(T, mtx.d_in), rn(T, mtx.d_out)
        e["Q"], e["P"] = rn(mtx.r, mtx.d_in, mtx.d_in ** -0.5), rn(mtx.d_out, mtx.r, mtx.r ** -0.5)
        e["z"], e["dzd"] = torch.zeros(mtx.r, device="cuda"), torch.ones(mtx.r, device="cuda")
        for name, rows, cols in (("H", T, mtx.r), ("Y", T, mtx.d_out), ("dX", T, mtx.d_in), ("dP", mtx.d_out, mtx.r),
                                 ("dQ", mtx.r, mtx.d_in), ("Pc", mtx.d_out, mtx.r), ("Qc", mtx.r, mtx.d_in),
                                 ("dPc", mtx.d_out, mtx.r), ("dQc", mtx.r, mtx.d_in)):
            e[name] = b.padded(rows, cols, bf)
        for name in ("dla", "zc", "dzc", "dlac"):
            e[name] = torch.zeros(mtx.r, device="cuda")
        e["idx"], e["pos"] = (torch.zeros(mtx.r, dtype=torch.int32, device="cuda") for _ in range(2))
        e["k"] = torch.zeros(1, dtype=torch.int32, device="cuda")
        e["ws"] = b.alloc_workspace(b.workspace_bytes(b.OP_BWD, T, mtx.d_in, mtx.d_out, mtx.r, b.BF16))
        es.append(e)
    fwd_d = b.problem_array([b.fwd_problem(e["X"], e["Q"], e["P"], e["z"], e["Y"], e["H"]) for e in es])
    bwd_d = b.problem_array([b.bwd_problem(e["dY"], e["X"], e["Q"], e["P"], e["z"], e["dzd"], e["H"], e["dX"], e["dP"], e["dQ"],
                                           e["dla"], e["ws"]) for e in es])
    gat = b.problem_array([b.active_gather_problem(e["z"], e["dzd"], e["P"], e["Q"], e["idx"], e["pos"], e["k"], e["zc"], e["dzc"],
                                                   e["Pc"], e["Qc"]) for e in es])
    fwd_a = b.problem_array([b.fwd_problem(e["X"], e["Qc"], e["Pc"], e["zc"], e["Y"], e["H"], r_dev=e["k"]) for e in es])
    bwd_a = b.problem_array([b.bwd_problem(e["dY"], e["X"], e["Qc"], e["Pc"], e["zc"], e["dzc"], e["H"], e["dX"], e["dPc"], e["dQc"],
                                           e["dlac"], e["ws"], r_dev=e["k"]) for e in es])
    sca = b.problem_array([b.active_scatter_problem(e["idx"], e["pos"], e["k"], e["m"].d_in, e["m"].d_out, e["m"].r, e["dPc"],
                                                    e["dQc"], e["dlac"], e["dP"], e["dQ"], e["dla"]) for e in es])

    def dense():
        b.gated_lowrank_fwd_grouped(fwd_d)
        b.gated_lowrank_bwd_grouped(bwd_d)

    def active_step():
        b.active_ranks_gather(gat)
        b.gated_lowrank_fwd_grouped(fwd_a)
        b.gated_lowrank_bwd_grouped(bwd_a)
        b.active_ranks_scatter(sca)

    print(f"\ntraining on the active rank components, one {w.name}-shaped layer ({len(es)} matrices, T={T}), graph replay")
    print(f"{'open gates':>11s} {'dense us':>9s} {'active us':>10s} {'speed-up':>9s}   (active = select + gather + fwd + bwd + scatter)")
    for frac in (1.0, 0.6, 0.3, 0.15, 0.05):
        for e in es:
            e["z"].copy_((torch.rand(e["m"].r, generator=g, device="cuda") < frac).float() * 0.7)
        td = timed(dense, iters=20, graph=True)
        ta = timed(active_step, iters=20, graph=True)
        print(f"{frac:11.2f} {td * 1e6:9.1f} {ta * 1e6:10.1f} {td / ta:9.2f}")


if __name__ == "__main__":
    main()
