"""The N > 1 path of bench.py on the CPU: the gradient buckets the benchmark builds for a workload (one per grouped
call, i.e. per layer) and the bucketed reducer, wired as bench.py wires them, on two gloo ranks."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1910_04732_b200 import dp
from paper_1910_04732_b200 import inputs as I


def bench_bucket_bounds(w: I.Workload, group: int):
    """Bucket bounds as bench.Job computes them (the same two helpers)."""
    return dp.bucket_bounds(dp.weight_gradient_sizes([m for _, _, m in w.all_matrices()]), group)


def test_bucket_bounds_of_the_bert_workload():
    w = I.WORKLOADS["bert"]
    bounds = bench_bucket_bounds(w, len(w.matrices))
    assert len(bounds) == w.layers + 1 == 13
    per_layer = 4 * 2 * 768 * 768 + 2 * (768 * 768 + 3072 * 768)
    assert all(b1 - b0 == per_layer for b0, b1 in zip(bounds, bounds[1:]))
    # ragged widths are padded to 8 elements per row
    txl = I.WORKLOADS["txl"]
    sizes = dp.weight_gradient_sizes([m for _, _, m in txl.all_matrices()][:1])
    assert sizes == [410 * 416 + 410 * 416]
    assert dp.bucket_bounds([3, 4, 5], 2) == [0, 7, 12] and dp.bucket_bounds([], 6) == [0]


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, bounds, n, out):
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g = torch.Generator().manual_seed(100 + rank)
    flat = torch.randn(n, generator=g)
    dla = torch.randn(97, generator=g)
    mine = flat.clone()
    red = dp.BucketedReducer(flat, bounds)
    for i in range(len(bounds) - 1):          # bench.Job.step(): a bucket is launched as soon as its layer's backward is issued
        red.launch(i)
    assert red.pending
    dp.allreduce_gradients([dla])             # bench.Job.finish(): dlog_alpha once per step, then wait for the buckets
    red.wait()
    gathered = [torch.zeros(n) for _ in range(world)]
    dist.all_gather(gathered, mine)
    want = sum(gathered)
    out[rank] = float((flat - want).abs().max())
    dist.destroy_process_group()


def test_twelve_layer_buckets_reduce_like_one_all_reduce():
    w = I.Workload("dp", "bf16", 64, 12, (I.Matrix("a", 16, 24, 8), I.Matrix("b", 24, 16, 8)), ("normal", 0.0, 1.0), 0.5)
    bounds = bench_bucket_bounds(w, len(w.matrices))
    assert len(bounds) == 13
    mgr = mp.Manager()
    out = mgr.dict()
    port = _free_port()
    mp.spawn(_worker, args=(2, port, bounds, bounds[-1], out), nprocs=2, join=True)
    assert out[0] < 1e-6 and out[1] < 1e-6
