"""Data-parallel decomposition of the layer on CPU (gloo, world_size 2): sharding by tokens with
one shared gate sample and one all-reduce of dP, dQ, dlog_alpha reproduces the full-batch gradients."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import flop_oracle as O
from paper_1910_04732_b200 import dp
from paper_1910_04732_b200 import inputs as I

HC = (I.BETA, I.GAMMA, I.ZETA)


def _worker(rank, world, port, T, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = I.Workload("dp", "f32", T, 1, (I.Matrix("w", 24, 40, 16),), ("normal", 0.5, 1.5), 0.5)
    prob = I.layer_problem(w, 0, 0, seed=3)
    seed, offset = dp.gate_stream(step=5)
    z, mask, dzd = O.gate_sample(prob["log_alpha"], *HC, seed=seed, offset=offset)      # same on every rank
    lo, cnt = dp.token_shard(T, rank, world)
    G = O.gated_lowrank_bwd(prob["dY"][lo:lo + cnt], prob["X"][lo:lo + cnt], prob["Q"], prob["P"], z, dzd)
    flat = torch.from_numpy(np.concatenate([G["dP"].ravel(), G["dQ"].ravel()]))
    dla = torch.from_numpy(G["dlog_alpha"].copy())
    dp.allreduce_gradients([flat, dla])
    masks = [torch.zeros(len(mask), dtype=torch.uint8) for _ in range(world)]
    dist.all_gather(masks, torch.from_numpy(mask.copy()))
    if rank == 0:
        full = O.gated_lowrank_bwd(prob["dY"], prob["X"], prob["Q"], prob["P"], z, dzd)
        want = np.concatenate([full["dP"].ravel(), full["dQ"].ravel()])
        ok = (np.allclose(flat.numpy(), want, rtol=1e-12, atol=1e-12)
              and np.allclose(dla.numpy(), full["dlog_alpha"], rtol=1e-12, atol=1e-12)
              and all(torch.equal(m, masks[0]) for m in masks))
        with open(out, "w") as f:
            f.write("ok" if ok else "mismatch")
    dist.barrier()
    dist.destroy_process_group()


def test_token_sharded_backward_with_one_allreduce(tmp_path):
    out = str(tmp_path / "result.txt")
    port = 29500 + (os.getpid() % 2000)
    mp.spawn(_worker, args=(2, port, 37, out), nprocs=2, join=True)      # 37 tokens: ranks get 19 and 18
    assert open(out).read() == "ok"


def test_token_shard_covers_every_token_once():
    for T, world in ((37, 2), (4096, 8), (5, 8), (0, 4)):
        spans = [dp.token_shard(T, r, world) for r in range(world)]
        assert spans[0][0] == 0 and sum(c for _, c in spans) == T
        for (s0, c0), (s1, _) in zip(spans, spans[1:]):
            assert s0 + c0 == s1
        assert max(c for _, c in spans) - min(c for _, c in spans) <= 1
    assert dp.gate_stream(3) == dp.gate_stream(3) and dp.gate_stream(3) != dp.gate_stream(4)


def _bucket_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g = torch.Generator().manual_seed(100 + rank)
    flat = torch.randn(1000, generator=g, dtype=torch.float64)
    mine = flat.clone()
    red = dp.BucketedReducer(flat, [0, 10, 10, 377, 1000])           # four buckets, one of them empty
    for i in reversed(range(red.n_buckets())):                       # backward order, as the layers finish
        red.launch(i)
    red.wait()
    parts = [torch.zeros(1000, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(parts, mine)
    if rank == 0:
        ok = torch.allclose(flat, sum(parts), rtol=0, atol=1e-12) and red.pending == []
        with open(out, "w") as f:
            f.write("ok" if ok else "mismatch")
    dist.barrier()
    dist.destroy_process_group()


def test_bucketed_reducer_sums_every_bucket(tmp_path):
    out = str(tmp_path / "bucket.txt")
    port = 31500 + (os.getpid() % 2000)
    mp.spawn(_bucket_worker, args=(2, port, out), nprocs=2, join=True)
    assert open(out).read() == "ok"


def test_bucketed_reducer_checks_bounds_and_is_a_no_op_alone():
    import pytest
    flat = torch.ones(8)
    for bad in ([1, 8], [0, 7], [0, 5, 3, 8]):
        with pytest.raises(ValueError):
            dp.BucketedReducer(flat, bad)
    red = dp.BucketedReducer(flat, [0, 4, 8])       # no process group: nothing to exchange
    red.launch(0); red.launch(1); red.wait()
    assert torch.equal(flat, torch.ones(8))
