"""Two gloo ranks on CPU: sharding the vectors, all-reducing the EMA statistics and applying
the update on every rank gives the single-process update.  (The arithmetic here is the
oracle's; what is under test is the host-side sharding and reduction used with N GPUs.)"""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import oracle
    import rvq_synth
    from paper_2410_15704_b200.dist import allreduce_stats, shard_range, stats_buffer
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = rvq_synth.key_cache(tokens=24, size=64, depth=3)
    lo, hi = shard_range(w.n, rank, world)
    x = w.x[lo:hi]
    enc = oracle.encode(x, w.codebooks, 32, w.layout)
    cnt, sm = oracle.ema_stats(x, enc["codes"], w.codebooks, w.layout)
    # the flat buffer the GPU benchmark uses: counts and sums in one collective
    flat, tc, ts = stats_buffer(*sm.shape)
    flat = flat.double()
    R_, K_, gd_ = sm.shape
    tc, ts = flat[:R_ * K_].view(R_, K_), flat[R_ * K_:].view(R_, K_, gd_)
    tc.copy_(torch.from_numpy(cnt)); ts.copy_(torch.from_numpy(sm))
    allreduce_stats(flat)
    n2, m2, cb = oracle.ema_normalise(tc.numpy(), ts.numpy(), np.ones(cnt.shape), w.codebooks.astype(np.float64), 0.9, 1e-5)
    np.save(os.path.join(out_dir, f"cb{rank}.npy"), cb)
    np.save(os.path.join(out_dir, f"cnt{rank}.npy"), tc.numpy())
    dist.destroy_process_group()


def test_sharded_ema_equals_single_process(tmp_path):
    import oracle
    import rvq_synth
    from paper_2410_15704_b200.dist import shard_range
    assert [shard_range(10, r, 3) for r in range(3)] == [(0, 4), (4, 7), (7, 10)]
    assert [shard_range(2, r, 4) for r in range(4)] == [(0, 1), (1, 2), (2, 2), (2, 2)]
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    w = rvq_synth.key_cache(tokens=24, size=64, depth=3)
    enc = oracle.encode(w.x, w.codebooks, 32, w.layout)
    ref = oracle.ema_update(w.x, enc["codes"], w.codebooks, np.ones((3, 64)), w.codebooks.astype(np.float64), 0.9, 1e-5, w.layout)
    for r in range(world):
        np.testing.assert_array_equal(np.load(tmp_path / f"cnt{r}.npy"), ref["count"])
        np.testing.assert_allclose(np.load(tmp_path / f"cb{r}.npy"), ref["codebooks"], rtol=0, atol=1e-12)


def test_bench_launch_plan_starts_one_rank_per_gpu(monkeypatch):
    """`python bench.py --gpus N` outside torchrun re-launches itself as N ranks on 127.0.0.1;
    inside torchrun (WORLD_SIZE set), for one GPU and for the reference arm it runs in place."""
    sys.path.insert(0, ROOT)
    import argparse
    import bench
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    args = argparse.Namespace(gpus=4, steps=7, warmup=2, impl="ours", tokens=None, no_cpu_baseline=False)
    plan = bench.launch_plan(args, argv0="bench.py", port=29512)
    assert plan[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=4" in plan
    assert plan[plan.index("--master-addr") + 1] == "127.0.0.1" and plan[plan.index("--master-port") + 1] == "29512"
    tail = plan[plan.index("bench.py"):]
    assert tail == ["bench.py", "--gpus", "4", "--impl", "ours", "--steps", "7", "--warmup", "2"]
    assert bench.launch_plan(argparse.Namespace(**{**vars(args), "gpus": 1})) is None
    assert bench.launch_plan(argparse.Namespace(**{**vars(args), "impl": "reference"})) is None
    monkeypatch.setenv("WORLD_SIZE", "4")
    assert bench.launch_plan(args) is None
