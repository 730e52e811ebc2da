"""Data-parallel sharding of the three passes over the minibatch S, checked on CPU
with two gloo ranks: fprop and bprop of a shard are the matching slices of the full
result (no exchange), accGrad's sum over S is the all-reduce(sum) of the per-rank
partial weight gradients -- the one collective `bench.py --gpus N` performs."""
import os
import socket

import numpy as np
import pytest


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import torch
    import torch.distributed as dist
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    s = wl.ConvShape("dp", 6, 3, 4, 9, 8, 3, 2, 16, cfg=9, point=1)
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    lo, hi = wl.shard_range(s.S, rank, world)
    y_loc = oracle.fprop(x[lo:hi], w)
    dx_loc = oracle.bprop(dy[lo:hi], w, s.h, s.w)
    dw = torch.from_numpy(oracle.accgrad(dy[lo:hi], x[lo:hi], s.kh, s.kw))
    dist.all_reduce(dw)                       # sum over ranks = sum over S
    np.savez(os.path.join(out_dir, "rank%d.npz" % rank), y=y_loc, dx=dx_loc, dw=dw.numpy(),
             lo=lo, hi=hi)
    dist.barrier()
    dist.destroy_process_group()


def test_s_sharding_with_allreduce_matches_unsharded(tmp_path):
    import torch.multiprocessing as mp
    import oracle
    from paper_1412_7580_b200 import workloads as wl
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    s = wl.ConvShape("dp", 6, 3, 4, 9, 8, 3, 2, 16, cfg=9, point=1)
    x, w, dy = wl.make_x(s), wl.make_w(s), wl.make_dy(s)
    y, dx, dw = oracle.fprop(x, w), oracle.bprop(dy, w, s.h, s.w), oracle.accgrad(dy, x, s.kh, s.kw)
    covered = 0
    for r in range(world):
        d = np.load(os.path.join(str(tmp_path), "rank%d.npz" % r))
        lo, hi = int(d["lo"]), int(d["hi"])
        covered += hi - lo
        np.testing.assert_array_equal(d["y"], y[lo:hi])
        np.testing.assert_array_equal(d["dx"], dx[lo:hi])
        np.testing.assert_allclose(d["dw"], dw, rtol=0, atol=1e-12)
    assert covered == s.S


@pytest.mark.parametrize("S,world", [(128, 8), (7, 2), (1, 4), (16, 3)])
def test_shard_ranges_partition_the_batch(S, world):
    from paper_1412_7580_b200 import workloads as wl
    edges = [wl.shard_range(S, r, world) for r in range(world)]
    assert edges[0][0] == 0 and edges[-1][1] == S
    for (a, b), (c, d) in zip(edges, edges[1:]):
        assert b == c and a <= b
    sizes = [b - a for a, b in edges]
    assert max(sizes) - min(sizes) <= 1
