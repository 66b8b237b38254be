"""The N > 1 path on CPU: two gloo ranks shard the element range of x*sin(a*x+b), evaluate their
shards, all-reduce the two summed gradients, and together reproduce the single-process result."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1707_08265_b200 import sharding
from paper_1707_08265_b200 import workloads as wl


def _rank_main(rank, world, port, n, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import interp      # stands in for the per-shard GPU evaluation in this CPU test
    x, a, b = wl.toy_feeds(n, 99)
    lo, hi = sharding.shard_range(n, rank, world)
    g, ids = wl.toy_function_grad(hi - lo)
    inputs, outs = [ids["x"], ids["a"], ids["b"]], [ids["dx"], ids["da"], ids["db"]]

    def evaluate():
        r = interp.run_function(g.desc, inputs, outs, [x[lo:hi], a, b])
        return [torch.from_numpy(np.atleast_1d(np.asarray(v, dtype=np.float64))) for v in r]

    res = sharding.run_sharded(evaluate, [1, 2], lambda t: dist.all_reduce(t))
    np.save(os.path.join(out_dir, "dx%d.npy" % rank), res[0].numpy())
    np.save(os.path.join(out_dir, "sums%d.npy" % rank), np.array([float(res[1]), float(res[2])]))
    dist.destroy_process_group()


def test_shard_ranges_tile_the_domain():
    for n in (1, 7, 4096, 100003):
        for world in (1, 2, 3, 8):
            edges = [sharding.shard_range(n, r, world) for r in range(world)]
            assert edges[0][0] == 0 and edges[-1][1] == n
            assert all(edges[r][1] == edges[r + 1][0] for r in range(world - 1))
            sizes = [hi - lo for lo, hi in edges]
            assert max(sizes) - min(sizes) <= 1


def test_two_ranks_reproduce_the_single_process_result(tmp_path):
    from oracle import interp
    n, world, port = 10007, 2, 29500 + os.getpid() % 2000
    mp.start_processes(_rank_main, args=(world, port, n, str(tmp_path)), nprocs=world, join=True, start_method="spawn")
    x, a, b = wl.toy_feeds(n, 99)
    g, ids = wl.toy_function_grad(n)
    dx, da, db = interp.run_function(g.desc, [ids["x"], ids["a"], ids["b"]], [ids["dx"], ids["da"], ids["db"]], [x, a, b])
    got_dx = np.concatenate([np.load(tmp_path / ("dx%d.npy" % r)) for r in range(world)])
    assert np.allclose(got_dx, dx, rtol=1e-15, atol=0)
    for r in range(world):
        s = np.load(tmp_path / ("sums%d.npy" % r))
        assert np.allclose(s, [float(da), float(db)], rtol=1e-12)
