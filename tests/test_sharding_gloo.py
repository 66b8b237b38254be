"""The N > 1 path on CPU: two gloo ranks shard the leading axis (the element range of x*sin(a*x+b), the
rows of a row DAG, the batch of the MLP), evaluate their shards, all-reduce what is a reduction over that
axis, and together reproduce the single-process result."""
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


def _rank_general(rank, world, port, which, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import interp      # stands in for the per-shard GPU evaluation in this CPU test
    desc, inputs, outs, feeds, extent = _case(which)
    lo, hi = sharding.shard_range(extent, rank, world)
    d = sharding.shard_desc(desc, extent, hi - lo)
    kinds = sharding.classify_outputs(desc, outs, extent)
    my = sharding.cut_feeds(desc, inputs, feeds, extent, lo, hi)

    def evaluate():
        r = interp.run_function(d, inputs, outs, my)
        return [torch.from_numpy(np.ascontiguousarray(np.atleast_1d(np.asarray(v, dtype=np.float64)))) for v in r]

    res = sharding.run_classified(evaluate, kinds, lambda t: dist.all_reduce(t), (hi - lo) / extent)
    for j, t in enumerate(res):
        np.save(os.path.join(out_dir, "%s_r%d_o%d.npy" % (which, rank, j)), t.numpy())
    dist.destroy_process_group()


def _case(which):
    from oracle import prune as oprune
    if which == "rows":
        R, C = 11, 24
        g, inputs, fetch = wl.random_row_dag(R, C, 3004, n_ops=48, n_fetch=2)
        wrts = [i for i in inputs if i in oprune.backward_marks(g.desc, fetch, inputs)]
        outs = fetch + g.grad(fetch, wrts)
        feeds = [a * np.float32(0.5) for a in wl.normal_feeds([g.shape(i) for i in inputs], 7)]
        return g.desc, inputs, outs, feeds, R
    batch = 10
    g, ids = wl.mlp(batch, 8, 16, 8)
    inputs = [ids[k] for k in ("X", "W1", "b1", "W2", "b2", "labels")]
    outs = [ids[k] for k in ("loss", "dW1", "db1", "dW2", "db2")]
    return g.desc, inputs, outs, list(wl.mlp_feeds(batch, 8, 16, 8, 5)), batch


def test_output_classes():
    desc, inputs, outs, feeds, R = _case("rows")
    kinds = sharding.classify_outputs(desc, outs, R)
    assert kinds[:2] == [sharding.LOCAL, sharding.LOCAL]
    assert sorted(set(kinds[2:])) in ([sharding.LOCAL, sharding.SUM], [sharding.LOCAL], [sharding.SUM])
    for o, k in zip(outs, kinds):
        assert (k == sharding.LOCAL) == (len(desc["tensors"][o]["shape"]) == 2)
    desc, inputs, outs, feeds, batch = _case("batch")
    assert sharding.classify_outputs(desc, outs, batch) == [sharding.MEAN] * 5
    g, ids = wl.toy_function_grad(100)
    assert sharding.classify_outputs(g.desc, [ids["f"], ids["dx"], ids["da"], ids["db"]], 100) == [sharding.LOCAL, sharding.LOCAL, sharding.SUM, sharding.SUM]


import pytest  # noqa: E402


@pytest.mark.parametrize("which", ["rows", "batch"])
def test_two_ranks_reproduce_row_and_batch_sharded_results(which, tmp_path):
    """Workload 5 split by rows (the [C] gradients are all-reduced) and workload 4 split by batch rows (loss and
    every gradient weighted by the rank's share and all-reduced): two ranks together equal one process (the
    batch halves, so the 1/M factors of the two runs differ by a power of two and the bf16 roundings agree)."""
    from oracle import interp
    world, port = 2, 31500 + os.getpid() % 2000 + (7 if which == "rows" else 0)
    mp.start_processes(_rank_general, args=(world, port, which, str(tmp_path)), nprocs=world, join=True, start_method="spawn")
    desc, inputs, outs, feeds, extent = _case(which)
    ref = interp.run_function(desc, inputs, outs, feeds)
    kinds = sharding.classify_outputs(desc, outs, extent)
    for j, (r, k) in enumerate(zip(ref, kinds)):
        parts = [np.load(tmp_path / ("%s_r%d_o%d.npy" % (which, rk, j))) for rk in range(world)]
        if k == sharding.LOCAL:
            got = np.concatenate(parts, axis=0)
            assert np.allclose(got, r, rtol=1e-12, atol=1e-12)
        else:
            for p in parts:          # every rank holds the reduced result
                tol = 1e-12 if which == "rows" else 1e-9
                assert np.allclose(p.reshape(np.shape(r)), r, rtol=tol, atol=tol * np.max(np.abs(r))), (j, k)
