"""The five benchmark workloads at full size on the GPU, against the oracle.

Where the oracle cannot evaluate the whole tensor in seconds, it is evaluated on sampled elements
(elementwise graphs) or sampled rows (row-reduction graph: rows are independent), and reductions
over all elements are checked at full size where the oracle can afford it."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import interp, prune as oprune
from paper_1707_08265_b200 import binding as B
from paper_1707_08265_b200 import workloads as wl
from test_gpu_vm import run_gpu, check, TOL32, TOLBF, to_dev

pytestmark = pytest.mark.gpu
SEEDS = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "config_seeds.json")))


def test_config1_toy_forward_two_targets():
    n = 1 << 20
    g, ids = wl.toy_function(n)
    x, a, b = wl.toy_feeds(n, wl.BASE_SEED + 1)
    inputs = [ids["x"], ids["a"], ids["b"]]
    (y,), f = run_gpu(g.desc, inputs, [ids["y"]], [x, a, None])
    want = oprune.function_sets(g.desc, inputs, [ids["y"]])
    assert f.marked() == want["marked"] and f.kept_ops()[0] == want["fwd_ops"] == [0]
    assert f.used_inputs() == [1, 1, 0]                                        # b, Add and Sin are gone
    check(y, interp.run_function(g.desc, inputs, [ids["y"]], [x, a, None])[0], TOL32, "y")
    (fv, y2), f2 = run_gpu(g.desc, inputs, [ids["f"], ids["y"]], [x, a, b])
    rf, ry = interp.run_function(g.desc, inputs, [ids["f"], ids["y"]], [x, a, b])
    assert all(f2.marked()[:7])
    check(fv, rf, TOL32, "f")
    check(y2, ry, TOL32, "y")


def test_config2_toy_gradients_full_size():
    n = 1 << 26
    g, ids = wl.toy_function_grad(n)
    x, a, b = wl.toy_feeds(n, wl.BASE_SEED + 2)
    inputs = [ids["x"], ids["a"], ids["b"]]
    outs = [ids["dx"], ids["da"], ids["db"]]
    got, f = run_gpu(g.desc, inputs, outs, [x, a, b])
    want = oprune.function_sets(g.desc, inputs, outs)
    fwd, gops, masks = f.kept_ops()
    assert f.marked() == want["marked"] and fwd == want["fwd_ops"] and gops == [k for (_, k, _) in want["grad_ops"]]
    ref = interp.run_function(g.desc, inputs, outs, [x, a, b])
    for gv, rv, name in zip(got, ref, ("dx", "da", "db")):
        check(gv, rv, TOL32, name)
    xd, ad, bd = x.astype(np.float64), float(a), float(b)
    u = ad * xd + bd
    check(got[0], np.sin(u) + ad * xd * np.cos(u), TOL32, "dx closed form")
    check(got[1], np.sum(xd * xd * np.cos(u)), TOL32, "da closed form")
    check(got[2], np.sum(xd * np.cos(u)), TOL32, "db closed form")


def test_config3_random_elementwise_dag_full_size():
    n = 1 << 27
    seed = SEEDS["random_dag"]["seed"]
    g, inputs, fetch = wl.random_dag(n, seed)
    want = oprune.function_sets(g.desc, inputs, fetch)
    gpu_in = [torch.empty(n, dtype=torch.float32, device="cuda").normal_(generator=torch.Generator("cuda").manual_seed(seed + k))
              for k in range(4)]
    outs = [torch.full((n,), float("nan"), dtype=torch.float32, device="cuda") for _ in fetch]
    f = B.Graph.from_desc(g.desc).function(inputs, fetch)
    assert f.marked() == want["marked"] and f.kept_ops()[0] == want["fwd_ops"] and f.used_inputs() == want["used_inputs"]
    f.run_torch([t if u else None for t, u in zip(gpu_in, f.used_inputs())], outs)
    assert f.status() == 0
    torch.cuda.synchronize()
    # elementwise graph: the oracle evaluates a sample of positions (several whole tiles, the tail,
    # and scattered elements) on the very same input values
    rng = np.random.default_rng(0)
    idx = np.unique(np.concatenate([np.arange(0, 3 * 4096), np.arange(n - 4099, n), rng.integers(0, n, 1 << 18)]))
    tidx = torch.from_numpy(idx).cuda()
    sample = [t[tidx].cpu().numpy() for t in gpu_in]
    gs, _, fs = wl.random_dag(idx.size, seed)
    ref = interp.run_function(gs.desc, inputs, fs, sample)
    for o, r in zip(outs, ref):
        assert torch.isfinite(o).all()
        check(o[tidx].cpu().numpy().astype(np.float64), r, TOL32, "config 3")


def test_config4_mlp_full_size():
    batch, d = 8192, 4096
    g, ids = wl.mlp(batch, d, d, d)
    feeds = list(wl.mlp_feeds(batch, d, d, d, wl.BASE_SEED + 4))
    inputs = [ids[k] for k in ("X", "W1", "b1", "W2", "b2", "labels")]
    outs = [ids[k] for k in ("loss", "dW1", "db1", "dW2", "db2")]
    got, f = run_gpu(g.desc, inputs, outs, feeds)
    want = oprune.function_sets(g.desc, inputs, outs)
    fwd, gops, masks = f.kept_ops()
    assert f.marked() == want["marked"] and fwd == want["fwd_ops"] and gops == [k for (_, k, _) in want["grad_ops"]]
    assert f.marked()[ids["side"]] == 0 and f.describe().count("gemm") == 5
    ref = interp.run_function(g.desc, inputs, outs, feeds)       # about 1.4e12 fp64 flop through BLAS
    for gv, rv, name in zip(got, ref, ("loss", "dW1", "db1", "dW2", "db2")):
        check(gv, rv, TOLBF, name)
        scale = np.max(np.abs(rv))
        assert np.max(np.abs(gv - rv)) <= 0.03 * scale + 1e-12, (name, np.max(np.abs(gv - rv)), scale)


def test_config5_row_dag_full_size():
    rows, cols = 16384, 4096
    seed = SEEDS["random_row_dag"]["seed"]
    g, inputs, fetch = wl.random_row_dag(rows, cols, seed)
    G = oprune.backward_marks(g.desc, fetch, inputs)
    wrts = [i for i in inputs if i in G]
    grads = g.grad(fetch, wrts)
    outs_ids = fetch + grads
    want = oprune.function_sets(g.desc, inputs, outs_ids)
    f = B.Graph.from_desc(g.desc).function(inputs, outs_ids)
    fwd, gops, masks = f.kept_ops()
    assert f.marked() == want["marked"] and fwd == want["fwd_ops"] and gops == [k for (_, k, _) in want["grad_ops"]]
    assert masks == [sum(1 << p for p in pos) for (_, _, pos) in want["grad_ops"]]
    gen = torch.Generator("cuda").manual_seed(seed)
    gpu_in = [torch.empty(tuple(g.shape(i)), dtype=torch.float32, device="cuda").normal_(generator=gen) for i in inputs]
    outs = [torch.full(tuple(g.shape(o)), float("nan"), dtype=torch.float32, device="cuda") for o in outs_ids]
    f.run_torch([t if u else None for t, u in zip(gpu_in, f.used_inputs())], outs)
    assert f.status() == 0
    torch.cuda.synchronize()
    # rows are independent (row sums stay inside a row): the oracle evaluates a subset of rows on
    # the same values; FULL-shaped outputs of those rows must match
    pick = np.unique(np.concatenate([[0, 1, rows - 1], np.random.default_rng(1).integers(0, rows, 29)]))
    sub_feeds = [t[torch.from_numpy(pick).cuda()].cpu().numpy() if t.dim() == 2 else t.cpu().numpy() for t in gpu_in]
    gs, in_s, fetch_s = wl.random_row_dag(len(pick), cols, seed)
    grads_s = gs.grad(fetch_s, wrts)
    ref = interp.run_function(gs.desc, in_s, fetch_s + grads_s, sub_feeds)
    for o, r, t in zip(outs, ref, outs_ids):
        assert torch.isfinite(o).all()
        if o.dim() == 2:
            check(o[torch.from_numpy(pick).cuda()].cpu().numpy().astype(np.float64), r, TOL32, "config 5 tensor %d" % t)
    # gradients of the [cols] inputs sum over all rows: checked against the oracle on a reduced row
    # count (the first 256 rows of the same inputs), where the oracle can afford every row
    r2 = 256
    g2, in2, fetch2 = wl.random_row_dag(r2, cols, seed)
    grads2 = g2.grad(fetch2, wrts)
    small_in = [t[:r2].contiguous() if t.dim() == 2 else t for t in gpu_in]
    f2 = B.Graph.from_desc(g2.desc).function(in2, fetch2 + grads2)
    outs2 = [torch.full(tuple(g2.shape(o)), float("nan"), dtype=torch.float32, device="cuda") for o in fetch2 + grads2]
    f2.run_torch([t if u else None for t, u in zip(small_in, f2.used_inputs())], outs2)
    torch.cuda.synchronize()
    ref2 = interp.run_function(g2.desc, in2, fetch2 + grads2, [t.cpu().numpy() for t in small_in])
    for o, r, t in zip(outs2, ref2, fetch2 + grads2):
        check(o.cpu().numpy().astype(np.float64), r, TOL32, "config 5 (256 rows) tensor %d" % t)
