"""The five benchmark workloads at full size on the GPU, against the oracle, every element of every
fetched tensor.

The two random graphs are too large for one pass of the NumPy interpreter, so the oracle runs over
chunks of the leading axis on the host's cores (oracle/chunked.py: elements of an elementwise graph and
rows of a row-reduction graph are independent; sums over that axis add up in fp64) and each chunk is
compared where it is computed."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import chunked, interp, prune as oprune
from paper_1707_08265_b200 import binding as B
from paper_1707_08265_b200 import workloads as wl
from test_gpu_vm import run_gpu, check, TOL32, TOLBF, to_dev, FLOOR_OK, C_COND

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
    for o in outs:
        assert torch.isfinite(o).all()
    # every element, in chunks of 2^21 over the host's cores, on the very same input values
    host_in = [t.cpu().numpy() if u else None for t, u in zip(gpu_in, f.used_inputs())]
    host_out = [o.cpu().numpy() for o in outs]
    res = chunked.run_chunked(g.desc, inputs, fetch, host_in, n, 1 << 21, compare=host_out, tol=TOL32, with_floor=True)
    for e, t in zip(res, fetch):
        allowed = 1.0 if e[6] <= FLOOR_OK else C_COND * e[6]      # see test_gpu_vm.check_conditioned
        print("config 3 tensor %d: worst error %.3g tolerances, CPU fp32 floor over all elements %.3g" % (t, e[1], e[6]))
        assert e[0] == "err" and e[1] <= allowed, "config 3 tensor %d: worst normalised error %.3g at element %d (got %r ref %r, floor %.3g)" % (
            t, e[1], e[2] + e[3], e[4], e[5], e[6])


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
    for o in outs:
        assert torch.isfinite(o).all()
    # rows are independent (row sums stay inside a row): the oracle runs over all 16384 rows in chunks of
    # 256 on the host's cores.  FULL-shaped outputs are compared chunk by chunk; the gradients of the
    # [cols] inputs are column sums over all rows: the chunks' shares are added in fp64 and compared whole.
    host_in = [t.cpu().numpy() if u else None for t, u in zip(gpu_in, f.used_inputs())]
    host_out = [o.cpu().numpy() if o.dim() == 2 else None for o in outs]
    res = chunked.run_chunked(g.desc, inputs, outs_ids, host_in, rows, 256, compare=host_out, tol=TOL32, with_floor=True)
    n_sums = 0
    for e, o, t in zip(res, outs, outs_ids):
        if e[0] == "err":
            # over 2^26 elements the tail of fp32 rounding shows: a tensor on which NumPy's own fp32 evaluation
            # leaves the tolerance somewhere is held to C_COND times that floor (test_gpu_vm.check_conditioned)
            allowed = 1.0 if e[6] <= FLOOR_OK else C_COND * e[6]
            print("config 5 tensor %d: worst error %.3g tolerances, CPU fp32 floor over all rows %.3g" % (t, e[1], e[6]))
            assert e[1] <= allowed, "config 5 tensor %d: worst normalised error %.3g in the chunk at row %d, offset %d (got %r ref %r, floor %.3g)" % (
                t, e[1], e[2], e[3], e[4], e[5], e[6])
        else:
            n_sums += 1
            check(o.cpu().numpy().astype(np.float64), e[1], TOL32, "config 5 column sums over all rows, tensor %d" % t)
    assert n_sums == sum(1 for w in wrts if len(g.shape(w)) == 1)
