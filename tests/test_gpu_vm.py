"""GPU parity of the graph VM against the oracle, through the C ABI (element by element, small
sizes that still span several tiles and a ragged tail)."""
import numpy as np
import pytest
import torch

from oracle import interp, prune as oprune
from paper_1707_08265_b200 import binding as B
from paper_1707_08265_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL32 = 1e-5      # max |gpu - ref| <= TOL32 * (1 + |ref|), ref evaluated in fp64
TOLBF = 1e-2      # outputs derived from bf16 contractions


def to_dev(a, dtype="f32"):
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype == "bf16":
        t = t.to(torch.bfloat16)
    return t.cuda()


def run_gpu(desc, inputs, outputs, feeds):
    g = B.Graph.from_desc(desc)
    f = g.function(inputs, outputs)
    dev_feeds = [to_dev(a, desc["tensors"][i]["dtype"]) for i, a in zip(inputs, feeds)]
    tdt = {"f32": torch.float32, "bf16": torch.bfloat16}
    outs = [torch.full(tuple(desc["tensors"][o]["shape"]), float("nan"), dtype=tdt[desc["tensors"][o]["dtype"]], device="cuda")
            for o in outputs]
    f.run_torch(dev_feeds, outs)
    assert f.status() == 0
    torch.cuda.synchronize()
    return [o.float().cpu().numpy().astype(np.float64) for o in outs], f


def check(got, ref, tol, what=""):
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    err = np.abs(got - ref) / (tol * (1 + np.abs(ref)))
    bad = ~(err <= 1)
    assert not bad.any(), "%s: worst normalised error %.3g at %s (got %r ref %r)" % (
        what, np.nanmax(err), np.argwhere(bad)[0], got[tuple(np.argwhere(bad)[0])], ref[tuple(np.argwhere(bad)[0])])
    return float(err.max()) if err.size else 0.0


@pytest.mark.parametrize("n", [1, 3, 4095, 4096, 4097, 3 * 4096 + 5, 1 << 20])
def test_toy_forward_and_pruned_input(n):
    g, ids = wl.toy_function(n)
    x, a, b = wl.toy_feeds(n, wl.BASE_SEED + 1)
    inputs = [ids["x"], ids["a"], ids["b"]]
    (y,), f = run_gpu(g.desc, inputs, [ids["y"]], [x, a, None])      # b pruned: its feed is NULL
    assert f.used_inputs() == [1, 1, 0]
    check(y, interp.run_function(g.desc, inputs, [ids["y"]], [x, a, None])[0], TOL32, "y")
    (fv, y), _ = run_gpu(g.desc, inputs, [ids["f"], ids["y"]], [x, a, b])
    rf, ry = interp.run_function(g.desc, inputs, [ids["f"], ids["y"]], [x, a, b])
    check(fv, rf, TOL32, "f")
    check(y, ry, TOL32, "y")


@pytest.mark.parametrize("n", [1, 5, 4096, 5 * 4096 + 17, 200 * 4096 + 1, 1 << 22])
def test_toy_gradients(n):
    g, ids = wl.toy_function_grad(n)
    x, a, b = wl.toy_feeds(n, wl.BASE_SEED + 2)
    inputs = [ids["x"], ids["a"], ids["b"]]
    outs = [ids["dx"], ids["da"], ids["db"]]
    got, f = run_gpu(g.desc, inputs, outs, [x, a, b])
    ref = interp.run_function(g.desc, inputs, outs, [x, a, b])
    for gv, rv, name in zip(got, ref, ("dx", "da", "db")):
        check(gv, rv, TOL32, name)
    # closed forms, independent of the interpreter
    xd, ad, bd = x.astype(np.float64), float(a), float(b)
    u = ad * xd + bd
    check(got[0], np.sin(u) + ad * xd * np.cos(u), TOL32, "dx closed form")
    check(got[1], np.sum(xd * xd * np.cos(u)), TOL32, "da closed form")
    check(got[2], np.sum(xd * np.cos(u)), TOL32, "db closed form")
    # fetching f as well changes nothing
    got2, _ = run_gpu(g.desc, inputs, [ids["f"]] + outs, [x, a, b])
    check(got2[0], xd * np.sin(u), TOL32, "f")
    assert np.array_equal(got2[1], got[0])


FLOOR_OK = 0.25   # CPU fp32 evaluation within a quarter of the tolerance: the tensor is held to the tolerance itself
C_COND = 16.0     # otherwise (floor f, in tolerances): held to C_COND * f tolerances


def fp32_floors(desc, inputs, outputs, feeds):
    """Per fetched tensor: how far the oracle's own arithmetic, instantiated in fp32 on the CPU (same plain
    loop, NumPy float32), lands from its fp64 result, in units of the tolerance.  A value above 1 says that
    the graph amplifies fp32 rounding beyond 1e-5 whatever evaluates it; such a tensor cannot be held to
    the plain tolerance, and is held to C_COND times its floor instead of not being compared at all."""
    ref = interp.run_function(desc, inputs, outputs, feeds)
    low = interp.run_function(desc, inputs, outputs, feeds, dtype=np.float32)
    floors = []
    for r, l in zip(ref, low):
        assert np.all(np.isfinite(r)), "the fp64 reference itself is not finite"
        floors.append(float(np.max(np.abs(l.astype(np.float64) - r) / (TOL32 * (1 + np.abs(r))))))
    return floors, ref


def check_conditioned(got, ref, floors, what):
    """Every tensor against the oracle: at the tolerance where fp32 can reach it (floor <= FLOOR_OK), else
    at C_COND * floor tolerances.  Returns the number of tensors held to the plain tolerance."""
    tight = 0
    for k, (gv, rv, fl) in enumerate(zip(got, ref, floors)):
        scale = 1.0 if fl <= FLOOR_OK else C_COND * fl
        tight += scale == 1.0
        check(gv, rv, TOL32 * scale, "%s tensor %d (fp32 floor %.3g)" % (what, k, fl))
    return tight


@pytest.mark.parametrize("seed", range(24))
def test_random_elementwise_dags(seed):
    n = 2 * 4096 + 77
    g, inputs, fetch = wl.random_dag(n, 1000 + seed, n_ops=64)
    feeds = wl.normal_feeds([[n]] * 4, 2000 + seed)
    floors, ref = fp32_floors(g.desc, inputs, fetch, feeds)
    got, f = run_gpu(g.desc, inputs, fetch, feeds)
    want = oprune.function_sets(g.desc, inputs, fetch)
    assert f.marked() == want["marked"] and f.kept_ops()[0] == want["fwd_ops"]
    check_conditioned(got, ref, floors, "seed %d" % seed)


@pytest.mark.parametrize("op", ["Add", "Sub", "Mul", "Div", "Sin", "Exp", "Tanh", "Sigmoid", "ReLU"])
def test_single_operators_forward_and_gradient(op):
    n = 4096 + 33
    gd = wl.GraphDesc()
    nin = 2 if op in wl.BINARY else 1
    ins = [gd.tensor("i%d" % k, [n]) for k in range(nin)]
    out = gd.op(op, ins, "out")
    w = gd.tensor("w", [n])
    obj = gd.op("Mul", [out, w], "obj")
    grads = gd.grad([obj], ins)
    rng = np.random.default_rng(5)
    scale = 6.0 if op == "Exp" else (30.0 if op == "Sin" else 3.0)
    feeds = [(rng.standard_normal(n) * scale).astype(np.float32) for _ in ins] + [rng.standard_normal(n).astype(np.float32)]
    feeds[0][:8] = [0.0, -0.0, 1e-6, -1e-6, 10.0, -10.0, 100.0, -100.0]
    inputs = ins + [w]
    got, _ = run_gpu(gd.desc, inputs, [out] + grads, feeds)
    ref = interp.run_function(gd.desc, inputs, [out] + grads, feeds)
    for gv, rv in zip(got, ref):
        check(gv, rv, TOL32, op)


@pytest.mark.parametrize("shape", [(1, 8), (5, 12), (7, 4096), (300, 1000), (3, 4095), (40, 130)])
def test_row_mode_broadcast_sum_mean(shape):
    R, C = shape
    gd = wl.GraphDesc()
    X = gd.tensor("X", [R, C]); r = gd.tensor("r", [C]); s = gd.tensor("s", [])
    t1 = gd.op("Mul", [X, r], "t1")
    t2 = gd.op("Sum", [t1], "t2")
    t3 = gd.op("Add", [t2, X], "t3")
    t4 = gd.op("Mean", [r], "t4")
    t5 = gd.op("Mul", [t3, t4], "t5")
    t6 = gd.op("Sub", [t5, s], "t6")
    t7 = gd.op("Tanh", [t6], "t7")
    dX, dr, ds = gd.grad([t7], [X, r, s])
    rng = np.random.default_rng(3)
    feeds = [rng.standard_normal((R, C)).astype(np.float32) * 0.3, rng.standard_normal(C).astype(np.float32) * 0.3,
             np.asarray(rng.standard_normal(), dtype=np.float32)]
    outs = [t7, t2, t4, dX, dr, ds]
    got, f = run_gpu(gd.desc, [X, r, s], outs, feeds)
    ref = interp.run_function(gd.desc, [X, r, s], outs, feeds)
    for gv, rv, name in zip(got, ref, ("t7", "t2", "t4", "dX", "dr", "ds")):
        check(gv, rv, TOL32, name)


@pytest.mark.parametrize("seed", range(10))
def test_random_row_dags_with_gradients(seed):
    R, C = 37, 520
    g, inputs, fetch = wl.random_row_dag(R, C, 3000 + seed, n_ops=48, n_fetch=2)
    G = oprune.backward_marks(g.desc, fetch, inputs)
    wrts = [i for i in inputs if i in G]
    grads = g.grad(fetch, wrts)
    shapes = [g.shape(i) for i in inputs]
    feeds = [a * np.float32(0.5) for a in wl.normal_feeds(shapes, 4000 + seed)]
    outs = fetch + grads
    floors, ref = fp32_floors(g.desc, inputs, outs, feeds)
    got, f = run_gpu(g.desc, inputs, outs, feeds)
    want = oprune.function_sets(g.desc, inputs, outs)
    fwd, gops, masks = f.kept_ops()
    assert f.marked() == want["marked"] and fwd == want["fwd_ops"] and gops == [k for (_, k, _) in want["grad_ops"]]
    check_conditioned(got, ref, floors, "seed %d" % seed)


@pytest.mark.parametrize("seed", range(8))
def test_random_row_dags_with_fed_intermediates(seed):
    """Sec. 3.1: any tensor can be fed.  Up to three tensors that operators produce (a full tensor, a broadcast
    row sum, whatever the draw gives) are listed among the inputs and fed with fresh values; forward values and
    the gradients with respect to the sources that keep a chain and to the given tensors themselves against the
    oracle, prune sets included."""
    R, C = 37, 520
    g, inputs, fetch = wl.random_row_dag(R, C, 3000 + seed, n_ops=48, n_fetch=2)
    kept = oprune.function_sets(g.desc, inputs, fetch)["fwd_ops"]
    rng = np.random.default_rng(seed)
    fed = sorted({g.desc["ops"][int(k)]["out"][0] for k in rng.choice(kept, size=min(3, len(kept)), replace=False)} - set(fetch))
    all_in = inputs + fed
    G = oprune.backward_marks(oprune.without_edges_into(g.desc, all_in), fetch, all_in)
    wrts = [i for i in all_in if i in G]
    grads = g.grad(fetch, wrts) if wrts else []
    feeds = [a * np.float32(0.5) for a in wl.normal_feeds([g.shape(i) for i in all_in], 4100 + seed)]
    outs = fetch + grads
    want = oprune.function_sets(g.desc, all_in, outs)
    feeds = [a if u else None for a, u in zip(feeds, want["used_inputs"])]
    floors, ref = fp32_floors(g.desc, all_in, outs, feeds)
    got, f = run_gpu(g.desc, all_in, outs, feeds)
    fwd, gops, masks = f.kept_ops()
    assert f.marked() == want["marked"] and fwd == want["fwd_ops"] and gops == [k for (_, k, _) in want["grad_ops"]]
    assert f.used_inputs() == want["used_inputs"]
    check_conditioned(got, ref, floors, "seed %d" % seed)


def test_register_pressure_spills_to_shared_and_global():
    # a wide fan-in: 40 live values force shared-memory slots and workspace spill slots
    n = 3 * 4096 + 9
    gd = wl.GraphDesc()
    x = gd.tensor("x", [n])
    vals = []
    cur = x
    for k in range(40):
        cur = gd.op("Sin" if k % 2 else "Tanh", [cur], "v%d" % k)
        vals.append(cur)
    acc = vals[0]
    for k, v in enumerate(vals[1:]):
        acc = gd.op("Add" if k % 3 else "Mul", [acc, v], "a%d" % k)
    (dx,) = gd.grad([acc], [x])
    xs = np.random.default_rng(1).standard_normal(n).astype(np.float32)
    got, f = run_gpu(gd.desc, [x], [acc, dx], [xs])
    assert "spill=0" not in f.describe()
    ref = interp.run_function(gd.desc, [x], [acc, dx], [xs])
    check(got[0], ref[0], TOL32, "acc")
    check(got[1], ref[1], TOL32, "dx")


def test_fetch_input_scalar_outputs_and_constants():
    n = 5000
    gd = wl.GraphDesc()
    x = gd.tensor("x", [n]); s = gd.tensor("s", [])
    t = gd.op("Sin", [s], "t")                      # scalar-only operator, fetched
    y = gd.op("Add", [x, t], "y")
    dx, ds = gd.grad([y], [x, s])                   # dx is the constant one, ds = n*cos(s)
    xs = np.random.default_rng(2).standard_normal(n).astype(np.float32)
    sv = np.asarray(0.7, dtype=np.float32)
    outs = [x, t, y, dx, ds]
    got, _ = run_gpu(gd.desc, [x, s], outs, [xs, sv])
    ref = interp.run_function(gd.desc, [x, s], outs, [xs, sv])
    for gv, rv, name in zip(got, ref, ("x", "t", "y", "dx", "ds")):
        check(gv, rv, TOL32, name)


@pytest.mark.parametrize("seed", [1, 2])
def test_dense_survival_row_dag_is_cut_into_segments(seed):
    """A 1024-operator row DAG fetched so that a quarter of its operators survive (about 255 forward and as many
    gradient operators, 40 fetched targets, gradients to every connected input): more memory operands than one VM
    program holds, so the lowering cuts the fused segment until every piece fits; values cross the pieces through
    the workspace.  Prune sets and operator order against the oracle, values under the conditioned tolerance."""
    from paper_1707_08265_b200 import binding as B
    R, C = 64, 520
    g, inputs, fetch = wl.random_row_dag(R, C, 9100 + seed, n_ops=1024, n_fetch=40)
    wrts = [i for i in inputs if i in oprune.backward_marks(g.desc, fetch, inputs)]
    outs = fetch + g.grad(fetch, wrts)
    feeds = [a * np.float32(0.5) for a in wl.normal_feeds([g.shape(i) for i in inputs], 9200 + seed)]
    ref64 = interp.run_function(g.desc, inputs, outs, feeds)
    finite = [k for k, r in enumerate(ref64) if np.all(np.isfinite(r)) and np.max(np.abs(r)) < 1e30]
    assert len(finite) >= len(outs) - 6          # a few of the 48 outputs overflow even in fp64 (chained sums of exponentials)
    got, f = run_gpu(g.desc, inputs, outs, feeds)
    want = oprune.function_sets(g.desc, inputs, outs)
    fwd, gops, masks = f.kept_ops()
    assert f.marked() == want["marked"] and fwd == want["fwd_ops"] and gops == [k for (_, k, _) in want["grad_ops"]]
    assert len(fwd) >= 250 and f.describe().count("vm[") >= 4
    low = interp.run_function(g.desc, inputs, outs, feeds, dtype=np.float32)
    tight = 0
    for k in finite:
        fl = float(np.max(np.abs(low[k].astype(np.float64) - ref64[k]) / (TOL32 * (1 + np.abs(ref64[k])))))
        if not np.isfinite(fl) or fl > 1e3:
            continue        # fp32 itself is off by more than 1 % there (sines of large exponentials and the like): nothing to hold a kernel to
        scale = 1.0 if fl <= FLOOR_OK else C_COND * fl
        tight += scale == 1.0
        check(got[k], ref64[k], TOL32 * scale, "seed %d output %d (fp32 floor %.3g)" % (seed, k, fl))
    assert tight >= len(finite) // 2
