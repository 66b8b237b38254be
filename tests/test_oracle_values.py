"""Pins for oracle/interp.py: closed forms, printed spot values, finite differences, library
cross-checks.  Each pin is chosen so that a dropped term, a wrong sign or a transposed operand
in the interpreter fails it."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import interp
from paper_1707_08265_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def read_golden(name):
    out = {}
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            out[k] = float(v)
    return out


def test_toy_spot_values():
    gold = read_golden("toy_spot_values.txt")
    g, ids = wl.toy_function_grad(1)
    inputs = [ids["x"], ids["a"], ids["b"]]
    outs = [ids[k] for k in ("f", "y", "dx", "da", "db")]
    f, y, dx, da, db = interp.run_function(g.desc, inputs, outs, [np.array([1.0]), np.array(1.0), np.array(0.0)])
    for got, key in ((f, "f"), (y, "y"), (dx, "dfdx"), (da, "dfda"), (db, "dfdb")):
        assert abs(float(np.ravel(got)[0]) - gold[key]) < 1e-9, key


def test_toy_closed_forms():
    n = 1000
    g, ids = wl.toy_function_grad(n)
    x, a, b = wl.toy_feeds(n, 7)
    inputs = [ids["x"], ids["a"], ids["b"]]
    outs = [ids[k] for k in ("f", "y", "dx", "da", "db")]
    f, y, dx, da, db = interp.run_function(g.desc, inputs, outs, [x, a, b])
    xd, ad, bd = x.astype(np.float64), float(a), float(b)
    u = ad * xd + bd
    assert np.allclose(f, xd * np.sin(u), rtol=1e-14, atol=1e-14)
    assert np.allclose(y, ad * xd, rtol=1e-15)
    assert np.allclose(dx, np.sin(u) + ad * xd * np.cos(u), rtol=1e-13, atol=1e-13)
    assert da.shape == () and db.shape == ()
    assert math.isclose(float(da), math.fsum(xd * xd * np.cos(u)), rel_tol=1e-12, abs_tol=1e-10)
    assert math.isclose(float(db), math.fsum(xd * np.cos(u)), rel_tol=1e-12, abs_tol=1e-10)


def test_toy_pruned_input_is_never_read():
    g, ids = wl.toy_function(5)
    x, a, b = wl.toy_feeds(5, 3)
    (y,) = interp.run_function(g.desc, [ids["x"], ids["a"], ids["b"]], [ids["y"]], [x, a, None])
    assert np.allclose(y, float(a) * x.astype(np.float64))


def _single_op_graph(type_, shapes):
    g = wl.GraphDesc()
    ins = [g.tensor("i%d" % k, s) for k, s in enumerate(shapes)]
    out = g.op(type_, ins, "out")
    return g, ins, out


KINKS = {"ReLU": [0.0], "Exp": [-10.0, 10.0]}


def test_fed_intermediate_closed_forms():
    """Sec. 3.1 (any tensor can be fed): with t2 given, f = x*sin(t2) whatever a and b are (they are not
    read), df/dx = sin(t2) alone (the chain through a*x is cut), and the gradient with respect to the
    given tensor is x*cos(t2).  With y given, df/db = sum x*cos(y+b)."""
    n = 257
    g = wl.toy_function(n)[0]
    ids = {t["name"]: i for i, t in enumerate(g.desc["tensors"])}
    dx, dt2, db = g.grad([ids["f"]], [ids["x"], ids["t2"], ids["b"]])
    x, a, b = wl.toy_feeds(n, 11)
    xd = x.astype(np.float64)
    t2 = np.random.default_rng(5).uniform(-3, 3, n)
    inputs = [ids["x"], ids["a"], ids["b"], ids["t2"]]
    f, gx, gt = interp.run_function(g.desc, inputs, [ids["f"], dx, dt2], [x, None, None, t2])
    assert np.allclose(f, xd * np.sin(t2), rtol=1e-15, atol=0)
    assert np.allclose(gx, np.sin(t2), rtol=1e-15, atol=0)
    assert np.allclose(gt, xd * np.cos(t2), rtol=1e-15, atol=0)
    with pytest.raises(ValueError):
        interp.run_function(g.desc, inputs, [db], [x, a, b, t2])
    yv = np.random.default_rng(6).uniform(-3, 3, n)
    inputs = [ids["x"], ids["a"], ids["b"], ids["y"]]
    (gb,) = interp.run_function(g.desc, inputs, [db], [x, None, b, yv])
    assert math.isclose(float(gb), math.fsum(xd * np.cos(yv + float(b))), rel_tol=1e-12)
    # feeding what the function itself would have computed changes nothing downstream
    full = interp.run_function(g.desc, inputs[:3], [ids["y"], ids["f"]], [x, a, b])
    (f2,) = interp.run_function(g.desc, inputs, [ids["f"]], [x, None, b, full[0]])
    assert np.array_equal(f2, full[1])


@pytest.mark.parametrize("type_,shapes", [
    ("Add", [[3, 4], [4]]), ("Sub", [[3, 4], [4]]), ("Sub", [[4], [3, 4]]), ("Mul", [[3, 4], []]),
    ("Mul", [[3, 4], [3, 4]]), ("Div", [[3, 4], [4]]), ("Div", [[4], [3, 4]]), ("Sin", [[3, 4]]),
    ("Exp", [[3, 4]]), ("Tanh", [[3, 4]]), ("Sigmoid", [[3, 4]]), ("ReLU", [[3, 4]]),
    ("Sum", [[3, 4]]), ("Mean", [[3, 4]]), ("Sum", [[4]]), ("Mean", [[4]]),
    ("Sqrt", [[3, 4]]), ("Reciprocal", [[3, 4]]),
])
def test_operator_gradients_match_finite_differences(type_, shapes):
    rng = np.random.default_rng(11)
    g, ins, out = _single_op_graph(type_, shapes)
    # weight the output with a fixed random tensor so that a gradient rule that ignores dy's
    # position (e.g. a wrong broadcast) is caught: obj = out * w
    w = g.tensor("w", g.shape(out))
    obj = g.op("Mul", [out, w], "obj")
    gids = g.grad([obj], ins)
    scale = 6.0 if type_ == "Exp" else 2.0
    feeds = [rng.standard_normal(size=s) * scale for s in shapes] + [rng.standard_normal(size=g.shape(out))]
    if type_ in ("Sqrt", "Reciprocal"):                      # positive arguments away from zero
        feeds[0] = np.abs(feeds[0]) + 0.3
    for f, s in zip(feeds, shapes):                          # keep away from kinks
        for kpt in KINKS.get(type_, []) + ([0.0] if type_ == "Div" else []):
            f[np.abs(f - kpt) < 1e-2] += 0.05
    inputs = ins + [w]
    got = interp.run_function(g.desc, inputs, gids, feeds)
    for wrt, gv in zip(ins, got):
        fd = interp.finite_difference(g.desc, inputs, feeds, [obj], wrt, h=1e-6)
        assert gv.shape == tuple(g.shape(wrt))
        assert np.allclose(gv, fd, rtol=2e-6, atol=2e-6), (type_, wrt, gv, fd)


def test_sqrt_reciprocal_closed_forms_and_updaters():
    # values: exact squares and powers of two; derivative of sqrt(x) * (1/x) = x^(-1/2) is -x^(-3/2)/2
    g, ins, out = _single_op_graph("Sqrt", [[4]])
    (v,) = interp.run_function(g.desc, ins, [out], [np.array([0.0, 1.0, 4.0, 2.25])])
    assert np.array_equal(v, [0.0, 1.0, 2.0, 1.5])
    g, ins, out = _single_op_graph("Reciprocal", [[3]])
    (v,) = interp.run_function(g.desc, ins, [out], [np.array([1.0, -4.0, 0.125])])
    assert np.array_equal(v, [1.0, -0.25, 8.0])
    gd = wl.GraphDesc()
    x = gd.tensor("x", [3])
    y = gd.op("Mul", [gd.op("Sqrt", [x], "s"), gd.op("Reciprocal", [x], "r")], "y")
    (dx,) = gd.grad([y], [x])
    xv = np.array([0.5, 1.0, 9.0])
    (got,) = interp.run_function(gd.desc, [x], [dx], [xv])
    assert np.allclose(got, -0.5 * xv ** -1.5, rtol=1e-14)
    # the updater graphs against their formulas written out (Sec. 3.2 names Momentum, RMSProp, Adam)
    rng = np.random.default_rng(4)
    W, gr, m, v = (rng.standard_normal(7) for _ in range(4))
    v = np.abs(v)
    lr, b1, b2, eps = 0.01, 0.9, 0.999, 1e-8
    u, ids = wl.updater([7], "adam")
    ins_ = [ids[k] for k in ("W", "g", "m", "v", "lr", "beta1", "one_minus_beta1", "beta2", "one_minus_beta2", "eps")]
    Wn, mn, vn = interp.run_function(u.desc, ins_, [ids["W_new"], ids["m_new"], ids["v_new"]],
                                     [W, gr, m, v] + [np.asarray(c) for c in (lr, b1, 1 - b1, b2, 1 - b2, eps)])
    m2, v2 = b1 * m + (1 - b1) * gr, b2 * v + (1 - b2) * gr * gr
    assert np.allclose(mn, m2, rtol=1e-15) and np.allclose(vn, v2, rtol=1e-15)
    assert np.allclose(Wn, W - lr * m2 / (np.sqrt(v2) + eps), rtol=1e-14)
    u, ids = wl.updater([7], "rmsprop")
    ins_ = [ids[k] for k in ("W", "g", "v", "lr", "rho", "one_minus_rho", "eps")]
    Wn, vn = interp.run_function(u.desc, ins_, [ids["W_new"], ids["v_new"]], [W, gr, v] + [np.asarray(c) for c in (lr, 0.9, 0.1, eps)])
    v2 = 0.9 * v + 0.1 * gr * gr
    assert np.allclose(vn, v2, rtol=1e-15) and np.allclose(Wn, W - lr * gr / (np.sqrt(v2) + eps), rtol=1e-14)


def test_same_operand_twice_and_fanout_accumulate():
    # f = (x*x) + x  ->  df/dx = 2x + 1 : Mul(n, n) contributions add, two consumers add
    g = wl.GraphDesc()
    x = g.tensor("x", [5])
    sq = g.op("Mul", [x, x], "sq")
    f = g.op("Add", [sq, x], "f")
    (dx,) = g.grad([f], [x])
    xv = np.linspace(-2, 2, 5)
    (got,) = interp.run_function(g.desc, [x], [dx], [xv])
    assert np.allclose(got, 2 * xv + 1, rtol=1e-15)


def test_kink_readings():
    # ReLU'(0) = 0; sgn(0) = 0 in the Div rule; Exp passes gradient at the clamp bounds
    for type_, xv, expect in (("ReLU", [0.0, -1.0, 2.0], [0.0, 0.0, 1.0]),
                              ("Exp", [-10.0, 10.0, 10.5, -11.0],
                               [math.exp(-10), math.exp(10), 0.0, 0.0])):
        g, ins, out = _single_op_graph(type_, [[len(xv)]])
        (dx,) = g.grad([out], ins)
        (got,) = interp.run_function(g.desc, ins, [dx], [np.array(xv)])
        assert np.allclose(got, expect, rtol=1e-15), type_
    g, ins, out = _single_op_graph("Div", [[2], [2]])
    da, db = g.grad([out], ins)
    ga, gb = interp.run_function(g.desc, ins, [da, db], [np.array([3.0, 3.0]), np.array([0.0, -1.0])])
    assert np.allclose(ga, [1.0, 0.5]) and np.allclose(gb, [0.0, 3.0 / 4.0])
    (val,) = interp.run_function(g.desc, ins, [out], [np.array([3.0, 3.0]), np.array([0.0, -1.0])])
    assert np.allclose(val, [3.0, 1.5])
    g, ins, out = _single_op_graph("Exp", [[3]])
    (val,) = interp.run_function(g.desc, ins, [out], [np.array([-50.0, 0.0, 50.0])])
    assert np.allclose(val, [math.exp(-10), 1.0, math.exp(10)], rtol=1e-15)


def test_sum_mean_closed_forms_and_fsum():
    g, ins, out = _single_op_graph("Sum", [[3, 7]])
    (v,) = interp.run_function(g.desc, ins, [out], [np.full((3, 7), 0.25)])
    assert v.shape == (3, 7) and np.all(v == 1.75)
    rng = np.random.default_rng(5)
    x = rng.standard_normal(size=(4, 1001)) * 1e3
    (v,) = interp.run_function(g2 := _single_op_graph("Sum", [[4, 1001]])[0].desc, [0], [1], [x])
    for r in range(4):
        assert math.isclose(v[r, 17], math.fsum(x[r]), rel_tol=1e-13)
        assert np.all(v[r] == v[r, 0])
    (v,) = interp.run_function(_single_op_graph("Mean", [[4, 1001]])[0].desc, [0], [1], [x])
    for r in range(4):
        assert math.isclose(v[r, 3], math.fsum(x[r]) / 1001, rel_tol=1e-13)
    (v,) = interp.run_function(_single_op_graph("Mean", [[6]])[0].desc, [0], [1], [np.arange(6.0)])
    assert v.shape == (6,) and np.all(v == 2.5)


def test_round_bf16_matches_library_conversion():
    rng = np.random.default_rng(9)
    x = np.concatenate([rng.standard_normal(4096) * 10.0 ** rng.integers(-8, 8, 4096),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895313892515355e38]]).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(interp.round_bf16(x), want)
    assert interp.round_bf16(x.astype(np.float64)).dtype == np.float64


def _ip_graph(m, k, n):
    g = wl.GraphDesc()
    X = g.tensor("X", [m, k])
    W = g.tensor("W", [n, k])
    Y = g.op("InnerProduct", [X, W], "Y", [m, n])
    return g, X, W, Y


def test_inner_product_identity_onehot_and_library():
    g, X, W, Y = _ip_graph(5, 4, 4)
    rng = np.random.default_rng(2)
    x = interp.round_bf16(rng.standard_normal((5, 4)))
    (y,) = interp.run_function(g.desc, [X, W], [Y], [x, np.eye(4)])
    assert np.array_equal(y, x)                               # identity weights
    g, X, W, Y = _ip_graph(5, 4, 3)
    w = np.zeros((3, 4)); w[0, 2] = 1; w[1, 0] = 1; w[2, 3] = 2
    (y,) = interp.run_function(g.desc, [X, W], [Y], [x, w])   # Y[m,n] = sum_k X[m,k] W[n,k]
    assert np.array_equal(y, np.stack([x[:, 2], x[:, 0], 2 * x[:, 3]], axis=1))
    g, X, W, Y = _ip_graph(33, 65, 17)
    x = interp.round_bf16(rng.standard_normal((33, 65))); w = interp.round_bf16(rng.standard_normal((17, 65)))
    (y,) = interp.run_function(g.desc, [X, W], [Y], [x, w])
    want = torch.matmul(torch.from_numpy(x), torch.from_numpy(w).T).numpy()
    assert np.allclose(y, want, rtol=1e-13, atol=1e-13)
    # operands that are not bf16 values are rounded before the contraction
    x2 = x + 1e-4
    (y2,) = interp.run_function(g.desc, [X, W], [Y], [x2, w])
    assert np.allclose(y2, interp.round_bf16(x2) @ w.T, rtol=1e-13, atol=1e-13)


def test_inner_product_gradients():
    g, X, W, Y = _ip_graph(3, 4, 2)
    wt = g.tensor("wt", [3, 2])
    obj = g.op("Mul", [Y, wt], "obj")
    dX, dW = g.grad([obj], [X, W])
    rng = np.random.default_rng(4)
    feeds = [rng.standard_normal((3, 4)), rng.standard_normal((2, 4)), rng.standard_normal((3, 2))]
    gx, gw = interp.run_function(g.desc, [X, W, wt], [dX, dW], feeds, bf16_contraction=False)
    for wrt, gv in ((X, gx), (W, gw)):
        fd = interp.finite_difference(g.desc, [X, W, wt], feeds, [obj], wrt, bf16_contraction=False)
        assert np.allclose(gv, fd, rtol=1e-6, atol=1e-6)
    # closed form with bf16 rounding on: dX = bf16(dY) @ bf16(W), dW = bf16(dY)^T @ bf16(X)
    gx, gw = interp.run_function(g.desc, [X, W, wt], [dX, dW], feeds)
    r = interp.round_bf16
    assert np.allclose(gx, r(feeds[2]) @ r(feeds[1]), rtol=1e-14)
    assert np.allclose(gw, r(feeds[2]).T @ r(feeds[0]), rtol=1e-14)


def test_bias_add_gradient_is_column_sum():
    g = wl.GraphDesc()
    Y = g.tensor("Y", [4, 3]); b = g.tensor("b", [3]); wt = g.tensor("wt", [4, 3])
    out = g.op("BiasAdd", [Y, b], "out", [4, 3])
    obj = g.op("Mul", [out, wt], "obj")
    dY, db = g.grad([obj], [Y, b])
    rng = np.random.default_rng(8)
    feeds = [rng.standard_normal((4, 3)), rng.standard_normal(3), rng.standard_normal((4, 3))]
    gy, gb = interp.run_function(g.desc, [Y, b, wt], [dY, db], feeds)
    assert np.allclose(gy, feeds[2]) and np.allclose(gb, feeds[2].sum(axis=0))
    (v,) = interp.run_function(g.desc, [Y, b, wt], [out], feeds)
    assert np.allclose(v, feeds[0] + feeds[1][None, :])


def _sce_graph(m, n):
    g = wl.GraphDesc()
    Z = g.tensor("Z", [m, n]); lab = g.tensor("lab", [m], "i32")
    L = g.op("SoftmaxCrossEntropy", [Z, lab], "L", [])
    (dZ,) = g.grad([L], [Z])
    return g, Z, lab, L, dZ


def test_softmax_cross_entropy_pins():
    g, Z, lab, L, dZ = _sce_graph(6, 4096)
    labels = np.arange(6, dtype=np.int32) * 7
    loss, dz = interp.run_function(g.desc, [Z, lab], [L, dZ], [np.full((6, 4096), 3.5), labels])
    assert math.isclose(float(loss), 8.3177661667, abs_tol=1e-9)          # ln 4096
    assert np.allclose(dz.sum(axis=1), 0, atol=1e-15)
    assert math.isclose(dz[2, 14], (1 / 4096 - 1) / 6, rel_tol=1e-12)
    g, Z, lab, L, dZ = _sce_graph(9, 13)
    rng = np.random.default_rng(6)
    z = rng.standard_normal((9, 13)) * 5 + 100.0                          # needs the max subtraction
    labels = rng.integers(0, 13, 9).astype(np.int32)
    loss, dz = interp.run_function(g.desc, [Z, lab], [L, dZ], [z, labels])
    zt = torch.from_numpy(z).requires_grad_(True)
    lt = torch.nn.functional.cross_entropy(zt, torch.from_numpy(labels).long())
    lt.backward()
    assert math.isclose(float(loss), float(lt.detach()), rel_tol=1e-12) and float(loss) >= 0
    assert np.allclose(dz, zt.grad.numpy(), rtol=1e-11, atol=1e-14)
    fd = interp.finite_difference(g.desc, [Z, lab], [z, labels], [L], Z, h=1e-6)
    assert np.allclose(dz, fd, rtol=1e-5, atol=1e-8)


def test_mlp_gradients_match_autograd_library():
    """Whole two-layer graph against torch autograd in fp64 with the same rounding points."""
    m, k, h, n = 16, 32, 24, 10
    g, ids = wl.mlp(m, k, h, n)
    X, W1, b1, W2, b2, labels = wl.mlp_feeds(m, k, h, n, 5)
    inputs = [ids[t] for t in ("X", "W1", "b1", "W2", "b2", "labels")]
    outs = [ids[t] for t in ("loss", "dW1", "db1", "dW2", "db2")]
    loss, dW1, db1, dW2, db2 = interp.run_function(g.desc, inputs, outs, [X, W1, b1, W2, b2, labels])

    class RoundBf16(torch.autograd.Function):     # value rounds, gradient passes (storage rounding)
        @staticmethod
        def forward(ctx, x):
            return x.float().to(torch.bfloat16).double()

        @staticmethod
        def backward(ctx, gy):
            return gy

    class RoundGrad(torch.autograd.Function):     # the gradient operand of a contraction is bf16
        @staticmethod
        def forward(ctx, x):
            return x.clone()

        @staticmethod
        def backward(ctx, gy):
            return gy.float().to(torch.bfloat16).double()

    t = lambda a: torch.from_numpy(a).double().requires_grad_(True)
    tX, tW1, tb1, tW2, tb2 = t(X), t(W1), t(b1), t(W2), t(b2)
    z1 = RoundGrad.apply(tX @ tW1.T)
    hh = RoundBf16.apply(torch.relu(z1 + tb1))
    z2 = RoundGrad.apply(hh @ tW2.T)
    z = RoundBf16.apply(z2 + tb2)
    lt = torch.nn.functional.cross_entropy(z, torch.from_numpy(labels).long())
    lt.backward()
    assert math.isclose(float(loss), float(lt.detach()), rel_tol=1e-12)
    for got, want in ((dW1, tW1.grad), (db1, tb1.grad), (dW2, tW2.grad), (db2, tb2.grad)):
        assert np.allclose(got, want.numpy(), rtol=1e-10, atol=1e-14)


def test_fp32_instance_runs_in_float32():
    g, inputs, fetch = wl.random_dag(64, 3, n_ops=16)
    feeds = wl.normal_feeds([[64]] * 4, 3)
    outs = interp.run_function(g.desc, inputs, fetch, feeds, dtype=np.float32)
    assert all(o.dtype == np.float32 for o in outs)


@pytest.mark.parametrize("workers", [1, 2])
def test_chunked_evaluation_equals_the_plain_one(workers):
    """oracle.chunked cuts the leading axis into independent chunks (rows of a row-reduction graph,
    elements of an elementwise one); values equal the unchunked interpreter's, sums over the axis add up."""
    from oracle import chunked, prune as oprune
    from paper_1707_08265_b200 import workloads as wl
    R, C = 23, 40
    g, inputs, fetch = wl.random_row_dag(R, C, 3004, n_ops=48, n_fetch=2)
    G = oprune.backward_marks(g.desc, fetch, inputs)
    wrts = [i for i in inputs if i in G]
    outs = fetch + g.grad(fetch, wrts)
    feeds = [a * np.float32(0.5) for a in wl.normal_feeds([g.shape(i) for i in inputs], 7)]
    ref = interp.run_function(g.desc, inputs, outs, feeds)
    res = chunked.run_chunked(g.desc, inputs, outs, feeds, R, 5, workers=workers)
    assert any(k == "sum" for k, *_ in res) and any(k == "val" for k, *_ in res)
    for (kind, v), r in zip(res, ref):
        assert np.allclose(v, r, rtol=1e-12, atol=1e-12), kind
    # comparison mode: the reference handed in as "got" gives zero error, a planted mistake is found
    cmp = [np.array(r) if len(np.shape(r)) == 2 else None for r in ref]
    bad = next(k for k, c in enumerate(cmp) if c is not None)
    cmp[bad][17, 3] += 1.0
    res = chunked.run_chunked(g.desc, inputs, outs, feeds, R, 5, workers=workers, compare=cmp)
    for k, e in enumerate(res):
        if e[0] == "err":
            assert (e[1] > 1 and e[2] == 15 and e[3] == 2 * C + 3) if k == bad else e[1] == 0.0
            assert e[6] == 0.0          # no floor was asked for
    # a flat elementwise graph with scalar gradients
    n = 1000
    g2, ids = wl.toy_function_grad(n)
    x, a, b = wl.toy_feeds(n, 3)
    ins, o2 = [ids["x"], ids["a"], ids["b"]], [ids["f"], ids["dx"], ids["da"], ids["db"]]
    ref2 = interp.run_function(g2.desc, ins, o2, [x, a, b])
    res2 = chunked.run_chunked(g2.desc, ins, o2, [x, a, b], n, 333, workers=workers)
    for (kind, v), r in zip(res2, ref2):
        assert np.allclose(v, r, rtol=1e-12, atol=1e-12)
