"""GPU checks that go beyond the benchmark graphs: the VM's elementary functions over dense sweeps
of arguments (every binade, both signs, the switch points of the implementations), and the weight
update run as a graph of its own (Sec. 3.2 of the paper), each against the fp64 oracle."""
import numpy as np
import pytest

from oracle import interp
from paper_1707_08265_b200 import workloads as wl
from test_gpu_vm import run_gpu, check, TOL32

pytestmark = pytest.mark.gpu


def sweep(lo_exp, hi_exp, per_binade=64):
    m = np.linspace(1.0, 2.0, per_binade, endpoint=False, dtype=np.float64)
    mag = np.concatenate([m * 2.0 ** e for e in range(lo_exp, hi_exp)])
    return np.concatenate([mag, -mag, [0.0, -0.0]]).astype(np.float32)


@pytest.mark.parametrize("op,lo,hi,extra", [
    ("Sin", -20, 128, [np.pi / 4, np.pi / 2, np.pi, 1e5 * np.pi, 1048576.0, 1048577.0, 6.4e6, 3.4028235e38]),   # every finite binade
    ("Exp", -20, 8, [10.0, -10.0, 9.9999, -9.9999, 10.0001, 88.0, -88.0]),   # clamp at +-10
    ("Tanh", -20, 8, [0.6, 0.5999999, 0.6000001, 9.0, 9.07, 9.1, 9.5, 10.0, 10.5, 20.0, 21.0, 90.0]),    # saturates exactly from 9.5 on at the latest
    ("Sigmoid", -20, 8, [86.0, -86.0, 88.7, -88.7, 100.0, -100.0]),
    ("Div", -20, 20, [1.0, -1.0]),
    ("Sqrt", -40, 60, [1.0, 4.0, 2.0, 3.0e38]),                              # positive arguments only (see below)
    ("Reciprocal", -60, 60, [1.0, -1.0, 3.0]),
])
def test_elementary_functions_over_dense_sweeps(op, lo, hi, extra):
    x = np.concatenate([sweep(lo, hi), np.asarray(extra, np.float32), -np.asarray(extra, np.float32)]).astype(np.float32)
    if op == "Sqrt":
        x = np.abs(x[x != 0])
    if op == "Reciprocal":
        x = x[x != 0]
    n = x.size
    gd = wl.GraphDesc()
    xi = gd.tensor("x", [n])
    ins = [xi]
    feeds = [x]
    if op == "Div":   # a / (1 + |b|): sweep b, a fixed to ones
        one = gd.tensor("one", [n])
        out = gd.op("Div", [one, xi], "out")
        ins = [one, xi]
        feeds = [np.ones(n, np.float32), x]
    else:
        out = gd.op(op, [xi], "out")
    grads = gd.grad([out], [xi])     # Sin -> cos, Exp -> exp*mask, Tanh -> 1-y^2, Sigmoid -> y(1-y), Div -> d/db
    got, _ = run_gpu(gd.desc, ins, [out] + grads, feeds)
    ref = interp.run_function(gd.desc, ins, [out] + grads, feeds)
    for gv, rv, what in zip(got, ref, ("value", "gradient")):
        check(gv, rv, TOL32, "%s %s" % (op, what))
    if op in ("Exp", "Sigmoid"):      # the hardware power of two is good to 2^-22: a few units in the last place overall
        big = np.abs(ref[0]) > 1e-30       # (a sigmoid below the normal range is flushed to zero)
        rel = np.abs(got[0] - ref[0])[big] / np.abs(ref[0])[big]
        assert np.max(rel) < 6e-7, np.max(rel)
    if op == "Tanh":      # a saturated tanh is exactly +-1 and its gradient exactly 0
        sat = np.abs(x) >= 9.5
        assert np.all(np.abs(got[0][sat]) == 1) and np.all(got[1][sat] == 0)


def updater_case(kind, shape, seed=11):
    g, ids = wl.updater(shape, kind)
    rng = np.random.default_rng(seed)
    W = rng.standard_normal(shape).astype(np.float32)
    grad = (rng.standard_normal(shape) * 0.1).astype(np.float32)
    m = (rng.standard_normal(shape) * 0.1).astype(np.float32)
    v = (rng.standard_normal(shape) ** 2 * 0.01).astype(np.float32)
    f32 = np.float32
    if kind == "adam":
        names = ("W", "g", "m", "v", "lr", "beta1", "one_minus_beta1", "beta2", "one_minus_beta2", "eps")
        feeds = [W, grad, m, v, f32(0.01), f32(0.9), f32(1) - f32(0.9), f32(0.999), f32(1) - f32(0.999), f32(1e-8)]
        outs = ("W_new", "m_new", "v_new")
    else:
        names = ("W", "g", "v", "lr", "rho", "one_minus_rho", "eps")
        feeds = [W, grad, v, f32(0.01), f32(0.9), f32(1) - f32(0.9), f32(1e-8)]
        outs = ("W_new", "v_new")
    return g, [ids[k] for k in names], [ids[k] for k in outs], feeds


@pytest.mark.parametrize("kind", ["rmsprop", "adam"])
@pytest.mark.parametrize("shape", [[5 * 4096 + 3], [300, 1000]])
def test_rmsprop_and_adam_updater_graphs(kind, shape):
    """Sec. 3.2 names the RMSProp and Adam updaters: each is one fused VM launch, equal to the oracle."""
    g, inputs, outs, feeds = updater_case(kind, shape)
    got, f = run_gpu(g.desc, inputs, outs, feeds)
    assert f.num_launches() == 1, f.describe()
    ref = interp.run_function(g.desc, inputs, outs, feeds)
    for gv, rv in zip(got, ref):
        check(gv, rv, TOL32, kind)


def test_adam_in_place_over_several_steps():
    """The state of the update (W, m, v) stays in device memory: the fetch pointers are the feed pointers
    (dragon_function_can_alias says that this function allows it), five steps with fresh gradients, against
    the oracle run five times on its own fp64 state."""
    import torch
    from paper_1707_08265_b200 import binding as B
    n = 7 * 4096 + 11
    g, inputs, outs, feeds = updater_case("adam", [n])
    f = B.Graph.from_desc(g.desc).function(inputs, outs)
    assert f.can_alias(0, 0) and f.can_alias(2, 1) and f.can_alias(3, 2)     # W, m, v
    assert not f.can_alias(3, 1)                                             # v is still read after m' has been written
    dev = [torch.from_numpy(np.ascontiguousarray(a)).cuda() for a in feeds]
    state64 = [feeds[0].astype(np.float64), feeds[2].astype(np.float64), feeds[3].astype(np.float64)]
    rng = np.random.default_rng(5)
    for step in range(5):
        grad = (rng.standard_normal(n) * 0.1).astype(np.float32)
        dev[1].copy_(torch.from_numpy(grad))
        f.run_torch(dev, [dev[0], dev[2], dev[3]])
        assert f.status() == 0
        ref = interp.run_function(g.desc, inputs, outs, [state64[0], grad, state64[1], state64[2]] + feeds[4:])
        state64 = [ref[0], ref[1], ref[2]]
    torch.cuda.synchronize()
    for t, r, name in zip((dev[0], dev[2], dev[3]), state64, ("W", "m", "v")):
        check(t.cpu().numpy().astype(np.float64), r, 5 * TOL32, "after five steps: " + name)


@pytest.mark.parametrize("kind", ["sgd", "momentum"])
@pytest.mark.parametrize("shape", [[5 * 4096 + 3], [300, 1000]])
def test_updater_graph(kind, shape):
    g, ids = wl.updater(shape, kind)
    rng = np.random.default_rng(11)
    W = rng.standard_normal(shape).astype(np.float32)
    grad = (rng.standard_normal(shape) * 0.1).astype(np.float32)
    lr, mu = np.float32(0.05), np.float32(0.9)
    if kind == "sgd":
        inputs, feeds, outs = [ids["W"], ids["g"], ids["lr"]], [W, grad, lr], [ids["W_new"]]
    else:
        v = (rng.standard_normal(shape) * 0.1).astype(np.float32)
        inputs, feeds, outs = [ids["W"], ids["g"], ids["lr"], ids["v"], ids["mu"]], [W, grad, lr, v, mu], [ids["W_new"], ids["v_new"]]
    got, f = run_gpu(g.desc, inputs, outs, feeds)
    assert f.num_launches() == 1, f.describe()     # one fused VM launch for the whole update
    ref = interp.run_function(g.desc, inputs, outs, feeds)
    for gv, rv in zip(got, ref):
        check(gv, rv, TOL32, kind)
    if kind == "sgd":                              # and against the formula written out
        assert np.allclose(got[0], W.astype(np.float64) - float(lr) * grad.astype(np.float64), rtol=0, atol=2e-6)


def test_sine_of_huge_arguments_is_exact_and_leaves_its_neighbours_alone():
    """Arguments beyond 2^20 in magnitude take the exact multi-word reduction and match the oracle like
    any other; inf and NaN give NaN; the other elements of the same thread (and of every other
    thread) are untouched by the rare path."""
    n = 2 * 4096 + 100
    x = np.random.default_rng(3).standard_normal(n).astype(np.float32)
    odd = {5: 7.0e6, 6: -1.0e30, 7: 4.8e8, 8: -22026.0 * 22026.0, 2049: np.inf, 4096 + 17: -np.inf, 4096 + 2048 + 3: np.nan,
           n - 1: 3.0e8, n - 2: 3.4028235e38, n - 3: -1048577.0}
    for k, v in odd.items():
        x[k] = v
    gd = wl.GraphDesc()
    xi = gd.tensor("x", [n])
    out = gd.op("Sin", [xi], "out")
    grads = gd.grad([out], [xi])
    (s, c), _ = run_gpu(gd.desc, [xi], [out] + grads, [x])
    fin = np.isfinite(x)
    xd = x.astype(np.float64)
    check(s[fin], np.sin(xd[fin]), TOL32, "sin")
    check(c[fin], np.cos(xd[fin]), TOL32, "cos")
    # far tighter than the tolerance: a few ulp, as for small arguments
    assert np.max(np.abs(s[fin] - np.sin(xd[fin]))) < 3e-7 and np.max(np.abs(c[fin] - np.cos(xd[fin]))) < 3e-7
    for k, v in odd.items():
        if not np.isfinite(v):
            assert np.isnan(s[k]) and np.isnan(c[k]), (k, s[k], c[k])


def test_sine_of_huge_arguments_in_every_lane_and_tail():
    """Random bit patterns of every exponent from 2^20 up, in all eight lanes of a thread, in full tiles and
    in a ragged tail, through the separate sin and cos instructions as well as the paired one."""
    n = 3 * 4096 + 777
    rng = np.random.default_rng(9)
    e = rng.integers(147, 255, n).astype(np.uint32)
    x = ((rng.integers(0, 2, n).astype(np.uint32) << 31) | (e << 23) | rng.integers(0, 1 << 23, n).astype(np.uint32)).view(np.float32)
    x[::3] = rng.standard_normal(x[::3].size).astype(np.float32) * 100        # mixed with ordinary arguments
    gd = wl.GraphDesc()
    xi = gd.tensor("x", [n])
    out = gd.op("Sin", [xi], "out")
    (s,), _ = run_gpu(gd.desc, [xi], [out], [x])                               # sin alone
    xd = x.astype(np.float64)
    assert np.max(np.abs(s - np.sin(xd))) < 3e-7
    grads = gd.grad([out], [xi])
    (c,), _ = run_gpu(gd.desc, [xi], grads, [x])                               # cos alone
    assert np.max(np.abs(c - np.cos(xd))) < 3e-7


@pytest.mark.parametrize("outer,inner,scale", [("Tanh", "Sigmoid", 1), ("Tanh", "Sin", 1), ("Tanh", "Tanh", 4), ("Exp", "Tanh", 8),
                                               ("Sigmoid", "Sin", 64), ("Exp", "Sin", 16)])
def test_forms_without_clamps_over_their_whole_proven_range(outer, inner, scale):
    """outer(scale * inner(x)): the lowering proves |argument| <= scale and, where that is inside the range in which
    the clamps of outer do nothing, emits the form without them (tanhb up to 4, sigmoidb up to 80, expcb up to 9.99).
    Values and gradients against the oracle over a dense sweep of x that drives the inner function to both ends of
    its range, inf and NaN included; scale 16 > 9.99 keeps the clamped exponential (and its mask) in the comparison."""
    gd = wl.GraphDesc()
    xs = np.concatenate([sweep(-12, 8, 48), np.linspace(-20, 20, 4001).astype(np.float32), [np.inf, -np.inf, np.nan]]).astype(np.float32)
    n = xs.size
    x = gd.tensor("x", [n]); w = gd.tensor("w", [n])
    v = gd.op(inner, [x], "inner")
    k = 1
    while k < scale:                                   # scale * v by doubling
        v = gd.op("Add", [v, v], "v%d" % k); k *= 2
    y = gd.op(outer, [v], "outer")
    (dx,) = gd.grad([gd.op("Mul", [y, w], "obj")], [x])
    ws = np.random.default_rng(3).standard_normal(n).astype(np.float32)
    got, f = run_gpu(gd.desc, [x, w], [y, dx], [xs, ws])
    want_b = {"Tanh": scale <= 4, "Sigmoid": scale <= 80, "Exp": scale <= 9}[outer]
    name = {"Tanh": "tanh", "Sigmoid": "sigmoid", "Exp": "expc"}[outer]
    # the inner function may itself be one of the three: look at the last occurrence
    plan = f.describe()
    assert (name + "b") in plan if want_b else (name + ";") in plan.replace(name + "b", "#"), plan
    from test_gpu_vm import FLOOR_OK, C_COND
    fin = np.isfinite(xs)
    with np.errstate(all="ignore"):
        ref = interp.run_function(gd.desc, [x, w], [y, dx], [xs, ws])
        low = interp.run_function(gd.desc, [x, w], [y, dx], [xs, ws], dtype=np.float32)
    for gv, rv, lv, what in zip(got, ref, low, ("value", "gradient")):
        # a composition that saturates amplifies fp32 rounding (e^(8 tanh x) near its ends): held to the plain
        # tolerance where the CPU fp32 instance of the same graph reaches it, else to C_COND times that floor
        floor = float(np.max(np.abs(lv[fin].astype(np.float64) - rv[fin]) / (TOL32 * (1 + np.abs(rv[fin])))))
        tol = TOL32 if floor <= FLOOR_OK else TOL32 * C_COND * floor
        check(gv[fin], rv[fin], tol, "%s(%d*%s) %s (fp32 floor %.3g)" % (outer, scale, inner, what, floor))
        if what == "value":
            assert np.isnan(gv[np.isnan(xs)]).all(), what             # NaN in, NaN out
