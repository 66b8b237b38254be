"""The workspace of Sec. 3.1 through the C ABI: tensors that live in device memory under a name, fed and
fetched by name, functions run against them by name; the updaters of Sec. 3.2 keep their state there
between runs; an intermediate tensor that one function leaves in the workspace is an input of the next."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import interp
from paper_1707_08265_b200 import binding as B
from paper_1707_08265_b200 import workloads as wl

TOL32 = 1e-5
TOLBF = 1e-2


def addr(a):
    return a.ctypes.data_as(ctypes.c_void_p).value


def feed(ws, name, a, dtype=None):
    a = np.asarray(a)
    shape = list(a.shape)                      # () for a scalar: ascontiguousarray would make it (1,)
    if dtype == B.BF16:
        t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16).contiguous()
        ws.feed(name, B.BF16, shape, t.data_ptr())
        torch.cuda.synchronize()
        return
    code = B.I32 if a.dtype == np.int32 else B.F32
    buf = np.ascontiguousarray(a, dtype=np.int32 if code == B.I32 else np.float32)
    ws.feed(name, code, shape, addr(buf))
    torch.cuda.synchronize()


def fetch(ws, name):
    p, dt, shape = ws.tensor(name)
    if dt == B.BF16:
        t = torch.empty(shape, dtype=torch.bfloat16)
        ws.fetch(name, t.data_ptr(), t.numel() * 2)
        torch.cuda.synchronize()
        return t.float().numpy().astype(np.float64)
    out = np.empty(shape, dtype=np.int32 if dt == B.I32 else np.float32)
    ws.fetch(name, addr(out), out.nbytes)
    torch.cuda.synchronize()
    return out.astype(np.float64)


def check(got, ref, tol, what):
    err = np.abs(got - ref) / (tol * (1 + np.abs(ref)))
    assert got.shape == np.shape(ref) and np.all(err <= 1), (what, float(np.max(err)))


def test_workspace_errors_without_touching_a_device():
    ws = B.Workspace()
    assert ws.nbytes() == 0
    buf = np.zeros(4, np.float32)
    with pytest.raises(B.DragonError) as e:
        ws.fetch("nothing", addr(buf), 16)
    assert e.value.code == B.ERR_MISSING_INPUT
    with pytest.raises(B.DragonError):
        ws.tensor("nothing")
    with pytest.raises(B.DragonError) as e:
        ws.feed("x", 9, [4], addr(buf))
    assert e.value.code == B.ERR_DTYPE
    with pytest.raises(B.DragonError) as e:
        ws.feed("x", B.F32, [0], addr(buf))
    assert e.value.code == B.ERR_SHAPE
    g, ids = wl.toy_function(8)
    f = B.Graph.from_desc(g.desc).function([ids["x"], ids["a"], ids["b"]], [ids["y"]])
    with pytest.raises(B.DragonError) as e:
        ws.run(f)
    assert e.value.code == B.ERR_MISSING_INPUT and "'x'" in str(e.value)
    ws.close()


@pytest.mark.gpu
def test_feed_fetch_by_name_and_shape_checks():
    ws = B.Workspace()
    x = np.arange(12, dtype=np.float32).reshape(3, 4)
    feed(ws, "x", x)
    assert np.array_equal(fetch(ws, "x"), x)
    p, dt, shape = ws.tensor("x")
    assert dt == B.F32 and shape == [3, 4] and p % 256 == 0
    feed(ws, "x", x + 1)                                   # feeding again overwrites in the same memory
    assert ws.tensor("x")[0] == p and np.array_equal(fetch(ws, "x"), x + 1)
    with pytest.raises(B.DragonError) as e:
        feed(ws, "x", np.zeros((4, 3), np.float32))
    assert e.value.code == B.ERR_SHAPE
    with pytest.raises(B.DragonError) as e:
        feed(ws, "x", np.zeros((3, 4), np.int32))
    assert e.value.code == B.ERR_DTYPE
    with pytest.raises(B.DragonError) as e:
        ws.fetch("x", addr(np.zeros(5, np.float32)), 20)
    assert e.value.code == B.ERR_SHAPE
    ws.feed("zeros", B.F32, [1000], 0)                     # created without a source: zero-filled
    assert not fetch(ws, "zeros").any()
    dev = torch.arange(1000, dtype=torch.float32, device="cuda")
    ws.feed("zeros", B.F32, [1000], dev.data_ptr())        # a device pointer is a source too
    assert np.array_equal(fetch(ws, "zeros"), np.arange(1000.0))
    # a function whose input has another shape than the tensor of that name is refused before anything runs
    g, ids = wl.toy_function(8)
    f = B.Graph.from_desc(g.desc).function([ids["x"], ids["a"], ids["b"]], [ids["y"]])
    feed(ws, "a", np.float32(2))
    with pytest.raises(B.DragonError) as e:
        ws.run(f)
    assert e.value.code == B.ERR_SHAPE and "'x'" in str(e.value)
    ws.close()


@pytest.mark.gpu
def test_pruned_input_need_not_exist_and_outputs_are_created():
    n = 3 * 4096 + 5
    g, ids = wl.toy_function(n)
    x, a, b = wl.toy_feeds(n, 5)
    inputs = [ids["x"], ids["a"], ids["b"]]
    ws = B.Workspace()
    feed(ws, "x", x); feed(ws, "a", a)                      # b is never fed: y = a*x does not need it (Sec. 2.2)
    f = B.Graph.from_desc(g.desc).function(inputs, [ids["y"]])
    ws.run(f)
    assert f.status() == 0
    check(fetch(ws, "y"), interp.run_function(g.desc, inputs, [ids["y"]], [x, a, None])[0], TOL32, "y")
    f2 = B.Graph.from_desc(g.desc).function(inputs, [ids["f"]])
    with pytest.raises(B.DragonError) as e:
        ws.run(f2)
    assert e.value.code == B.ERR_MISSING_INPUT and "'b'" in str(e.value)
    feed(ws, "b", b)
    ws.run(f2, ["result"])                                  # bound to another name than the graph's
    check(fetch(ws, "result"), interp.run_function(g.desc, inputs, [ids["f"]], [x, a, b])[0], TOL32, "f")
    with pytest.raises(B.DragonError):
        ws.tensor("f")
    ws.close()


@pytest.mark.gpu
def test_adam_state_lives_in_the_workspace():
    """Sec. 3.2: the updater is a graph of its own; its outputs W', m', v' are bound to the names W, m, v.  The
    function allows the overwrite in place, so the three tensors keep their addresses and the workspace does
    not grow; six steps with fresh gradients against the oracle iterated on its own fp64 state."""
    n = 9 * 4096 + 7
    g, ids = wl.updater([n], "adam")
    names = ("W", "g", "m", "v", "lr", "beta1", "one_minus_beta1", "beta2", "one_minus_beta2", "eps")
    inputs = [ids[k] for k in names]
    outs = [ids[k] for k in ("W_new", "m_new", "v_new")]
    f = B.Graph.from_desc(g.desc).function(inputs, outs)
    rng = np.random.default_rng(2)
    W0 = rng.standard_normal(n).astype(np.float32)
    f32 = np.float32
    hyper = [f32(0.01), f32(0.9), f32(1) - f32(0.9), f32(0.999), f32(1) - f32(0.999), f32(1e-8)]
    ws = B.Workspace()
    feed(ws, "W", W0)
    ws.feed("m", B.F32, [n], 0); ws.feed("v", B.F32, [n], 0)          # moments start at zero
    for k, val in zip(names[4:], hyper):
        feed(ws, k, val)
    state = [W0.astype(np.float64), np.zeros(n), np.zeros(n)]
    addr0, size0 = None, None
    for step in range(6):
        grad = (rng.standard_normal(n) * 0.1).astype(np.float32)
        feed(ws, "g", grad)
        ws.run(f, ["W", "m", "v"])
        assert f.status() == 0
        if step == 0:
            addr0, size0 = [ws.tensor(k)[0] for k in ("W", "m", "v")], ws.nbytes()
        state = interp.run_function(g.desc, inputs, outs, [state[0], grad, state[1], state[2]] + hyper)
    assert [ws.tensor(k)[0] for k in ("W", "m", "v")] == addr0 and ws.nbytes() == size0
    for k, ref in zip(("W", "m", "v"), state):
        check(fetch(ws, k), ref, 6 * TOL32, "after six steps: " + k)
    ws.close()


@pytest.mark.gpu
def test_an_update_that_cannot_run_in_place_goes_through_a_second_buffer():
    """W' = W - lr * g / (1 + |row sum of g*W|) over [R, C] is a row program: a thread block reads a whole
    row of W before it writes, and other rows are in flight, so the library does not promise an in-place
    run.  The workspace writes W' to a second buffer and lets the name W point to it; the two buffers
    alternate from step to step and the values follow the oracle."""
    R, C = 50, 777
    gd = wl.GraphDesc()
    W = gd.tensor("W", [R, C]); G = gd.tensor("g", [R, C]); lr = gd.tensor("lr", [])
    s = gd.op("Sum", [gd.op("Mul", [G, W], "gw")], "s")
    upd = gd.op("Mul", [lr, gd.op("Div", [G, s], "scaled")], "upd")
    Wn = gd.op("Sub", [W, upd], "W_new")
    inputs = [W, G, lr]
    f = B.Graph.from_desc(gd.desc).function(inputs, [Wn])
    assert f.can_alias(0, 0) == 0
    rng = np.random.default_rng(4)
    w0 = rng.standard_normal((R, C)).astype(np.float32)
    ws = B.Workspace()
    feed(ws, "W", w0); feed(ws, "lr", np.float32(0.1))
    ref = w0.astype(np.float64)
    seen = []
    for step in range(4):
        grad = rng.standard_normal((R, C)).astype(np.float32)
        feed(ws, "g", grad)
        ws.run(f, ["W"])
        assert f.status() == 0
        seen.append(ws.tensor("W")[0])
        (ref,) = interp.run_function(gd.desc, inputs, [Wn], [ref, grad, np.float32(0.1)])
        check(fetch(ws, "W"), ref, (step + 1) * TOL32, "step %d" % step)
    assert seen[0] != seen[1] and seen[0] == seen[2] and seen[1] == seen[3]
    ws.close()
    # two outputs cannot be bound to one name
    g2, ids2 = wl.updater([8], "momentum")
    f2 = B.Graph.from_desc(g2.desc).function([ids2[k] for k in ("W", "g", "lr", "v", "mu")], [ids2["W_new"], ids2["v_new"]])
    ws2 = B.Workspace()
    for k in ("W", "g", "v"):
        feed(ws2, k, np.zeros(8, np.float32))
    feed(ws2, "lr", np.float32(1)); feed(ws2, "mu", np.float32(1))
    with pytest.raises(B.DragonError) as e:
        ws2.run(f2, ["same", "same"])
    assert e.value.code == B.ERR_INVALID_ARG
    ws2.run(f2, ["W", "v"])
    ws2.close()


@pytest.mark.gpu
def test_two_functions_meet_in_the_workspace_at_an_intermediate_tensor():
    """Sec. 3.1: feed and fetch any tensor.  The first function leaves h (the first layer's activations) in the
    workspace; the second lists h among its inputs, so its graph starts there: the loss and the second layer's
    gradients equal those of the function that computes everything at once."""
    batch, d_in, d_hid, d_out = 256, 192, 320, 136
    g, ids = wl.mlp(batch, d_in, d_hid, d_out)
    X, W1, b1, W2, b2, labels = wl.mlp_feeds(batch, d_in, d_hid, d_out, 21)
    ws = B.Workspace()
    for name, a in (("X", X), ("W1", W1), ("b1", b1), ("W2", W2), ("b2", b2)):
        feed(ws, name, a, B.BF16)
    feed(ws, "labels", labels)
    G = B.Graph.from_desc(g.desc)
    first = G.function([ids["X"], ids["W1"], ids["b1"]], [ids["h"]])
    second = G.function([ids["h"], ids["W2"], ids["b2"], ids["labels"]], [ids["loss"], ids["dW2"], ids["db2"]])
    assert second.kept_ops()[0] == [4, 5, 6]
    ws.run(first)
    ws.run(second)
    assert first.status() == 0 and second.status() == 0
    inputs = [ids[k] for k in ("X", "W1", "b1", "W2", "b2", "labels")]
    ref = interp.run_function(g.desc, inputs, [ids["h"], ids["loss"], ids["dW2"], ids["db2"]], [X, W1, b1, W2, b2, labels])
    names = ("h", "loss", g.desc["tensors"][ids["dW2"]]["name"], g.desc["tensors"][ids["db2"]]["name"])
    for name, rv in zip(names, ref):
        got = fetch(ws, name)
        check(got, rv, TOLBF, name)
        assert np.max(np.abs(got - rv)) <= 0.03 * np.max(np.abs(rv)) + 1e-12, name
    ws.close()


@pytest.mark.gpu
def test_training_loop_inside_the_workspace():
    """The training graph and one SGD updater graph per parameter (Sec. 3.2: separate graphs, neither is cyclic)
    share tensors by name: the training function leaves loss and the four gradients in the workspace, each
    updater reads its parameter and that gradient and writes the parameter.  Nothing but the scalar loss leaves
    the device.  The loss falls, and its trajectory follows the oracle doing the same steps on its own state."""
    batch, d_in, d_hid, d_out = 128, 64, 128, 16
    g, ids = wl.mlp(batch, d_in, d_hid, d_out)
    X, W1, b1, W2, b2, labels = wl.mlp_feeds(batch, d_in, d_hid, d_out, 31)
    train_in = [ids[k] for k in ("X", "W1", "b1", "W2", "b2", "labels")]
    train_out = [ids[k] for k in ("loss", "dW1", "db1", "dW2", "db2")]
    train = B.Graph.from_desc(g.desc).function(train_in, train_out)
    params = {"W1": W1, "b1": b1, "W2": W2, "b2": b2}
    updaters = {}
    for p, val in params.items():
        gd = wl.GraphDesc()
        P = gd.tensor(p, list(val.shape), "bf16")
        dP = gd.tensor(g.desc["tensors"][ids["d" + p]]["name"], list(val.shape), "f32")
        lr = gd.tensor("lr", [])
        Pn = gd.op("Sub", [P, gd.op("Mul", [lr, dP], "step")], p + "_new", out_dtype="bf16")
        updaters[p] = (gd, [P, dP, lr], Pn, B.Graph.from_desc(gd.desc).function([P, dP, lr], [Pn]))
    ws = B.Workspace()
    feed(ws, "X", X, B.BF16); feed(ws, "labels", labels); feed(ws, "lr", np.float32(0.5))
    for p, val in params.items():
        feed(ws, p, val, B.BF16)
    ref_params = {p: v.astype(np.float64) for p, v in params.items()}
    losses, ref_losses = [], []
    for step in range(8):
        ws.run(train)
        for p, (gd, ins, out, fn) in updaters.items():
            ws.run(fn, [p])
        losses.append(float(fetch(ws, "loss")))
        r = interp.run_function(g.desc, train_in, train_out,
                                [X, ref_params["W1"], ref_params["b1"], ref_params["W2"], ref_params["b2"], labels])
        ref_losses.append(float(r[0]))
        for p, grad in zip(("W1", "b1", "W2", "b2"), r[1:]):
            gd, ins, out, fn = updaters[p]
            (ref_params[p],) = interp.run_function(gd.desc, ins, [out], [ref_params[p], grad, np.float32(0.5)])
    assert train.status() == 0
    assert losses[-1] < 0.7 * losses[0], losses
    for a, b in zip(losses, ref_losses):
        assert abs(a - b) <= 2e-2 * (1 + abs(b)), (losses, ref_losses)
    ws.close()
