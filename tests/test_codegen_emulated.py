"""The emitted VM programs, executed by the NumPy emulator of the instruction set and compared with
the oracle: checks lowering, dead-code removal, slot allocation (register slots, shared-memory
slots, spill slots), fusion peepholes and reduced outputs on the CPU."""
import numpy as np
import pytest

from oracle import interp, prune as oprune
from paper_1707_08265_b200 import binding as B
from paper_1707_08265_b200 import workloads as wl
from vm_emulator import run_step


def emulate(desc, inputs, outputs, feeds):
    f = B.Graph.from_desc(desc).function(inputs, outputs)
    assert f.num_launches() <= 2, f.describe()
    step = f.vm_step(0)
    shapes = {j: tuple(desc["tensors"][o]["shape"]) for j, o in enumerate(outputs)}
    out, colout, scalout = run_step(step, feeds, shapes, nr=step["n_regs"])
    for kind, acc, pos in step["reduced"]:
        out[pos] = np.asarray(colout[acc] if kind == 0 else scalout[acc], dtype=np.float64).reshape(shapes[pos])
    return [out[j] for j in range(len(outputs))], f


def close(a, b):
    return np.allclose(a, b, rtol=1e-9, atol=1e-9)


def test_toy_function_programs():
    n = 300
    g, ids = wl.toy_function_grad(n)
    x, a, b = wl.toy_feeds(n, 5)
    inputs = [ids["x"], ids["a"], ids["b"]]
    for outs in ([ids["dx"], ids["da"], ids["db"]], [ids["f"], ids["y"]], [ids["f"], ids["dx"], ids["db"]], [ids["da"]]):
        got, f = emulate(g.desc, inputs, outs, [x, a, b])
        ref = interp.run_function(g.desc, inputs, outs, [x, a, b])
        for gv, rv in zip(got, ref):
            assert close(gv, rv), f.describe()


@pytest.mark.parametrize("seed", range(30))
def test_random_elementwise_programs(seed):
    n = 97
    g, inputs, fetch = wl.random_dag(n, 500 + seed, n_ops=64, n_fetch=3)
    feeds = [a * 0.5 for a in wl.normal_feeds([[n]] * 4, 600 + seed)]
    grads = g.grad(fetch, [i for i in inputs if i in oprune.backward_marks(g.desc, fetch, inputs)])
    outs = fetch + grads
    got, f = emulate(g.desc, inputs, outs, feeds)
    ref = interp.run_function(g.desc, inputs, outs, feeds)
    for gv, rv in zip(got, ref):
        ok = np.isfinite(rv)
        assert np.allclose(gv[ok], rv[ok], rtol=1e-7, atol=1e-7), f.describe()


@pytest.mark.parametrize("seed", range(20))
def test_random_row_programs(seed):
    R, C = 5, 24
    g, inputs, fetch = wl.random_row_dag(R, C, 700 + seed, n_ops=80, n_fetch=3)
    wrts = [i for i in inputs if i in oprune.backward_marks(g.desc, fetch, inputs)]
    grads = g.grad(fetch, wrts)
    feeds = [a * 0.5 for a in wl.normal_feeds([g.shape(i) for i in inputs], 800 + seed)]
    outs = fetch + grads
    got, f = emulate(g.desc, inputs, outs, feeds)
    ref = interp.run_function(g.desc, inputs, outs, feeds)
    # the emulator computes in fp64 but the program's constants are fp32 (1/24 is not representable: a mean is
    # off by 3e-8 relative, and a row sum behind it multiplies that by up to the row length)
    for gv, rv in zip(got, ref):
        ok = np.isfinite(rv)
        assert np.allclose(gv[ok], rv[ok], rtol=2e-6, atol=1e-6), f.describe()


def test_register_pressure_program():
    n = 50
    gd = wl.GraphDesc()
    x = gd.tensor("x", [n])
    vals, cur = [], x
    for k in range(40):
        cur = gd.op("Sin" if k % 2 else "Tanh", [cur], "v%d" % k)
        vals.append(cur)
    acc = vals[0]
    for k, v in enumerate(vals[1:]):
        acc = gd.op("Add" if k % 3 else "Mul", [acc, v], "a%d" % k)
    (dx,) = gd.grad([acc], [x])
    xs = np.random.default_rng(1).standard_normal(n).astype(np.float32)
    got, f = emulate(gd.desc, [x], [acc, dx], [xs])
    assert f.vm_step(0)["n_spill"] > 0 and f.vm_step(0)["n_smem"] > 0
    ref = interp.run_function(gd.desc, [x], [acc, dx], [xs])
    assert close(got[0], ref[0]) and close(got[1], ref[1])
