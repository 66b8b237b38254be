"""The two execution tiers of a graph-VM program on the GPU: the interpreter kernel and the kernel specialised
for the program (the same leaves as straight-line code).  Both must return the same bits, whatever the
program: flat and row programs, ragged tails, reductions, spills, several segments, the general sine
reduction, the chunked host-buffer run.  (The parity tests proper run the default tier, the specialised
one, against the oracle; the equality here carries their verdict over to the interpreter.)"""
import numpy as np
import pytest
import torch

from oracle import prune as oprune
from paper_1707_08265_b200 import binding as B
from paper_1707_08265_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def bits(t):
    return t.detach().cpu().contiguous().view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32).numpy()


def run_tier(desc, inputs, outputs, dev_feeds, tier):
    f = B.Graph.from_desc(desc).function(inputs, outputs)
    n_vm = sum(f.vm_step(k) is not None for k in range(f.num_launches() + 4))
    if tier:
        assert f.specialize(2) == n_vm and f.num_specialized() == n_vm, f.describe()
    else:
        f.specialize(0)
    tdt = {"f32": torch.float32, "bf16": torch.bfloat16}
    outs = [torch.full(tuple(desc["tensors"][o]["shape"]), float("nan"), dtype=tdt[desc["tensors"][o]["dtype"]], device="cuda") for o in outputs]
    f.run_torch(dev_feeds, outs)
    assert f.status() == 0
    torch.cuda.synchronize()
    assert f.num_specialized() == (n_vm if tier else 0) and "interpreted" not in f.describe()
    return outs, f


def same_bits(desc, inputs, outputs, feeds, what):
    dev = [None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda() for a in feeds]
    a, _ = run_tier(desc, inputs, outputs, dev, 0)
    b, f = run_tier(desc, inputs, outputs, dev, 1)
    for k, (x, y) in enumerate(zip(a, b)):
        assert np.array_equal(bits(x), bits(y)), "%s: output %d differs between the tiers" % (what, k)
    return f


@pytest.mark.parametrize("n", [1, 4095, 3 * 4096 + 5, (1 << 22) + 77])
def test_toy_gradients_same_bits(n):
    g, ids = wl.toy_function_grad(n)
    x, a, b = wl.toy_feeds(n, 3)
    same_bits(g.desc, [ids["x"], ids["a"], ids["b"]], [ids["f"], ids["dx"], ids["da"], ids["db"]], [x, a, b], "toy")


@pytest.mark.parametrize("seed", range(8))
def test_random_elementwise_dags_same_bits(seed):
    n = 5 * 4096 + 77
    g, inputs, fetch = wl.random_dag(n, 1000 + seed, n_ops=64)
    same_bits(g.desc, inputs, fetch, wl.normal_feeds([[n]] * 4, 2000 + seed), "dag %d" % seed)


@pytest.mark.parametrize("seed", range(8))
def test_random_row_dags_with_gradients_same_bits(seed):
    R, C = 300, 520 if seed % 2 else 4096
    g, inputs, fetch = wl.random_row_dag(R, C, 3000 + seed, n_ops=48, n_fetch=2)
    G = oprune.backward_marks(g.desc, fetch, inputs)
    grads = g.grad(fetch, [i for i in inputs if i in G])
    feeds = [a * np.float32(0.5) for a in wl.normal_feeds([g.shape(i) for i in inputs], 4000 + seed)]
    same_bits(g.desc, inputs, fetch + grads, feeds, "rows %d" % seed)


def test_many_operators_kept_several_segments_same_bits():
    R, C = 64, 4096
    g, inputs, fetch = wl.random_row_dag(R, C, 77, n_ops=1024, n_fetch=24)
    feeds = [a * np.float32(0.5) for a in wl.normal_feeds([g.shape(i) for i in inputs], 5)]
    f = same_bits(g.desc, inputs, fetch, feeds, "1024 operators")
    assert f.num_specialized() >= 1


def test_spills_and_shared_memory_slots_same_bits():
    n = 3 * 4096 + 9
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
    f = same_bits(gd.desc, [x], [acc, dx], [np.random.default_rng(1).standard_normal(n).astype(np.float32)], "spills")
    assert "spill=0" not in f.describe()


def test_huge_sine_arguments_take_the_general_reduction_in_both_tiers():
    n = 4096 * 2 + 11
    gd = wl.GraphDesc()
    x = gd.tensor("x", [n])
    s = gd.op("Sin", [x], "s")
    t = gd.op("Mul", [s, gd.op("Sin", [gd.op("Mul", [x, x], "xx")], "s2")], "t")
    (dx,) = gd.grad([t], [x])
    rng = np.random.default_rng(9)
    xs = (rng.standard_normal(n) * np.exp2(rng.integers(-3, 60, n))).astype(np.float32)
    xs[5], xs[6], xs[4097] = np.inf, np.nan, -3.0e38
    same_bits(gd.desc, [x], [s, t, dx], [xs], "sine")


@pytest.mark.parametrize("kind", ["sgd", "momentum", "rmsprop", "adam"])
def test_updaters_same_bits(kind):
    from test_gpu_math_and_updater import updater_case
    n = 6 * 4096 + 3
    if kind in ("rmsprop", "adam"):
        g, inputs, outs, feeds = updater_case(kind, [n])
    else:
        g, ids = wl.updater([n], kind)
        rng = np.random.default_rng(1)
        names = ("W", "g", "lr") if kind == "sgd" else ("W", "g", "lr", "v", "mu")
        vals = {"W": rng.standard_normal(n), "g": rng.standard_normal(n), "v": rng.standard_normal(n), "lr": 0.05, "mu": 0.9}
        inputs, feeds = [ids[k] for k in names], [np.asarray(vals[k], dtype=np.float32) for k in names]
        outs = [ids["W_new"]] + ([ids["v_new"]] if kind == "momentum" else [])
    same_bits(g.desc, inputs, outs, feeds, kind)


def test_host_buffer_run_in_chunks_same_bits():
    """dragon_run_host cuts a flat elementwise function into chunks with copies on streams of its own; the
    specialised kernel takes the same parameters as the interpreter, chunk by chunk."""
    n = (1 << 23) + 4096 * 3 + 17
    g, ids = wl.toy_function_grad(n)
    inputs, outputs = [ids["x"], ids["a"], ids["b"]], [ids["dx"], ids["da"], ids["db"]]
    x, a, b = wl.toy_feeds(n, 4)
    res = []
    for tier in (0, 1):
        f = B.Graph.from_desc(g.desc).function(inputs, outputs)
        f.specialize(2 if tier else 0)
        f.ensure_workspace()
        staging = torch.empty(f.staging_bytes() + 256, dtype=torch.uint8, device="cuda")
        base = (staging.data_ptr() + 255) & ~255
        hx = torch.from_numpy(x).pin_memory(); ha = torch.tensor(float(a)).pin_memory(); hb = torch.tensor(float(b)).pin_memory()
        outs = [torch.full((n,), float("nan")).pin_memory(), torch.zeros(()).pin_memory(), torch.zeros(()).pin_memory()]
        f.run_host([hx.data_ptr(), ha.data_ptr(), hb.data_ptr()], [o.data_ptr() for o in outs], base, f.staging_bytes(),
                   torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert f.status() == 0 and f.num_specialized() == tier
        res.append([o.clone() for o in outs])
    for k in range(3):
        assert np.array_equal(bits(res[0][k]), bits(res[1][k])), k


def test_without_an_assembler_the_interpreter_runs_and_says_so(monkeypatch):
    """A driver without the PTX assembler (simulated on the host): in the default mode the program stays with
    the interpreter, the plan says why, the results are the oracle's; asking for specialisation outright fails."""
    from oracle import interp
    monkeypatch.setenv("DRAGON_VM_NO_ASSEMBLER", "1")
    n = 3 * 4096 + 5
    g, ids = wl.toy_function_grad(n)
    inputs, outputs = [ids["x"], ids["a"], ids["b"]], [ids["dx"], ids["da"], ids["db"]]
    x, a, b = wl.toy_feeds(n, 3)
    f = B.Graph.from_desc(g.desc).function(inputs, outputs)
    f.specialize(1)
    dev = [torch.from_numpy(np.ascontiguousarray(v)).cuda() for v in (x, a, b)]
    outs = [torch.full(tuple(g.shape(o)), float("nan"), device="cuda") for o in outputs]
    f.run_torch(dev, outs)
    assert f.status() == 0 and f.num_specialized() == 0
    assert "runs interpreted: no assembler" in f.describe()
    ref = interp.run_function(g.desc, inputs, outputs, [x, a, b])
    for o, r in zip(outs, ref):
        assert np.all(np.abs(o.cpu().numpy() - r) <= 1e-5 * (1 + np.abs(r)))
    f2 = B.Graph.from_desc(g.desc).function(inputs, outputs)
    with pytest.raises(B.DragonError) as e:
        f2.specialize(2)
    assert e.value.code == B.ERR_CUDA and "no assembler" in str(e.value)
