"""Host side of the library through the C ABI, no GPU: exported symbols, error codes, prune sets
and operator order against the oracle (bit-exact), linear-time pruning of a long chain."""
import ctypes
import os
import re
import time

import numpy as np
import pytest

from oracle import prune as oprune
from paper_1707_08265_b200 import binding as B
from paper_1707_08265_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "dragon.h")).read()
    names = set(re.findall(r"\b(dragon_[a-z_]+)\s*\(", header))
    assert len(names) >= 20
    L = ctypes.CDLL(B.LIB_PATH)
    for n in sorted(names):
        assert hasattr(L, n), n
    assert names == set(B._SIGNATURES), names ^ set(B._SIGNATURES)


def compare_sets(desc, inputs, outputs):
    want = oprune.function_sets(desc, inputs, outputs)
    g = B.Graph.from_desc(desc)
    f = g.function(inputs, outputs)
    fwd, gops, masks = f.kept_ops()
    assert f.marked() == want["marked"]
    assert fwd == want["fwd_ops"]
    assert gops == [k for (_, k, _) in want["grad_ops"]]
    assert masks == [sum(1 << p for p in pos) for (_, _, pos) in want["grad_ops"]]
    assert f.used_inputs() == want["used_inputs"]
    return f


def test_paper_example_through_the_c_abi():
    g, ids = wl.toy_function_grad(1 << 12)
    inputs = [ids["x"], ids["a"], ids["b"]]
    f = compare_sets(g.desc, inputs, [ids["y"]])
    assert f.used_inputs() == [1, 1, 0] and f.kept_ops()[0] == [0]      # b is redundant (Sec. 2.2)
    compare_sets(g.desc, inputs, [ids["f"], ids["y"]])
    compare_sets(g.desc, inputs, [ids["dx"], ids["da"], ids["db"]])
    compare_sets(g.desc, inputs, [ids["db"]])
    compare_sets(g.desc, inputs, [ids["f"], ids["da"]])


@pytest.mark.parametrize("seed", range(12))
def test_random_dag_prune_sets_match_oracle(seed):
    g, inputs, fetch = wl.random_dag(1000, seed, n_ops=40)
    compare_sets(g.desc, inputs, fetch)
    compare_sets(g.desc, inputs, fetch[:1])


@pytest.mark.parametrize("seed", range(8))
def test_random_row_dag_with_gradients_matches_oracle(seed):
    g, inputs, fetch = wl.random_row_dag(8, 16, seed, n_ops=60)
    G = oprune.backward_marks(g.desc, fetch, inputs)
    wrts = [i for i in inputs if i in G]
    grads = g.grad(fetch, wrts)
    compare_sets(g.desc, inputs, fetch + grads)
    compare_sets(g.desc, inputs, grads[:1])
    compare_sets(g.desc, inputs, fetch[:1] + grads[-1:])


def test_mlp_prune_sets():
    g, ids = wl.mlp(64, 32, 32, 16)
    inputs = [ids[k] for k in ("X", "W1", "b1", "W2", "b2", "labels")]
    f = compare_sets(g.desc, inputs, [ids[k] for k in ("loss", "dW1", "db1", "dW2", "db2")])
    plan = f.describe()
    assert plan.count("gemm") == 5                      # two forward, dW2, dH, dW1; no dX of layer 1
    compare_sets(g.desc, inputs, [ids["loss"]])
    compare_sets(g.desc, inputs, [ids["dW2"]])


def test_two_gradient_stages():
    g, ids = wl.toy_function(16)
    s0 = g.grad([ids["f"]], [ids["x"], ids["b"]])
    s1 = g.grad([ids["y"]], [ids["a"]])
    inputs = [ids["x"], ids["a"], ids["b"]]
    compare_sets(g.desc, inputs, s0 + s1)
    f = compare_sets(g.desc, inputs, s1)
    assert f.used_inputs() == [1, 1, 0]


def test_error_codes():
    g = B.Graph()
    x = g.add_tensor("x", B.F32, [4, 8])
    r = g.add_tensor("r", B.F32, [8])
    bad = g.add_tensor("bad", B.F32, [7])
    lab = g.add_tensor("lab", B.I32, [4])
    y = g.add_tensor("y", B.F32, [4, 8])
    y2 = g.add_tensor("y2", B.F32, [4, 9])

    def code(fn):
        with pytest.raises(B.DragonError) as e:
            fn()
        return e.value.code

    assert code(lambda: g.add_tensor("x", B.F32, [1])) == B.ERR_INVALID_ARG           # duplicate name
    assert code(lambda: g.add_tensor("z", 7, [1])) == B.ERR_DTYPE
    assert code(lambda: g.add_tensor("z", B.F32, [0])) == B.ERR_SHAPE
    assert code(lambda: g.add_op(B.OPS["Add"], [x, bad], [y])) == B.ERR_SHAPE          # no broadcast
    assert code(lambda: g.add_op(B.OPS["Add"], [x, r], [y2])) == B.ERR_SHAPE           # declared != inferred
    assert code(lambda: g.add_op(B.OPS["Add"], [x, lab], [y])) == B.ERR_DTYPE
    assert code(lambda: g.add_op(B.OPS["Add"], [x, y], [y])) == B.ERR_NOT_SSA          # reads its own output
    assert code(lambda: g.add_op(99, [x, r], [y])) == B.ERR_INVALID_ARG
    assert g.add_op(B.OPS["Add"], [x, r], [y]) == 0
    assert code(lambda: g.add_op(B.OPS["Add"], [x, r], [y])) == B.ERR_NOT_SSA          # second producer
    z = g.add_tensor("z", B.F32, [4, 8])
    assert code(lambda: g.add_grad([y], [bad])) == B.ERR_NO_PATH
    (dr,) = g.add_grad([y], [r])
    assert code(lambda: g.add_op(B.OPS["Sin"], [dr], [z])) == B.ERR_UNSUPPORTED        # gradient tensors are terminal
    with pytest.raises(B.DragonError):
        g.function([r], [y])                                                           # x is needed but not listed
    assert b"not among the inputs" in B.lib().dragon_last_error()
    f = g.function([x, r, y], [y])                                                     # y is given: nothing is computed
    assert f.used_inputs() == [0, 0, 1] and f.kept_ops()[0] == []
    with pytest.raises(B.DragonError):
        g.function([x, r, dr], [y])                                                    # a gradient tensor cannot be fed
    with pytest.raises(B.DragonError) as e:
        g.function([x, r, y], [dr])                                                    # the only chain r -> y is cut
    assert "no chain is left" in str(e.value)
    f = g.function([x, r, bad], [y, dr])
    assert f.used_inputs() == [1, 1, 0]
    assert f.workspace_bytes() > 0 and f.num_launches() >= 1
    with pytest.raises(B.DragonError) as e:
        f.run([0, 0, 0], [0, 0])                                                       # no workspace yet
    assert e.value.code == B.ERR_WORKSPACE


def test_long_chain_prunes_in_linear_time_without_recursion():
    def build(n):
        g = B.Graph()
        prev = g.add_tensor("x", B.F32, [8])
        for k in range(n):
            nxt = g.add_tensor("t%d" % k, B.F32, [8])
            g.add_op(B.OPS["Tanh"] if k % 2 else B.OPS["Sin"], [prev], [nxt])
            prev = nxt
        return g, prev

    lib = B.lib()
    times = []
    for n in (50000, 200000):
        g, last = build(n)
        dx = g.add_grad([last], [0])
        ins = (ctypes.c_int32 * 1)(0)
        outs = (ctypes.c_int32 * 2)(last, dx[0])
        # only the two prunes are timed here: lowering a 200000-operator fused segment is not the claim
        t0 = time.perf_counter()
        ok = lib.dragon_add_grad(g.h, (ctypes.c_int32 * 1)(last), 1, (ctypes.c_int32 * 1)(0), 1, (ctypes.c_int32 * 1)())
        times.append(time.perf_counter() - t0)
        assert ok == 0
    assert times[1] < 12 * times[0] + 0.05


def test_limits_are_reported_not_faulted():
    # a row reduction over rows longer than one tile is refused at compile time
    g = B.Graph()
    x = g.add_tensor("x", B.F32, [4, 5000])
    y = g.add_tensor("y", B.F32, [4, 5000])
    g.add_op(B.OPS["Sum"], [x], [y])
    with pytest.raises(B.DragonError):
        g.function([x], [y])
    assert b"rows longer than" in B.lib().dragon_last_error()
    # the same shape without a row operation is a flat elementwise function and compiles
    g2 = B.Graph()
    x2 = g2.add_tensor("x", B.F32, [4, 5000])
    y2 = g2.add_tensor("y", B.F32, [4, 5000])
    g2.add_op(B.OPS["Tanh"], [x2], [y2])
    f = g2.function([x2], [y2])
    assert "vm[flat" in f.describe() and " n=20000 " in f.describe()
    # fetching the same tensor twice is refused
    with pytest.raises(B.DragonError):
        g2.function([x2], [y2, y2])


def test_bias_relu_after_a_product_fuse_into_its_epilogue():
    """Lowering: a segment that only adds a row vector to an InnerProduct's result, clamps and rounds
    it, becomes the product's epilogue; a second reader of the product prevents it."""
    from paper_1707_08265_b200 import workloads as wl
    g, ids = wl.mlp(256, 128, 192, 64)
    inputs = [ids[k] for k in ("X", "W1", "b1", "W2", "b2", "labels")]
    f = B.Graph.from_desc(g.desc).function(inputs, [ids[k] for k in ("loss", "dW1", "db1", "dW2", "db2")])
    text = f.describe()
    assert text.count("+bias") == 2 and text.count("relu") == 1 and text.count("*step") == 1, text
    assert " step;" not in text and " mul " not in text, text          # the mask is applied in the product's epilogue
    assert "gld" not in text.split("softmax")[0], text          # no elementwise launch before the loss
    # the pre-activation fetched as well: the first product keeps a launch of its own
    f2 = B.Graph.from_desc(g.desc).function(inputs, [ids["loss"], ids["z1"]])
    assert f2.describe().count("+bias") == 1, f2.describe()


@pytest.mark.parametrize("bias_first", [True, False])
def test_epilogue_fusion_needs_the_bias_in_memory_before_the_product_runs(bias_first):
    from paper_1707_08265_b200 import workloads as wl
    m, n, k = 64, 128, 64
    gd = wl.GraphDesc()
    X = gd.tensor("X", [m, k], "bf16"); W = gd.tensor("W", [n, k], "bf16"); b = gd.tensor("b", [n], "f32")
    if bias_first:
        tb = gd.op("Tanh", [b], "tb")
    Z = gd.op("InnerProduct", [X, W], "Z", [m, n], "f32")
    if not bias_first:
        tb = gd.op("Tanh", [b], "tb")
    Y = gd.op("BiasAdd", [Z, tb], "Y", [m, n], "f32")
    f = B.Graph.from_desc(gd.desc).function([X, W, b], [Y])
    text = f.describe()
    assert ("+bias" in text) == bias_first, text


@pytest.mark.parametrize("n_scalars", [8, 9, 10, 14, 30])
def test_many_reduced_outputs_fit_the_finishing_launch_or_are_refused(n_scalars):
    """Gradients with respect to k scalars are k sums over the whole domain.  One segment holds 4 scalar
    accumulators, 5 pinned register slots and, beyond those, pinned shared-memory slots; the finishing
    launch has a job table sized for all of them.  Up to 20 sums are one program with exactly k jobs (and
    compute the right sums, checked on the instruction-set emulator); more are cut into several programs."""
    from vm_emulator import run_step
    n = 3 * 4096 + 5
    gd = wl.GraphDesc()
    x = gd.tensor("x", [n])
    ss = [gd.tensor("s%d" % k, []) for k in range(n_scalars)]
    acc = None
    for k, s in enumerate(ss):
        t = gd.op("Mul", [s, gd.op("Sin" if k % 2 else "Tanh", [x], "u%d" % k)], "t%d" % k)
        acc = t if acc is None else gd.op("Add", [acc, t], "a%d" % k)
    grads = gd.grad([acc], ss)
    f = B.Graph.from_desc(gd.desc).function([x] + ss, grads)
    steps = [st for st in (f.vm_step(i) for i in range(16)) if st]
    assert sum(len(st["reduced"]) for st in steps) == n_scalars and all(len(st["reduced"]) <= 20 for st in steps)
    if n_scalars > 20:      # more than one program holds: the lowering cut the segment in two
        assert len(steps) >= 2
        return
    step = steps[0]
    assert len(steps) == 1
    rng = np.random.default_rng(n_scalars)
    feeds = [rng.standard_normal(n)] + [rng.standard_normal() for _ in ss]
    _, _, scal = run_step(step, feeds, {})
    for k in range(n_scalars):
        want = float(np.sum(np.sin(feeds[0]) if k % 2 else np.tanh(feeds[0])))
        kind, accidx, pos = step["reduced"][[r[2] for r in step["reduced"]].index(k)]
        assert kind == 1 and abs(scal[accidx] - want) <= 1e-9 * (1 + abs(want)), (k, scal[accidx], want)


@pytest.mark.parametrize("seed", range(60))
def test_multi_output_operators_are_pruned_by_the_library_like_by_the_oracle(seed):
    """Sec. 2.2: an operator connects each of its inputs to each of its outputs.  Tiny DAGs with one- and
    two-output opaque operators and one or two gradient stages, replayed through the C ABI: marks, kept
    operators, masks and used inputs equal the oracle's (which is itself pinned by path enumeration); a
    function that keeps an opaque operator compiles and refuses to run."""
    from test_oracle_prune import tiny_dag_with_stages
    rng = np.random.default_rng(9000 + seed)
    d, fetch = tiny_dag_with_stages(rng)
    f = compare_sets(d, [0, 1, 2], fetch)
    if f.kept_ops()[0]:
        assert "not executable" in f.describe() and f.num_launches() == 0
        with pytest.raises(B.DragonError) as e:
            f.run([0, 0, 0], [0] * len(fetch))
        assert e.value.code == B.ERR_UNSUPPORTED and "opaque" in str(e.value)


@pytest.mark.parametrize("seed", range(60))
def test_fed_intermediates_are_pruned_by_the_library_like_by_the_oracle(seed):
    """Sec. 3.1: any tensor can be fed.  The same tiny DAGs with one or two produced tensors among the inputs:
    the library's sets equal the oracle's (pinned by path enumeration on the graph without the edges into the
    given tensors), and a fetched gradient that has lost its chains is refused with NO_PATH by both."""
    from test_oracle_prune import tiny_dag_with_stages
    rng = np.random.default_rng(9000 + seed)
    d, fetch = tiny_dag_with_stages(rng)
    n_fwd = len(d["tensors"]) - sum(len(st["wrts"]) for st in d["grads"])
    fed = [int(t) for t in rng.choice(np.arange(3, n_fwd), size=int(rng.integers(1, 3)), replace=False)]
    inputs = [0, 1, 2] + fed
    try:
        oprune.function_sets(d, inputs, fetch)
    except ValueError:
        with pytest.raises(B.DragonError) as e:
            B.Graph.from_desc(d).function(inputs, fetch)
        assert "no chain is left" in str(e.value)
        return
    compare_sets(d, inputs, fetch)


@pytest.mark.parametrize("seed", range(8))
def test_fed_intermediates_in_random_row_dags_with_gradients(seed):
    g, inputs, fetch = wl.random_row_dag(8, 16, seed, n_ops=60)
    kept = oprune.function_sets(g.desc, inputs, fetch)["fwd_ops"]
    rng = np.random.default_rng(seed)
    fed = sorted({g.desc["ops"][int(k)]["out"][0] for k in rng.choice(kept, size=min(3, len(kept)), replace=False)} - set(fetch))
    G = oprune.backward_marks(oprune.without_edges_into(g.desc, inputs + fed), fetch, inputs + fed)
    wrts = [i for i in inputs + fed if i in G]
    grads = g.grad(fetch, wrts) if wrts else []
    f = compare_sets(g.desc, inputs + fed, fetch + grads)
    assert "not executable" not in f.describe()
    for t in fed:                                       # what produced a given tensor is kept only for other readers
        k = next(k for k, op in enumerate(g.desc["ops"]) if t in op["out"])
        assert k not in f.kept_ops()[0]


def test_an_opaque_operator_that_is_pruned_away_does_not_stop_execution():
    g = B.Graph()
    x = g.add_tensor("x", B.F32, [100])
    y = g.add_tensor("y", B.F32, [100])
    u = g.add_tensor("u", B.F32, [7])
    v = g.add_tensor("v", B.F32, [3, 3])
    g.add_op(B.OPS["Tanh"], [x], [y])
    g.add_op(B.OPS["Opaque"], [x, y], [u, v])                  # two outputs of arbitrary declared shapes
    f = g.function([x], [y])
    assert f.kept_ops()[0] == [0] and f.marked() == [1, 1, 0, 0] and "vm[" in f.describe()
    f2 = g.function([x], [v])
    assert f2.kept_ops()[0] == [0, 1] and f2.marked() == [1, 1, 0, 1]     # u is an un-colored output of a kept operator
    with pytest.raises(B.DragonError) as e:
        g.add_op(B.OPS["Tanh"], [x], [u, v])                   # executable types have one output
    assert e.value.code == B.ERR_INVALID_ARG
    w = g.add_tensor("w", B.F32, [7])
    with pytest.raises(B.DragonError) as e:
        g.add_op(B.OPS["Opaque"], [x], [w, w])
    assert e.value.code == B.ERR_NOT_SSA


def test_elementwise_chains_behind_a_product_run_in_its_epilogue():
    """Lowering: a chain of elementwise operators whose only tensor of the product's shape is the product itself
    (plus constants, scalars, row vectors and other tensors already in memory) becomes the contraction's
    epilogue program: one launch, the fp32 product never reaches memory.  A second reader of the product, or an
    operand that is computed after the product, keeps the separate elementwise launch."""
    m, n, k = 200, 136, 72
    gd = wl.GraphDesc()
    X = gd.tensor("X", [m, k], "bf16"); W = gd.tensor("W", [n, k], "bf16")
    T = gd.op("Tanh", [gd.op("InnerProduct", [X, W], "Y", [m, n], "f32")], "T", out_dtype="bf16")
    f = B.Graph.from_desc(gd.desc).function([X, W], [T])
    assert f.num_launches() == 1 and "epilogue: tanh, rbf16" in f.describe(), f.describe()
    gd = wl.GraphDesc()
    X = gd.tensor("X", [m, k], "bf16"); W = gd.tensor("W", [n, k], "bf16"); b = gd.tensor("b", [n]); side = gd.tensor("side", [m, n])
    s = gd.tensor("s", [])
    A = gd.op("BiasAdd", [gd.op("InnerProduct", [X, W], "Z", [m, n], "f32"), b], "A", [m, n], "f32")
    O = gd.op("Mul", [gd.op("Sigmoid", [A], "S"), side], "O")
    P = gd.op("Sub", [s, O], "P")
    f = B.Graph.from_desc(gd.desc).function([X, W, b, side, s], [P])
    assert f.num_launches() == 1 and "epilogue: add row, sigmoid, mul full, rsub s" in f.describe(), f.describe()
    f = B.Graph.from_desc(gd.desc).function([X, W, b, side, s], [P, A])          # A fetched too: two readers of the chain
    assert "epilogue" not in f.describe() and f.num_launches() == 2, f.describe()
    # the side operand is itself computed by a later step than the product: no fusion
    gd = wl.GraphDesc()
    X = gd.tensor("X", [m, k], "bf16"); W = gd.tensor("W", [n, k], "bf16"); raw = gd.tensor("raw", [m, n])
    Y = gd.op("InnerProduct", [X, W], "Y", [m, n], "f32")
    side = gd.op("Sum", [raw], "side")                                             # a row-mode segment of its own, after the product
    O = gd.op("Mul", [gd.op("Tanh", [Y], "T"), side], "O")
    f = B.Graph.from_desc(gd.desc).function([X, W, raw], [O])
    assert "epilogue" not in f.describe(), f.describe()


def test_clamps_are_left_out_only_where_the_argument_is_proven_in_range():
    """Interval analysis over the micro-operations: tanh of a sigmoid, of a sine, of a product of two bounded values
    takes the form without clamps, tanh of a fed tensor or of a sum that can exceed the range does not; the clamped
    exponential of a bounded argument likewise, and of 12 * tanh(x) (up to 12 > 10) not."""
    def plan(build):
        gd = wl.GraphDesc()
        x = gd.tensor("x", [5000]); y = gd.tensor("y", [5000])
        out = build(gd, x, y)
        return B.Graph.from_desc(gd.desc).function([x, y], [out]).describe()

    def twelve(gd, v):      # 12 * v as a sum of doublings, no constant operand needed
        v2 = gd.op("Add", [v, v], "v2"); v4 = gd.op("Add", [v2, v2], "v4"); v8 = gd.op("Add", [v4, v4], "v8")
        return gd.op("Add", [v8, v4], "v12")

    assert "tanhb" in plan(lambda gd, x, y: gd.op("Tanh", [gd.op("Sigmoid", [x], "s")], "t"))
    assert "tanhb" in plan(lambda gd, x, y: gd.op("Tanh", [gd.op("Sin", [x], "s")], "t"))
    assert "tanhb" in plan(lambda gd, x, y: gd.op("Tanh", [gd.op("Mul", [gd.op("Sin", [x], "s"), gd.op("Tanh", [y], "u")], "p")], "t"))
    p = plan(lambda gd, x, y: gd.op("Tanh", [x], "t"))
    assert "tanh;" in p and "tanhb" not in p
    p = plan(lambda gd, x, y: gd.op("Tanh", [gd.op("Add", [gd.op("Sin", [x], "s"), y], "a")], "t"))
    assert "tanhb" not in p
    p = plan(lambda gd, x, y: gd.op("Tanh", [twelve(gd, gd.op("Sin", [x], "s"))], "t"))
    assert "tanhb" not in p                                              # |12 sin x| <= 12 > 4
    assert "sigmoidb" in plan(lambda gd, x, y: gd.op("Sigmoid", [twelve(gd, gd.op("Sin", [x], "s"))], "t"))     # 12 <= 80
    assert "expcb" in plan(lambda gd, x, y: gd.op("Exp", [gd.op("Tanh", [x], "s")], "t"))
    p = plan(lambda gd, x, y: gd.op("Exp", [twelve(gd, gd.op("Tanh", [x], "s"))], "t"))
    assert "expcb" not in p and "expc;" in p
    # a ReLU keeps the upper bound open, a division by 1 + |b| keeps the numerator's bound
    assert "tanhb" not in plan(lambda gd, x, y: gd.op("Tanh", [gd.op("ReLU", [x], "r")], "t"))
    assert "tanhb" in plan(lambda gd, x, y: gd.op("Tanh", [gd.op("Div", [gd.op("Sigmoid", [x], "s"), y], "d")], "t"))
