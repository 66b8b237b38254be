"""Pins for oracle/prune.py: brute-force path enumeration, the y = a*x example of Sec. 2.2,
the coloring invariants of Sec. 2.1, the operator order of Sec. 3.2."""
import numpy as np
import pytest

from oracle import prune, brute
from paper_1707_08265_b200 import workloads as wl


def tiny_dag(rng, n_src=3, n_ops=6):
    """Random DAG with one- and two-output operators."""
    tensors, ops = [{"name": "s%d" % i, "dtype": "f32", "shape": []} for i in range(n_src)], []
    for k in range(n_ops):
        nin = int(rng.integers(1, 3))
        nout = int(rng.integers(1, 3))
        ins = [int(rng.integers(len(tensors))) for _ in range(nin)]
        outs = []
        for j in range(nout):
            tensors.append({"name": "t%d_%d" % (k, j), "dtype": "f32", "shape": []})
            outs.append(len(tensors) - 1)
        ops.append({"type": "Opaque", "in": ins, "out": outs})
    return {"tensors": tensors, "ops": ops, "grads": []}


@pytest.mark.parametrize("seed", range(40))
def test_forward_marks_equal_bruteforce(seed):
    rng = np.random.default_rng(seed)
    d = tiny_dag(rng)
    n = len(d["tensors"])
    targets = [int(t) for t in rng.choice(n, size=int(rng.integers(1, 3)), replace=False)]
    assert prune.forward_marks(d, targets) == brute.forward_marks_bruteforce(d, targets)


@pytest.mark.parametrize("seed", range(40))
def test_backward_marks_equal_bruteforce(seed):
    rng = np.random.default_rng(1000 + seed)
    d = tiny_dag(rng)
    n = len(d["tensors"])
    objs = [int(t) for t in rng.choice(n, size=int(rng.integers(1, 3)), replace=False)]
    wrts = [int(t) for t in rng.choice(n, size=int(rng.integers(1, 3)), replace=False)]
    assert prune.backward_marks(d, objs, wrts) == brute.backward_marks_bruteforce(d, objs, wrts)


def test_backward_marks_keeps_side_chain_to_wrt():
    # obj -> {wrt, c}, c -> wrt in the gradient direction, i.e. forward edges wrt -> c -> obj and
    # wrt -> obj: c lies on a chain between the two and must be marked whichever child comes first.
    d = {"tensors": [{"name": n, "dtype": "f32", "shape": []} for n in ("wrt", "c", "obj")],
         "ops": [{"type": "Opaque", "in": [0], "out": [1]}, {"type": "Opaque", "in": [0, 1], "out": [2]}],
         "grads": []}
    assert prune.backward_marks(d, [2], [0]) == {0, 1, 2}
    assert prune.backward_marks(d, [2], [2]) == {2}          # obj == wrt: the single node
    assert prune.backward_marks(d, [1], [2]) == set()        # no chain


def test_paper_example_b_is_redundant():
    g, ids = wl.toy_function(8)
    inputs = [ids["x"], ids["a"], ids["b"]]
    s = prune.function_sets(g.desc, inputs, [ids["y"]])
    marked = {i for i, m in enumerate(s["marked"]) if m}
    assert marked == {ids["x"], ids["a"], ids["y"]}          # b, t2, t3, f stay un-colored
    assert s["fwd_ops"] == [0]                               # only Mul(a, x); Add, Sin, Mul removed
    assert s["used_inputs"] == [1, 1, 0]
    s = prune.function_sets(g.desc, inputs, [ids["f"], ids["y"]])
    assert all(s["marked"]) and s["fwd_ops"] == [0, 1, 2, 3] and s["used_inputs"] == [1, 1, 1]


@pytest.mark.parametrize("seed", range(20))
def test_coloring_invariants(seed):
    rng = np.random.default_rng(2000 + seed)
    d = tiny_dag(rng, n_ops=10)
    n = len(d["tensors"])
    targets = [int(t) for t in rng.choice(n, size=2, replace=False)]
    s = prune.function_sets(d, list(range(3)), targets)
    m = s["marked"]
    for k, op in enumerate(d["ops"]):
        kept = k in s["fwd_ops"]
        assert kept == any(m[o] for o in op["out"])          # removed iff all outputs un-colored
        if kept:
            assert all(m[i] for i in op["in"])               # every parent of a marked tensor is marked
    assert s["fwd_ops"] == sorted(s["fwd_ops"])              # creating order


def test_toy_gradient_stage_order_and_masks():
    g, ids = wl.toy_function_grad(8)
    inputs = [ids["x"], ids["a"], ids["b"]]
    s = prune.function_sets(g.desc, inputs, [ids["dx"], ids["da"], ids["db"]])
    assert s["fwd_ops"] == [0, 1, 2, 3]
    # inverse creating order; Mul(x,t3): both operands; Sin; Add(y,b): both; Mul(a,x): both
    assert s["grad_ops"] == [(0, 3, (0, 1)), (0, 2, (0,)), (0, 1, (0, 1)), (0, 0, (0, 1))]
    assert all(s["marked"])
    # only df/db fetched: the a-branch of Mul(a,x) is not solved, x only through Mul(x,t3)'s t3 side
    s = prune.function_sets(g.desc, inputs, [ids["db"]])
    assert s["grad_ops"] == [(0, 3, (1,)), (0, 2, (0,)), (0, 1, (1,))]
    assert s["marked"][ids["dx"]] == 0 and s["marked"][ids["da"]] == 0 and s["marked"][ids["db"]] == 1
    # forward-only fetch: no gradient operator survives
    s = prune.function_sets(g.desc, inputs, [ids["f"]])
    assert s["grad_ops"] == [] and s["marked"][ids["dx"]] == 0


def test_mlp_prune_drops_side_branch_and_input_gradient():
    g, ids = wl.mlp(4, 8, 8, 8)
    inputs = [ids[k] for k in ("X", "W1", "b1", "W2", "b2", "labels")]
    outs = [ids[k] for k in ("loss", "dW1", "db1", "dW2", "db2")]
    s = prune.function_sets(g.desc, inputs, outs)
    assert s["marked"][ids["side"]] == 0
    assert 0 not in s["fwd_ops"]                              # Tanh(X) is operator 0
    gops = {k: pos for (_, k, pos) in s["grad_ops"]}
    assert gops[1] == (1,)                                    # InnerProduct#1: dW1 only, no dX
    assert gops[4] == (0, 1)                                  # InnerProduct#2: dH and dW2
    assert [k for (_, k, _) in s["grad_ops"]] == [6, 5, 4, 3, 2, 1]
    assert s["used_inputs"] == [1] * 6


def test_gradient_without_path_is_rejected():
    g, ids = wl.toy_function(4)
    g.grad([ids["y"]], [ids["b"]])                            # y = a*x does not depend on b
    with pytest.raises(ValueError):
        prune.function_sets(g.desc, [ids["x"], ids["a"], ids["b"]], [g.desc["grads"][0]["grad_ids"][0]])


def tiny_dag_with_stages(rng):
    """A tiny DAG (one- and two-output operators) with one or two gradient stages whose derivative targets
    all have a chain to an objective, and a random set of fetched forward and gradient tensors."""
    while True:
        d = tiny_dag(rng, n_src=3, n_ops=int(rng.integers(3, 6)))
        n = len(d["tensors"])
        if n > 12:
            continue
        stages = []
        for s in range(int(rng.integers(1, 3))):
            objs = [int(t) for t in rng.choice(n, size=int(rng.integers(1, 3)), replace=False)]
            cand = [w for w in range(n) if brute.backward_marks_bruteforce(d, set(objs), {w})]
            if not cand:
                break
            wrts = [int(w) for w in rng.choice(cand, size=min(len(cand), int(rng.integers(1, 4))), replace=False)]
            stages.append((objs, wrts))
        else:
            break
    for s, (objs, wrts) in enumerate(stages):
        gids = []
        for w in wrts:
            d["tensors"].append({"name": "grad%d/%d" % (s, w), "dtype": "f32", "shape": []})
            gids.append(len(d["tensors"]) - 1)
        d["grads"].append({"objs": objs, "wrts": wrts, "grad_ids": gids})
    total = len(d["tensors"])
    fetch = [int(t) for t in rng.choice(total, size=int(rng.integers(1, 4)), replace=False)]
    return d, fetch


@pytest.mark.parametrize("seed", range(120))
def test_function_sets_equal_bruteforce_on_the_two_stage_dag(seed):
    """oracle.prune.function_sets against the explicit two-stage DAG of Sec. 2.3 with every path that
    ends in a fetched node walked edge by edge (anchor and seed edges written out): marks, kept
    forward operators, kept gradient operators with the operand gradients they produce."""
    rng = np.random.default_rng(7000 + seed)
    d, fetch = tiny_dag_with_stages(rng)
    inputs = [0, 1, 2]
    got = prune.function_sets(d, inputs, fetch)
    want = brute.function_sets_bruteforce(d, inputs, fetch)
    assert got == want


def test_bruteforce_function_sets_on_the_paper_example():
    # the pin of the pin: fetching only df/db drops the a-side of Mul(a, x) (worked out by hand)
    g, ids = wl.toy_function_grad(8)
    inputs = [ids["x"], ids["a"], ids["b"]]
    s = brute.function_sets_bruteforce(g.desc, inputs, [ids["db"]])
    assert s["grad_ops"] == [(0, 3, (1,)), (0, 2, (0,)), (0, 1, (1,))]
    assert s["marked"][ids["dx"]] == 0 and s["marked"][ids["da"]] == 0 and s["marked"][ids["db"]] == 1
    assert s["fwd_ops"] == [0, 1, 2, 3] and s["used_inputs"] == [1, 1, 1]
    s = brute.function_sets_bruteforce(g.desc, inputs, [ids["y"]])
    assert s["fwd_ops"] == [0] and s["used_inputs"] == [1, 1, 0] and s["grad_ops"] == []


# ---- fed intermediates (Sec. 3.1: any tensor can be fed by name) -----------------------------------

@pytest.mark.parametrize("seed", range(120))
def test_function_sets_with_fed_intermediates_equal_bruteforce(seed):
    """The same brute-force comparison when some of the listed inputs are tensors that an operator
    produces: the walk over explicit edges simply has no edge into a given tensor.  Fetched gradients
    whose derivative target keeps no chain are rejected by both."""
    rng = np.random.default_rng(9000 + seed)
    d, fetch = tiny_dag_with_stages(rng)
    n_fwd = len(d["tensors"]) - sum(len(st["wrts"]) for st in d["grads"])
    fed = [int(t) for t in rng.choice(np.arange(3, n_fwd), size=int(rng.integers(1, 3)), replace=False)]
    inputs = [0, 1, 2] + fed
    alias = {gid: (s, w) for s, st in enumerate(d["grads"]) for w, gid in zip(st["wrts"], st["grad_ids"])}
    given = set(inputs)
    cut = {"tensors": d["tensors"], "grads": d["grads"],
           "ops": [dict(op, out=[y for y in op["out"] if y not in given]) for op in d["ops"]]}
    dead = [t for t in fetch if t in alias and
            not brute.backward_marks_bruteforce(cut, set(d["grads"][alias[t][0]]["objs"]), {alias[t][1]})]
    if dead:
        with pytest.raises(ValueError):
            prune.function_sets(d, inputs, fetch)
        fetch = [t for t in fetch if t not in dead]
        if not fetch:
            return
    got = prune.function_sets(d, inputs, fetch)
    want = brute.function_sets_bruteforce(d, inputs, fetch)
    assert got == want
    # no operator is kept for the sake of a given tensor alone, and a given tensor has no marked parent through it
    for k in got["fwd_ops"]:
        assert any(got["marked"][y] for y in d["ops"][k]["out"] if y not in given)


def test_feeding_the_argument_of_the_sine_by_hand():
    """The function of Sec. 2.2 with t2 = a*x + b given instead of computed (worked out by hand):
    f = x*sin(t2) needs x and t2 only, so Mul(a, x) and Add(y, b) go and a, b are never read; df/dx keeps
    the one chain x -> f (the chain through y is cut), so only the gradient operator of the last Mul
    stays and it produces the x side alone; df/da and df/db have no chain left."""
    g, ids = wl.toy_function_grad(8)
    inputs = [ids["x"], ids["a"], ids["b"], ids["t2"]]
    s = prune.function_sets(g.desc, inputs, [ids["f"], ids["dx"]])
    assert s["fwd_ops"] == [2, 3] and s["used_inputs"] == [1, 0, 0, 1]
    assert s["grad_ops"] == [(0, 3, (0,))]
    assert [s["marked"][ids[k]] for k in ("y", "t2", "t3", "f", "dx", "da", "db")] == [0, 1, 1, 1, 1, 0, 0]
    assert s == brute.function_sets_bruteforce(g.desc, inputs, [ids["f"], ids["dx"]])
    for dead in ("da", "db"):
        with pytest.raises(ValueError):
            prune.function_sets(g.desc, inputs, [ids[dead]])
    # given y instead: the chain b -> t2 -> t3 -> f is alive, a's is not
    inputs = [ids["x"], ids["a"], ids["b"], ids["y"]]
    s = prune.function_sets(g.desc, inputs, [ids["db"], ids["dx"]])
    assert s["fwd_ops"] == [1, 2, 3] and s["used_inputs"] == [1, 0, 1, 1]
    assert s["grad_ops"] == [(0, 3, (0, 1)), (0, 2, (0,)), (0, 1, (1,))]
