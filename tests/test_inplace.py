"""Algorithm 3 (in-place structures, Sec. 2.4): pins for the oracle, the library's rename
dictionary against the oracle (bit-exact), and the memory sharing of the tensors that cross
kernels (no two tensors that are alive at the same time share bytes, except an in-place pair)."""
import numpy as np
import pytest

from oracle import inplace, prune as oprune
from paper_1707_08265_b200 import binding as B
from paper_1707_08265_b200 import workloads as wl
from test_oracle_prune import tiny_dag


def test_chain_through_a_binary_operator_and_a_fork():
    # x0 -> x1 -> x2, (x2, x3) -> x4, x4 -> x5 and x4 -> x6: the structure x0..x4 is one path of
    # only-children (x3 has x4 as its only child too, but x4 is taken); x4 has two children, so
    # x5 and x6 start structures of their own
    d = {"tensors": [{}] * 7, "ops": [{"in": [0], "out": [1]}, {"in": [1], "out": [2]}, {"in": [2, 3], "out": [4]},
                                      {"in": [4], "out": [5]}, {"in": [4], "out": [6]}]}
    assert inplace.rename_dictionary(d, range(7), range(5)) == {0: 0, 1: 0, 2: 0, 3: 3, 4: 0, 5: 5, 6: 6}


def test_pruned_operators_do_not_count_as_children():
    # x0 feeds two operators; when the second is pruned x0 has one child left and x1 joins x0
    d = {"tensors": [{}] * 3, "ops": [{"in": [0], "out": [1]}, {"in": [0], "out": [2]}]}
    assert inplace.rename_dictionary(d, [0, 1, 2], [0, 1]) == {0: 0, 1: 1, 2: 2}
    assert inplace.rename_dictionary(d, [0, 1], [0]) == {0: 0, 1: 0}


@pytest.mark.parametrize("seed", range(60))
def test_algorithm_equals_the_definition_on_tiny_dags(seed):
    rng = np.random.default_rng(4000 + seed)
    d = tiny_dag(rng, n_src=3, n_ops=7)
    n = len(d["tensors"])
    targets = [int(t) for t in rng.choice(n, size=int(rng.integers(1, 4)), replace=False)]
    marked = sorted(oprune.forward_marks(d, targets))
    kept = [k for k, op in enumerate(d["ops"]) if any(o in marked for o in op["out"])]
    rd = inplace.rename_dictionary(d, marked, kept)
    assert rd == inplace.rename_dictionary_bruteforce(d, marked, kept)
    assert set(rd) == set(marked) and all(rd[x] <= x for x in rd) and all(rd[rd[x]] == rd[x] for x in rd)


@pytest.mark.parametrize("seed", range(12))
def test_library_rename_dictionary_matches_the_oracle(seed):
    g, inputs, fetch = wl.random_dag(64, 6000 + seed, n_ops=48)
    f = B.Graph.from_desc(g.desc).function(inputs, fetch)
    want = oprune.function_sets(g.desc, inputs, fetch)
    marked = [t for t, m in enumerate(want["marked"]) if m]
    # the definition written out (no shared walk state), not the step-by-step form the library also follows
    rd = inplace.rename_dictionary_bruteforce(g.desc, marked, want["fwd_ops"])
    got = f.rename_dictionary()
    assert got == [rd.get(t, -1) for t in range(len(got))]
    assert rd == inplace.rename_dictionary(g.desc, marked, want["fwd_ops"])


def test_toy_function_structures():
    g, ids = wl.toy_function(16)      # t1 = a*x, t2 = t1 + b, t3 = sin(t2), f = x*t3
    f = B.Graph.from_desc(g.desc).function([ids["x"], ids["a"], ids["b"]], [ids["f"]])
    rd = f.rename_dictionary()
    # x has two children (t1 and f): it starts nothing beyond itself; a -> t1 -> t2 -> t3 -> f is one structure
    assert rd[ids["x"]] == ids["x"] and rd[ids["f"]] == ids["a"] and rd[ids["b"]] == ids["b"]


def overlaps(a, b):
    return a[0] < b[0] + b[1] and b[0] < a[0] + a[1]


@pytest.mark.parametrize("hidden", [256, 512])
def test_workspace_tensors_share_memory_only_when_one_is_dead(hidden):
    g, ids = wl.mlp(128, 256, hidden, 128)
    inputs = [ids[k] for k in ("X", "W1", "b1", "W2", "b2", "labels")]
    outputs = [ids[k] for k in ("loss", "dW1", "db1", "dW2", "db2")]
    f = B.Graph.from_desc(g.desc).function(inputs, outputs)
    check_sharing(f.workspace_tensors(), expect_reuse=False)


def test_regions_of_dead_tensors_are_used_again():
    # products read twice by what follows (so that it cannot run in their epilogue): every fp32 product dies in
    # the step after it
    g = wl.GraphDesc()
    X = g.tensor("X", [128, 256], "bf16"); labels = g.tensor("labels", [128], "i32")
    cur = X
    for k in range(3):
        W = g.tensor("W%d" % k, [256, 256], "bf16")
        z = g.op("InnerProduct", [cur, W], "z%d" % k, [128, 256], "f32")
        cur = g.op("Add", [g.op("Tanh", [z], "u%d" % k), g.op("Sin", [z], "v%d" % k)], "t%d" % k, out_dtype="bf16")
    loss = g.op("SoftmaxCrossEntropy", [cur, labels], "loss", [], "f32")
    ins = [t for t in range(len(g.desc["tensors"])) if g.desc["tensors"][t]["name"][0] in "XWl" and g.desc["tensors"][t]["name"] != "loss"]
    f = B.Graph.from_desc(g.desc).function(ins, [loss])
    assert "epilogue" not in f.describe()
    check_sharing(f.workspace_tensors(), expect_reuse=True)


def check_sharing(ts, expect_reuse):
    assert len(ts) >= 4
    own = sum((b + 255) // 256 * 256 for _, b, _, _, _ in ts)
    span = max(o + b for o, b, _, _, _ in ts) - min(o for o, _, _, _, _ in ts)
    assert span <= own
    if expect_reuse:
        assert span < own, "no region is used twice"
    for i, a in enumerate(ts):
        for b in ts[i + 1:]:
            alive_together = a[2] <= b[3] and b[2] <= a[3]
            if alive_together and overlaps(a, b):
                # only an output written in place over an input that dies in that very step
                first, second = (a, b) if a[2] <= b[2] else (b, a)
                assert second[4] == 1 and first[3] == second[2] and first[0] == second[0] and first[1] == second[1]


def test_elementwise_step_writes_in_place_over_a_dying_input():
    # z = X * W^T (a kernel of its own), y = relu(z) * 2 in fp32 (an elementwise kernel), loss on y
    g = wl.GraphDesc()
    X = g.tensor("X", [64, 128], "bf16"); W = g.tensor("W", [128, 128], "bf16"); labels = g.tensor("labels", [64], "i32")
    z = g.op("InnerProduct", [X, W], "z", [64, 128], "f32")
    y = g.op("Add", [g.op("ReLU", [z], "r"), g.op("ReLU", [z], "r2")], "y")
    loss = g.op("SoftmaxCrossEntropy", [y, labels], "loss", [], "f32")
    f = B.Graph.from_desc(g.desc).function([X, W, labels], [loss])
    ts = f.workspace_tensors()
    assert any(t[4] == 1 for t in ts), f.describe()
