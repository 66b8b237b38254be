"""Several gradient stages in one function: d o_i / d w_j kept apart per objective (Sec. 2.3, the
enumeration of (objective, wrt) pairs of Algorithm 2), all stages sharing one forward sweep.

CPU part: the oracle's per-pair gradients against central differences and against linearity in the
objective; the host compiler's program for a multi-stage function run on the ISA emulator.
GPU part: Jacobian-style fetches (one stage per objective) through the C-ABI against the oracle."""
import numpy as np
import pytest

from oracle import interp, prune as oprune
from paper_1707_08265_b200 import binding as B
from paper_1707_08265_b200 import workloads as wl


def three_objectives(n):
    g = wl.GraphDesc()
    x = g.tensor("x", [n])
    w = g.tensor("w", [n])
    a = g.tensor("a", [])
    t = g.op("Mul", [a, x], "t")
    u = g.op("Add", [t, w], "u")
    o1 = g.op("Sin", [u], "o1")
    o2 = g.op("Exp", [t], "o2")
    o3 = g.op("Mul", [o1, w], "o3")
    return g, [x, w, a], [o1, o2, o3]


def attach_pairs(g, objs, inputs):
    """One stage per objective, wrts = the inputs Algorithm 2 connects to it."""
    stages = []
    for o in objs:
        G = oprune.backward_marks(g.desc, [o], inputs)
        wrts = [i for i in inputs if i in G]
        stages.append((o, wrts, g.grad([o], wrts)))
    return stages


def test_oracle_per_pair_gradients_match_central_differences():
    n = 5
    g, inputs, objs = three_objectives(n)
    stages = attach_pairs(g, objs, inputs)
    assert [len(w) for (_, w, _) in stages] == [3, 2, 3]          # exp(a*x) does not depend on w
    rng = np.random.default_rng(11)
    feeds = [rng.standard_normal(n), rng.standard_normal(n), np.float64(0.6)]
    outs = [gid for (_, _, gids) in stages for gid in gids]
    got = interp.run_function(g.desc, inputs, outs, feeds)
    k = 0
    h = 1e-6
    for (o, wrts, _) in stages:
        for w in wrts:
            pos = inputs.index(w)
            base = np.asarray(feeds[pos], dtype=np.float64)
            fd = np.zeros(base.shape)
            for j in range(base.size):
                d = np.zeros(base.size)
                d[j] = h
                hi = list(feeds)
                lo = list(feeds)
                hi[pos] = (base.reshape(-1) + d).reshape(base.shape)
                lo[pos] = (base.reshape(-1) - d).reshape(base.shape)
                fh = interp.run_function(g.desc, inputs, [o], hi)[0].sum()
                fl = interp.run_function(g.desc, inputs, [o], lo)[0].sum()
                fd.reshape(-1)[j] = (fh - fl) / (2 * h)
            assert np.allclose(got[k], fd, rtol=1e-6, atol=1e-8), (o, w)
            k += 1


def test_oracle_stage_of_several_objectives_is_the_sum_of_its_pairs():
    n = 9
    g, inputs, objs = three_objectives(n)
    x, w, a = inputs
    pair = [g.grad([o], [x, a]) for o in (objs[0], objs[2])]
    both = g.grad([objs[0], objs[2]], [x, a])
    rng = np.random.default_rng(5)
    feeds = [rng.standard_normal(n), rng.standard_normal(n), np.float64(-0.3)]
    outs = pair[0] + pair[1] + both
    r = interp.run_function(g.desc, inputs, outs, feeds)
    assert np.allclose(r[0] + r[2], r[4], rtol=1e-12, atol=1e-12)
    assert np.allclose(r[1] + r[3], r[5], rtol=1e-12, atol=1e-12)


def test_pruned_sets_per_stage_are_the_per_pair_marks():
    g, inputs, fetch = wl.random_row_dag(3, 8, 77, n_ops=40, n_fetch=3)
    stages = attach_pairs(g, fetch, inputs)
    outs = [gid for (_, _, gids) in stages for gid in gids]
    want = oprune.function_sets(g.desc, inputs, outs)
    f = B.Graph.from_desc(g.desc).function(inputs, outs)
    fwd, gops, masks = f.kept_ops()
    assert f.marked() == want["marked"] and fwd == want["fwd_ops"]
    assert gops == [k for (_, k, _) in want["grad_ops"]]
    # each stage keeps exactly the operators on a path from one of its wrts to its objective
    for s, (o, wrts, _) in enumerate(stages):
        G = oprune.backward_marks(g.desc, [o], wrts)
        on_path = sorted(k for k, op in enumerate(g.desc["ops"]) if op["out"][0] in G)
        assert sorted(k for (st, k, _) in want["grad_ops"] if st == s) == on_path


def emulate(g, inputs, outs, feeds):
    from test_codegen_emulated import emulate as run_emulated
    got, f = run_emulated(g.desc, inputs, outs, feeds)
    return f, got


def test_emulated_multi_stage_program_shares_the_forward_sweep():
    n = 4096 + 13
    g, inputs, objs = three_objectives(n)
    stages = attach_pairs(g, objs, inputs)
    outs = list(objs) + [gid for (_, _, gids) in stages for gid in gids]
    feeds = [a.astype(np.float32) for a in wl.normal_feeds([[n], [n]], 21)] + [np.float32(0.45)]
    f, got = emulate(g, inputs, outs, feeds)
    ref = interp.run_function(g.desc, inputs, outs, feeds)
    for gv, rv in zip(got, ref):
        assert np.allclose(gv, rv, rtol=1e-9, atol=1e-9)
    text = f.describe()
    # one forward evaluation of sin(u) and of exp(t) serves the fetch and every stage that needs it
    assert text.count(" expc") == 1 and (text.count(" sin") + text.count(" sincos") + text.count(" cossin")) <= 2


@pytest.mark.parametrize("seed", range(6))
def test_emulated_jacobian_style_row_dag(seed):
    R, C = 5, 24
    g, inputs, fetch = wl.random_row_dag(R, C, 8100 + seed, n_ops=36, n_fetch=3)
    stages = attach_pairs(g, fetch, inputs)
    outs = list(fetch) + [gid for (_, _, gids) in stages for gid in gids]
    feeds = [a * np.float32(0.5) for a in wl.normal_feeds([g.shape(i) for i in inputs], 8200 + seed)]
    ref = interp.run_function(g.desc, inputs, outs, feeds)
    _, got = emulate(g, inputs, outs, feeds)
    for gv, rv, o in zip(got, ref, outs):
        ok = np.isfinite(rv)
        assert np.allclose(gv[ok], rv[ok], rtol=1e-7, atol=1e-7), o


def test_emulated_per_objective_program_of_the_large_row_dag():
    """The 1024-operator row DAG with one stage per objective, at its full row length: the emitted
    program (wide build, shared-memory slots, a workspace spill slot, three column sums) evaluated in
    fp64 by the emulator equals the oracle to rounding, ill-conditioned outputs included."""
    import json
    import os
    seed = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "config_seeds.json")))["random_row_dag"]["seed"]
    g, inputs, fetch = wl.random_row_dag(3, 4096, seed)
    stages = attach_pairs(g, fetch, inputs)
    outs = list(fetch) + [gid for (_, _, gids) in stages for gid in gids]
    feeds = wl.normal_feeds([g.shape(i) for i in inputs], 5)
    ref = interp.run_function(g.desc, inputs, outs, feeds)
    _, got = emulate(g, inputs, outs, feeds)
    for gv, rv, o in zip(got, ref, outs):
        assert np.allclose(gv, rv, rtol=1e-9, atol=1e-9), o


# ---- GPU ---------------------------------------------------------------------------------------

@pytest.mark.gpu
@pytest.mark.parametrize("seed", range(6))
def test_gpu_jacobian_style_row_dag(seed):
    from test_gpu_vm import run_gpu, fp32_floors, check_conditioned
    R, C = 41, (2056, 1547)[seed % 2]
    g, inputs, fetch = wl.random_row_dag(R, C, 8300 + seed, n_ops=48, n_fetch=3)
    stages = attach_pairs(g, fetch, inputs)
    outs = list(fetch) + [gid for (_, _, gids) in stages for gid in gids]
    feeds = [a * np.float32(0.5) for a in wl.normal_feeds([g.shape(i) for i in inputs], 8400 + seed)]
    floors, ref = fp32_floors(g.desc, inputs, outs, feeds)
    got, f = run_gpu(g.desc, inputs, outs, feeds)
    want = oprune.function_sets(g.desc, inputs, outs)
    fwd, gops, masks = f.kept_ops()
    assert f.marked() == want["marked"] and fwd == want["fwd_ops"] and gops == [k for (_, k, _) in want["grad_ops"]]
    check_conditioned(got, ref, floors, "seed %d" % seed)


@pytest.mark.gpu
def test_gpu_three_objectives_flat_with_ragged_tail():
    from test_gpu_vm import run_gpu, check, TOL32
    n = 300 * 4096 + 1234
    g, inputs, objs = three_objectives(n)
    stages = attach_pairs(g, objs, inputs)
    outs = list(objs) + [gid for (_, _, gids) in stages for gid in gids]
    feeds = [a.astype(np.float32) for a in wl.normal_feeds([[n], [n]], 31)] + [np.asarray(0.45, dtype=np.float32)]
    got, f = run_gpu(g.desc, inputs, outs, feeds)
    assert f.num_launches() <= 2
    ref = interp.run_function(g.desc, inputs, outs, feeds)
    for gv, rv, o in zip(got, ref, outs):
        check(gv, rv, TOL32, "tensor %d" % o)
    # closed forms of the pairs (u = a x + w): d sin(u)/dw = cos(u); d exp(a x)/da = sum x exp(a x);
    # d (w sin u)/dw = sin u + w cos u
    x, w, a = feeds[0].astype(np.float64), feeds[1].astype(np.float64), 0.45
    a = float(np.float32(a))
    u = a * x + w
    k = len(objs)
    check(got[k + 1], np.cos(u), TOL32, "d o1 / d w")
    check(got[k + 4], np.sum(x * np.exp(a * x)), TOL32, "d o2 / d a")
    check(got[k + 6], np.sin(u) + w * np.cos(u), TOL32, "d o3 / d w")


@pytest.mark.gpu
def test_gpu_jacobian_style_row_dag_full_size():
    """The row DAG of the fifth workload at [16384, 4096] with one gradient stage per objective, in the
    launch configuration the benchmark times.  Rows are independent (row sums stay inside a row), so the
    oracle evaluates a sample of rows on the same values; FULL-shaped outputs of those rows must match."""
    import json
    import os
    import torch
    from test_gpu_vm import check, TOL32, C_COND, FLOOR_OK
    rows, cols = 16384, 4096
    seed = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "config_seeds.json")))["random_row_dag"]["seed"]

    def build(r):
        g, inputs, fetch = wl.random_row_dag(r, cols, seed)
        outs = list(fetch)
        for o in fetch:
            G = oprune.backward_marks(g.desc, [o], inputs)
            outs += g.grad([o], [i for i in inputs if i in G])
        return g, inputs, outs

    g, inputs, outs_ids = build(rows)
    f = B.Graph.from_desc(g.desc).function(inputs, outs_ids)
    want = oprune.function_sets(g.desc, inputs, outs_ids)
    fwd, gops, masks = f.kept_ops()
    assert f.marked() == want["marked"] and fwd == want["fwd_ops"] and gops == [k for (_, k, _) in want["grad_ops"]]
    gen = torch.Generator("cuda").manual_seed(seed)
    gpu_in = [torch.empty(tuple(g.shape(i)), dtype=torch.float32, device="cuda").normal_(generator=gen) for i in inputs]
    outs = [torch.full(tuple(g.shape(o)), float("nan"), dtype=torch.float32, device="cuda") for o in outs_ids]
    f.run_torch([t if u else None for t, u in zip(gpu_in, f.used_inputs())], outs)
    assert f.status() == 0
    torch.cuda.synchronize()
    pick = np.unique(np.concatenate([[0, 1, rows - 1], np.random.default_rng(2).integers(0, rows, 13)]))
    tp = torch.from_numpy(pick).cuda()
    sub = [t[tp].cpu().numpy() if t.dim() == 2 else t.cpu().numpy() for t in gpu_in]
    gs, in_s, outs_s = build(len(pick))
    ref, v64, _ = interp.run_function(gs.desc, in_s, outs_s, sub, return_all=True)
    low, v32, _ = interp.run_function(gs.desc, in_s, outs_s, sub, dtype=np.float32, return_all=True)
    # Rows in which fp32 cannot decide a kink: an operand of ReLU (kink at 0), of Exp (the clamp at +-10) or the
    # divisor of Div (|b| at 0) lies closer to the kink than 64 times the distance between the fp32 and the
    # fp64 evaluation of that very operand (typically a row sum that cancels to almost nothing).  There the
    # operator's value or derivative jumps, any fp32 evaluation may land on either side, and the whole row is
    # affected through the row sums; such rows are set aside and counted, all others are compared.
    undecided = np.zeros(len(pick), bool)
    for k in oprune.function_sets(gs.desc, in_s, outs_s)["fwd_ops"]:
        op = gs.desc["ops"][k]
        kinks = {"ReLU": (0, [0.0]), "Div": (1, [0.0]), "Exp": (0, [-10.0, 10.0])}.get(op["type"])
        if kinks is None:
            continue
        x64, x32 = v64[op["in"][kinks[0]]], v32[op["in"][kinks[0]]].astype(np.float64)
        dev = np.abs(x32 - x64)
        for c in kinks[1]:
            near = (np.abs(x64 - c) <= 64 * dev) & (dev > 0)
            if near.ndim == 2:
                undecided |= near.any(axis=1)
            elif near.any():
                undecided[:] = True
    assert undecided.sum() <= 2, "fp32 cannot decide a kink in %d of %d sampled rows" % (undecided.sum(), len(pick))
    keep = ~undecided
    n_full = n_tight = 0
    for o, r, l, t in zip(outs, ref, low, outs_ids):
        assert torch.isfinite(o).all()
        if o.dim() == 2:
            # A tensor on which NumPy's own fp32 evaluation leaves the tolerance is held to C_COND times that
            # floor (the emitted program for it is exact when run in fp64: the emulated tests), every other
            # tensor to the tolerance itself.
            floor = float(np.max((np.abs(l.astype(np.float64) - r) / (TOL32 * (1 + np.abs(r))))[keep]))
            scale = 1.0 if floor <= FLOOR_OK else C_COND * floor
            n_full += 1
            n_tight += scale == 1.0
            check(o[tp].cpu().numpy().astype(np.float64)[keep], r[keep], TOL32 * scale, "tensor %d (fp32 floor %.3g)" % (t, floor))
    assert n_full >= 4 and n_tight >= n_full - 1
