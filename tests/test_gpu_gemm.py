"""GPU parity of the tensor-core contraction and of the whole two-layer graph (InnerProduct, BiasAdd,
ReLU, SoftmaxCrossEntropy, forward + backward) against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import interp
from paper_1707_08265_b200 import workloads as wl
from test_gpu_vm import run_gpu, check, TOLBF, TOL32

pytestmark = pytest.mark.gpu


def bf16able(a):
    return torch.from_numpy(a.astype(np.float32)).to(torch.bfloat16).float().numpy()


@pytest.mark.parametrize("m,n,k,dt", [(128, 128, 64, "f32"), (128, 128, 512, "f32"), (256, 384, 448, "bf16"),
                                      (200, 136, 72, "f32"), (1, 8, 8, "f32"), (300, 520, 1000, "bf16"),
                                      (1024, 1024, 2048, "f32")])
def test_inner_product_forward(m, n, k, dt):
    gd = wl.GraphDesc()
    X = gd.tensor("X", [m, k], "bf16"); W = gd.tensor("W", [n, k], "bf16")
    Y = gd.op("InnerProduct", [X, W], "Y", [m, n], dt)
    rng = np.random.default_rng(m + n + k)
    x = bf16able(rng.standard_normal((m, k))); w = bf16able(rng.standard_normal((n, k)) / np.sqrt(k))
    (got,), f = run_gpu(gd.desc, [X, W], [Y], [x, w])
    (ref,) = interp.run_function(gd.desc, [X, W], [Y], [x, w])
    # fp32 accumulation of exact bf16 products: far inside the bf16-contraction tolerance
    check(got, ref, TOLBF if dt == "bf16" else 2e-5, "Y")
    # a transposed or shifted operand would not survive this: one-hot weights pick columns of X
    if n <= k:
        sel = np.zeros((n, k), dtype=np.float32)
        sel[np.arange(n), (np.arange(n) * 7) % k] = 1
        (got,), _ = run_gpu(gd.desc, [X, W], [Y], [x, sel])
        assert np.array_equal(got, x[:, (np.arange(n) * 7) % k].astype(np.float64))


@pytest.mark.parametrize("m,n,k", [(128, 128, 128), (96, 40, 72), (512, 256, 320)])
def test_inner_product_gradients(m, n, k):
    gd = wl.GraphDesc()
    X = gd.tensor("X", [m, k], "bf16"); W = gd.tensor("W", [n, k], "bf16"); G = gd.tensor("G", [m, n], "f32")
    Y = gd.op("InnerProduct", [X, W], "Y", [m, n], "f32")
    obj = gd.op("Mul", [Y, G], "obj")
    dX, dW = gd.grad([obj], [X, W])
    rng = np.random.default_rng(k)
    feeds = [bf16able(rng.standard_normal((m, k))), bf16able(rng.standard_normal((n, k))), bf16able(rng.standard_normal((m, n)))]
    got, f = run_gpu(gd.desc, [X, W, G], [dX, dW], feeds)
    ref = interp.run_function(gd.desc, [X, W, G], [dX, dW], feeds)
    check(got[0], ref[0], 1e-4, "dX")
    check(got[1], ref[1], 1e-4, "dW")


def mlp_case(batch, d_in, d_hid, d_out, seed):
    g, ids = wl.mlp(batch, d_in, d_hid, d_out)
    feeds = list(wl.mlp_feeds(batch, d_in, d_hid, d_out, seed))
    inputs = [ids[k] for k in ("X", "W1", "b1", "W2", "b2", "labels")]
    outs = [ids[k] for k in ("loss", "dW1", "db1", "dW2", "db2")]
    return g, ids, inputs, outs, feeds


@pytest.mark.parametrize("shape", [(128, 128, 128, 128), (256, 192, 320, 136), (1024, 512, 512, 1000)])
def test_mlp_forward_backward(shape):
    g, ids, inputs, outs, feeds = mlp_case(*shape, seed=wl.BASE_SEED + 4)
    got, f = run_gpu(g.desc, inputs, outs, feeds)
    assert f.used_inputs() == [1] * 6 and f.marked()[ids["side"]] == 0       # Tanh(X) pruned
    assert f.describe().count("gemm") == 5                                     # no dX of layer 1
    ref = interp.run_function(g.desc, inputs, outs, feeds)
    for gv, rv, name in zip(got, ref, ("loss", "dW1", "db1", "dW2", "db2")):
        check(gv, rv, TOLBF, name)
        scale = np.max(np.abs(rv))
        assert np.max(np.abs(gv - rv)) <= 0.03 * scale + 1e-12, (name, np.max(np.abs(gv - rv)), scale)


def test_mlp_with_the_hidden_activations_given():
    """Sec. 3.1: feeding h (the output of the first layer) makes it a source of the function: the first
    contraction, its bias and ReLU go, X, W1 and b1 are never read, the second layer's loss and gradients
    are computed from the given h, and the gradient with respect to h itself can be fetched."""
    batch, d_in, d_hid, d_out = 256, 192, 320, 136
    g, ids = wl.mlp(batch, d_in, d_hid, d_out)
    (dh,) = g.grad([ids["loss"]], [ids["h"]])
    feeds = list(wl.mlp_feeds(batch, d_in, d_hid, d_out, 77))
    hv = bf16able(np.abs(np.random.default_rng(8).standard_normal((batch, d_hid))))
    inputs = [ids[k] for k in ("X", "W1", "b1", "W2", "b2", "labels", "h")]
    outs = [ids["loss"], ids["dW2"], ids["db2"], dh]
    fd = [None, None, None, feeds[3], feeds[4], feeds[5], hv]
    got, f = run_gpu(g.desc, inputs, outs, fd)
    assert f.used_inputs() == [0, 0, 0, 1, 1, 1, 1] and f.kept_ops()[0] == [4, 5, 6]
    assert f.describe().count("gemm") == 3, f.describe()                       # z2, dW2, dh
    ref = interp.run_function(g.desc, inputs, outs, fd)
    for gv, rv, name in zip(got, ref, ("loss", "dW2", "db2", "dh")):
        check(gv, rv, TOLBF, name)
        assert np.max(np.abs(gv - rv)) <= 0.03 * np.max(np.abs(rv)) + 1e-12, name
    # the first layer's gradients have lost their chain in this function
    from paper_1707_08265_b200 import binding as B
    with pytest.raises(B.DragonError) as e:
        B.Graph.from_desc(g.desc).function(inputs, [ids["dW1"]])
    assert "no chain is left" in str(e.value)


def test_mlp_out_of_range_label_sets_status_and_does_not_fault():
    g, ids, inputs, outs, feeds = mlp_case(128, 128, 128, 128, seed=3)
    feeds[5] = feeds[5].copy(); feeds[5][7] = 4096
    from paper_1707_08265_b200 import binding as B
    from test_gpu_vm import to_dev
    fn = B.Graph.from_desc(g.desc).function(inputs, outs)
    dev = [to_dev(a, g.desc["tensors"][i]["dtype"]) for i, a in zip(inputs, feeds)]
    o = [torch.empty(tuple(g.shape(t)), dtype=torch.float32, device="cuda") for t in outs]
    fn.run_torch(dev, o)
    assert fn.status() == B.ERR_INVALID_ARG


def test_unsupported_contraction_length_is_an_error_not_a_fault():
    from paper_1707_08265_b200 import binding as B
    from test_gpu_vm import to_dev
    gd = wl.GraphDesc()
    X = gd.tensor("X", [16, 12], "bf16"); W = gd.tensor("W", [8, 12], "bf16")     # K = 12 is not a multiple of 8
    Y = gd.op("InnerProduct", [X, W], "Y", [16, 8], "f32")
    f = B.Graph.from_desc(gd.desc).function([X, W], [Y])
    out = torch.zeros(16, 8, device="cuda")
    with pytest.raises(B.DragonError) as e:
        f.run_torch([to_dev(np.zeros((16, 12), np.float32), "bf16"), to_dev(np.zeros((8, 12), np.float32), "bf16")], [out])
    assert e.value.code == B.ERR_UNSUPPORTED


@pytest.mark.parametrize("m,n,k,bias_dt,relu,out_dt", [
    (128, 128, 64, "f32", False, "f32"), (256, 384, 448, "bf16", True, "bf16"), (200, 136, 72, "bf16", True, "f32"),
    (300, 520, 1000, "f32", True, "bf16"), (70, 40, 72, "bf16", False, "bf16"), (1024, 1024, 512, "bf16", True, "bf16")])
def test_bias_and_relu_run_in_the_epilogue_of_the_product(m, n, k, bias_dt, relu, out_dt):
    """Y = [ReLU](X W^T + b): one launch, the fp32 product never written; ragged tiles in m and n."""
    gd = wl.GraphDesc()
    X = gd.tensor("X", [m, k], "bf16"); W = gd.tensor("W", [n, k], "bf16"); b = gd.tensor("b", [n], bias_dt)
    Z = gd.op("InnerProduct", [X, W], "Z", [m, n], "f32")
    last_dt = out_dt if not relu else "f32"
    Y = gd.op("BiasAdd", [Z, b], "A", [m, n], last_dt)
    if relu:
        Y = gd.op("ReLU", [Y], "Y", out_dtype=out_dt)
    rng = np.random.default_rng(m * 3 + n)
    x = bf16able(rng.standard_normal((m, k))); w = bf16able(rng.standard_normal((n, k)) / np.sqrt(k))
    bv = bf16able(rng.standard_normal(n))
    (got,), f = run_gpu(gd.desc, [X, W, b], [Y], [x, w, bv])
    assert f.num_launches() == 1 and "+bias" in f.describe() and ("relu" in f.describe()) == relu, f.describe()
    (ref,) = interp.run_function(gd.desc, [X, W, b], [Y], [x, w, bv])
    check(got, ref, TOLBF if out_dt == "bf16" else 2e-5, "Y")
    if relu:
        assert (got >= 0).all() and (got == 0).any() and (got > 0).any()


def test_product_that_is_also_fetched_keeps_its_own_launch():
    m, n, k = 128, 128, 64
    gd = wl.GraphDesc()
    X = gd.tensor("X", [m, k], "bf16"); W = gd.tensor("W", [n, k], "bf16"); b = gd.tensor("b", [n], "f32")
    Z = gd.op("InnerProduct", [X, W], "Z", [m, n], "f32")
    Y = gd.op("BiasAdd", [Z, b], "Y", [m, n], "f32")
    rng = np.random.default_rng(9)
    feeds = [bf16able(rng.standard_normal((m, k))), bf16able(rng.standard_normal((n, k))), bf16able(rng.standard_normal(n))]
    got, f = run_gpu(gd.desc, [X, W, b], [Y, Z], feeds)
    assert "+bias" not in f.describe()
    ref = interp.run_function(gd.desc, [X, W, b], [Y, Z], feeds)
    check(got[0], ref[0], 2e-5, "Y")
    check(got[1], ref[1], 2e-5, "Z")


@pytest.mark.parametrize("m,n,k", [(128, 256, 128), (200, 136, 72), (70, 40, 1000)])
def test_relu_backward_runs_in_the_epilogue_of_the_product(m, n, k):
    """H = ReLU(X W1^T + b) in bf16, Y = H W2^T, objective sum(Y * G): dZ1 = (G W2) * step(H) comes out of
    the product's epilogue, db = column sums of dZ1, dW1 = dZ1^T X.  Ragged tiles in every extent."""
    gd = wl.GraphDesc()
    X = gd.tensor("X", [m, k], "bf16"); W1 = gd.tensor("W1", [n, k], "bf16"); b = gd.tensor("b", [n], "bf16")
    W2 = gd.tensor("W2", [n, n], "bf16"); G = gd.tensor("G", [m, n], "f32")
    Z = gd.op("InnerProduct", [X, W1], "Z", [m, n], "f32")
    A = gd.op("BiasAdd", [Z, b], "A", [m, n], "f32")
    H = gd.op("ReLU", [A], "H", out_dtype="bf16")
    Y = gd.op("InnerProduct", [H, W2], "Y", [m, n], "f32")
    obj = gd.op("Mul", [Y, G], "obj")
    dW1, db = gd.grad([obj], [W1, b])
    rng = np.random.default_rng(n + k)
    feeds = [bf16able(rng.standard_normal((m, k))), bf16able(rng.standard_normal((n, k)) / np.sqrt(k)),
             bf16able(rng.standard_normal(n) * 0.1), bf16able(rng.standard_normal((n, n)) / np.sqrt(n)),
             bf16able(rng.standard_normal((m, n)))]
    ins = [X, W1, b, W2, G]
    got, f = run_gpu(gd.desc, ins, [dW1, db], feeds)
    assert "*step" in f.describe() and "step;" not in f.describe(), f.describe()
    ref = interp.run_function(gd.desc, ins, [dW1, db], feeds)
    check(got[0], ref[0], TOLBF, "dW1")
    # dZ1 is stored in bf16 (it is an operand of the next product), but its column sums are taken in the product's
    # epilogue from the fp32 values before that rounding ("+colsum" in the plan), as the oracle sums them
    assert "+colsum" in f.describe(), f.describe()
    check(got[1], ref[1], 1e-4, "db")


@pytest.mark.parametrize("bias_first", [True, False])
def test_computed_bias_before_or_after_the_product(bias_first):
    m, n, k = 64, 128, 64
    gd = wl.GraphDesc()
    X = gd.tensor("X", [m, k], "bf16"); W = gd.tensor("W", [n, k], "bf16"); b = gd.tensor("b", [n], "f32")
    if bias_first:
        tb = gd.op("Tanh", [b], "tb")
    Z = gd.op("InnerProduct", [X, W], "Z", [m, n], "f32")
    if not bias_first:
        tb = gd.op("Tanh", [b], "tb")
    Y = gd.op("BiasAdd", [Z, tb], "Y", [m, n], "f32")
    rng = np.random.default_rng(4)
    feeds = [bf16able(rng.standard_normal((m, k))), bf16able(rng.standard_normal((n, k))), rng.standard_normal(n).astype(np.float32)]
    (got,), f = run_gpu(gd.desc, [X, W, b], [Y], feeds)
    (ref,) = interp.run_function(gd.desc, [X, W, b], [Y], feeds)
    check(got, ref, 2e-5, "Y")


@pytest.mark.parametrize("m", [128, 256])             # one CTA per tile; a pair of CTAs on one tile
@pytest.mark.parametrize("k", [64, 320])
def test_a_pipeline_wait_that_runs_out_is_reported_and_the_next_run_is_correct(k, m, monkeypatch):
    """Failure detection without a fault: the producer of the contraction leaves out the loads of its first
    stage (test hook), so the consumer's first wait is for a signal that nothing sends; with the pipeline's
    budget shortened to about a millisecond the wait runs out, the kernel records DRAGON_ERR_TIMEOUT, lets
    the copies that are in flight land (that wait keeps its full budget), frees its tensor memory and
    returns by itself.  The context stays usable: the same function run again without the hook is correct."""
    from paper_1707_08265_b200 import binding as B
    n = 256                                           # one output tile; k = 320: later stages are really loaded
    # m = 256: the pair kernel; both CTAs leave out their first loads, the first CTA's consumer gives up, the second
    # CTA's epilogue gives up on its own budget, both meet at the cluster barrier and free their tensor memory
    gd = wl.GraphDesc()
    X = gd.tensor("X", [m, k], "bf16"); W = gd.tensor("W", [n, k], "bf16")
    Y = gd.op("InnerProduct", [X, W], "Y", [m, n], "f32")
    rng = np.random.default_rng(k)
    x = bf16able(rng.standard_normal((m, k))); w = bf16able(rng.standard_normal((n, k)) / np.sqrt(k))
    f = B.Graph.from_desc(gd.desc).function([X, W], [Y])
    dx, dw = torch.from_numpy(x).to(torch.bfloat16).cuda(), torch.from_numpy(w).to(torch.bfloat16).cuda()
    out = torch.full((m, n), float("nan"), dtype=torch.float32, device="cuda")
    monkeypatch.setenv("DRAGON_GEMM_WAIT_BUDGET", "2000000")
    monkeypatch.setenv("DRAGON_GEMM_DROP_FIRST_LOAD", "1")
    f.run_torch([dx, dw], [out])
    assert f.status() == B.ERR_TIMEOUT
    monkeypatch.delenv("DRAGON_GEMM_WAIT_BUDGET")
    monkeypatch.delenv("DRAGON_GEMM_DROP_FIRST_LOAD")
    f.run_torch([dx, dw], [out])
    assert f.status() == 0
    torch.cuda.synchronize()
    (ref,) = interp.run_function(gd.desc, [X, W], [Y], [x, w])
    check(out.cpu().numpy().astype(np.float64), ref, 2e-5, "Y after the timed-out run")


@pytest.mark.parametrize("m,n,k", [(200, 136, 72), (256, 512, 128), (1, 8, 8), (300, 1000, 264)])
def test_elementwise_chain_in_the_epilogue_of_a_product(m, n, k):
    """InnerProduct -> Tanh -> bf16, and InnerProduct -> BiasAdd -> Sigmoid -> Mul(side tensor) -> scalar - (.),
    each as ONE launch (the chain runs on the accumulator registers before the store), against the oracle at
    ragged and at aligned sizes; bf16 and fp32 side operands."""
    rng = np.random.default_rng(m + k)
    x = bf16able(rng.standard_normal((m, k))); w = bf16able(rng.standard_normal((n, k)) / np.sqrt(k))
    gd = wl.GraphDesc()
    X = gd.tensor("X", [m, k], "bf16"); W = gd.tensor("W", [n, k], "bf16")
    T = gd.op("Tanh", [gd.op("InnerProduct", [X, W], "Y", [m, n], "f32")], "T", out_dtype="bf16")
    (got,), f = run_gpu(gd.desc, [X, W], [T], [x, w])
    assert f.num_launches() == 1 and "epilogue" in f.describe()
    (ref,) = interp.run_function(gd.desc, [X, W], [T], [x, w])
    check(got, ref, TOLBF, "tanh in the epilogue")
    for side_dtype in ("f32", "bf16"):
        gd = wl.GraphDesc()
        X = gd.tensor("X", [m, k], "bf16"); W = gd.tensor("W", [n, k], "bf16"); b = gd.tensor("b", [n], side_dtype)
        side = gd.tensor("side", [m, n], side_dtype); s = gd.tensor("s", [])
        A = gd.op("BiasAdd", [gd.op("InnerProduct", [X, W], "Z", [m, n], "f32"), b], "A", [m, n], "f32")
        P = gd.op("Sub", [s, gd.op("Mul", [gd.op("Sigmoid", [A], "S"), side], "O")], "P")
        feeds = [x, w, bf16able(rng.standard_normal(n)), bf16able(rng.standard_normal((m, n))), np.asarray(0.75, np.float32)]
        (got,), f = run_gpu(gd.desc, [X, W, b, side, s], [P], feeds)
        want = "epilogue: add row, sigmoid, mul %s, rsub s" % ("row" if m == 1 else "full")     # a one-row tensor is a row vector
        assert f.num_launches() == 1 and want in f.describe(), f.describe()
        (ref,) = interp.run_function(gd.desc, [X, W, b, side, s], [P], feeds)
        check(got, ref, 2e-5, "bias, sigmoid, side operand, scalar in the epilogue (%s)" % side_dtype)


@pytest.mark.parametrize("pair", ["0", "1"])
@pytest.mark.parametrize("m,n,k", [(136, 104, 64), (264, 256, 72), (520, 264, 136), (128, 256, 64), (1024, 136, 200)])
def test_both_kernel_forms_at_the_edges_of_a_pair_tile(m, n, k, pair, monkeypatch):
    """The product kernel exists for one CTA per 128 x 256 tile and for a pair of CTAs per 256 x 256 tile.  Shapes that
    leave the pair's second CTA eight rows of A, no row of B at all (n <= 128), or a last tile that is mostly empty, in
    both forms, forward with bias and ReLU and all three gradients (the transposed-operand variants and the column
    sums of the bias gradient), against the oracle."""
    monkeypatch.setenv("DRAGON_GEMM_PAIR", pair)
    gd = wl.GraphDesc()
    X = gd.tensor("X", [m, k], "bf16"); W = gd.tensor("W", [n, k], "bf16"); b = gd.tensor("b", [n], "f32"); G = gd.tensor("G", [m, n], "f32")
    Y = gd.op("ReLU", [gd.op("BiasAdd", [gd.op("InnerProduct", [X, W], "Z", [m, n], "f32"), b], "A", [m, n], "f32")], "Y")
    obj = gd.op("Mul", [Y, G], "obj")
    dX, dW, db = gd.grad([obj], [X, W, b])
    rng = np.random.default_rng(m + n + k)
    feeds = [bf16able(rng.standard_normal((m, k))), bf16able(rng.standard_normal((n, k)) / np.sqrt(k)), bf16able(rng.standard_normal(n)),
             bf16able(rng.standard_normal((m, n)))]
    got, f = run_gpu(gd.desc, [X, W, b, G], [Y, dX, dW, db], feeds)
    ref = interp.run_function(gd.desc, [X, W, b, G], [Y, dX, dW, db], feeds)
    for gv, rv, name in zip(got, ref, ("Y", "dX", "dW", "db")):
        check(gv, rv, 1e-4 if name != "Y" else 2e-5, "%s (pair=%s)" % (name, pair))
