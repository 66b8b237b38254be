"""Seeded synthetic graphs and tensors for the five benchmark workloads.

This module holds no arithmetic of the method: it only writes graph
descriptions (plain dicts, the format documented in ``GraphDesc``) and draws
input values.  Both the CUDA library's tests and the CPU checker are driven
from these descriptions, so it imports neither.

Workloads (sizes are arguments so that tests can shrink them):
  toy_function        f = x*sin(a*x+b) and y = a*x, the example of Sec. 2.2
  toy_function_grad   the same with the gradient stage objs={f}, wrts={x,a,b} (Sec. 2.3)
  random_dag          random elementwise DAG (64 operators over 4 inputs by default)
  mlp                 InnerProduct/BiasAdd/ReLU/InnerProduct/BiasAdd/SoftmaxCrossEntropy
                      with an unused Tanh side branch and gradients for weights and biases
  random_row_dag      random broadcast/row-reduction DAG over [R,C] and [C] tensors, with
                      gradients for every input
"""
import numpy as np

BASE_SEED = 170708265

UNARY = ("Sin", "Exp", "Tanh", "Sigmoid", "ReLU")
BINARY = ("Add", "Sub", "Mul", "Div")
ROWRED = ("Sum", "Mean")


class GraphDesc:
    """Builder of the neutral graph description.

    ``desc`` = {"tensors": [{"name","dtype","shape"}], "ops": [{"type","in","out"}],
    "grads": [{"objs","wrts","grad_ids"}]}; ids are list positions (creation order).
    """

    def __init__(self):
        self.desc = {"tensors": [], "ops": [], "grads": []}

    def tensor(self, name, shape, dtype="f32"):
        self.desc["tensors"].append({"name": name, "dtype": dtype, "shape": [int(s) for s in shape]})
        return len(self.desc["tensors"]) - 1

    def shape(self, t):
        return self.desc["tensors"][t]["shape"]

    def op(self, type_, ins, out_name, out_shape=None, out_dtype="f32"):
        if out_shape is None:
            out_shape = _broadcast_shape([self.shape(i) for i in ins])
        o = self.tensor(out_name, out_shape, out_dtype)
        self.desc["ops"].append({"type": type_, "in": [int(i) for i in ins], "out": [o]})
        return o

    def grad(self, objs, wrts):
        gids = []
        s = len(self.desc["grads"])
        for w in wrts:
            t = self.desc["tensors"][w]
            gids.append(self.tensor("grad%d/%s" % (s, t["name"]), t["shape"], "f32"))
        self.desc["grads"].append({"objs": list(objs), "wrts": list(wrts), "grad_ids": gids})
        return gids


def _broadcast_shape(shapes):
    rank = max(len(s) for s in shapes)
    out = [1] * rank
    for s in shapes:
        s = [1] * (rank - len(s)) + list(s)
        for k, d in enumerate(s):
            if d != 1:
                assert out[k] in (1, d), shapes
                out[k] = d
    return out


def toy_function(n):
    """Sec. 2.2: tensors x, a, b, t1 = a*x (this is y), t2 = t1+b, t3 = sin(t2), f = x*t3."""
    g = GraphDesc()
    x = g.tensor("x", [n])
    a = g.tensor("a", [])
    b = g.tensor("b", [])
    y = g.op("Mul", [a, x], "y")
    t2 = g.op("Add", [y, b], "t2")
    t3 = g.op("Sin", [t2], "t3")
    f = g.op("Mul", [x, t3], "f")
    return g, {"x": x, "a": a, "b": b, "y": y, "t2": t2, "t3": t3, "f": f}


def toy_function_grad(n):
    g, ids = toy_function(n)
    dx, da, db = g.grad([ids["f"]], [ids["x"], ids["a"], ids["b"]])
    ids.update(dx=dx, da=da, db=db)
    return g, ids


def toy_feeds(n, seed):
    rng = np.random.default_rng(seed)
    x = rng.uniform(-4.0, 4.0, size=n).astype(np.float32)
    a = np.float32(rng.standard_normal())
    b = np.float32(rng.standard_normal())
    return x, np.asarray(a, dtype=np.float32), np.asarray(b, dtype=np.float32)


def random_dag(n, seed, n_inputs=4, n_ops=64, n_fetch=2):
    """Random elementwise DAG: operator types uniform over BINARY+UNARY, each operand uniform
    over the inputs and the earlier operator nodes; fetches are drawn without replacement
    among operator nodes that nothing consumes."""
    rng = np.random.default_rng(seed)
    g = GraphDesc()
    nodes = [g.tensor("in%d" % k, [n]) for k in range(n_inputs)]
    inputs = list(nodes)
    kinds = BINARY + UNARY
    for k in range(n_ops):
        t = kinds[int(rng.integers(len(kinds)))]
        nin = 2 if t in BINARY else 1
        ins = [nodes[int(rng.integers(len(nodes)))] for _ in range(nin)]
        nodes.append(g.op(t, ins, "n%d" % k))
    consumed = {i for op in g.desc["ops"] for i in op["in"]}
    sinks = [t for t in nodes[n_inputs:] if t not in consumed]
    pick = rng.choice(len(sinks), size=min(n_fetch, len(sinks)), replace=False)
    fetch = [sinks[int(p)] for p in sorted(pick)]
    return g, inputs, fetch


def normal_feeds(shapes, seed):
    rng = np.random.default_rng(seed)
    return [rng.standard_normal(size=s, dtype=np.float32) for s in shapes]


def mlp(batch, d_in, d_hidden, d_out):
    """Two-layer perceptron with a side branch Tanh(X) that no target needs."""
    g = GraphDesc()
    X = g.tensor("X", [batch, d_in], "bf16")
    W1 = g.tensor("W1", [d_hidden, d_in], "bf16")
    b1 = g.tensor("b1", [d_hidden], "bf16")
    W2 = g.tensor("W2", [d_out, d_hidden], "bf16")
    b2 = g.tensor("b2", [d_out], "bf16")
    labels = g.tensor("labels", [batch], "i32")
    side = g.op("Tanh", [X], "side", out_dtype="bf16")
    z1 = g.op("InnerProduct", [X, W1], "z1", [batch, d_hidden], "f32")
    a1 = g.op("BiasAdd", [z1, b1], "a1", [batch, d_hidden], "f32")
    h = g.op("ReLU", [a1], "h", out_dtype="bf16")
    z2 = g.op("InnerProduct", [h, W2], "z2", [batch, d_out], "f32")
    z = g.op("BiasAdd", [z2, b2], "z", [batch, d_out], "bf16")
    loss = g.op("SoftmaxCrossEntropy", [z, labels], "loss", [], "f32")
    dW1, db1, dW2, db2 = g.grad([loss], [W1, b1, W2, b2])
    ids = dict(X=X, W1=W1, b1=b1, W2=W2, b2=b2, labels=labels, side=side, z1=z1, a1=a1, h=h,
               z2=z2, z=z, loss=loss, dW1=dW1, db1=db1, dW2=dW2, db2=db2)
    return g, ids


def mlp_feeds(batch, d_in, d_hidden, d_out, seed):
    """float32 arrays holding bf16-representable values (truncated mantissas), plus int32 labels."""
    rng = np.random.default_rng(seed)

    def bf16able(a):
        u = a.astype(np.float32).view(np.uint32)
        return ((u + 0x8000) & 0xFFFF0000).astype(np.uint32).view(np.float32)

    X = bf16able(rng.standard_normal(size=(batch, d_in), dtype=np.float32))
    W1 = bf16able(rng.standard_normal(size=(d_hidden, d_in), dtype=np.float32) / np.float32(np.sqrt(d_in)))
    b1 = bf16able(rng.standard_normal(size=(d_hidden,), dtype=np.float32) / np.float32(np.sqrt(d_in)))
    W2 = bf16able(rng.standard_normal(size=(d_out, d_hidden), dtype=np.float32) / np.float32(np.sqrt(d_hidden)))
    b2 = bf16able(rng.standard_normal(size=(d_out,), dtype=np.float32) / np.float32(np.sqrt(d_hidden)))
    labels = rng.integers(0, d_out, size=batch).astype(np.int32)
    return X, W1, b1, W2, b2, labels


def random_row_dag(rows, cols, seed, n_full=6, n_row=2, n_ops=1024, n_fetch=4):
    """Random DAG over FULL [rows, cols] and ROW [cols] tensors; operator types uniform over
    BINARY+UNARY+ROWRED; fetches drawn among FULL-shaped operator nodes nothing consumes.
    The gradient stage (objs = fetches, wrts = the inputs connected to a fetch) is attached by
    the caller with ``g.grad(fetch, wrts)``: which inputs are connected is the pruner's
    business, and this module holds none of it."""
    rng = np.random.default_rng(seed)
    g = GraphDesc()
    nodes = [g.tensor("full%d" % k, [rows, cols]) for k in range(n_full)]
    nodes += [g.tensor("row%d" % k, [cols]) for k in range(n_row)]
    inputs = list(nodes)
    kinds = BINARY + UNARY + ROWRED
    for k in range(n_ops):
        t = kinds[int(rng.integers(len(kinds)))]
        nin = 2 if t in BINARY else 1
        ins = [nodes[int(rng.integers(len(nodes)))] for _ in range(nin)]
        nodes.append(g.op(t, ins, "n%d" % k))
    consumed = {i for op in g.desc["ops"] for i in op["in"]}
    sinks = [t for t in nodes[len(inputs):] if t not in consumed and len(g.shape(t)) == 2]
    pick = rng.choice(len(sinks), size=min(n_fetch, len(sinks)), replace=False)
    fetch = [sinks[int(p)] for p in sorted(pick)]
    return g, inputs, fetch


def updater(shape, kind="sgd"):
    """The weight update as a graph of its own (Sec. 3.2 of the paper: the updater is split from the
    training graph so that neither becomes cyclic; it names Momentum, RMSProp and Adam).
      sgd:      W' = W - lr*g
      momentum: v' = mu*v + g,  W' = W - lr*v'
      rmsprop:  v' = rho*v + (1-rho)*g*g,  W' = W - lr * g / (sqrt(v') + eps)
      adam:     m' = beta1*m + (1-beta1)*g,  v' = beta2*v + (1-beta2)*g*g,  W' = W - lr * m' / (sqrt(v') + eps)
                (lr and eps carry the bias corrections of the step: lr_t = lr*sqrt(1-beta2^t)/(1-beta1^t))
    The hyper-parameters are scalar tensors, 1-x fed beside x; returns (graph, ids)."""
    g = GraphDesc()
    ids = {"W": g.tensor("W", shape), "g": g.tensor("g", shape)}

    def scalars(*names):
        for n in names:
            ids[n] = g.tensor(n, [])

    def decayed(state, keep, mix, value, name):      # keep*state + mix*value
        return g.op("Add", [g.op("Mul", [ids[keep], ids[state]], name + "_keep"), g.op("Mul", [ids[mix], value], name + "_mix")], name)

    if kind == "sgd":
        scalars("lr")
        step = g.op("Mul", [ids["lr"], ids["g"]], "step")
    elif kind == "momentum":
        ids["lr"] = g.tensor("lr", [])
        ids["v"] = g.tensor("v", shape)
        ids["mu"] = g.tensor("mu", [])
        ids["v_new"] = g.op("Add", [g.op("Mul", [ids["mu"], ids["v"]], "mv"), ids["g"]], "v_new")
        step = g.op("Mul", [ids["lr"], ids["v_new"]], "step")
    elif kind in ("rmsprop", "adam"):
        if kind == "adam":
            ids["m"] = g.tensor("m", shape)
        ids["v"] = g.tensor("v", shape)
        if kind == "adam":
            scalars("lr", "beta1", "one_minus_beta1", "beta2", "one_minus_beta2", "eps")
            ids["m_new"] = decayed("m", "beta1", "one_minus_beta1", ids["g"], "m_new")
            num, keep, mix = ids["m_new"], "beta2", "one_minus_beta2"
        else:
            scalars("lr", "rho", "one_minus_rho", "eps")
            num, keep, mix = ids["g"], "rho", "one_minus_rho"
        ids["v_new"] = decayed("v", keep, mix, g.op("Mul", [ids["g"], ids["g"]], "g2"), "v_new")
        den = g.op("Add", [g.op("Sqrt", [ids["v_new"]], "root"), ids["eps"]], "den")
        step = g.op("Mul", [g.op("Mul", [ids["lr"], num], "lr_num"), g.op("Reciprocal", [den], "inv")], "step")
    else:
        raise ValueError(kind)
    ids["W_new"] = g.op("Sub", [ids["W"], step], "W_new")
    return g, ids
