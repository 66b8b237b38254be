"""Node-at-a-time interpreter of a pruned function: forward values and reverse-mode gradients.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

The paper fixes the graph model and the execution order (Sec. 3.2: kept forward
operators in creating order, gradient operators in inverse order) but gives no
operator semantics; those below are this project's reading of the operator
names.  Everything is evaluated with NumPy in ``dtype`` (float64 by default;
float32 gives the "CPU fp32 floor" used for conditioning checks), one whole
tensor per operator, no fusion, no reordering.

  Add, Sub, Mul      a+b, a-b, a*b with NumPy broadcasting
  Div(a, b)          a / (1 + |b|)
  Sin, Tanh, Sigmoid, ReLU   the usual; Exp(x) = exp(clip(x, -10, 10))
  Sqrt, Reciprocal   sqrt(x), 1/x (the updaters of Sec. 3.2 divide by a root: RMSProp, Adam)
  Sum, Mean          over the last axis, result broadcast back to the operand's shape
  InnerProduct(X, W) X[M,K] @ W[N,K]^T; operands are rounded to bf16 first (the
                     contraction consumes bf16), products and sums are wide
  BiasAdd(Y, b)      Y[m,n] + b[n]
  SoftmaxCrossEntropy(Z, labels)  scalar  -(1/M) sum_m log softmax(Z[m,:])[labels[m]]

Gradient rules (dy = gradient of the output): Add (dy,dy); Sub (dy,-dy);
Mul (dy*b, dy*a); Div (dy/(1+|b|), -dy*a*sgn(b)/(1+|b|)^2) with sgn(0)=0;
Sin dy*cos x; Exp dy*y*[-10<=x<=10]; Tanh dy*(1-y^2); Sigmoid dy*y*(1-y);
ReLU dy*[x>0]; Sqrt dy/(2y); Reciprocal -dy*y^2; Sum: row-sum of dy broadcast back; Mean: the same / C;
InnerProduct dX = dY@W, dW = dY^T@X (dY rounded to bf16 first);
BiasAdd (dy, column sums of dy); SoftmaxCrossEntropy dZ = dL*(softmax - onehot)/M.
A gradient with respect to a broadcast operand is summed over the broadcast
axes; contributions from several consumers add (reverse mode, Sec. 2.3); the
seed is one for every element of every objective of the stage.

A forward tensor declared bf16 is rounded to bf16 (round to nearest even, taken
on the float32 image of the value) when it is produced.
"""
import numpy as np

from .prune import function_sets


def round_bf16(a):
    """Round to bfloat16 (nearest even), result returned in the dtype of ``a``."""
    a = np.asarray(a)
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16) << 16
    nan = np.isnan(f)
    out = r.astype(np.uint32).view(np.float32)
    out = np.where(nan, np.float32(np.nan), out)
    return out.astype(a.dtype if a.dtype.kind == "f" else np.float32)


def _unbroadcast(g, shape):
    """Sum ``g`` over the axes along which a tensor of ``shape`` was broadcast."""
    shape = tuple(shape)
    while g.ndim > len(shape):
        g = g.sum(axis=0)
    for ax, (gs, ts) in enumerate(zip(g.shape, shape)):
        if ts == 1 and gs != 1:
            g = g.sum(axis=ax, keepdims=True)
    return g.reshape(shape)


def _forward(op, ins, dtype, bf16_contraction=True):
    t = op["type"]
    if t == "Add":
        return ins[0] + ins[1]
    if t == "Sub":
        return ins[0] - ins[1]
    if t == "Mul":
        return ins[0] * ins[1]
    if t == "Div":
        return ins[0] / (1 + np.abs(ins[1]))
    if t == "Sin":
        return np.sin(ins[0])
    if t == "Exp":
        return np.exp(np.clip(ins[0], -10, 10))
    if t == "Tanh":
        return np.tanh(ins[0])
    if t == "Sigmoid":
        return 1 / (1 + np.exp(-ins[0]))
    if t == "ReLU":
        return np.maximum(ins[0], 0)
    if t == "Sqrt":
        return np.sqrt(ins[0])
    if t == "Reciprocal":
        return 1 / ins[0]
    if t == "Sum":
        return np.broadcast_to(ins[0].sum(axis=-1, keepdims=True), ins[0].shape).copy()
    if t == "Mean":
        return np.broadcast_to(ins[0].mean(axis=-1, keepdims=True), ins[0].shape).copy()
    if t == "InnerProduct":
        rb = round_bf16 if bf16_contraction else (lambda a: a)
        return rb(ins[0]) @ rb(ins[1]).T
    if t == "BiasAdd":
        return ins[0] + ins[1][None, :]
    if t == "SoftmaxCrossEntropy":
        z, lab = ins[0], ins[1].astype(np.int64)
        zs = z - z.max(axis=1, keepdims=True)
        lse = np.log(np.exp(zs).sum(axis=1))
        return np.asarray(-(zs[np.arange(z.shape[0]), lab] - lse).mean(), dtype=dtype)
    raise ValueError("unknown operator type %r" % t)


def _backward(op, ins, out, dy, pos, bf16_contraction=True):
    """Gradients with respect to the operand positions in ``pos`` (un-reduced, operand-broadcast)."""
    t = op["type"]
    g = {}
    if t == "Add":
        for p in pos:
            g[p] = dy
    elif t == "Sub":
        for p in pos:
            g[p] = dy if p == 0 else -dy
    elif t == "Mul":
        for p in pos:
            g[p] = dy * ins[1 - p]
    elif t == "Div":
        den = 1 + np.abs(ins[1])
        for p in pos:
            g[p] = dy / den if p == 0 else -dy * ins[0] * np.sign(ins[1]) / (den * den)
    elif t == "Sin":
        g[0] = dy * np.cos(ins[0])
    elif t == "Exp":
        g[0] = dy * out * ((ins[0] >= -10) & (ins[0] <= 10))
    elif t == "Tanh":
        g[0] = dy * (1 - out * out)
    elif t == "Sigmoid":
        g[0] = dy * out * (1 - out)
    elif t == "ReLU":
        g[0] = dy * (ins[0] > 0)
    elif t == "Sqrt":
        g[0] = dy / (2 * out)
    elif t == "Reciprocal":
        g[0] = -dy * out * out
    elif t in ("Sum", "Mean"):
        r = np.broadcast_to(np.broadcast_to(dy, ins[0].shape).sum(axis=-1, keepdims=True), ins[0].shape)
        g[0] = r / ins[0].shape[-1] if t == "Mean" else r.copy()
    elif t == "InnerProduct":
        rb = round_bf16 if bf16_contraction else (lambda a: a)
        d = rb(dy)
        for p in pos:
            g[p] = d @ rb(ins[1]) if p == 0 else d.T @ rb(ins[0])
    elif t == "BiasAdd":
        for p in pos:
            g[p] = dy if p == 0 else dy.sum(axis=0)
    elif t == "SoftmaxCrossEntropy":
        z, lab = ins[0], ins[1].astype(np.int64)
        zs = z - z.max(axis=1, keepdims=True)
        e = np.exp(zs)
        sm = e / e.sum(axis=1, keepdims=True)
        sm[np.arange(z.shape[0]), lab] -= 1
        g[0] = dy * sm / z.shape[0]
    else:
        raise ValueError("unknown operator type %r" % t)
    return g


def run_function(desc, inputs, outputs, feeds, dtype=np.float64, return_all=False,
                 bf16_contraction=True):
    """Evaluate ``function(inputs, outputs)`` on ``feeds`` (arrays, order of ``inputs``).

    Pruned inputs may be fed as None.  ``bf16_contraction=False`` switches off the bf16
    rounding of InnerProduct operands (used only by the finite-difference pins, which need
    a differentiable function).  Returns the fetched arrays in the order of
    ``outputs`` (and, with ``return_all``, the dict of every forward value and the
    per-stage gradient dicts as well).
    """
    tensors, ops, grads = desc["tensors"], desc["ops"], desc.get("grads", [])
    sets = function_sets(desc, inputs, outputs)
    val = {}
    for i, f in zip(inputs, feeds):
        if sets["marked"][i]:
            a = np.asarray(f)
            val[i] = a if tensors[i]["dtype"] == "i32" else a.astype(dtype)
            assert tuple(val[i].shape) == tuple(tensors[i]["shape"]), (i, val[i].shape)
    for k in sets["fwd_ops"]:                       # creating order
        op = ops[k]
        with np.errstate(over="ignore", invalid="ignore"):
            y = _forward(op, [val[i] for i in op["in"]], dtype, bf16_contraction)
        (o,) = op["out"]
        y = np.asarray(y, dtype=dtype)
        if tensors[o]["dtype"] == "bf16":
            y = round_bf16(y)
        assert tuple(y.shape) == tuple(tensors[o]["shape"]), (k, y.shape, tensors[o]["shape"])
        val[o] = y
    gval = [dict() for _ in grads]
    for s, g in enumerate(grads):
        for o in g["objs"]:
            gval[s][o] = np.ones(tensors[o]["shape"], dtype=dtype)
    for (s, k, pos) in sets["grad_ops"]:            # inverse order inside a stage
        op = ops[k]
        (o,) = op["out"]
        dy = gval[s][o]
        ins = [val[i] for i in op["in"]]
        wanted = {op["in"][q] for q in pos}           # Op(n, n): both positions contribute to dn
        contrib = _backward(op, ins, val[o], dy, [p for p, i in enumerate(op["in"]) if i in wanted],
                            bf16_contraction)
        for p, gp in contrib.items():
            x = op["in"][p]
            gp = _unbroadcast(np.asarray(gp, dtype=dtype), tensors[x]["shape"])
            gval[s][x] = gval[s][x] + gp if x in gval[s] else gp
    grad_node = {}
    for s, g in enumerate(grads):
        for w, gid in zip(g["wrts"], g["grad_ids"]):
            grad_node[gid] = (s, w)
    res = []
    for t in outputs:
        if t in grad_node:
            s, w = grad_node[t]
            res.append(gval[s][w])
        else:
            res.append(val[t])
    if return_all:
        return res, val, gval
    return res


def finite_difference(desc, inputs, feeds, objs, wrt, h=1e-6, bf16_contraction=True):
    """Central differences of sum(all elements of all objs) with respect to input ``wrt``, in fp64."""
    k = inputs.index(wrt)
    base = [None if f is None else np.array(f, dtype=np.float64 if np.asarray(f).dtype.kind == "f" else None)
            for f in feeds]
    x = base[k]
    g = np.zeros_like(x)
    flat, gflat = x.reshape(-1), g.reshape(-1)

    def total():
        return sum(float(np.sum(v)) for v in run_function(desc, inputs, list(objs), base,
                                                              bf16_contraction=bf16_contraction))

    for j in range(flat.size):
        old = flat[j]
        step = h * max(1.0, abs(old))
        flat[j] = old + step
        up = total()
        flat[j] = old - step
        dn = total()
        flat[j] = old
        gflat[j] = (up - dn) / (2 * step)
    return g
