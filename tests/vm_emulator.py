"""A NumPy emulator of the graph-VM instruction set (csrc/vm_isa.h), for checking on the CPU what the
host compiler emits.  It executes one VM step over the whole domain at once: every "V-wide" value
is an array over all domain elements ([n] in flat mode, [rows, cols] in row mode), so tiling and
thread layout play no role.  Arithmetic is float64; it checks the *program*, not fp32 rounding.
Single-step functions only (feeds and fetches as memory operands)."""
import numpy as np

STRIDE = 8   # case id of a register-operand instruction = index * STRIDE + register slot
J = ["ldr", "str", "add", "sub", "rsub", "mul", "divp", "rdivp", "addto", "accum", "fmaur", "rtos", "stor", "spillr", "fillr",
     "gldr", "sincosr", "cossinr", "macc0", "macc1", "macc2", "macc3", "ldswr", "ldswar",
     "stld0", "stld1", "stld2", "stld3", "stld4", "stld5", "stld6", "stld7", "ldswarf", "fmaurst}loop", "strlds"]
P = ["ldu", "addu", "subu", "rsubu", "mulu", "divpu", "rdivpu", "fmau", "lds", "sts", "adds", "subs", "rsubs", "muls", "divps",
     "rdivps", "sin", "cos", "sincos", "cossin", "expc", "tanh", "sigmoid", "relu", "neg", "step", "clampmask", "onemsq", "yomy", "divpgb",
     "rbf16", "rowsum", "gld", "gst", "gldf", "gstf", "fill", "spill", "uload", "uconst", "loop{", "}loop", "colout", "scalout",
     "sacc0", "sacc1", "sacc2", "sacc3", "ascal0", "ascal1", "ascal2", "ascal3", "glda0", "glda", "ldsw", "ldswa", "gstf}loop", "glda0h", "ldswah", "rowsumu", "accums", "sqrt", "rcp", "tanhb", "sigmoidb", "expcb", "end"]


def _bf16(a):
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    r = (((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16).astype(np.uint32)
    return r.view(np.float32).astype(np.float64)


def run_step(step, feeds, fetch_shapes, nr=STRIDE):
    """step: dict from Function.vm_step; feeds: arrays by feed position; returns {fetch position: array}."""
    code, ops = step["code"], step["operands"]
    shape = (step["n"], step["cols"]) if step["row_mode"] else (step["n"],)
    first_plain = len(J) * STRIDE
    A = [0.0] * 4   # scalar accumulators

    def divp(a, b):
        return a / (1 + np.abs(b))

    acc = np.zeros(shape)
    R = [np.zeros(shape) for _ in range(nr)]
    S, G, U = {}, {}, {}
    out, colout, scalout = {}, {}, {}
    binops = {"add": lambda a, b: a + b, "sub": lambda a, b: a - b, "rsub": lambda a, b: b - a, "mul": lambda a, b: a * b,
              "divp": divp, "rdivp": lambda a, b: divp(b, a)}

    def load(i):
        where, pos, kind, dtype = ops[i]
        assert where == 0, "the emulator handles feeds only"
        a = np.asarray(feeds[pos], dtype=np.float64)
        if kind == 1:
            return np.broadcast_to(a.reshape(1, -1), shape).copy()
        return a.reshape(shape).copy()

    pc = 0
    while True:
        w = code[pc]; pc += 1
        cs, arg = w & 1023, w >> 14
        if cs < first_plain:
            name, k = J[cs // STRIDE], cs % STRIDE
            assert k < nr, "register slot %d beyond the %d of this build" % (k, nr)
            if name == "ldr": acc = R[k].copy()
            elif name == "str": R[k] = acc.copy()
            elif name in binops: acc = binops[name](acc, R[k])
            elif name in ("addto", "accum"): R[k] = R[k] + acc
            elif name == "fmaur": acc = acc * U[arg] + R[k]
            elif name == "rtos": S[arg] = R[k].copy()
            elif name == "stor": R[k] = S[arg].copy()
            elif name == "spillr": G[arg] = R[k].copy()
            elif name == "fillr": R[k] = G[arg].copy()
            elif name == "gldr": acc = load(arg); R[k] = acc.copy()
            elif name in ("ldswr", "ldswar"): acc = load(arg & 63); R[k] = acc.copy(); S[arg >> 6] = acc.copy()
            elif name == "strlds": R[k] = acc.copy(); acc = S[arg].copy()
            elif name == "ldswarf":
                R[k] = load(arg & 63); S[(arg >> 6) & 15] = R[k].copy()
                acc = R[k] * U[arg >> 10] + U[(arg >> 10) + 1]
            elif name == "fmaurst}loop":
                acc = acc * U[arg & 511] + R[k]
                where, pos, kind, dtype = ops[arg >> 9]
                assert where == 1 and kind == 0 and dtype == 0
                out[pos] = np.array(acc, dtype=np.float64).reshape(fetch_shapes[pos])
            elif name == "sincosr": R[k] = np.cos(acc); acc = np.sin(acc)
            elif name == "cossinr": R[k] = np.sin(acc); acc = np.cos(acc)
            elif name.startswith("macc"): A[int(name[4])] += float((acc * R[k]).sum())
            elif name.startswith("stld"):
                assert int(name[4]) < nr
                R[int(name[4])] = acc.copy(); acc = R[k].copy()
            else: raise ValueError(name)
            continue
        name = P[cs - first_plain]
        if name == "ldu": acc = np.full(shape, U[arg])
        elif name[:-1] in binops and name.endswith("u"): acc = binops[name[:-1]](acc, U[arg])
        elif name == "fmau": acc = acc * U[arg & 511] + U[arg >> 9]
        elif name == "lds": acc = S[arg].copy()
        elif name == "sts": S[arg] = acc.copy()
        elif name[:-1] in binops and name.endswith("s") and name not in ("cos",): acc = binops[name[:-1]](acc, S[arg])
        elif name == "sin": acc = np.sin(acc)
        elif name == "cos": acc = np.cos(acc)
        elif name == "sincos": S[arg] = np.cos(acc); acc = np.sin(acc)
        elif name == "cossin": S[arg] = np.sin(acc); acc = np.cos(acc)
        elif name == "expc": acc = np.exp(np.clip(acc, -10, 10))
        elif name == "tanh": acc = np.tanh(acc)
        elif name == "tanhb":
            assert np.all(np.abs(acc[np.isfinite(acc)]) <= 4.01), "tanhb outside its proven range"
            acc = np.tanh(acc)
        elif name == "sigmoidb":
            assert np.all(np.abs(acc[np.isfinite(acc)]) <= 80.0), "sigmoidb outside its proven range"
            acc = 1 / (1 + np.exp(-acc))
        elif name == "expcb":
            assert np.all(np.abs(acc[np.isfinite(acc)]) <= 10.0), "expcb outside its proven range"
            acc = np.exp(acc)
        elif name == "sigmoid": acc = 1 / (1 + np.exp(-acc))
        elif name == "relu": acc = np.maximum(acc, 0)
        elif name == "neg": acc = -acc
        elif name == "step": acc = (acc > 0).astype(np.float64)
        elif name == "clampmask": acc = ((acc >= -10) & (acc <= 10)).astype(np.float64)
        elif name == "onemsq": acc = 1 - acc * acc
        elif name == "yomy": acc = acc * (1 - acc)
        elif name == "divpgb": acc = -np.sign(acc) / (1 + np.abs(acc)) ** 2
        elif name == "rbf16": acc = _bf16(acc)
        elif name == "rowsum": acc = np.broadcast_to(acc.sum(axis=-1, keepdims=True), shape).copy()
        elif name == "rowsumu": acc = np.broadcast_to(acc.sum(axis=-1, keepdims=True), shape).copy() * U[arg >> 3]
        elif name in ("gld", "gldf"): acc = load(arg)
        elif name in ("gst", "gstf", "gstf}loop"):
            where, pos, kind, dtype = ops[arg]
            assert where == 1
            v = acc if kind == 0 else (acc[0] if kind == 1 else acc.reshape(-1)[0])
            out[pos] = np.array(_bf16(v) if dtype == 1 else v, dtype=np.float64).reshape(fetch_shapes[pos])
        elif name == "fill": acc = G[arg].copy()
        elif name == "spill": G[arg] = acc.copy()
        elif name == "uload":
            where, pos, kind, dtype = ops[arg >> 9]
            U[arg & 511] = float(np.asarray(feeds[pos]).reshape(-1)[0])
        elif name == "uconst":
            U[arg] = float(np.array([code[pc]], dtype=np.uint32).view(np.float32)[0]); pc += 1
        elif name in ("loop{", "}loop"): pass
        elif name == "colout": colout[arg] = acc.sum(axis=0)
        elif name == "scalout": scalout[arg] = acc.sum()
        elif name in ("glda0", "glda", "glda0h"): pass      # the copy itself is modelled at the read
        elif name == "ldswah": acc = load(arg & 63)
        elif name in ("ldsw", "ldswa"): acc = load(arg & 63); S[arg >> 6] = acc.copy()
        elif name == "accums": S[arg] = S[arg] + acc
        elif name == "sqrt": acc = np.sqrt(acc)
        elif name == "rcp": acc = 1 / acc
        elif name.startswith("sacc"): A[int(name[4])] += float(acc.sum())
        elif name.startswith("ascal"): scalout[arg] = A[int(name[5])]
        elif name == "end": break
        else: raise ValueError(name)
    return out, colout, scalout
