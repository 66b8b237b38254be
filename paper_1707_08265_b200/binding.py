"""Thin ctypes binding of libdragon.so: same names as include/dragon.h, argument marshalling only.

Every step of the evaluated path runs in the library's CUDA kernels; nothing here computes.
The library must have been built (``python -m paper_1707_08265_b200.build`` or
``__graft_entry__.build()``); loading fails loudly otherwise.
"""
import ctypes
import os

HERE = os.path.dirname(os.path.abspath(__file__))
# DRAGON_LIB names another build of the same library (the sanitizer build of build.build_sanitized)
LIB_PATH = os.environ.get("DRAGON_LIB") or os.path.join(HERE, "libdragon.so")

OK = 0
ERR_INVALID_ARG, ERR_SHAPE, ERR_DTYPE, ERR_NOT_SSA, ERR_MISSING_INPUT = -1, -2, -3, -4, -5
ERR_NO_PATH, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = -6, -7, -8, -9, -10
F32, BF16, I32 = 0, 1, 2
DTYPES = {"f32": F32, "bf16": BF16, "i32": I32}
OPS = {"Add": 0, "Sub": 1, "Mul": 2, "Div": 3, "Sin": 4, "Exp": 5, "Tanh": 6, "Sigmoid": 7, "ReLU": 8,
       "Sum": 9, "Mean": 10, "InnerProduct": 11, "BiasAdd": 12, "SoftmaxCrossEntropy": 13, "Sqrt": 14,
       "Reciprocal": 15, "Opaque": 16}

_lib = None

_c = ctypes
_SIGNATURES = {
    "dragon_graph_create": (_c.c_void_p, []),
    "dragon_graph_destroy": (None, [_c.c_void_p]),
    "dragon_add_tensor": (_c.c_int32, [_c.c_void_p, _c.c_char_p, _c.c_int, _c.c_int, _c.POINTER(_c.c_int64)]),
    "dragon_add_op": (_c.c_int32, [_c.c_void_p, _c.c_int, _c.POINTER(_c.c_int32), _c.c_int, _c.POINTER(_c.c_int32),
                                   _c.c_int, _c.POINTER(_c.c_double), _c.c_int]),
    "dragon_add_grad": (_c.c_int, [_c.c_void_p, _c.POINTER(_c.c_int32), _c.c_int, _c.POINTER(_c.c_int32), _c.c_int,
                                   _c.POINTER(_c.c_int32)]),
    "dragon_graph_num_tensors": (_c.c_int, [_c.c_void_p]),
    "dragon_graph_num_ops": (_c.c_int, [_c.c_void_p]),
    "dragon_function": (_c.c_void_p, [_c.c_void_p, _c.POINTER(_c.c_int32), _c.c_int, _c.POINTER(_c.c_int32), _c.c_int]),
    "dragon_function_destroy": (None, [_c.c_void_p]),
    "dragon_function_specialize": (_c.c_int, [_c.c_void_p, _c.c_int]),
    "dragon_function_num_specialized": (_c.c_int, [_c.c_void_p]),
    "dragon_function_vm_ptx": (_c.c_int, [_c.c_void_p, _c.c_int, _c.c_char_p, _c.c_int]),
    "dragon_verify_vm_program": (_c.c_int, [_c.POINTER(_c.c_uint32), _c.c_int, _c.c_int, _c.c_int, _c.c_int, _c.c_int, _c.c_int,
                                            _c.c_int, _c.c_int, _c.c_int]),
    "dragon_workspace_create": (_c.c_void_p, []),
    "dragon_workspace_destroy": (None, [_c.c_void_p]),
    "dragon_workspace_feed": (_c.c_int, [_c.c_void_p, _c.c_char_p, _c.c_int, _c.c_int, _c.POINTER(_c.c_int64), _c.c_void_p,
                                         _c.c_void_p]),
    "dragon_workspace_fetch": (_c.c_int, [_c.c_void_p, _c.c_char_p, _c.c_void_p, _c.c_size_t, _c.c_void_p]),
    "dragon_workspace_tensor": (_c.c_void_p, [_c.c_void_p, _c.c_char_p, _c.POINTER(_c.c_int), _c.POINTER(_c.c_int),
                                              _c.POINTER(_c.c_int64)]),
    "dragon_workspace_bytes": (_c.c_size_t, [_c.c_void_p]),
    "dragon_workspace_run": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.POINTER(_c.c_char_p), _c.c_void_p]),
    "dragon_function_marked": (_c.c_int, [_c.c_void_p, _c.POINTER(_c.c_uint8), _c.c_int]),
    "dragon_function_kept_ops": (_c.c_int, [_c.c_void_p, _c.POINTER(_c.c_int32), _c.c_int, _c.POINTER(_c.c_int),
                                            _c.POINTER(_c.c_int32), _c.POINTER(_c.c_uint32), _c.c_int, _c.POINTER(_c.c_int)]),
    "dragon_function_used_inputs": (_c.c_int, [_c.c_void_p, _c.POINTER(_c.c_uint8), _c.c_int]),
    "dragon_function_can_alias": (_c.c_int, [_c.c_void_p, _c.c_int, _c.c_int]),
    "dragon_function_num_launches": (_c.c_int, [_c.c_void_p]),
    "dragon_function_describe": (_c.c_int, [_c.c_void_p, _c.c_char_p, _c.c_int]),
    "dragon_function_vm_step": (_c.c_int, [_c.c_void_p, _c.c_int, _c.POINTER(_c.c_int64), _c.POINTER(_c.c_uint32), _c.c_int,
                                           _c.POINTER(_c.c_int64), _c.c_int, _c.POINTER(_c.c_int64), _c.c_int]),
    "dragon_function_workspace_bytes": (_c.c_size_t, [_c.c_void_p]),
    "dragon_function_set_workspace": (_c.c_int, [_c.c_void_p, _c.c_void_p, _c.c_size_t]),
    "dragon_run": (_c.c_int, [_c.c_void_p, _c.POINTER(_c.c_void_p), _c.POINTER(_c.c_void_p), _c.c_void_p]),
    "dragon_function_status": (_c.c_int, [_c.c_void_p]),
    "dragon_function_staging_bytes": (_c.c_size_t, [_c.c_void_p]),
    "dragon_run_host": (_c.c_int, [_c.c_void_p, _c.POINTER(_c.c_void_p), _c.POINTER(_c.c_void_p), _c.c_void_p,
                                   _c.c_size_t, _c.c_void_p]),
    "dragon_function_rename_dictionary": (_c.c_int, [_c.c_void_p, _c.POINTER(_c.c_int32), _c.c_int]),
    "dragon_function_workspace_tensors": (_c.c_int, [_c.c_void_p, _c.POINTER(_c.c_int64), _c.c_int]),
    "dragon_function_profile": (_c.c_int, [_c.c_void_p, _c.c_int, _c.c_int]),
    "dragon_function_profile_read": (_c.c_int, [_c.c_void_p, _c.POINTER(_c.c_double), _c.POINTER(_c.c_int)]),
    "dragon_softmax_ce_loss_static": (_c.c_int, [_c.c_void_p, _c.c_int, _c.c_void_p, _c.c_int, _c.c_int, _c.c_void_p, _c.c_void_p]),
    "dragon_host_math": (_c.c_int, [_c.c_int, _c.POINTER(_c.c_float), _c.POINTER(_c.c_float), _c.c_int]),
    "dragon_last_error": (_c.c_char_p, []),
}


def lib():
    """The loaded library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libdragon.so is missing: build it with `python -m paper_1707_08265_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


class DragonError(RuntimeError):
    def __init__(self, code, where):
        msg = lib().dragon_last_error()
        super().__init__("%s failed with code %d: %s" % (where, code, msg.decode() if msg else ""))
        self.code = code


def _ids(seq):
    arr = (_c.c_int32 * max(1, len(seq)))(*seq)
    return arr


class Graph:
    """dragon_graph_t: tensors and operators in creation order."""

    def __init__(self):
        self.h = lib().dragon_graph_create()
        if not self.h:
            raise MemoryError("dragon_graph_create")

    def close(self):
        if self.h:
            lib().dragon_graph_destroy(self.h)
            self.h = None

    __del__ = close

    def add_tensor(self, name, dtype, shape):
        shp = (_c.c_int64 * max(1, len(shape)))(*shape)
        r = lib().dragon_add_tensor(self.h, name.encode(), dtype, len(shape), shp)
        if r < 0:
            raise DragonError(r, "dragon_add_tensor")
        return r

    def add_op(self, op_type, ins, outs):
        r = lib().dragon_add_op(self.h, op_type, _ids(ins), len(ins), _ids(outs), len(outs), None, 0)
        if r < 0:
            raise DragonError(r, "dragon_add_op")
        return r

    def add_grad(self, objs, wrts):
        out = (_c.c_int32 * max(1, len(wrts)))()
        r = lib().dragon_add_grad(self.h, _ids(objs), len(objs), _ids(wrts), len(wrts), out)
        if r < 0:
            raise DragonError(r, "dragon_add_grad")
        return list(out[:len(wrts)])

    def num_tensors(self):
        return lib().dragon_graph_num_tensors(self.h)

    def num_ops(self):
        return lib().dragon_graph_num_ops(self.h)

    def function(self, inputs, outputs):
        return Function(self, inputs, outputs)

    @staticmethod
    def from_desc(desc):
        """Replays a graph description (see workloads.GraphDesc) through the C ABI.  Tensors,
        operators and gradient stages are created in the same order, so ids coincide."""
        g = Graph()
        grad_ids = {gid for st in desc.get("grads", []) for gid in st["grad_ids"]}
        stage_first = {st["grad_ids"][0]: st for st in desc.get("grads", []) if st["grad_ids"]}
        producer = {}
        for k, op in enumerate(desc["ops"]):
            for o in op["out"]:
                producer[o] = k
        next_op = 0
        for t, ti in enumerate(desc["tensors"]):
            if t in grad_ids:
                if t in stage_first:
                    st = stage_first[t]
                    got = g.add_grad(st["objs"], st["wrts"])
                    assert got == list(st["grad_ids"]), (got, st["grad_ids"])
                continue
            tid = g.add_tensor(ti["name"], DTYPES[ti["dtype"]], ti["shape"])
            assert tid == t
            # operators whose outputs are all declared can be appended now (creation order)
            while next_op < len(desc["ops"]) and max(desc["ops"][next_op]["out"]) <= t:
                op = desc["ops"][next_op]
                oid = g.add_op(OPS[op["type"]], op["in"], op["out"])
                assert oid == next_op
                next_op += 1
        assert next_op == len(desc["ops"])
        return g


class Function:
    """dragon_function_t: the pruned, compiled function(inputs, outputs)."""

    def __init__(self, graph, inputs, outputs):
        self.n_in, self.n_out = len(inputs), len(outputs)
        self.n_tensors = graph.num_tensors()
        self.n_ops = graph.num_ops()
        self.h = lib().dragon_function(graph.h, _ids(inputs), len(inputs), _ids(outputs), len(outputs))
        if not self.h:
            raise DragonError(-1, "dragon_function")
        self._ws = None

    def close(self):
        if self.h:
            lib().dragon_function_destroy(self.h)
            self.h = None

    __del__ = close

    def marked(self):
        buf = (_c.c_uint8 * self.n_tensors)()
        r = lib().dragon_function_marked(self.h, buf, self.n_tensors)
        if r < 0:
            raise DragonError(r, "dragon_function_marked")
        return list(buf)

    def kept_ops(self):
        cap = 2 * self.n_ops * 4 + 8
        fwd = (_c.c_int32 * cap)()
        gops = (_c.c_int32 * cap)()
        mask = (_c.c_uint32 * cap)()
        nf, ng = _c.c_int(), _c.c_int()
        r = lib().dragon_function_kept_ops(self.h, fwd, cap, _c.byref(nf), gops, mask, cap, _c.byref(ng))
        if r < 0:
            raise DragonError(r, "dragon_function_kept_ops")
        assert nf.value <= cap and ng.value <= cap
        return list(fwd[:nf.value]), list(gops[:ng.value]), list(mask[:ng.value])

    def used_inputs(self):
        buf = (_c.c_uint8 * max(1, self.n_in))()
        r = lib().dragon_function_used_inputs(self.h, buf, self.n_in)
        if r < 0:
            raise DragonError(r, "dragon_function_used_inputs")
        return list(buf[:self.n_in])

    def can_alias(self, input_pos, output_pos):
        r = lib().dragon_function_can_alias(self.h, input_pos, output_pos)
        if r < 0:
            raise DragonError(r, "dragon_function_can_alias")
        return bool(r)

    def num_launches(self):
        return lib().dragon_function_num_launches(self.h)

    def describe(self):
        buf = _c.create_string_buffer(1 << 16)
        lib().dragon_function_describe(self.h, buf, len(buf))
        return buf.value.decode()

    def vm_step(self, step):
        """Instruction stream and operand table of a graph-VM step, or None for another kind of step."""
        info = (_c.c_int64 * 10)()
        if lib().dragon_function_vm_step(self.h, step, info, None, 0, None, 0, None, 0) < 0:
            return None
        code = (_c.c_uint32 * max(1, info[0]))()
        ops = (_c.c_int64 * max(4, 4 * info[3]))()
        red = (_c.c_int64 * max(3, 3 * info[8]))()
        lib().dragon_function_vm_step(self.h, step, info, code, info[0], ops, info[3], red, info[8])
        return {"code": list(code[:info[0]]), "row_mode": bool(info[1]), "cols": info[2], "n": info[6] | (info[7] << 32),
                "n_spill": info[4], "n_smem": info[5], "n_regs": info[9],
                "operands": [tuple(ops[4 * i:4 * i + 4]) for i in range(info[3])],
                "reduced": [tuple(red[3 * i:3 * i + 3]) for i in range(info[8])]}

    def specialize(self, mode=2):
        """0: interpreter; 1: specialised kernels from the first run on (default); 2: specialise now."""
        r = lib().dragon_function_specialize(self.h, mode)
        if r < 0:
            raise DragonError(r, "dragon_function_specialize")
        return r

    def num_specialized(self):
        return lib().dragon_function_num_specialized(self.h)

    def vm_ptx(self, step):
        """PTX text of the specialised kernel of a graph-VM step (no GPU needed)."""
        n = lib().dragon_function_vm_ptx(self.h, step, None, 0)
        if n < 0:
            raise DragonError(n, "dragon_function_vm_ptx")
        buf = _c.create_string_buffer(n + 1)
        lib().dragon_function_vm_ptx(self.h, step, buf, n + 1)
        return buf.value.decode()

    def rename_dictionary(self):
        """Algorithm 3: per tensor id the ancestor it may be renamed to (-1: not marked)."""
        rd = (_c.c_int32 * max(1, self.n_tensors))()
        r = lib().dragon_function_rename_dictionary(self.h, rd, self.n_tensors)
        if r < 0:
            raise DragonError(r, "dragon_function_rename_dictionary")
        return list(rd[:self.n_tensors])

    def workspace_tensors(self):
        """[(offset, bytes, first step, last step, in place)] of the tensors that cross kernels."""
        n = lib().dragon_function_workspace_tensors(self.h, None, 0)
        buf = (_c.c_int64 * max(5, 5 * n))()
        lib().dragon_function_workspace_tensors(self.h, buf, n)
        return [tuple(buf[5 * i:5 * i + 5]) for i in range(n)]

    def workspace_bytes(self):
        return lib().dragon_function_workspace_bytes(self.h)

    def set_workspace(self, dev_ptr, nbytes):
        r = lib().dragon_function_set_workspace(self.h, dev_ptr, nbytes)
        if r < 0:
            raise DragonError(r, "dragon_function_set_workspace")

    def run(self, feed_ptrs, fetch_ptrs, stream=0):
        feeds = (_c.c_void_p * max(1, self.n_in))(*[p or None for p in feed_ptrs])
        fetches = (_c.c_void_p * max(1, self.n_out))(*fetch_ptrs)
        r = lib().dragon_run(self.h, feeds, fetches, stream)
        if r < 0:
            raise DragonError(r, "dragon_run")

    def status(self):
        return lib().dragon_function_status(self.h)

    def staging_bytes(self):
        return lib().dragon_function_staging_bytes(self.h)

    def run_host(self, host_feed_ptrs, host_fetch_ptrs, staging_ptr, staging_bytes, stream=0):
        feeds = (_c.c_void_p * max(1, self.n_in))(*[p or None for p in host_feed_ptrs])
        fetches = (_c.c_void_p * max(1, self.n_out))(*host_fetch_ptrs)
        r = lib().dragon_run_host(self.h, feeds, fetches, staging_ptr, staging_bytes, stream)
        if r < 0:
            raise DragonError(r, "dragon_run_host")

    def profile(self, step, capacity=1024):
        r = lib().dragon_function_profile(self.h, step, capacity)
        if r < 0:
            raise DragonError(r, "dragon_function_profile")

    def profile_read(self):
        ms, runs = _c.c_double(), _c.c_int()
        r = lib().dragon_function_profile_read(self.h, _c.byref(ms), _c.byref(runs))
        if r < 0:
            raise DragonError(r, "dragon_function_profile_read")
        return ms.value, runs.value

    # ---- convenience for torch tensors (device memory and streams only) ----
    def ensure_workspace(self):
        import torch
        if self._ws is None:
            nbytes = max(256, self.workspace_bytes())
            self._ws = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
            base = (self._ws.data_ptr() + 255) & ~255
            self.set_workspace(base, nbytes)

    def run_torch(self, feeds, fetches, stream=None):
        """feeds / fetches: lists of CUDA torch tensors (None for a pruned input)."""
        import torch
        self.ensure_workspace()
        s = stream if stream is not None else torch.cuda.current_stream()
        self.run([0 if t is None else t.data_ptr() for t in feeds], [t.data_ptr() for t in fetches], s.cuda_stream)


class Workspace:
    """dragon_workspace_t: named tensors that stay in device memory between runs (feed, fetch, run by name)."""

    def __init__(self):
        self.h = lib().dragon_workspace_create()
        if not self.h:
            raise DragonError(-1, "dragon_workspace_create")

    def close(self):
        if self.h:
            lib().dragon_workspace_destroy(self.h)
            self.h = None

    __del__ = close

    def feed(self, name, dtype, shape, src_ptr, stream=0):
        """src_ptr: address of host or device memory holding the tensor (0 creates it zero-filled)."""
        arr = (_c.c_int64 * max(1, len(shape)))(*shape)
        r = lib().dragon_workspace_feed(self.h, name.encode(), dtype, len(shape), arr, src_ptr or None, stream)
        if r < 0:
            raise DragonError(r, "dragon_workspace_feed")

    def fetch(self, name, dst_ptr, nbytes, stream=0):
        r = lib().dragon_workspace_fetch(self.h, name.encode(), dst_ptr, nbytes, stream)
        if r < 0:
            raise DragonError(r, "dragon_workspace_fetch")

    def tensor(self, name):
        """(device address, dtype, shape) of a named tensor."""
        dt, rk = _c.c_int(), _c.c_int()
        shp = (_c.c_int64 * 2)()
        p = lib().dragon_workspace_tensor(self.h, name.encode(), _c.byref(dt), _c.byref(rk), shp)
        if not p:
            raise DragonError(-1, "dragon_workspace_tensor")
        return p, dt.value, list(shp[:rk.value])

    def nbytes(self):
        return lib().dragon_workspace_bytes(self.h)

    def run(self, function, output_names=None, stream=0):
        """output_names: None, or one name (or None) per output of the function."""
        names = None
        if output_names is not None:
            assert len(output_names) == function.n_out
            names = (_c.c_char_p * function.n_out)(*[None if n is None else n.encode() for n in output_names])
        r = lib().dragon_workspace_run(self.h, function.h, names, stream)
        if r < 0:
            raise DragonError(r, "dragon_workspace_run")


def verify_vm_program(code, loop_start, register_slots, n_operands, n_smem, n_spill, n_colacc, n_scalacc, row_mode):
    """dragon_verify_vm_program: raises DragonError (INVALID_ARG) naming the first bad word."""
    arr = (_c.c_uint32 * max(1, len(code)))(*code)
    r = lib().dragon_verify_vm_program(arr, len(code), loop_start, register_slots, n_operands, n_smem, n_spill, n_colacc,
                                       n_scalacc, int(bool(row_mode)))
    if r < 0:
        raise DragonError(r, "dragon_verify_vm_program")


def softmax_ce_loss_static(logits_ptr, dtype, labels_ptr, rows, cols, loss_ptr, stream=0):
    """dragon_softmax_ce_loss_static: allocation-free mean cross-entropy (device pointers)."""
    r = lib().dragon_softmax_ce_loss_static(logits_ptr, dtype, labels_ptr, rows, cols, loss_ptr, stream)
    if r < 0:
        raise DragonError(r, "dragon_softmax_ce_loss_static")


def host_math(fn, x):
    import numpy as np
    x = np.ascontiguousarray(x, dtype=np.float32)
    y = np.empty_like(x)
    r = lib().dragon_host_math(fn, x.ctypes.data_as(_c.POINTER(_c.c_float)), y.ctypes.data_as(_c.POINTER(_c.c_float)), x.size)
    if r < 0:
        raise DragonError(r, "dragon_host_math")
    return y
