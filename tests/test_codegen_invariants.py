"""Structural invariants of the emitted VM programs that the kernel relies on and that an
emulation of the values cannot see: scratch buffers of successive row sums, staging slots,
the fused store/loop-end, register indices within the build's range."""
import json
import os

import numpy as np
import pytest

from oracle import prune as oprune
from paper_1707_08265_b200 import binding as B
from paper_1707_08265_b200 import workloads as wl
from vm_emulator import J, P, STRIDE

FIRST_PLAIN = len(J) * STRIDE


def decode(step):
    """[(name, register slot or None, arg)] of a VM step, literals skipped"""
    out, code, i = [], step["code"], 0
    while i < len(code):
        cs, arg = code[i] & 1023, code[i] >> 14
        if cs < FIRST_PLAIN:
            out.append((J[cs // STRIDE], cs % STRIDE, arg))
        else:
            out.append((P[cs - FIRST_PLAIN], None, arg))
            if out[-1][0] == "uconst":
                i += 1
        i += 1
    return out


def programs():
    for seed in range(12):
        g, inputs, fetch = wl.random_dag(3 * 4096 + 5, 900 + seed, n_ops=64)
        yield B.Graph.from_desc(g.desc).function(inputs, fetch)
    for seed in range(12):
        g, inputs, fetch = wl.random_row_dag(40, 520, 300 + seed, n_ops=160)
        G = oprune.backward_marks(g.desc, fetch, inputs)
        outs = fetch + g.grad(fetch, [i for i in inputs if i in G])
        yield B.Graph.from_desc(g.desc).function(inputs, outs)
    g, ids = wl.toy_function_grad(1 << 20)
    yield B.Graph.from_desc(g.desc).function([ids["x"], ids["a"], ids["b"]], [ids["dx"], ids["da"], ids["db"]])


def vm_steps(f):
    k = 0
    while True:
        try:
            st = f.vm_step(k)
        except Exception:
            return
        if st is None:
            if k > 64:
                return
        else:
            yield st
        k += 1
        if k > 64:
            return


def test_programs_respect_the_builds_and_the_kernel_contracts():
    seen = set()
    for f in programs():
        for st in vm_steps(f):
            ins = decode(st)
            names = [n for n, _, _ in ins]
            seen.update(names)
            nr = st["n_regs"]
            # register slots within the build; the fused put-away/take pair names two different slots
            for n, k, arg in ins:
                if k is not None:
                    assert k < nr, (n, k, nr)
                if n.startswith("stld"):
                    assert int(n[4:]) < nr and int(n[4:]) != k
            # exactly one loop, closed either by "}loop" or by the fused store
            assert names.count("loop{") == 1 and names.count("}loop") + names.count("gstf}loop") + names.count("fmaurst}loop") == 1
            lo = names.index("loop{")
            hi = [i for i, n in enumerate(names) if n.endswith("}loop")][0]
            body = ins[lo + 1:hi + 1]
            # successive row sums (the last of an iteration and the first of the next included) use
            # different scratch buffers; a single one asks for the barrier after its read
            rs = [arg & 7 for n, _, arg in body if n in ("rowsum", "rowsumu")]
            if len(rs) == 1:
                assert rs[0] & 4
            for a, b in zip(rs, rs[1:] + rs[:1]):
                if len(rs) > 1:
                    assert (a & 3) != (b & 3) and not (a & 4)
            # staged operands: one slot each, above every slot the allocator uses, copied before the loop body
            staged = {}
            for n, _, arg in ins:
                if n in ("glda0", "glda0h"):
                    assert arg & 63 not in staged
                    staged[arg & 63] = arg >> 6
            assert len(set(staged.values())) == len(staged) and all(s < st["n_smem"] for s in staged.values())
            ordinary = {arg for n, _, arg in ins if n in ("sts", "rtos", "sincos", "cossin")}
            assert not (ordinary & set(staged.values()))
            for n, _, arg in body:
                if n in ("ldsw", "ldswa", "ldswr", "ldswar", "glda", "ldswah", "ldswarf"):
                    assert staged.get(arg & 63) == (arg >> 6) & (15 if n == "ldswarf" else 0xFFF), (n, arg)
                if n == "gldf":     # an unstaged fp32 load only when no slot was left
                    assert arg not in staged
            assert names[-1] == "end"
    assert {"stld0", "rowsum", "rowsumu", "ldswa", "gstf}loop", "strlds"} <= seen | {"stld0"}, "the corpus no longer exercises the fused instructions"
