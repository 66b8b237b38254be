"""Static verification of graph-VM instruction streams (csrc/verify.cpp), no GPU.

The compiler verifies every program it emits, so the programs of real functions pass; here each kind of index
an instruction can name is pushed out of range in an otherwise valid program, and the structure is broken in
each way the verifier knows, and every such stream must be refused with a message that names the word."""
import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, os.path.join(ROOT, "paper_1707_08265_b200"))
import vm_ptxgen as gen  # noqa: E402

from oracle import prune as oprune  # noqa: E402
from paper_1707_08265_b200 import binding as B  # noqa: E402
from paper_1707_08265_b200 import workloads as wl  # noqa: E402

FIRST_PLAIN = gen.JOINT_STRIDE * len(gen.JOINT)


def plain(name):
    return FIRST_PLAIN + gen.PLAIN.index(name)


def joint(name, slot):
    return gen.JOINT.index(name) * gen.JOINT_STRIDE + slot


def word(case, arg=0):
    return case | (arg << 14)


def program_of(g, inputs, outputs):
    f = B.Graph.from_desc(g.desc).function(inputs, outputs)
    k = next(k for k in range(f.num_launches() + 4) if f.vm_step(k) is not None)
    st = f.vm_step(k)
    ptx = f.vm_ptx(k)
    import re
    loop_start = int(re.findall(r"mov\.u32 %arg, \d+;\n\tbra\.uni \$I_(\d+);\n\$le_", ptx)[0])
    limits = dict(register_slots=st["n_regs"], n_operands=len(st["operands"]), n_smem=st["n_smem"], n_spill=st["n_spill"],
                  n_colacc=sum(1 for r in st["reduced"] if r[0] == 0), n_scalacc=sum(1 for r in st["reduced"] if r[0] == 1),
                  row_mode=st["row_mode"])
    return list(st["code"]), loop_start, limits


def verify(code, loop_start, L):
    B.verify_vm_program(code, loop_start, L["register_slots"], L["n_operands"], L["n_smem"], L["n_spill"], L["n_colacc"],
                        L["n_scalacc"], L["row_mode"])


def refused(code, loop_start, L, what):
    with pytest.raises(B.DragonError) as e:
        verify(code, loop_start, L)
    assert e.value.code == B.ERR_INVALID_ARG and what in str(e.value), str(e.value)


def cases():
    g, ids = wl.toy_function_grad(1 << 16)
    yield program_of(g, [ids["x"], ids["a"], ids["b"]], [ids["dx"], ids["da"], ids["db"]])
    g, inputs, fetch = wl.random_dag(3 * 4096 + 5, 1003, n_ops=64)
    yield program_of(g, inputs, fetch)
    g, inputs, fetch = wl.random_row_dag(37, 520, 3002, n_ops=48, n_fetch=2)
    G = oprune.backward_marks(g.desc, fetch, inputs)
    yield program_of(g, inputs, fetch + g.grad(fetch, [i for i in inputs if i in G]))


def test_compiled_programs_pass_and_tight_limits_do_not():
    for code, loop_start, L in cases():
        verify(code, loop_start, L)
        # the limits the compiler reports are the ones the program needs: one less of anything it uses is refused
        for key, what in (("n_operands", "memory operand"), ("n_smem", "shared-memory slot")):
            if L[key] > 0:
                refused(code, loop_start, dict(L, **{key: L[key] - 1}), what)
        if L["n_scalacc"]:
            refused(code, loop_start, dict(L, n_scalacc=L["n_scalacc"] - 1), "scalar accumulator")
        if L["n_colacc"]:
            refused(code, loop_start, dict(L, n_colacc=L["n_colacc"] - 1), "column accumulator")
        if L["row_mode"]:
            refused(code, loop_start, dict(L, row_mode=False), "row sum in a flat program")


def hand_program():
    """uload; loop{; glda0; ldswa; mulu; gstf}loop; end — y = a*x as in the compiler's own output."""
    code = [word(plain("uload"), 0 | (0 << 9)), word(plain("loop_begin")), word(plain("glda0"), 1 | (0 << 6)),
            word(plain("ldswa"), 1 | (0 << 6)), word(plain("mulu"), 0), word(plain("gstfl"), 2), word(plain("end"))]
    L = dict(register_slots=3, n_operands=3, n_smem=1, n_spill=0, n_colacc=0, n_scalacc=0, row_mode=False)
    return code, 3, L


def test_every_kind_of_index_is_range_checked():
    code, ls, L = hand_program()
    verify(code, ls, L)

    def with_word(pos, w):
        c = list(code)
        c[pos] = w
        return c

    refused(with_word(4, word(1000)), ls, L, "case id")
    refused(with_word(4, word(joint("mul", 3))), ls, L, "register slot")                     # dense build: slots 0..2
    verify(with_word(4, word(joint("mul", 6))), ls, dict(L, register_slots=7))              # fine in the wide build
    refused(with_word(4, word(joint("stld5", 0))), ls, L, "register slot")
    refused(with_word(4, word(plain("mulu"), 512)), ls, L, "uniform")
    verify(with_word(4, word(plain("fmau"), 3 | (511 << 9))), ls, L)        # both fields are 9 bits wide: every value is a uniform
    refused(with_word(4, word(plain("lds"), 1)), ls, L, "shared-memory slot")
    refused(with_word(4, word(joint("rtos", 1), 1)), ls, L, "shared-memory slot")
    refused(with_word(4, word(joint("strlds", 0), 7)), ls, L, "shared-memory slot")
    refused(with_word(4, word(plain("accums"), 2)), ls, L, "shared-memory slot")
    refused(with_word(4, word(plain("gld"), 3)), ls, L, "memory operand")
    refused(with_word(5, word(plain("gstfl"), 40)), ls, L, "memory operand")
    refused(with_word(3, word(plain("ldswa"), 5 | (0 << 6))), ls, L, "memory operand")
    refused(with_word(3, word(plain("ldswa"), 1 | (1 << 6))), ls, L, "shared-memory slot")
    refused(with_word(0, word(plain("uload"), 0 | (9 << 9))), ls, L, "memory operand")
    refused(with_word(4, word(plain("fill"), 0)), ls, L, "spill slot")
    refused(with_word(4, word(joint("spillr", 0), 0)), ls, L, "spill slot")
    refused(with_word(4, word(joint("fmaur", 0), 512)), ls, L, "uniform")
    refused(with_word(4, word(joint("gldr", 0), 3)), ls, L, "memory operand")
    verify(with_word(4, word(joint("ldswarf", 0), 1 | (0 << 6) | (255 << 10))), ls, L)    # u is 8 bits wide: U[u], U[u + 1] exist
    refused(with_word(4, word(joint("ldswarf", 0), 1 | (1 << 6) | (4 << 10))), ls, L, "shared-memory slot")
    refused(with_word(5, word(joint("fmaurstl", 0), 0 | (3 << 9))), ls, L, "memory operand")
    refused(with_word(4, word(plain("colout"), 0)), ls, L, "column accumulator")
    refused(with_word(4, word(plain("ascal1"), 0)), ls, L, "scalar accumulator")
    refused(with_word(4, word(plain("rowsum"), 0)), ls, L, "row sum in a flat program")
    refused(with_word(4, word(plain("rowsum"), 9)), ls, dict(L, row_mode=True), "row-sum argument")
    refused(with_word(4, word(plain("rowsumu"), 0 | (700 << 3))), ls, dict(L, row_mode=True), "uniform")
    verify(with_word(4, word(plain("rowsum"), 5)), ls, dict(L, row_mode=True))


def test_structure_is_checked():
    code, ls, L = hand_program()
    refused(code[:-1], ls, L, "does not end with the end instruction")
    refused(code + [word(plain("relu"))], ls, L, "behind the end")
    verify(code + [word(plain("end"))], ls, L)                                    # padding with end words is allowed
    refused(code[:5] + [word(plain("gstf"), 2)] + code[6:], ls, L, "not closed by a loop end")
    refused(code[:1] + code[2:], ls - 1, L, "behind a loop_begin")
    refused(code, 1, L, "behind a loop_begin")                                    # the body cannot start at the loop_begin itself
    refused(code, 40, L, "behind a loop_begin")
    refused(code[:4] + [word(plain("loop_begin"))] + code[4:], ls, L, "second loop_begin")
    refused(code[:5] + [word(plain("loop_end"))] + code[5:], ls, L, "second loop end")
    # a uconst takes the next word as data: a literal that looks like an instruction is not one ...
    lit = word(1000)
    ok = [word(plain("uconst"), 3), lit] + code
    verify(ok, ls + 2, L)
    # ... the body cannot start inside it, and the stream cannot stop before it
    refused(ok, 1, L, "behind a loop_begin")
    refused([word(plain("loop_begin")), word(plain("loop_end")), word(plain("uconst"), 0)], 1, L, "without its literal")
    refused([], 0, L, "empty program")
    refused(code, ls, dict(L, register_slots=5), "no kernel build")
    refused(code, ls, dict(L, n_operands=41), "limits")


@pytest.mark.parametrize("seed", range(6))
def test_random_single_word_damage_is_caught_or_harmless(seed):
    """Flip the argument field of one word of a real program to a huge value: either the verifier refuses the
    stream, or the instruction takes no argument (its leaf never looks at the field)."""
    takes_no_arg = {plain(n) for n in ("sin", "cos", "expc", "tanh", "sigmoid", "relu", "neg", "step", "clampmask", "onemsq", "yomy",
                                       "divpgb", "rbf16", "loop_begin", "loop_end", "end", "sacc0", "sacc1", "sacc2", "sacc3", "sqrt", "rcp", "tanhb", "sigmoidb", "expcb")}
    for j in ("ldr", "str", "add", "sub", "rsub", "mul", "divp", "rdivp", "addto", "accum", "sincosr", "cossinr", "macc0", "macc1", "macc2",
              "macc3") + tuple("stld%d" % k for k in range(8)):
        takes_no_arg |= {joint(j, s) for s in range(8)}
    rng = np.random.default_rng(seed)
    progs = list(cases())
    code, ls, L = progs[seed % len(progs)]
    uconst = plain("uconst")
    is_literal = [False] * len(code)
    for i, w in enumerate(code):
        if (w & 1023) == uconst and not is_literal[i]:
            is_literal[i + 1] = True
    for _ in range(40):
        i = int(rng.integers(len(code)))
        if is_literal[i]:
            continue
        bad = list(code)
        bad[i] = (bad[i] & 1023) | (0x3FFFF << 14)
        if (code[i] & 1023) in takes_no_arg:
            verify(bad, ls, L)
        else:
            with pytest.raises(B.DragonError):
                verify(bad, ls, L)
