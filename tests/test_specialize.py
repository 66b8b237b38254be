"""Specialised kernels of graph-VM programs, host side (no GPU): the C++ stitcher (csrc/specialize.cpp) against
the generator's own Python twin, text for text; the PTX of the programs of the toy function, random DAGs, row
DAGs with gradients and the updaters through the assembler; what must not be left in a specialised kernel."""
import os
import shutil
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, os.path.join(ROOT, "paper_1707_08265_b200"))
import vm_ptxgen as gen  # noqa: E402

from oracle import prune as oprune  # noqa: E402
from paper_1707_08265_b200 import binding as B  # noqa: E402
from paper_1707_08265_b200 import workloads as wl  # noqa: E402

_TEMPLATES = {}


def templates(n_regs):
    if n_regs not in _TEMPLATES:
        name, nr, ctas, threads = next(v for v in gen.VARIANTS if v[1] == n_regs)
        _TEMPLATES[n_regs] = gen.Kernel(name, nr, ctas, threads, template=True).build_templates()
    return _TEMPLATES[n_regs]


def loop_start_of(code, ptx):
    """The first instruction of the per-tile body: where the loop end's leaf of the C++ text jumps back to
    (the library does not export the index); it lies behind the loop_begin instruction."""
    import re
    targets = set(re.findall(r"mov\.u32 %arg, \d+;\n\tbra\.uni \$I_(\d+);\n\$le_", ptx))
    assert len(targets) == 1, targets
    k = int(targets.pop())
    ids = [w & 1023 for w in code]
    assert k > ids.index(gen.JOINT_STRIDE * len(gen.JOINT) + gen.PLAIN.index("loop_begin"))
    return k


def programs():
    out = []
    g, ids = wl.toy_function_grad(1 << 20)
    out.append(("toy", g, [ids["x"], ids["a"], ids["b"]], [ids["dx"], ids["da"], ids["db"]]))
    g, inputs, fetch = wl.random_dag(3 * 4096 + 5, 1003, n_ops=64)
    out.append(("dag", g, inputs, fetch))
    g, inputs, fetch = wl.random_row_dag(37, 520, 3002, n_ops=48, n_fetch=2)
    G = oprune.backward_marks(g.desc, fetch, inputs)
    out.append(("rows", g, inputs, fetch + g.grad(fetch, [i for i in inputs if i in G])))
    g, ids = wl.updater([70000], "adam")
    names = ("W", "g", "m", "v", "lr", "beta1", "one_minus_beta1", "beta2", "one_minus_beta2", "eps")
    out.append(("adam", g, [ids[k] for k in names], [ids[k] for k in ("W_new", "m_new", "v_new")]))
    return out


def vm_steps(f):
    return [k for k in range(f.num_launches() + 4) if f.vm_step(k) is not None]


@pytest.mark.parametrize("case", programs(), ids=lambda c: c[0])
def test_stitcher_equals_the_generators_twin_and_the_ptx_assembles(case, tmp_path):
    name, g, inputs, outputs = case
    f = B.Graph.from_desc(g.desc).function(inputs, outputs)
    steps = vm_steps(f)
    assert steps
    ptxas = shutil.which("ptxas") or "/usr/local/cuda/bin/ptxas"
    for k in steps:
        st = f.vm_step(k)
        ptx = f.vm_ptx(k)
        twin = gen.specialise(templates(st["n_regs"]), st["code"], loop_start_of(st["code"], ptx))
        assert ptx == twin
        assert "#" not in ptx                                   # every placeholder was filled
        assert "brx.idx.uni" not in ptx and "ld.shared.v2.u32 {%case, %arg}" not in ptx      # no dispatch, no fetch
        assert ptx.count("$I_%d:" % (len(st["code"]) - 1)) == 1 and ptx.count(".entry dragon_vm_spec") == 1
        if os.path.exists(ptxas):
            p = tmp_path / ("%s_%d.ptx" % (name, k))
            p.write_text(ptx)
            r = subprocess.run([ptxas, "-arch=sm_100a", "-O3", "-v", str(p), "-o", str(tmp_path / "o.cubin")], capture_output=True, text=True)
            assert r.returncode == 0, r.stderr[-2000:]
            regs = int(r.stderr.split("Used ")[1].split(" registers")[0])
            assert regs <= (64 if st["n_regs"] == 3 else 128), regs     # 2 x 512 or 1 x 512 threads per SM


def test_explicit_rounding_everywhere():
    """The two tiers agree bit for bit only if the assembler can never contract a multiplication of one leaf
    with an addition of another: every fp32 add, sub and mul of the generated code names its rounding."""
    import re
    text = gen.generate() + gen.templates_source()
    loose = re.findall(r"\b(?:add|sub|mul)\.(?:ftz\.)?f32(?:x2)? ", text)
    assert not loose, loose[:5]


def test_vm_ptx_of_a_step_that_is_not_a_vm_program_is_refused():
    g, ids = wl.mlp(128, 128, 128, 128)
    inputs = [ids[k] for k in ("X", "W1", "b1", "W2", "b2", "labels")]
    f = B.Graph.from_desc(g.desc).function(inputs, [ids["loss"]])
    with pytest.raises(B.DragonError) as e:
        f.vm_ptx(0)
    assert e.value.code == B.ERR_INVALID_ARG
    assert f.num_specialized() == 0
    assert f.specialize(0) == 0 and f.specialize(1) == 0     # setting the tier needs no device
