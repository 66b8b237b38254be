"""The PTX generator of the graph-VM kernel against the instruction-set header: same instruction
lists in the same order, same parameter-block offsets, and PTX that the assembler accepts."""
import os
import re
import shutil
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_1707_08265_b200", "csrc")
sys.path.insert(0, os.path.join(ROOT, "paper_1707_08265_b200"))
import vm_ptxgen as gen  # noqa: E402

FIELDS = {"code": "P_CODE", "spill": "P_SPILL", "colpart": "P_COLPART", "scalpart": "P_SCALPART", "status": "P_STATUS",
          "n": "P_N", "n_code": "P_NCODE", "row_mode": "P_ROWMODE", "cols": "P_COLS", "n_spill": "P_NSPILL",
          "n_tiles": "P_NTILES", "loop_start": "P_LOOPSTART", "grid": "P_GRID", "n_full_tiles": "P_NFULL", "status_clear": "P_STATUSCLEAR", "tile_stride_bytes": "P_STRIDE",
          "full_end_bytes": "P_FULLEND", "next_end_bytes": "P_NEXTEND", "all_end_bytes": "P_ALLEND", "operand": "P_OPERAND"}


def _enum(body):
    body = re.sub(r"//.*", "", body)
    return [m.lower() for m in re.findall(r"\b[JP]_(\w+)", body)]


def test_instruction_lists_match_the_header():
    h = open(os.path.join(CSRC, "vm_isa.h")).read()
    joint = _enum(re.search(r"enum Joint : int \{(.*?)J_COUNT", h, re.S).group(1))
    plain = _enum(re.search(r"enum Plain : int \{(.*?)P_COUNT_", h, re.S).group(1))
    rename = {"spill": "spillr", "fill": "fillr"}
    assert [rename.get(j, j) for j in joint] == gen.JOINT
    assert plain == gen.PLAIN
    assert int(re.search(r"kJointStride = (\d+)", h).group(1)) == gen.JOINT_STRIDE
    assert int(re.search(r"kVmScalarAccs = (\d+)", h).group(1)) == gen.N_SACC
    wide, dense = re.search(r"kVmRegsWide = (\d+), kVmRegsDense = (\d+)", h).groups()
    assert set(gen.VARIANTS) == {("dragon_vm_wide", int(wide), 1, 512), ("dragon_vm_dense", int(dense), 2, 512)}
    threads, vec = re.search(r"DRAGON_VM_THREADS (\d+)", h).group(1), re.search(r"DRAGON_VM_VEC (\d+)", h).group(1)
    assert int(threads) * int(vec) == gen.TILE


def test_parameter_block_offsets(tmp_path):
    fields = {f: getattr(gen, c) for f, c in FIELDS.items() if hasattr(gen, c)}
    assert {"code", "n", "operand", "grid"} <= set(fields)
    src = tmp_path / "off.cpp"
    src.write_text('#include <cstddef>\n#include <cstdio>\n#include "vm_isa.h"\nint main() {\n' +
                   "".join('  std::printf("%s %%zu\\n", offsetof(dragon::vm::Params, %s));\n' % (f, f) for f in fields) +
                   '  std::printf("size %zu\\n", sizeof(dragon::vm::Params));\n  return 0;\n}\n')
    exe = tmp_path / "off"
    subprocess.run(["g++", "-std=c++17", "-I", CSRC, str(src), "-o", str(exe)], check=True)
    got = dict(l.split() for l in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.splitlines())
    for f, off in fields.items():
        assert int(got[f]) == off, f
    assert int(got["size"]) == gen.P_SIZE


def test_generated_ptx_assembles(tmp_path):
    ptxas = shutil.which("ptxas") or "/usr/local/cuda/bin/ptxas"
    if not os.path.exists(ptxas):
        pytest.skip("no ptxas on this machine")
    ptx = tmp_path / "vm.ptx"
    ptx.write_text(gen.generate())
    r = subprocess.run([ptxas, "-arch=sm_100a", "-O3", "-v", str(ptx), "-o", str(tmp_path / "vm.cubin")], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    used = dict(re.findall(r"Compiling entry function '(\w+)'.*?Used (\d+) registers", r.stderr, re.S))
    assert int(used["dragon_vm_dense"]) <= 64 and int(used["dragon_vm_wide"]) <= 128   # 2 x 512 and 1 x 512 threads per SM
