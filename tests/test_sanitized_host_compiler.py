"""The host compiler (both prunes, lowering, segmentation, slot allocation, code generation) under
AddressSanitizer and UndefinedBehaviorSanitizer: the library is rebuilt with the host-only sources (prune, lower, codegen, specialize, verify)
instrumented and the host-side tests run against it in a child process with the sanitizer runtime
preloaded.  Any report (heap overflow, use after free, signed overflow, misaligned access, ...) fails."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_host_compiler_tests_are_clean_under_asan_and_ubsan():
    asan = subprocess.run(["gcc", "-print-file-name=libasan.so"], capture_output=True, text=True).stdout.strip()
    if not os.path.isabs(asan) or not os.path.exists(asan):
        pytest.skip("no AddressSanitizer runtime on this machine")
    sys.path.insert(0, ROOT)
    from paper_1707_08265_b200 import build
    lib = build.build_sanitized()
    env = dict(os.environ, DRAGON_LIB=lib, LD_PRELOAD=asan,
               ASAN_OPTIONS="detect_leaks=0:abort_on_error=0:exitcode=99", UBSAN_OPTIONS="print_stacktrace=1:halt_on_error=1:exitcode=98")
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "not gpu", "-p", "no:cacheprovider",
                        "tests/test_host_compiler.py", "tests/test_codegen_emulated.py", "tests/test_codegen_invariants.py",
                        "tests/test_inplace.py", "tests/test_gradient_stages.py", "tests/test_verify_program.py", "tests/test_specialize.py"],
                       cwd=ROOT, env=env, capture_output=True, text=True, timeout=1500)
    out = r.stdout + r.stderr
    assert "AddressSanitizer" not in out and "runtime error:" not in out, out[-4000:]
    assert r.returncode == 0, out[-4000:]
    assert "libdragon_san.so" in lib and " passed" in r.stdout
