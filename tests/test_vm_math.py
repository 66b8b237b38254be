"""Accuracy sweep of the VM's elementary functions (host instantiation of csrc/vm_math.h, reached
through dragon_host_math) against fp64.  The device build differs only in the reciprocal and the
power of two (rcp.approx, about one ulp; ex2.approx, 2^-22 relative: swept on the GPU in
tests/test_gpu_math_and_updater.py); the polynomials, reductions and constants are the same code."""
import numpy as np

from paper_1707_08265_b200 import binding as B

SIN, COS = B.OPS["Sin"], 100 + B.OPS["Sin"]


def rel(y, r):
    return np.abs(y.astype(np.float64) - r) / np.maximum(np.abs(r), 1e-300)


def test_sin_cos_small_and_medium_arguments():
    x = np.concatenate([np.linspace(-100, 100, 1_000_001), np.linspace(-1e-3, 1e-3, 10001), [0.0, -0.0]]).astype(np.float32)
    xd = x.astype(np.float64)
    for fn, ref in ((SIN, np.sin), (COS, np.cos)):
        y, r = B.host_math(fn, x), ref(xd)
        assert np.max(np.abs(y - r)) < 1.5e-7
        big = np.abs(r) > 1e-3
        assert np.max(rel(y, r)[big]) < 2.5e-7            # about two ulp
    tiny = np.float32([1e-30, -3e-20, 1e-10])
    assert np.array_equal(B.host_math(SIN, tiny), tiny)      # sin x = x to the last bit near zero
    x = (np.float32(10) ** np.linspace(2, 5, 300001)).astype(np.float32)
    for fn, ref in ((SIN, np.sin), (COS, np.cos)):
        assert np.max(np.abs(B.host_math(fn, x) - ref(x.astype(np.float64)))) < 3e-7


def test_sin_cos_huge_arguments_are_exact():
    # up to 2^20 the two-constant reduction; beyond, the multi-word one: every finite fp32 argument is
    # within a few ulp of the fp64 value (NumPy's fp64 sin reduces exactly)
    x = (np.float32(10) ** np.linspace(5, 6.8, 100001)).astype(np.float32)
    for fn, ref in ((SIN, np.sin), (COS, np.cos)):
        assert np.max(np.abs(B.host_math(fn, x) - ref(x.astype(np.float64)))) < 3e-7
    rng = np.random.default_rng(1)
    n = 400000
    bits = (rng.integers(0, 2, n).astype(np.uint32) << 31) | (rng.integers(147, 255, n).astype(np.uint32) << 23) | rng.integers(0, 1 << 23, n).astype(np.uint32)
    x = np.concatenate([bits.view(np.float32), np.float32([1048576.0, 1048577.0, -1048577.0, 3.4028235e38, -3.4028235e38, 1e30, 4.8e8])])
    xd = x.astype(np.float64)
    for fn, ref in ((SIN, np.sin), (COS, np.cos)):
        y, r = B.host_math(fn, x), ref(xd)
        assert np.max(np.abs(y - r)) < 2e-7
        big = np.abs(r) > 1e-3
        assert np.max(rel(y, r)[big]) < 2.5e-7
    # the closest an fp32 number comes to a multiple of pi/2 is still resolved (a relative, not absolute, matter)
    k = np.argsort(np.abs(np.sin(xd)))[:100]
    assert np.max(rel(B.host_math(SIN, x[k]), np.sin(xd[k]))) < 2.5e-7
    y = B.host_math(SIN, np.float32([np.inf, -np.inf, np.nan]))
    assert np.all(np.isnan(y))
    y = B.host_math(COS, np.float32([np.inf, -np.inf, np.nan]))
    assert np.all(np.isnan(y))


def test_exp_tanh_sigmoid_div():
    x = np.linspace(-12, 12, 1_000_001).astype(np.float32)
    assert np.max(rel(B.host_math(B.OPS["Exp"], x), np.exp(np.clip(x.astype(np.float64), -10, 10)))) < 2e-7
    x = np.concatenate([np.linspace(-20, 20, 1_000_001), np.linspace(-1e-3, 1e-3, 10001)]).astype(np.float32)
    r = np.tanh(x.astype(np.float64))
    y = B.host_math(B.OPS["Tanh"], x)
    assert np.max(rel(y, r)[r != 0]) < 4e-7 and np.all(np.abs(y) <= 1)     # about 5 ulp, never beyond +-1
    assert np.sqrt(np.mean(rel(y, r)[r != 0] ** 2)) < 1e-7
    t = B.host_math(B.OPS["Tanh"], np.float32([np.nan, np.inf, -np.inf, 0.0, 1e-30]))
    assert np.isnan(t[0]) and t[1] == 1 and t[2] == -1 and t[3] == 0 and t[4] == np.float32(1e-30)
    # saturation is exact: from 9.3 on (tanh rounds to +-1 in fp32 from 9.02 on; in between the result is within
    # one rounding step of it) the result is +-1, so 1 - y^2 is 0
    x = np.concatenate([np.linspace(9.3, 200, 400001), [1e10, 3e38]]).astype(np.float32)
    assert np.all(B.host_math(B.OPS["Tanh"], x) == 1) and np.all(B.host_math(B.OPS["Tanh"], -x) == -1)
    x = np.linspace(-80, 80, 1_000_001).astype(np.float32)
    assert np.max(rel(B.host_math(B.OPS["Sigmoid"], x), 1 / (1 + np.exp(-x.astype(np.float64))))) < 3e-7
    y = B.host_math(B.OPS["Sigmoid"], np.float32([-200, 200]))
    assert y[0] < 1e-37 and y[1] == 1
    x = np.linspace(-50, 50, 100001).astype(np.float32)
    assert np.max(rel(B.host_math(B.OPS["Div"], x), 1 / (1 + np.abs(x.astype(np.float64))))) < 2e-7
