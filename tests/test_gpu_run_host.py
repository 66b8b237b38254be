"""dragon_run_host (host buffers in, host buffers out) against the device-resident run: the plain
path and the chunked one that overlaps copy-in, kernel and copy-out for large elementwise functions."""
import numpy as np
import pytest
import torch

from oracle import interp
from paper_1707_08265_b200 import binding as B
from paper_1707_08265_b200 import workloads as wl
from test_gpu_vm import check, TOL32

pytestmark = pytest.mark.gpu


def host_run(f, feeds, out_shapes, repeats=1):
    f.ensure_workspace()
    nbytes = f.staging_bytes()
    stg = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
    stg_ptr = (stg.data_ptr() + 255) & ~255
    hf = [torch.from_numpy(np.ascontiguousarray(a)).pin_memory() for a in feeds]
    ho = [torch.full(tuple(s), float("nan"), dtype=torch.float32).pin_memory() for s in out_shapes]
    stream = torch.cuda.Stream()
    for _ in range(repeats):
        f.run_host([t.data_ptr() for t in hf], [t.data_ptr() for t in ho], stg_ptr, nbytes, stream.cuda_stream)
    stream.synchronize()
    assert f.status() == 0
    return [t.numpy().astype(np.float64) for t in ho]


# 5000 tiles: above 16 x (2 CTAs x 148 SMs), so the run is chunked; 600 tiles and a tiny case: the plain path
@pytest.mark.parametrize("n", [5000 * 4096 + 77, 600 * 4096 + 5, 1000])
def test_host_run_matches_device_run_and_oracle(n):
    g, ids = wl.toy_function_grad(n)
    x, a, b = wl.toy_feeds(n, 31)
    inputs = [ids["x"], ids["a"], ids["b"]]
    outputs = [ids["dx"], ids["da"], ids["db"]]
    f = B.Graph.from_desc(g.desc).function(inputs, outputs)
    got = host_run(f, [x, a, b], [g.shape(o) for o in outputs], repeats=2)      # twice: the staging area is reused
    dev = [torch.from_numpy(np.ascontiguousarray(v)).cuda() for v in (x, a, b)]
    outs = [torch.empty(tuple(g.shape(o)), dtype=torch.float32, device="cuda") for o in outputs]
    f.run_torch(dev, outs)
    torch.cuda.synchronize()
    assert np.array_equal(got[0], outs[0].cpu().numpy().astype(np.float64))      # same kernel, same bits per element
    for gv, o in zip(got[1:], outs[1:]):                                           # sums: another grouping of the partials
        assert abs(gv - o.item()) <= 1e-6 * (1 + abs(o.item()))
    m = min(n, 1 << 16)                                                            # and the oracle on a prefix (dx) ...
    ref = interp.run_function(g.desc, inputs, outputs, [x, a, b]) if n <= (1 << 22) else None
    if ref is not None:
        for gv, rv in zip(got, ref):
            check(gv, rv, TOL32, "host run n=%d" % n)
    else:
        xs = x[:m].astype(np.float64)
        u = float(a) * xs + float(b)
        check(got[0][:m], np.sin(u) + float(a) * xs * np.cos(u), TOL32, "dx prefix")
        xd = x.astype(np.float64)
        ud = float(a) * xd + float(b)
        check(got[1], np.sum(xd * xd * np.cos(ud)), TOL32, "da")
        check(got[2], np.sum(xd * np.cos(ud)), TOL32, "db")


def test_host_run_of_an_updater_is_chunked_and_exact():
    n = 4800 * 4096
    g, ids = wl.updater([n], "momentum")
    rng = np.random.default_rng(3)
    W, grad, v = (rng.standard_normal(n).astype(np.float32) for _ in range(3))
    lr, mu = np.float32(0.05), np.float32(0.9)
    inputs, outputs = [ids["W"], ids["g"], ids["lr"], ids["v"], ids["mu"]], [ids["W_new"], ids["v_new"]]
    f = B.Graph.from_desc(g.desc).function(inputs, outputs)
    got = host_run(f, [W, grad, lr, v, mu], [[n], [n]])
    ref = interp.run_function(g.desc, inputs, outputs, [W, grad, lr, v, mu])
    for gv, rv in zip(got, ref):
        check(gv, rv, TOL32, "updater")
