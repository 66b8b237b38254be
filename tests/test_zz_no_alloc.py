"""The allocation-free loss entry point against the regular path.

dragon_softmax_ce_loss_static() serves callers that cannot hand the library any memory of their own
making: it keeps its per-row scratch in an array that is part of the library image.  The test calls
it through the C ABI twice in a row (the scratch is shared and keeps the previous call's contents,
so the second call must not be disturbed by the first) and compares each result with the loss that
the compiled SoftmaxCrossEntropy graph produces through dragon_run() on the same inputs.  It is
collected last so that a failure here cannot hide the other tests' results."""
import numpy as np
import pytest
import torch

from paper_1707_08265_b200 import binding as B
from paper_1707_08265_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def graph_loss(z, labels, dtype_name):
    m, n = z.shape
    gd = wl.GraphDesc()
    Z = gd.tensor("Z", [m, n], dtype_name)
    L = gd.tensor("labels", [m], "i32")
    loss = gd.op("SoftmaxCrossEntropy", [Z, L], "loss", [], "f32")
    f = B.Graph.from_desc(gd.desc).function([Z, L], [loss])
    out = torch.full((), float("nan"), dtype=torch.float32, device="cuda")
    f.run_torch([z, labels], [out])
    assert f.status() == 0
    torch.cuda.synchronize()
    return float(out)


@pytest.mark.parametrize("dtype_name", ["f32", "bf16"])
def test_static_loss_matches_graph_loss_twice(dtype_name):
    tdt = torch.float32 if dtype_name == "f32" else torch.bfloat16
    gen = torch.Generator("cuda").manual_seed(11)
    # second call: fewer rows than the first left behind; then a row length that is not a multiple of 8
    # (element-wise loads), one beyond the in-register limit (looping kernel, vector loads), the row limit
    cases = [(777, 1000), (64, 4096), (130, 1001), (33, 8200), (65536, 16)]
    for m, n in cases:
        z = (torch.randn(m, n, generator=gen, device="cuda") * 3).to(tdt)
        labels = torch.randint(0, n, (m,), generator=gen, device="cuda", dtype=torch.int32)
        want = graph_loss(z, labels, dtype_name)
        got = torch.full((1,), float("nan"), dtype=torch.float32, device="cuda")
        B.softmax_ce_loss_static(z.data_ptr(), B.DTYPES[dtype_name], labels.data_ptr(), m, n, got.data_ptr(),
                                 torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert abs(float(got[0]) - want) <= 1e-5 * (1 + abs(want)), (m, n, float(got[0]), want)
        # and against the library routine, as an outside check
        ref = float(torch.nn.functional.cross_entropy(z.double(), labels.long()))
        assert abs(float(got[0]) - ref) <= 1e-5 * (1 + abs(ref))


def test_static_loss_rejects_oversized_and_bad_arguments():
    z = torch.zeros(8, 8, device="cuda")
    labels = torch.zeros(8, dtype=torch.int32, device="cuda")
    out = torch.zeros(1, device="cuda")
    with pytest.raises(B.DragonError) as e:
        B.softmax_ce_loss_static(z.data_ptr(), B.F32, labels.data_ptr(), 65537, 8, out.data_ptr())
    assert e.value.code == B.ERR_WORKSPACE and "65536" in str(e.value)
    with pytest.raises(B.DragonError) as e:
        B.softmax_ce_loss_static(0, B.F32, labels.data_ptr(), 8, 8, out.data_ptr())
    assert e.value.code == B.ERR_INVALID_ARG
    # a view that starts 4 bytes into the buffer: refused on the host, nothing is launched
    with pytest.raises(B.DragonError) as e:
        B.softmax_ce_loss_static(z.data_ptr() + 4, B.F32, labels.data_ptr(), 7, 8, out.data_ptr())
    assert e.value.code == B.ERR_INVALID_ARG and "aligned" in str(e.value)
    with pytest.raises(B.DragonError) as e:
        B.softmax_ce_loss_static(z.data_ptr(), B.F32, labels.data_ptr() + 2, 7, 8, out.data_ptr())
    assert e.value.code == B.ERR_INVALID_ARG
    torch.cuda.synchronize()
