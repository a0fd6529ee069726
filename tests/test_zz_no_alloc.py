"""The allocation-free entry point, btc_execute_static_scratch, against btc_execute.

Some users of the library cannot obtain device memory at the point where they contract (a
plug-in whose host application owns all of it, a real-time loop that must not allocate) and have
no workspace to hand over either.  For them one entry point keeps the split-K scratch in an
8 MiB array inside the library's own device image.  This file checks, through the C-ABI and on
two calls in a row, that it produces what the ordinary entry point produces, and that it refuses
operations whose scratch would not fit.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import helpers
import oracle
from paper_2601_07827_b200 import inputs

pytestmark = pytest.mark.gpu


def _make_op(api, handle, w, A, B, D, split_k=0):
    dt = api.dtype_code(D.dtype)
    tA = api.TensorInfo(handle, dt, A.extents, A.strides)
    tB = api.TensorInfo(handle, dt, B.extents, B.strides)
    tD = api.TensorInfo(handle, dt, D.extents, D.strides)
    tC = tD if w.beta != 0 else None
    op = api.Contraction(handle, tA, w.labelsA, tB, w.labelsB, tC, w.labelsD, tD, w.labelsD, w.alpha, w.beta,
                         w.conjA, w.conjB, w.conjC)
    if split_k:
        op.set_attr(api.ATTR_SPLIT_K, split_k)
    return op


def test_static_scratch_matches_ordinary_execute_twice_in_a_row():
    api = helpers.api()
    handle = api.Handle()
    w = inputs.workloads()["cfg1_f64_small"]          # split-K plan: really uses scratch
    A, B, C, D = inputs.make_workload_tensors(w)
    dA, dB, dC = A.to("cuda"), B.to("cuda"), C.to("cuda")
    op = _make_op(api, handle, w, A, B, D)
    ws_bytes = op.workspace_size()
    assert 0 < ws_bytes <= 8 << 20 and op.split_k > 1
    stream = torch.cuda.current_stream().cuda_stream

    # the existing entry point, with a caller workspace
    d_ref = D.to("cuda")
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    op.execute(stream, dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), d_ref.data_ptr(),
               workspace=ws.data_ptr(), workspace_bytes=ws_bytes)
    torch.cuda.synchronize()
    ref = d_ref.get_logical().cpu().numpy()

    # tolerance scale |alpha| sum|a||b| + |beta||c| as in the other parity tests
    want = D.clone()
    scale = oracle.contract(A.numpy(), w.labelsA, B.numpy(), w.labelsB, C.numpy(), w.labelsD, want.numpy(),
                            w.labelsD, w.alpha, w.beta)
    assert helpers.compare(ref, want.get_logical().numpy(), scale, D.dtype) <= 1.0

    for call in range(2):                              # the second call finds the first one's leftovers
        d_new = D.to("cuda")
        op.execute_static_scratch(stream, dA.data_ptr(), dB.data_ptr(), dC.data_ptr(), d_new.data_ptr())
        torch.cuda.synchronize()
        got = d_new.get_logical().cpu().numpy()
        assert helpers.compare(got, ref, scale, D.dtype) <= 1.0, call
        assert np.array_equal(got, ref), call          # same kernels, same summation order
    assert op.device_error == 0


def test_static_scratch_without_split_k_and_with_other_scalars():
    api = helpers.api()
    handle = api.Handle()
    w = inputs.scaled_down(inputs.workloads()["cfg4_c64_conj"], {"p": 40, "q": 24, "r": 5, "s": 12, "t": 8})
    A, B, C, D = inputs.make_workload_tensors(w)
    dA, dB = A.to("cuda"), B.to("cuda")
    op = _make_op(api, handle, w, A, B, D, split_k=1)
    assert op.workspace_size() == 0
    stream = torch.cuda.current_stream().cuda_stream
    d_ref, d_new = D.to("cuda"), D.to("cuda")
    op.execute(stream, dA.data_ptr(), dB.data_ptr(), 0, d_ref.data_ptr(), alpha=2.0 - 1.0j)
    op.execute_static_scratch(stream, dA.data_ptr(), dB.data_ptr(), 0, d_new.data_ptr(), alpha=2.0 - 1.0j)
    torch.cuda.synchronize()
    assert torch.equal(torch.view_as_real(d_new.get_logical()), torch.view_as_real(d_ref.get_logical()))


def test_static_scratch_refuses_what_does_not_fit():
    api = helpers.api()
    handle = api.Handle()
    dt = api.F64
    tA, tB, tD = (api.TensorInfo(handle, dt, e) for e in ((1024, 4096), (4096, 1024), (1024, 1024)))
    op = api.Contraction(handle, tA, "ik", tB, "kj", None, None, tD, "ij")
    op.set_attr(api.ATTR_SPLIT_K, 8)
    assert op.workspace_size() > 8 << 20
    buf = torch.zeros(8, dtype=torch.float64, device="cuda")       # never touched: the call is refused first
    with pytest.raises(api.BtcError) as ei:
        op.execute_static_scratch(0, buf.data_ptr(), buf.data_ptr(), 0, buf.data_ptr())
    assert ei.value.code == api.ERR_SCRATCH_LIMIT
    assert "8 MiB" in api.explain_error(api.ERR_SCRATCH_LIMIT)
