"""Shared helpers of the GPU parity tests: run one contraction through the C-ABI on the GPU and
through the CPU oracle on the same seeded inputs, and compare element by element.

Acceptance: |d_gpu - d_oracle| <= tol * scale with scale = |alpha| sum|a||b| + |beta||c| from the
oracle; tol = 1e-12 for 64-bit parts and 1e-5 for 32-bit parts; exact equality where scale == 0.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2601_07827_b200 import inputs

TOL = {torch.float32: 1e-5, torch.complex64: 1e-5, torch.float64: 1e-12, torch.complex128: 1e-12}


def api():
    from paper_2601_07827_b200 import build
    build.build()
    from paper_2601_07827_b200 import api as _api
    return _api


def compare(got: np.ndarray, want: np.ndarray, scale: np.ndarray, dtype) -> float:
    """Returns the largest error in units of tol * scale (must be <= 1)."""
    err = np.abs(got.astype(np.complex128) - want.astype(np.complex128))
    assert not np.any(np.isnan(err)), "NaN in result"
    zero = scale == 0
    assert np.all(err[zero] == 0)
    if np.all(zero):
        return 0.0
    return float(np.max(err[~zero] / (TOL[dtype] * scale[~zero])))


def canary_intact(before: torch.Tensor, after: torch.Tensor, touched: torch.Tensor) -> bool:
    """Every buffer position outside `touched` still holds its NaN canary bit pattern."""
    mask = torch.ones(before.numel(), dtype=torch.bool)
    mask[touched] = False
    width = {4: torch.int32, 8: torch.int64, 16: torch.int64}[before.element_size()]
    b = before.view(width).reshape(before.numel(), -1)[mask]
    a = after.view(width).reshape(after.numel(), -1)[mask]
    return bool(torch.equal(a, b))


def run_case(handle, A, la, B, lb, C, D, ld, alpha=1.0, beta=0.0, conjA=False, conjB=False, conjC=False,
             kernel=0, split_k=0, host_path=False, want_status=False, variant=-1, pre_reduce=None):
    """A, B, C, D are inputs.StridedTensor on the CPU; D is not modified.  Returns
    (worst error in tolerance units, status dict or None, GPU result buffer on the CPU)."""
    _api = api()
    in_place = C is D
    dA, dB = A.to("cuda"), B.to("cuda")
    dD = D.to("cuda")
    dC = dD if in_place else (C.to("cuda") if C is not None else None)
    status = None
    if host_path:
        hD = D.clone()
        hC = hD if in_place else C
        dt = _api.dtype_code(D.dtype)
        tA = _api.TensorInfo(handle, dt, A.extents, A.strides)
        tB = _api.TensorInfo(handle, dt, B.extents, B.strides)
        tD = _api.TensorInfo(handle, dt, D.extents, D.strides)
        tC = _api.TensorInfo(handle, dt, C.extents, C.strides) if C is not None else None
        op = _api.Contraction(handle, tA, la, tB, lb, tC, ld, tD, ld, alpha, beta, conjA, conjB, conjC)
        if kernel:
            op.set_attr(_api.ATTR_KERNEL, kernel)
        op.execute_host(0, A.data_ptr(), B.data_ptr(), hC.data_ptr() if hC is not None else 0, hD.data_ptr())
        result = hD.buffer
    else:
        op, status = _api.contract(handle, dA, la, dB, lb, dC, dD, ld, alpha, beta, conjA, conjB, conjC,
                                   stream=torch.cuda.current_stream().cuda_stream, kernel=kernel,
                                   split_k=split_k, want_status=want_status, variant=variant, pre_reduce=pre_reduce)
        torch.cuda.synchronize()
        # no bounded wait gave up; in builds with offset checks (BTC_CHECK_OFFSETS=1): no offset left its tensor
        assert op.device_error == 0, op.device_error
        result = dD.buffer.cpu()

    # oracle on the same inputs
    want = D.clone()
    wantC = want if in_place else C
    scale = oracle.contract(A.numpy(), la, B.numpy(), lb, wantC.numpy() if wantC is not None else None, ld,
                            want.numpy(), ld, alpha, beta, conjA=conjA, conjB=conjB, conjC=conjC)
    pos = D.offsets()
    got = result[pos].numpy()
    ref = want.buffer[pos].numpy()
    worst = compare(got, ref, scale, D.dtype)
    assert canary_intact(D.buffer, result, pos), "bytes outside D's elements were modified"
    return worst, status, result


def workload_case(handle, w: inputs.Workload, **kw):
    A, B, C, D = inputs.make_workload_tensors(w)
    return run_case(handle, A, w.labelsA, B, w.labelsB, C, D, w.labelsD, w.alpha, w.beta,
                    w.conjA, w.conjB, w.conjC, **kw)


def random_tensor(seed, extents, strides, dtype, dist=("uniform", 1.0)):
    flat = inputs.logical_values(seed, extents, dtype, *dist)
    return inputs.place(flat, extents, strides, dtype)
