"""GPU parity for operations whose tensors do not share one element type (Sec. "Challenge: Datatypes"):
real operands among complex ones, and 32-bit storage with sums kept in fp64 (the compute precision an
operation may ask for, Sec. "Tensor Operation Descriptors"), against the mixed-type CPU oracle."""
import numpy as np
import pytest
import torch

import helpers
import oracle
from paper_2601_07827_b200 import inputs

pytestmark = pytest.mark.gpu

PAIRS = [(torch.float64, torch.complex128), (torch.float32, torch.complex64)]
SHAPES = {
    # name: (labelsA, labelsB, labelsD, extents)
    "matrix_product": ("ik", "kj", "ij", dict(i=70, j=45, k=33)),
    "batch_and_permuted_output": ("hik", "kjh", "jih", dict(h=3, i=20, j=17, k=12)),
    "isolated_and_repeated_labels": ("ikkx", "kj", "ij", dict(i=15, j=14, k=9, x=4)),
    "outer_product": ("i", "j", "ij", dict(i=40, j=30)),
}


def _ext(labels, table):
    return tuple(table[l] for l in labels)


def _run(api, handle, A, la, B, lb, C, D, ld, alpha, beta, **kw):
    dA, dB, dD = A.to("cuda"), B.to("cuda"), D.to("cuda")
    dC = C.to("cuda") if C is not None else None
    op, status = api.contract(handle, dA, la, dB, lb, dC, dD, ld, alpha, beta, want_status=True,
                              stream=torch.cuda.current_stream().cuda_stream, **kw)
    torch.cuda.synchronize()
    assert op.device_error == 0
    return dD.buffer.cpu(), status, op


@pytest.mark.parametrize("real,cplx", PAIRS)
@pytest.mark.parametrize("which", ["A", "B", "C", "AB", "ABC"])
@pytest.mark.parametrize("shape", list(SHAPES))
def test_real_operands_among_complex_ones(real, cplx, which, shape):
    api = helpers.api()
    handle = api.Handle()
    la, lb, ld, ext = SHAPES[shape]
    tA, tB, tC = (real if x in which else cplx for x in "ABC")
    A = helpers.random_tensor(201, _ext(la, ext), None, tA)
    B = helpers.random_tensor(202, _ext(lb, ext), None, tB)
    C = helpers.random_tensor(203, _ext(ld, ext), None, tC)
    D = inputs.place(None, _ext(ld, ext), None, cplx)
    alpha, beta = complex(0.75, -1.25), complex(-0.5, 0.25)
    got, status, op = _run(api, handle, A, la, B, lb, C, D, ld, alpha, beta, conjA=True, conjB=True, conjC=True)
    assert status["kernel"] == api.KERNEL_GENERIC
    want = D.clone()
    scale = oracle.contract_mixed(A.numpy(), la, B.numpy(), lb, C.numpy(), ld, want.numpy(), ld, alpha, beta,
                                  conjA=True, conjB=True, conjC=True)
    pos = D.offsets()
    assert helpers.compare(got[pos].numpy(), want.buffer[pos].numpy(), scale, cplx) <= 1.0


@pytest.mark.parametrize("dtype", [torch.float32, torch.complex64])
def test_32_bit_storage_with_sums_kept_in_fp64(dtype):
    """BTC_PRECISION_FP64_SUMS: the result is the wide sum rounded once, i.e. within one unit in the last place
    of the oracle's (long double sums) and far inside the 1e-5 bound; the default plan of the same operation
    (three TF32 products, fp32 sums) is visibly further away on a long sum."""
    api = helpers.api()
    handle = api.Handle()
    ext = dict(i=40, j=24, k=4096)
    A = helpers.random_tensor(211, _ext("ki", ext), None, dtype)
    B = helpers.random_tensor(212, _ext("kj", ext), None, dtype)
    D = inputs.place(None, _ext("ij", ext), None, dtype)
    want = D.clone()
    scale = oracle.contract_mixed(A.numpy(), "ki", B.numpy(), "kj", None, "ij", want.numpy(), "ij", 1.0, 0.0)
    pos = D.offsets()
    ref = want.buffer[pos].numpy().astype(np.complex128)
    dt = api.dtype_code(dtype)
    tA, tB, tD = (api.TensorInfo(handle, dt, x.extents, x.strides) for x in (A, B, D))
    op = api.Contraction(handle, tA, "ki", tB, "kj", None, "ij", tD, "ij", 1.0, 0.0)
    dA, dB = A.to("cuda"), B.to("cuda")
    errs = {}
    for precision in (api.PRECISION_FP64_SUMS, api.PRECISION_DEFAULT):
        op.set_attr(api.ATTR_COMPUTE_PRECISION, precision)
        assert (op.kernel == api.KERNEL_GENERIC) == (precision == api.PRECISION_FP64_SUMS)
        dD = D.to("cuda")
        need = op.workspace_size()
        ws = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda")
        op.execute(torch.cuda.current_stream().cuda_stream, dA.data_ptr(), dB.data_ptr(), 0, dD.data_ptr(),
                   workspace=ws.data_ptr(), workspace_bytes=need)
        torch.cuda.synchronize()
        got = dD.buffer.cpu()[pos].numpy().astype(np.complex128)
        errs[precision] = np.abs(got - ref)
        assert helpers.compare(dD.buffer.cpu()[pos].numpy(), want.buffer[pos].numpy(), scale, dtype) <= 1.0
    ulp = 2.0 ** -23 * np.maximum(np.abs(ref), 1e-30)
    assert np.all(errs[api.PRECISION_FP64_SUMS] <= 1.5 * ulp)
    assert errs[api.PRECISION_DEFAULT].max() > 4 * errs[api.PRECISION_FP64_SUMS].max()


def test_unsupported_mixes_are_refused():
    api = helpers.api()
    handle = api.Handle()
    t = lambda dt, ext: api.TensorInfo(handle, dt, ext)
    with pytest.raises(api.BtcError) as ei:      # 32- with 64-bit parts
        api.Contraction(handle, t(api.F32, (4, 5)), "ik", t(api.F64, (5, 3)), "kj", None, "ij", t(api.F64, (4, 3)), "ij")
    assert ei.value.code == api.ERR_NOT_SUPPORTED
    with pytest.raises(api.BtcError) as ei:      # a real result of a complex input
        api.Contraction(handle, t(api.C64, (4, 5)), "ik", t(api.F64, (5, 3)), "kj", None, "ij", t(api.F64, (4, 3)), "ij")
    assert ei.value.code == api.ERR_NOT_SUPPORTED


REAL_VIEW_SHAPES = {
    # large enough for a tiled plan of the real contraction
    "matrix_product": ("ki", "kj", "ij", dict(i=192, j=160, k=96)),
    "batch_and_permuted_output": ("hik", "kjh", "jih", dict(h=3, i=96, j=80, k=64)),
    "isolated_label": ("ikx", "kj", "ij", dict(i=128, j=96, k=48, x=3)),
}


@pytest.mark.parametrize("real,cplx", PAIRS)
@pytest.mark.parametrize("which", ["A", "B"])
@pytest.mark.parametrize("shape", list(REAL_VIEW_SHAPES))
def test_one_real_input_runs_the_tiled_kernels_through_real_views(real, cplx, which, shape):
    """One real and one complex input, real scalars, nothing conjugated: the complex tensors are read as real
    tensors with one more mode and the tiled kernels of the part type run; with a complex alpha the same
    operation object falls back to the per-element kernel.  Both against the mixed-type oracle."""
    api = helpers.api()
    handle = api.Handle()
    la, lb, ld, ext = REAL_VIEW_SHAPES[shape]
    tA, tB = (real if x in which else cplx for x in "AB")
    A = helpers.random_tensor(221, _ext(la, ext), None, tA)
    B = helpers.random_tensor(222, _ext(lb, ext), None, tB)
    C = helpers.random_tensor(223, _ext(ld, ext), None, cplx)
    D = inputs.place(None, _ext(ld, ext), None, cplx)
    pos = D.offsets()
    for alpha, beta, tiled in ((0.75, -0.5, True), (complex(0.75, -1.25), -0.5, False)):
        got, status, op = _run(api, handle, A, la, B, lb, C, D, ld, alpha, beta)
        assert (status["kernel"] == api.KERNEL_TILED) == tiled, status
        want = D.clone()
        scale = oracle.contract_mixed(A.numpy(), la, B.numpy(), lb, C.numpy(), ld, want.numpy(), ld, alpha, beta)
        assert helpers.compare(got[pos].numpy(), want.buffer[pos].numpy(), scale, cplx) <= 1.0
