"""Pointer-array batched execution (btc_execute_batched): every entry must equal the single execute of
the same operation on that entry's buffers bit for bit (same plan, same summation order), and entry 0
and the last entry are checked against the CPU oracle."""
import numpy as np
import pytest
import torch

import helpers
import oracle
from paper_2601_07827_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def api():
    return helpers.api()


@pytest.fixture(scope="module")
def handle(api):
    return api.Handle()


def _ext(labels, table):
    return tuple(table[l] for l in labels)


CASES = {
    # name: (dtype, labelsA, labelsB, labelsD, extents, beta, count)
    "f64_split_k": (torch.float64, "acid", "dbcj", "abij", dict(a=8, b=8, c=8, d=8, i=8, j=8), 0.5, 5),
    "f32_network": (torch.float32, "axbycwde", "wfygxhij", "afbgchdiej", {l: 2 for l in "abcdefghijxyw"} | dict(a=4, f=4, x=4), 0.0, 7),
    "f32_own_batch_label": (torch.float32, "hik", "hkj", "ijh", dict(h=3, i=70, j=50, k=40), 0.0, 4),
    "c128_conj": (torch.complex128, "spt", "tqsr", "pqr", dict(p=40, q=24, r=3, s=12, t=8), 0.0, 3),
    "c64_in_place": (torch.complex64, "ik", "kj", "ij", dict(i=150, j=70, k=33), 1.0, 3),
    "f32_tcgen05_persistent": (torch.float32, "ki", "kj", "ij", dict(i=300, j=200, k=96), 0.0, 3, 21),
    "generic_kernel_loop": (torch.float64, "i", "j", "ij", dict(i=5, j=3), 0.0, 4),
    "case4_loop": (torch.float64, "ikx", "kj", "ij", dict(i=40, j=30, k=20, x=3), 0.0, 3),
}


@pytest.mark.parametrize("name", list(CASES))
def test_batched_equals_single_executes(api, handle, name):
    dtype, la, lb, ld, ext, beta, count = CASES[name][:7]
    variant = CASES[name][7] if len(CASES[name]) > 7 else -1
    cplx = dtype.is_complex
    alpha = complex(0.75, -0.5) if cplx else 0.75
    As = [helpers.random_tensor(100 + 3 * i, _ext(la, ext), None, dtype) for i in range(count)]
    Bs = [helpers.random_tensor(101 + 3 * i, _ext(lb, ext), None, dtype) for i in range(count)]
    Cs = [helpers.random_tensor(102 + 3 * i, _ext(ld, ext), None, dtype) for i in range(count)]
    in_place = name.endswith("in_place")
    dt = api.dtype_code(dtype)
    tA = api.TensorInfo(handle, dt, As[0].extents, As[0].strides)
    tB = api.TensorInfo(handle, dt, Bs[0].extents, Bs[0].strides)
    tD = api.TensorInfo(handle, dt, Cs[0].extents, Cs[0].strides)
    op = api.Contraction(handle, tA, la, tB, lb, tD if beta else None, ld, tD, ld, alpha, beta, conjA=cplx)
    if variant >= 0:      # a bulk-copy variant of the tcgen05 kernel: the batched call must run its gathering twin
        op.set_attr(api.ATTR_KERNEL, api.KERNEL_TILED)
        op.set_attr(api.ATTR_VARIANT, variant)
    # entries carved out of one pool per tensor, so that C[i] - C[0] == D[i] - D[0]
    n = Cs[0].buffer.numel()
    poolC = torch.stack([c.buffer for c in Cs]).cuda()
    poolD1 = poolC.clone() if in_place else torch.full_like(poolC, float("nan"))
    poolD2 = poolD1.clone()
    dA = [a.to("cuda") for a in As]
    dB = [b.to("cuda") for b in Bs]
    esz = Cs[0].buffer.element_size()
    ptrs = lambda pool: [pool.data_ptr() + i * n * esz for i in range(count)]
    pC1 = ptrs(poolD1) if in_place else ptrs(poolC)
    pC2 = ptrs(poolD2) if in_place else ptrs(poolC)
    stream = torch.cuda.current_stream().cuda_stream
    ws_bytes = op.workspace_size()
    ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device="cuda")
    for i in range(count):
        op.execute(stream, dA[i].data_ptr(), dB[i].data_ptr(), pC1[i] if beta else 0, ptrs(poolD1)[i],
                   workspace=ws.data_ptr(), workspace_bytes=ws_bytes)
    bws_bytes = op.batched_workspace_size(count)
    bws = torch.empty(max(bws_bytes, 256), dtype=torch.uint8, device="cuda")
    op.execute_batched(stream, [a.data_ptr() for a in dA], [b.data_ptr() for b in dB], pC2 if beta else None,
                       ptrs(poolD2), workspace=bws.data_ptr(), workspace_bytes=bws_bytes)
    torch.cuda.synchronize()
    assert torch.equal(poolD1.view(torch.uint8), poolD2.view(torch.uint8))
    got = poolD2.cpu()
    for i in (0, count - 1):
        want = Cs[i].clone()
        scale = oracle.contract(As[i].numpy(), la, Bs[i].numpy(), lb, want.numpy() if beta else None, ld, want.numpy(), ld,
                                alpha, beta, conjA=cplx)
        pos = Cs[i].offsets()
        assert helpers.compare(got[i][pos].numpy(), want.buffer[pos].numpy(), scale, dtype) <= 1.0


def test_batch_hint_drops_split_k(api, handle):
    """A small problem is split along K to fill the GPU when it runs alone; told that it will run over a long
    pointer array the planner keeps K whole (no partial sums in the workspace), and the batched result still
    matches the oracle."""
    dtype, la, lb, ld = torch.float64, "acid", "dbcj", "abij"
    ext = dict(a=8, b=8, c=8, d=8, i=8, j=8)
    count = 6
    As = [helpers.random_tensor(300 + 2 * i, _ext(la, ext), None, dtype) for i in range(count)]
    Bs = [helpers.random_tensor(301 + 2 * i, _ext(lb, ext), None, dtype) for i in range(count)]
    D0 = inputs.place(None, _ext(ld, ext), None, dtype)
    dt = api.dtype_code(dtype)
    tA, tB, tD = (api.TensorInfo(handle, dt, x.extents, x.strides) for x in (As[0], Bs[0], D0))
    op = api.Contraction(handle, tA, la, tB, lb, None, ld, tD, ld, 1.0, 0.0)
    assert op.split_k > 1
    alone = op.batched_workspace_size(count)
    op.set_attr(api.ATTR_BATCH_HINT, 512)
    assert op.split_k == 1 and op.batched_workspace_size(count) < alone
    dA, dB = [a.to("cuda") for a in As], [b.to("cuda") for b in Bs]
    pool = torch.full((count, D0.buffer.numel()), float("nan"), dtype=dtype, device="cuda")
    need = op.batched_workspace_size(count)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda")
    op.execute_batched(torch.cuda.current_stream().cuda_stream, [a.data_ptr() for a in dA], [b.data_ptr() for b in dB], None,
                       [pool.data_ptr() + i * D0.buffer.numel() * 8 for i in range(count)], workspace=ws.data_ptr(),
                       workspace_bytes=need)
    torch.cuda.synchronize()
    got = pool.cpu()
    for i in range(count):
        want = D0.clone()
        scale = oracle.contract(As[i].numpy(), la, Bs[i].numpy(), lb, None, ld, want.numpy(), ld, 1.0, 0.0)
        pos = D0.offsets()
        assert helpers.compare(got[i][pos].numpy(), want.buffer[pos].numpy(), scale, dtype) <= 1.0


def test_batched_argument_errors(api, handle):
    ext = dict(i=64, j=64, k=64)
    A = helpers.random_tensor(1, _ext("ik", ext), None, torch.float32).to("cuda")
    B = helpers.random_tensor(2, _ext("kj", ext), None, torch.float32).to("cuda")
    D = inputs.place(None, _ext("ij", ext), None, torch.float32).to("cuda")
    dt = api.dtype_code(torch.float32)
    tA, tB, tD = (api.TensorInfo(handle, dt, x.extents, x.strides) for x in (A, B, D))
    op = api.Contraction(handle, tA, "ik", tB, "kj", None, "ij", tD, "ij", 1.0, 0.0)
    need = op.batched_workspace_size(2)
    assert need >= 3 * 2 * 8
    with pytest.raises(api.BtcError) as e:
        op.execute_batched(0, [A.data_ptr()] * 2, [B.data_ptr()] * 2, None, [D.data_ptr()] * 2, workspace=0, workspace_bytes=0)
    assert e.value.code == api.ERR_WORKSPACE_TOO_SMALL
    ws = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(api.BtcError) as e:
        op.execute_batched(0, [A.data_ptr(), 0], [B.data_ptr()] * 2, None, [D.data_ptr()] * 2, workspace=ws.data_ptr(),
                           workspace_bytes=need)
    assert e.value.code == api.ERR_INVALID_ARGUMENT
