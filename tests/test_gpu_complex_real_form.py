"""complex64 contractions large enough to run in their real form on the fp32 tensor-core kernels (the
smaller input expanded to 2 x 2 real blocks, the other tensors read as float tensors with one more
mode): conjugations, complex alpha, real beta with C, either input as the expanded one, a batch label,
and the cases that must stay on the complex kernels.  Oracle at sampled elements."""
import numpy as np
import pytest
import torch

import helpers
import oracle

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
    # name: (labelsA, labelsB, labelsD, extents, conjA, conjB, alpha, beta, expect real form)
    "a_small_conj_a": ("ki", "kj", "ij", dict(i=256, j=4096, k=320), True, False, 0.5 - 0.25j, 0.0, True),
    "b_small_conj_b": ("ik", "jk", "ij", dict(i=4096, j=256, k=320), False, True, 1.0 + 0.0j, 0.0, True),
    "both_conj_real_beta": ("ki", "jk", "ji", dict(i=512, j=2048, k=256), True, True, -1.5 + 2.0j, 0.75, True),
    "batch_label": ("hki", "hkj", "ijh", dict(h=3, i=256, j=2048, k=192), False, False, 1.0 + 1.0j, 0.0, True),
    "complex_beta_stays_complex": ("ki", "kj", "ij", dict(i=256, j=4096, k=320), False, False, 1.0 + 0.0j, 0.5 + 0.5j, False),
}


# strides (elements) per tensor for the cases that are not dense column-major: padding, a reversed mode
STRIDES = {
    "padded_and_reversed": ((-1, 330), (1, 336), (264, -1)),
}
CASES["padded_and_reversed"] = ("ki", "kj", "ji", dict(i=256, j=2048, k=320), True, False, 0.5 + 0.5j, -0.25, True)


@pytest.mark.parametrize("name", list(CASES))
def test_complex64_real_form(api, handle, name):
    la, lb, ld, ext, conjA, conjB, alpha, beta, real_form = CASES[name]
    dtype = torch.complex64
    sA, sB, sD = STRIDES.get(name, (None, None, None))
    A = helpers.random_tensor(11, _ext(la, ext), sA, dtype)
    B = helpers.random_tensor(12, _ext(lb, ext), sB, dtype)
    D = helpers.random_tensor(13, _ext(ld, ext), sD, dtype)
    use_c = beta != 0.0
    dA, dB, dD = A.to("cuda"), B.to("cuda"), D.to("cuda")
    op, status = api.contract(handle, dA, la, dB, lb, dD if use_c else None, dD, ld, alpha, beta, conjA, conjB, False,
                              stream=torch.cuda.current_stream().cuda_stream, want_status=True)
    torch.cuda.synchronize()
    assert op.device_error == 0
    assert (10 <= status["variant"] <= 21) == real_form, status
    total = D.numel()
    rng = np.random.default_rng(5)
    want = np.unique(np.concatenate([rng.integers(0, total, size=3000), np.arange(2048)]))
    d_stub = np.zeros(1, dtype=np.complex64)
    hC = D if use_c else None
    vals, scale = oracle.contract(A.numpy(), la, B.numpy(), lb, hC.numpy() if hC is not None else None, ld, d_stub, ld,
                                  alpha, beta, conjA=conjA, conjB=conjB, conjC=False, want=want,
                                  layouts={"D": (D.extents, D.strides)})
    pos = np.full(want.shape, D.origin, dtype=np.int64)
    rem = want.copy()
    for e, s in zip(D.extents, D.strides):
        pos += (rem % e) * s
        rem //= e
    got = dD.buffer.cpu()[torch.from_numpy(pos)].numpy()
    assert helpers.compare(got, vals, scale, dtype) <= 1.0
    assert helpers.canary_intact(D.buffer, dD.buffer.cpu(), D.offsets()), "bytes outside D's elements were modified"


def test_without_room_in_the_workspace_the_complex_kernels_run(api, handle):
    la, lb, ld, ext = "ki", "kj", "ij", dict(i=2048, j=4096, k=192)     # many tiles: the complex plan itself needs no scratch
    dtype = torch.complex64
    A = helpers.random_tensor(21, _ext(la, ext), None, dtype).to("cuda")
    B = helpers.random_tensor(22, _ext(lb, ext), None, dtype).to("cuda")
    D1 = helpers.random_tensor(23, _ext(ld, ext), None, dtype).to("cuda")
    D2 = helpers.random_tensor(23, _ext(ld, ext), None, dtype).to("cuda")
    dt = api.dtype_code(dtype)
    info = lambda t: api.TensorInfo(handle, dt, t.extents, t.strides)
    op = api.Contraction(handle, info(A), la, info(B), lb, None, ld, info(D1), ld, 1.0, 0.0)
    need = op.workspace_size()
    assert need > 0 and 10 <= op.variant <= 21          # planned in its real form
    stream = torch.cuda.current_stream().cuda_stream
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    st1 = op.execute(stream, A.data_ptr(), B.data_ptr(), 0, D1.data_ptr(), workspace=ws.data_ptr(), workspace_bytes=need, want_status=True)
    st2 = op.execute(stream, A.data_ptr(), B.data_ptr(), 0, D2.data_ptr(), want_status=True)       # no workspace at all
    torch.cuda.synchronize()
    assert op.device_error == 0
    assert 10 <= st1["variant"] <= 21 and not (10 <= st2["variant"] <= 21), (st1, st2)
    # two different summation schemes of the same contraction: equal within the tolerance's scale
    a, b = D1.buffer[D1.offsets()], D2.buffer[D2.offsets()]
    scale = float(ext["k"]) * 1.0
    assert float((a - b).abs().max()) <= 2e-5 * scale
