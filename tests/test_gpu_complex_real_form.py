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


@pytest.mark.parametrize("name", list(CASES))
def test_complex64_real_form(api, handle, name):
    la, lb, ld, ext, conjA, conjB, alpha, beta, real_form = CASES[name]
    dtype = torch.complex64
    A = helpers.random_tensor(11, _ext(la, ext), None, dtype)
    B = helpers.random_tensor(12, _ext(lb, ext), None, dtype)
    D = helpers.random_tensor(13, _ext(ld, ext), None, dtype)
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
