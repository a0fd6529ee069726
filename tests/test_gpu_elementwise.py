"""GPU parity of the binary / unary operation C := alpha op(A) + beta op(B) against the CPU oracle:
element by element on the same seeded inputs, through the C-ABI.

Acceptance as for the contraction: |c_gpu - c_oracle| <= tol * scale, scale = |alpha| sum|a| +
|beta||b| from the oracle, tol = 1e-12 (64-bit parts) / 1e-5 (32-bit parts); bit-exact where the
operation only moves data (alpha = 1, beta = 0, nothing summed)."""
import numpy as np
import pytest
import torch

import helpers
import oracle
from paper_2601_07827_b200 import inputs

pytestmark = pytest.mark.gpu

REAL_AND_COMPLEX = [torch.float32, torch.float64, torch.complex64, torch.complex128]


@pytest.fixture(scope="module")
def api():
    return helpers.api()


@pytest.fixture(scope="module")
def handle(api):
    return api.Handle()


def _ext(labels, table):
    return tuple(table[l] for l in labels)


def run_elementwise(api, handle, A, la, B, C, lc, alpha=1.0, beta=0.0, conjA=False, conjB=False):
    """A, B, C: inputs.StridedTensor on the CPU (C not modified).  Returns (worst error in tolerance
    units, kernel id, whether GPU and oracle agree bit for bit)."""
    in_place = B is C
    dA = A.to("cuda")
    dC = C.to("cuda")
    dB = dC if in_place else (B.to("cuda") if B is not None else None)
    op = api.elementwise(handle, dA, la, dB, dC, lc, alpha, beta, conjA, conjB,
                         stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    result = dC.buffer.cpu()
    want = C.clone()
    wantB = want if in_place else B
    scale = oracle.elementwise(A.numpy(), la, wantB.numpy() if wantB is not None else None, want.numpy(), lc,
                               alpha, beta, conjA=conjA, conjB=conjB)
    pos = C.offsets()
    got, ref = result[pos].numpy(), want.buffer[pos].numpy()
    worst = helpers.compare(got, ref, scale, C.dtype)
    assert helpers.canary_intact(C.buffer, result, pos), "bytes outside C's elements were modified"
    return worst, op.kernel, bool(np.array_equal(got, ref))


CASES = {
    # name: (labelsA, labelsC, extents, B present)
    "copy": ("ijk", "ijk", dict(i=37, j=29, k=5), False),
    "axpby": ("ij", "ij", dict(i=300, j=70), True),
    "transpose_2d": ("ij", "ji", dict(i=130, j=75), False),
    "permute_4d": ("abcd", "dbac", dict(a=33, b=12, c=40, d=50), True),
    "permute_fast_label_moves_to_the_middle": ("abc", "cab", dict(a=70, b=9, c=65), False),
    "reduce_slow_labels": ("ixjy", "ji", dict(i=40, j=33, x=5, y=6), True),
    "reduce_fast_label": ("xij", "ij", dict(i=50, j=20, x=70), False),
    "reduce_everything": ("ijk", "", dict(i=17, j=9, k=33), False),
    "broadcast": ("i", "xiy", dict(i=45, x=7, y=11), True),
    "broadcast_scalar": ("", "ij", dict(i=40, j=33), False),
    "diagonal": ("ii", "i", dict(i=77), False),
    "semi_diagonal_transposed": ("iji", "ji", dict(i=40, j=36), True),
    "trace": ("kk", "", dict(k=90), False),
    "reduce_and_transpose": ("ixj", "ji", dict(i=64, j=48, x=7), True),
}


@pytest.mark.parametrize("dtype", REAL_AND_COMPLEX)
@pytest.mark.parametrize("name", list(CASES))
def test_elementwise_categories(api, handle, name, dtype):
    la, lc, ext, with_b = CASES[name]
    A = helpers.random_tensor(201, _ext(la, ext), None, dtype)
    B = helpers.random_tensor(202, _ext(lc, ext), None, dtype) if with_b else None
    C = inputs.place(None, _ext(lc, ext), None, dtype)
    cplx = dtype.is_complex
    alpha = complex(0.75, -1.25) if cplx else 0.75
    beta = (complex(-0.5, 0.25) if cplx else -0.5) if with_b else 0.0
    worst, _, _ = run_elementwise(api, handle, A, la, B, C, lc, alpha, beta, conjA=cplx, conjB=cplx)
    assert worst <= 1.0, worst


@pytest.mark.parametrize("dtype", REAL_AND_COMPLEX)
def test_pure_permutation_is_bit_exact_and_uses_the_tiled_kernel(api, handle, dtype):
    ext = dict(a=96, b=40, c=50)
    A = helpers.random_tensor(211, _ext("abc", ext), None, dtype)
    C = inputs.place(None, _ext("cba", ext), None, dtype)
    worst, kernel, exact = run_elementwise(api, handle, A, "abc", None, C, "cba")
    assert worst == 0.0 and exact and kernel == api.EW_KERNEL_TRANSPOSING
    C2 = inputs.place(None, _ext("abc", ext), None, dtype)
    worst, kernel, exact = run_elementwise(api, handle, A, "abc", None, C2, "abc")
    assert exact and kernel == api.EW_KERNEL_DIRECT


@pytest.mark.parametrize("dtype", [torch.float64, torch.complex64])
def test_strides_negative_zero_padded_in_place(api, handle, dtype):
    ext = dict(i=70, j=45, k=6)
    # A: negative stride on i, padded; zero stride on k (a replicated operand)
    A = helpers.random_tensor(221, _ext("ikj", ext), (-1, 0, 75), dtype)
    B = helpers.random_tensor(222, _ext("ji", ext), (2, -95), dtype)
    C = inputs.place(None, _ext("ji", ext), (1, 47), dtype)
    worst, _, _ = run_elementwise(api, handle, A, "ikj", B, C, "ji", 1.5, 0.5)
    assert worst <= 1.0
    # in place: B is C
    X = helpers.random_tensor(223, _ext("ji", ext), (1, 47), dtype)
    worst, _, _ = run_elementwise(api, handle, A, "ikj", X, X, "ji", 2.0, -1.0)
    assert worst <= 1.0


def test_alpha_or_beta_zero_do_not_read_their_operand(api, handle):
    ext = dict(i=40, j=30)
    nanA = inputs.place(None, _ext("ij", ext), None, torch.float64)        # all canary NaNs
    B = helpers.random_tensor(231, _ext("ji", ext), None, torch.float64)
    C = inputs.place(None, _ext("ji", ext), None, torch.float64)
    worst, _, exact = run_elementwise(api, handle, nanA, "ij", B, C, "ji", 0.0, 2.0)
    assert worst <= 1.0 and exact
    A = helpers.random_tensor(232, _ext("ij", ext), None, torch.float64)
    nanB = inputs.place(None, _ext("ji", ext), None, torch.float64)
    worst, _, exact = run_elementwise(api, handle, A, "ij", nanB, C, "ji", 1.0, 0.0)
    assert worst <= 1.0 and exact


def test_error_codes(api, handle):
    def code(fn):
        with pytest.raises(api.BtcError) as ei:
            fn()
        return ei.value.code

    t = lambda e, s=None: api.TensorInfo(handle, api.F64, e, s)
    assert code(lambda: api.Elementwise(handle, t((3, 4)), "ij", None, t((4, 5)), "ji")) == api.ERR_EXTENT_MISMATCH
    assert code(lambda: api.Elementwise(handle, t((3, 4)), "ii", None, t((3,)), "i")) == api.ERR_EXTENT_MISMATCH
    assert code(lambda: api.Elementwise(handle, t((3, 4)), "ij", t((3, 4)), t((4, 3)), "ji", 1.0, 1.0)) == api.ERR_C_D_MISMATCH
    assert code(lambda: api.Elementwise(handle, t((3, 4)), "ij", None, t((4, 3)), "ji", 1.0, 1.0)) == api.ERR_INVALID_ARGUMENT
    assert code(lambda: api.Elementwise(handle, t((3, 4)), "ij", None, t((3, 3)), "ii")) == api.ERR_NOT_SUPPORTED
    assert code(lambda: api.Elementwise(handle, t((3, 4)), "ij", None, t((4, 3), (1, 2)), "ji")) == api.ERR_D_ALIASING
    assert code(lambda: api.Elementwise(handle, t((3, 4)), "ij", None,
                                        api.TensorInfo(handle, api.F32, (4, 3)), "ji")) == api.ERR_NOT_SUPPORTED
