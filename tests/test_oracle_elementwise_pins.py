"""Pins of the CPU oracle for C := alpha * op(A) + beta * op(B) (Sec. "Unary and Binary Operations")
against things fixed outside it: numpy's own permutation / reduction / broadcasting / diagonal
routines, explicit Python loops written from the definition, closed forms and invariants.  A
dropped term, a wrong sign, a transposed index or a missed stride fails at least one of them."""
import itertools

import numpy as np
import pytest

import oracle

DTYPES = [np.float32, np.float64, np.complex64, np.complex128]


def rnd(rng, shape, dtype, order="F"):
    x = rng.uniform(-1, 1, size=shape)
    if np.issubdtype(dtype, np.complexfloating):
        x = x + 1j * rng.uniform(-1, 1, size=shape)
    return np.asarray(x, dtype=dtype, order=order)


def tol(dtype):
    return 1e-5 if np.dtype(dtype) in (np.dtype(np.float32), np.dtype(np.complex64)) else 1e-13


@pytest.mark.parametrize("dtype", DTYPES)
def test_permutation_equals_numpy_transpose(dtype):
    rng = np.random.default_rng(1)
    A = rnd(rng, (3, 4, 5, 2), dtype)
    for perm in itertools.permutations(range(4)):
        labels = "ijkl"
        lc = "".join(labels[p] for p in perm)
        C = np.zeros(tuple(A.shape[p] for p in perm), dtype=dtype, order="F")
        oracle.elementwise(A, labels, None, C, lc, 1.0, 0.0)
        assert np.array_equal(C, np.transpose(A, perm))          # a pure copy is exact


@pytest.mark.parametrize("dtype", DTYPES)
def test_axpby_with_two_layouts(dtype):
    rng = np.random.default_rng(2)
    A = rnd(rng, (6, 5), dtype, order="C")                       # row-major A
    B = rnd(rng, (5, 6), dtype, order="F")
    C = np.zeros((5, 6), dtype=dtype, order="F")
    alpha, beta = (0.75, -1.5)
    oracle.elementwise(A, "ij", B, C, "ji", alpha, beta)
    want = alpha * A.T.astype(np.complex128) + beta * B.astype(np.complex128)
    assert np.max(np.abs(C - want)) <= tol(dtype) * 4


@pytest.mark.parametrize("dtype", DTYPES)
def test_reduction_over_labels_only_in_A_equals_numpy_sum(dtype):
    rng = np.random.default_rng(3)
    A = rnd(rng, (4, 3, 5, 6), dtype)                            # i x j y
    C = np.zeros((5, 4), dtype=dtype, order="F")                 # j i
    oracle.elementwise(A, "ixjy", None, C, "ji", 2.0, 0.0)
    want = 2.0 * np.einsum("ixjy->ji", A.astype(np.complex128))
    assert np.max(np.abs(C - want)) <= tol(dtype) * 40
    # all labels of A summed: rank-0 result
    c0 = np.zeros((), dtype=dtype)
    oracle.elementwise(A, "ixjy", None, c0, "", 1.0, 0.0)
    assert abs(c0 - A.astype(np.complex128).sum()) <= tol(dtype) * 400


@pytest.mark.parametrize("dtype", DTYPES)
def test_broadcast_along_labels_only_in_C(dtype):
    rng = np.random.default_rng(4)
    A = rnd(rng, (4,), dtype)
    B = rnd(rng, (3, 4, 2), dtype)
    C = np.zeros((3, 4, 2), dtype=dtype, order="F")
    oracle.elementwise(A, "i", B, C, "xiy", 1.0, 1.0)
    want = np.broadcast_to(A[None, :, None], (3, 4, 2)) + B
    assert np.max(np.abs(C - want)) <= tol(dtype) * 4
    # rank-0 A broadcast everywhere
    a0 = np.asarray(rnd(rng, (), dtype))
    oracle.elementwise(a0, "", None, C, "xiy", 3.0, 0.0)
    assert np.max(np.abs(C - 3.0 * a0)) <= tol(dtype) * 4


@pytest.mark.parametrize("dtype", DTYPES)
def test_repeated_labels_in_A_address_the_diagonal(dtype):
    rng = np.random.default_rng(5)
    A = rnd(rng, (5, 5), dtype)
    d = np.zeros((5,), dtype=dtype)
    oracle.elementwise(A, "ii", None, d, "i", 1.0, 0.0)
    assert np.array_equal(d, np.diagonal(A))
    t = np.zeros((), dtype=dtype)
    oracle.elementwise(A, "kk", None, t, "", 1.0, 0.0)           # isolated and repeated: the trace
    assert abs(t - np.trace(A.astype(np.complex128))) <= tol(dtype) * 10
    A3 = rnd(rng, (4, 3, 4), dtype)
    C = np.zeros((3, 4), dtype=dtype, order="F")
    oracle.elementwise(A3, "iji", None, C, "ji", 1.0, 0.0)       # semi-diagonal
    assert np.array_equal(C, np.einsum("iji->ji", A3))


def test_explicit_loops_from_the_definition():
    """C[c, a, z] = alpha * sum_{x, y} conj(A[a, x, c, y, x]) + beta * conj(B[c, a, z]) written as
    plain loops (x repeated and isolated, y isolated, z broadcast)."""
    rng = np.random.default_rng(6)
    ea, ex, ec, ey, ez = 3, 2, 4, 3, 2
    A = rnd(rng, (ea, ex, ec, ey, ex), np.complex128)
    B = rnd(rng, (ec, ea, ez), np.complex128)
    C = np.zeros((ec, ea, ez), dtype=np.complex128, order="F")
    alpha, beta = complex(0.5, -2.0), complex(-1.0, 0.25)
    oracle.elementwise(A, "axcyx", B, C, "caz", alpha, beta, conjA=True, conjB=True)
    want = np.zeros_like(C)
    for c in range(ec):
        for a in range(ea):
            for z in range(ez):
                s = 0
                for x in range(ex):
                    for y in range(ey):
                        s += np.conj(A[a, x, c, y, x])
                want[c, a, z] = alpha * s + beta * np.conj(B[c, a, z])
    assert np.max(np.abs(C - want)) <= 1e-13


def test_small_integers_are_exact():
    rng = np.random.default_rng(7)
    for dtype in (np.float32, np.float64):
        A = np.asfortranarray(rng.integers(-8, 9, size=(5, 4, 3)).astype(dtype))
        B = np.asfortranarray(rng.integers(-8, 9, size=(3, 5)).astype(dtype))
        C = np.zeros((3, 5), dtype=dtype, order="F")
        oracle.elementwise(A, "ijk", B, C, "ki", 3.0, -2.0)
        assert np.array_equal(C, 3.0 * A.sum(1).T - 2.0 * B)


def test_strides_negative_zero_padded_and_in_place():
    rng = np.random.default_rng(8)
    base = rnd(rng, (8, 7), np.float64)
    A = base[::-1, ::2]                                           # negative and stride-2 view
    buf = np.full((10, 6), np.nan, order="F")
    C = buf[1:9, 1:5]                                             # padded C inside a canary frame
    oracle.elementwise(A, "ij", None, C, "ij", 1.0, 0.0)
    assert np.array_equal(C, A)
    assert np.isnan(buf[0]).all() and np.isnan(buf[9]).all() and np.isnan(buf[:, 0]).all() and np.isnan(buf[:, 5]).all()
    # zero stride in A = replication
    row = rnd(rng, (4,), np.float64)
    Az = np.lib.stride_tricks.as_strided(row, shape=(8, 4), strides=(0, 8))
    oracle.elementwise(Az, "ij", None, C, "ij", 1.0, 0.0)
    assert np.array_equal(C, np.broadcast_to(row, (8, 4)))
    # in place: B is C
    X = rnd(rng, (8, 4), np.float64)
    X0 = X.copy()
    oracle.elementwise(A, "ij", X, X, "ij", 2.0, 0.5)
    assert np.allclose(X, 2.0 * A + 0.5 * X0, rtol=0, atol=1e-14)


def test_identities_and_scale():
    rng = np.random.default_rng(9)
    A = rnd(rng, (4, 5), np.float64)
    B = rnd(rng, (5, 4), np.float64)
    C = np.zeros((5, 4), order="F")
    # beta == 0: B is never read (NaNs in it do not propagate); alpha == 0: A is never read
    oracle.elementwise(A, "ij", np.full((5, 4), np.nan, order="F"), C, "ji", 1.0, 0.0)
    assert np.array_equal(C, A.T)
    oracle.elementwise(np.full((4, 5), np.nan, order="F"), "ij", B, C, "ji", 0.0, 2.0)
    assert np.array_equal(C, 2.0 * B)
    # linearity in alpha, beta
    C1, C2 = np.zeros((5, 4), order="F"), np.zeros((5, 4), order="F")
    oracle.elementwise(A, "ij", B, C1, "ji", 1.5, -0.5)
    oracle.elementwise(A, "ij", None, C2, "ji", 1.5, 0.0)
    assert np.allclose(C1, C2 - 0.5 * B, rtol=0, atol=1e-15)
    # scale = |alpha| sum |a| + |beta| |b|
    A3 = rnd(rng, (4, 3, 5), np.complex128)
    B3 = rnd(rng, (5, 4), np.complex128)
    C3 = np.zeros((5, 4), dtype=np.complex128, order="F")
    scale = oracle.elementwise(A3, "ixj", B3, C3, "ji", complex(0, 2), complex(3, 4))
    want = 2.0 * np.abs(A3).sum(1).T + 5.0 * np.abs(B3)
    assert np.allclose(scale.reshape((5, 4), order="F"), want, rtol=1e-12)
    # sampled mode returns the same values and leaves C alone
    keep = C3.copy()
    idx = [0, 7, 19, 3]
    vals, sc = oracle.elementwise(A3, "ixj", B3, C3, "ji", complex(0, 2), complex(3, 4), want=idx)
    assert np.array_equal(C3, keep)
    assert np.array_equal(vals, C3.reshape(-1, order="F")[idx]) and np.allclose(sc, scale[idx])
    # relabelling changes nothing
    C4 = np.zeros_like(C3)
    oracle.elementwise(A3, "pqr", B3, C4, "rp", complex(0, 2), complex(3, 4))
    assert np.array_equal(C4, C3)


def test_error_codes():
    A = np.zeros((3, 4), order="F")
    C = np.zeros((4, 3), order="F")

    def code(fn):
        with pytest.raises(oracle.OracleError) as ei:
            fn()
        return ei.value.code

    assert code(lambda: oracle.elementwise(A, "ij", None, np.zeros((4, 5), order="F"), "ji")) == oracle.ERR_EXTENT_MISMATCH
    assert code(lambda: oracle.elementwise(np.zeros((3, 4)), "ii", None, C, "ji")) == oracle.ERR_EXTENT_MISMATCH
    assert code(lambda: oracle.elementwise(A, "ij", np.zeros((3, 4), order="F"), C, "ji", 1.0, 1.0)) == oracle.ERR_B_C_MISMATCH
    assert code(lambda: oracle.elementwise(A, "ij", None, C, "ji", 1.0, 1.0)) == oracle.ERR_B_C_MISMATCH
    assert code(lambda: oracle.elementwise(A, "ij", None, np.zeros((3, 3), order="F"), "ii")) == oracle.ERR_NOT_SUPPORTED
    assert code(lambda: oracle.elementwise(A, "ij", None, C, "ji", layouts={"C": ((4, 3), (1, 2))})) == oracle.ERR_C_ALIASING
    assert code(lambda: oracle.elementwise(A, "ij", None, C, "ji", layouts={"C": ((4, 3), (0, 1))})) == oracle.ERR_C_ALIASING
    assert code(lambda: oracle.elementwise(A, "ij", None, C, "ji", layouts={"A": ((3, 0), (1, 3))})) == oracle.ERR_INVALID_EXTENT
