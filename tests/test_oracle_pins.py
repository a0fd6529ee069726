"""Pins for the CPU oracle: it is checked against things other than itself.

The paper prints no numeric worked example, so the pins are: loops written out by hand in this
file for the paper's index-form examples (Cases 1-4), the matrix-product special case against an
independent triple loop and numpy's matmul, closed forms, identities, invariances, conjugation
properties, exactly representable integer inputs (bit-exact), brute force on tiny tensors, and the
error cases of the paper's test list (items 26-28).
"""
import itertools

import numpy as np
import pytest

import oracle

DTYPES = [np.float32, np.float64, np.complex64, np.complex128]
RTOL = {np.float32: 1e-5, np.float64: 1e-12, np.complex64: 1e-5, np.complex128: 1e-12}


def rnd(rng, shape, dtype, order="F"):
    x = rng.uniform(-1, 1, size=shape)
    if np.issubdtype(dtype, np.complexfloating):
        x = x + 1j * rng.uniform(-1, 1, size=shape)
    return np.asarray(x, dtype=dtype, order=order)


def ints(rng, shape, dtype, order="F"):
    x = rng.integers(-8, 9, size=shape).astype(np.float64)
    if np.issubdtype(dtype, np.complexfloating):
        x = x + 1j * rng.integers(-8, 9, size=shape)
    return np.asarray(x, dtype=dtype, order=order)


def run(A, la, B, lb, C, ld, alpha=1.0, beta=0.0, D=None, **kw):
    """Oracle call returning (D, scale); D is a fresh column-major array unless given."""
    ext = {}
    for t, l in ((A, la), (B, lb)):
        for e, ch in zip(t.shape, l):
            ext[ch] = e
    if D is None:
        D = np.full([ext[ch] for ch in ld], np.nan, dtype=A.dtype, order="F")
    scale = oracle.contract(A, la, B, lb, C, ld, D, ld, alpha, beta, **kw)
    return D, scale


def close(got, want, scale, dtype, factor=4.0):
    """|got - want| <= factor * tol * scale element-wise (scale flat, column-major)."""
    err = np.abs(np.asarray(got, dtype=np.complex128) - np.asarray(want, dtype=np.complex128))
    bound = factor * RTOL[dtype] * scale.reshape(got.shape, order="F") + 1e-300
    return bool(np.all(err <= bound))


# ---------------------------------------------------------------- matrix product (Case 1)
@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("order", ["F", "C"])
def test_matrix_product_equals_triple_loop_and_matmul(dtype, order):
    rng = np.random.default_rng(1)
    m, n, k = 5, 4, 7
    A, B, C = rnd(rng, (m, k), dtype, order), rnd(rng, (k, n), dtype, order), rnd(rng, (m, n), dtype, order)
    alpha, beta = dtype(1.5), dtype(-0.25)
    D = np.full((m, n), np.nan, dtype=dtype, order=order)
    D, scale = run(A, "ik", B, "kj", C, "ij", alpha, beta, D=D)
    want = np.zeros((m, n), dtype=np.complex128)
    for i in range(m):          # the well-known triple loop
        for j in range(n):
            s = 0.0
            for kk in range(k):
                s += complex(A[i, kk]) * complex(B[kk, j])
            want[i, j] = complex(alpha) * s + complex(beta) * complex(C[i, j])
    assert close(D, want, scale, dtype)
    lib = alpha * (A.astype(np.complex128) @ B.astype(np.complex128)) + beta * C
    assert close(D, lib, scale, dtype)


def test_transposed_operand_is_not_confused():
    # A[k,i] given: a transposed-operand mistake would produce A^T-less result
    rng = np.random.default_rng(2)
    A, B = rnd(rng, (6, 3), np.float64), rnd(rng, (6, 4), np.float64)
    D, scale = run(A, "ki", B, "kj", None, "ij")
    assert close(D, A.T @ B, scale, np.float64)
    D2, scale2 = run(A, "ki", B, "kj", None, "ji")
    assert close(D2, B.T @ A, scale2, np.float64)


# ---------------------------------------------------------------- the paper's index-form examples
def test_case1_example_written_out():
    # D[delta,gamma] = alpha sum_{k,l} A[k,l,j] B[l,i,k] + beta C[i,j]   (Case 1 example)
    rng = np.random.default_rng(3)
    ea, eb, eg, ed = 3, 2, 4, 3
    A, B, C = rnd(rng, (ea, eb, eg), np.float64), rnd(rng, (eb, ed, ea), np.float64), rnd(rng, (ed, eg), np.float64)
    D, scale = run(A, "abg", B, "bda", C, "dg", 2.0, -1.5)
    want = np.zeros((ed, eg))
    for i in range(ed):
        for j in range(eg):
            s = 0.0
            for k in range(ea):
                for l in range(eb):
                    s += A[k, l, j] * B[l, i, k]
            want[i, j] = 2.0 * s - 1.5 * C[i, j]
    assert close(D, want, scale, np.float64)


def test_case2_example_written_out():
    # D[delta,alpha] = alpha sum_k A[i,k] B[k,j,i] + beta C[j,i]          (Case 2 example)
    rng = np.random.default_rng(4)
    ea, eb, ed = 3, 4, 2
    A, B, C = rnd(rng, (ea, eb), np.complex128), rnd(rng, (eb, ed, ea), np.complex128), rnd(rng, (ed, ea), np.complex128)
    al, be = 0.5 + 1j, -0.25j
    D, scale = run(A, "ab", B, "bda", C, "da", al, be)
    want = np.zeros((ed, ea), dtype=np.complex128)
    for i in range(ea):
        for j in range(ed):
            s = 0.0
            for k in range(eb):
                s += A[i, k] * B[k, j, i]
            want[j, i] = al * s + be * C[j, i]
    assert close(D, want, scale, np.complex128)


def test_case3_example_written_out():
    # D[delta,alpha] = alpha sum_k A[k,i,k] B[k,j,i] + beta C[j,i]        (Case 3 example)
    rng = np.random.default_rng(5)
    ea, eb, ed = 3, 4, 2
    A, B, C = rnd(rng, (eb, ea, eb), np.float64), rnd(rng, (eb, ed, ea), np.float64), rnd(rng, (ed, ea), np.float64)
    D, scale = run(A, "bab", B, "bda", C, "da", 1.25, 0.75)
    want = np.zeros((ed, ea))
    for i in range(ea):
        for j in range(ed):
            s = 0.0
            for k in range(eb):
                s += A[k, i, k] * B[k, j, i]
            want[j, i] = 1.25 * s + 0.75 * C[j, i]
    assert close(D, want, scale, np.float64)


def test_case4_example_written_out():
    # D[delta,alpha] = alpha sum_k A[k,i,k] (sum_l B[k,l,j,l,i]) + beta C[j,i]   (Case 4 example)
    rng = np.random.default_rng(6)
    ea, eb, eg, ed = 3, 2, 3, 2
    A = rnd(rng, (eb, ea, eb), np.float64)
    B = rnd(rng, (eb, eg, ed, eg, ea), np.float64)
    C = rnd(rng, (ed, ea), np.float64)
    D, scale = run(A, "bab", B, "bgdga", C, "da", -2.0, 1.0)
    want = np.zeros((ed, ea))
    for i in range(ea):
        for j in range(ed):
            s = 0.0
            for k in range(eb):
                inner = 0.0
                for l in range(eg):
                    inner += B[k, l, j, l, i]
                s += A[k, i, k] * inner
            want[j, i] = -2.0 * s + C[j, i]
    assert close(D, want, scale, np.float64)


def test_case4_equals_prereduced_case2():
    rng = np.random.default_rng(7)
    A = rnd(rng, (3, 4, 5), np.float64)      # labels i k x  (x isolated in A)
    B = rnd(rng, (4, 2, 3), np.float64)      # labels k y j  (y isolated in B)
    D, scale = run(A, "ikx", B, "kyj", None, "ij")
    Ar = np.asfortranarray(A.sum(axis=2))
    Br = np.asfortranarray(B.sum(axis=1))
    D2, _ = run(Ar, "ik", Br, "kj", None, "ij")
    assert close(D, D2, scale, np.float64)


# ---------------------------------------------------------------- exact arithmetic and brute force
@pytest.mark.parametrize("dtype", DTYPES)
def test_small_integers_are_bit_exact(dtype):
    rng = np.random.default_rng(8)
    A, B, C = ints(rng, (4, 5, 3), dtype), ints(rng, (5, 3, 6), dtype), ints(rng, (6, 4), dtype)
    D, _ = run(A, "ikl", B, "klj", C, "ji", dtype(2), dtype(-3))
    want = 2 * np.einsum("ikl,klj->ji", A.astype(np.complex128), B.astype(np.complex128)) - 3 * C
    assert np.array_equal(D.astype(np.complex128), want)
    Dn, _ = run(A, "ikl", B, "klj", C, "ji", dtype(2), dtype(-3), native_acc=True)
    assert np.array_equal(Dn, D)


def test_brute_force_all_small_label_patterns():
    """Every way of assigning labels from {a,b,c} to a rank-2 A, rank-2 B and rank<=2 D (that the
    definition allows) against sums written over all label values in Python."""
    rng = np.random.default_rng(9)
    ext = {"a": 2, "b": 3, "c": 2}
    count = 0
    for la in itertools.product("abc", repeat=2):
        for lb in itertools.product("abc", repeat=2):
            for rd in (0, 1, 2):
                for ld in itertools.permutations("abc", rd):
                    if not set(ld) <= set(la) | set(lb):
                        continue
                    A = ints(rng, [ext[x] for x in la], np.float64)
                    B = ints(rng, [ext[x] for x in lb], np.float64)
                    D = np.full([ext[x] for x in ld], np.nan, order="F")
                    oracle.contract(A, la, B, lb, None, ld, D, ld, 1.0, 0.0)
                    labels = sorted(set(la) | set(lb))
                    want = np.zeros([ext[x] for x in ld])
                    for vals in itertools.product(*[range(ext[x]) for x in labels]):
                        v = dict(zip(labels, vals))
                        want[tuple(v[x] for x in ld)] += (A[tuple(v[x] for x in la)] *
                                                         B[tuple(v[x] for x in lb)])
                    assert np.array_equal(D, want), (la, lb, ld)
                    count += 1
    assert count > 300


# ---------------------------------------------------------------- closed forms
@pytest.mark.parametrize("dtype", DTYPES)
def test_all_ones(dtype):
    A, B, C = np.ones((3, 4, 5), dtype, order="F"), np.ones((5, 4, 2), dtype, order="F"), np.ones((2, 3), dtype, order="F")
    D, _ = run(A, "ikl", B, "lkj", C, "ji", dtype(2), dtype(7))
    assert np.all(D == 2 * 20 + 7)


def test_rank_one_separable():
    rng = np.random.default_rng(10)
    u, v, v2, w = (rng.uniform(-1, 1, n) for n in (4, 6, 6, 5))
    A = np.asfortranarray(np.outer(u, v))
    B = np.asfortranarray(np.outer(v2, w))
    D, scale = run(A, "ik", B, "kj", None, "ij", 3.0)
    assert close(D, 3.0 * (v @ v2) * np.outer(u, w), scale, np.float64)


@pytest.mark.parametrize("dtype", DTYPES)
def test_outer_product_full_contraction_hadamard(dtype):
    rng = np.random.default_rng(11)
    a, b = rnd(rng, (3, 2), dtype), rnd(rng, (4,), dtype)
    D, scale = run(a, "ij", b, "k", None, "kij", dtype(2))                 # no contracted label
    want = 2 * np.einsum("ij,k->kij", a.astype(np.complex128), b.astype(np.complex128))
    assert close(D, want, scale, dtype)
    x, y = rnd(rng, (3, 4), dtype), rnd(rng, (4, 3), dtype)
    D0, s0 = run(x, "ij", y, "ji", None, "")                               # everything contracted
    assert D0.shape == () and close(D0, np.sum(x.astype(np.complex128) * y.T), s0, dtype)
    h1, h2 = rnd(rng, (3, 4), dtype), rnd(rng, (3, 4), dtype)
    Dh, sh = run(h1, "ij", h2, "ij", None, "ij")                           # pure Hadamard
    assert close(Dh, h1.astype(np.complex128) * h2, sh, dtype)


def test_zero_mode_operands():
    s = np.array(2.5)
    T = np.asfortranarray(np.arange(6.0).reshape(2, 3))
    D, _ = run(s, "", T, "ij", None, "ji")
    assert np.array_equal(D, 2.5 * T.T)
    D2, _ = run(s, "", np.array(4.0), "", np.array(1.0), "", 2.0, 3.0)
    assert D2 == 2.0 * 10.0 + 3.0


# ---------------------------------------------------------------- identities
@pytest.mark.parametrize("dtype", DTYPES)
def test_alpha_zero_and_beta_zero(dtype):
    rng = np.random.default_rng(12)
    A, B, C = rnd(rng, (3, 4), dtype), rnd(rng, (4, 5), dtype), rnd(rng, (3, 5), dtype)
    nanA, nanB = np.full_like(A, np.nan), np.full_like(B, np.nan)
    D, _ = run(nanA, "ik", nanB, "kj", C, "ij", dtype(0), dtype(2))        # A, B never read
    assert np.array_equal(D, 2 * C)
    D1, s1 = run(A, "ik", B, "kj", np.full_like(C, np.nan), "ij", dtype(1), dtype(0))   # C never read
    assert close(D1, A.astype(np.complex128) @ B, s1, dtype)
    D2, _ = run(A, "ik", B, "kj", None, "ij", dtype(1), dtype(0))
    assert np.array_equal(D1, D2)


def test_linearity_in_alpha_beta():
    rng = np.random.default_rng(13)
    A, B, C = rnd(rng, (3, 4, 2), np.complex128), rnd(rng, (4, 2, 5), np.complex128), rnd(rng, (5, 3), np.complex128)
    al, be = 0.3 - 2j, 1.5 + 0.5j
    D, scale = run(A, "ikl", B, "klj", C, "ji", al, be)
    D10, _ = run(A, "ikl", B, "klj", None, "ji", 1.0, 0.0)
    assert close(D, al * D10 + be * C, scale, np.complex128)


def test_in_place_c_equals_d():
    rng = np.random.default_rng(14)
    A, B, C = rnd(rng, (3, 4), np.float64), rnd(rng, (4, 5), np.float64), rnd(rng, (3, 5), np.float64)
    want = 2 * A @ B + 0.5 * C
    scale = oracle.contract(A, "ik", B, "kj", C, "ij", C, "ij", 2.0, 0.5)
    assert close(C, want, scale, np.float64)


def test_scale_is_sum_of_moduli():
    rng = np.random.default_rng(15)
    A, B, C = rnd(rng, (3, 4), np.complex128), rnd(rng, (4, 5), np.complex128), rnd(rng, (3, 5), np.complex128)
    al, be = 3 - 4j, 0.5j
    _, scale = run(A, "ik", B, "kj", C, "ij", al, be, conjA=True)
    want = 5.0 * (np.abs(A) @ np.abs(B)) + 0.5 * np.abs(C)
    assert np.allclose(scale.reshape(3, 5, order="F"), want, rtol=1e-14)


def test_sampled_evaluation_matches_full():
    rng = np.random.default_rng(16)
    A, B, C = rnd(rng, (3, 4, 2), np.float32), rnd(rng, (4, 2, 5), np.float32), rnd(rng, (5, 3), np.float32)
    D, scale = run(A, "ikl", B, "klj", C, "ji", 2.0, 1.0)
    want_idx = [0, 7, 14, 3]
    Dd = np.full((5, 3), np.nan, np.float32, order="F")
    vals, sc = oracle.contract(A, "ikl", B, "klj", C, "ji", Dd, "ji", 2.0, 1.0, want=want_idx)
    assert np.all(np.isnan(Dd))
    assert np.array_equal(vals, D.reshape(-1, order="F")[want_idx])
    assert np.array_equal(sc, scale[want_idx])


@pytest.mark.parametrize("dtype", DTYPES)
def test_native_accumulator_within_tolerance_of_wide(dtype):
    rng = np.random.default_rng(17)
    A, B = rnd(rng, (6, 300), dtype), rnd(rng, (300, 5), dtype)
    D, scale = run(A, "ik", B, "kj", None, "ij")
    Dn, _ = run(A, "ik", B, "kj", None, "ij", native_acc=True)
    eps = np.finfo(dtype).eps
    err = np.abs(D.astype(np.complex128) - Dn)
    assert np.all(err <= 300 * eps * scale.reshape(6, 5, order="F"))
    assert oracle.long_double_mant_dig() >= 64   # the wide fp64 accumulator really is wider


# ---------------------------------------------------------------- invariances
def test_relabelling_is_bit_identical():
    rng = np.random.default_rng(18)
    A, B = rnd(rng, (3, 4, 2), np.float32), rnd(rng, (2, 5, 4), np.float32)
    D1, _ = run(A, "ikl", B, "ljk", None, "ji")
    D2, _ = run(A, [907, -3, 2**40], B, [2**40, 11, -3], None, [11, 907])
    assert np.array_equal(D1, D2)


def test_memory_order_permutation_leaves_logical_result():
    rng = np.random.default_rng(19)
    A = rnd(rng, (3, 4, 2), np.float64, "F")
    B = rnd(rng, (2, 5, 4), np.float64, "F")
    D1, scale = run(A, "ikl", B, "ljk", None, "ji")
    A2 = np.ascontiguousarray(A)            # same logical tensor, row-major memory
    B2 = np.ascontiguousarray(B)
    D2 = np.full((5, 3), np.nan, order="C")
    D2, _ = run(A2, "ikl", B2, "ljk", None, "ji", D=D2)
    assert close(D1, D2, scale, np.float64)
    # permuting D's labels permutes D (paper's test item 4)
    D3, scale3 = run(A, "ikl", B, "ljk", None, "ij")
    assert close(D3, D1.T, scale3, np.float64)


def test_commutativity_swap_a_and_b():
    rng = np.random.default_rng(20)
    A, B, C = rnd(rng, (3, 4, 2), np.complex64), rnd(rng, (2, 5, 4), np.complex64), rnd(rng, (5, 3), np.complex64)
    D1, scale = run(A, "ikl", B, "ljk", C, "ji", 1 + 1j, 2.0, conjA=True)
    D2, _ = run(B, "ljk", A, "ikl", C, "ji", 1 + 1j, 2.0, conjB=True)
    assert close(D1, D2, scale, np.complex64)


def test_negative_stride_is_reversed_copy():
    rng = np.random.default_rng(21)
    A, B = rnd(rng, (4, 5), np.float64), rnd(rng, (5, 3), np.float64)
    D1, scale = run(A[::-1, ::-1], "ik", B[::-1, :], "kj", None, "ij")
    D2, _ = run(np.asfortranarray(A[::-1, ::-1].copy()), "ik", np.asfortranarray(B[::-1, :].copy()), "kj", None, "ij")
    assert close(D1, D2, scale, np.float64)
    assert close(D1, A[::-1, ::-1] @ B[::-1, :], scale, np.float64)
    # negative stride in D
    Dbuf = np.full((4, 3), np.nan, order="F")
    run(A, "ik", B, "kj", None, "ij", D=Dbuf[::-1, :])
    assert close(Dbuf[::-1, :], A @ B, scale, np.float64)


def test_zero_stride_is_replication():
    rng = np.random.default_rng(22)
    a, B = rnd(rng, (4,), np.float64), rnd(rng, (5, 3), np.float64)
    A0 = np.lib.stride_tricks.as_strided(a, shape=(4, 5), strides=(a.itemsize, 0))
    D1, scale = run(A0, "ik", B, "kj", None, "ij")
    D2, _ = run(np.asfortranarray(np.repeat(a[:, None], 5, axis=1)), "ik", B, "kj", None, "ij")
    assert close(D1, D2, scale, np.float64)


def test_subtensors_and_padded_strides():
    rng = np.random.default_rng(23)
    big = rnd(rng, (7, 8, 6), np.float32)
    A = big[1:5, 2:7, 3]                    # fewer modes than the parent, offset base
    Bbig = rnd(rng, (9, 6), np.float32)
    B = Bbig[2:7, ::2]                      # stride 2 on a mode
    Dbig = np.full((6, 5), np.nan, np.float32, order="F")
    Dv = Dbig[:4, 1:4]
    run(A, "ik", B, "kj", None, "ij", D=Dv)
    _, scale = run(np.asfortranarray(A.copy()), "ik", np.asfortranarray(B.copy()), "kj", None, "ij")
    assert close(Dv, A.astype(np.float64) @ B.astype(np.float64), scale, np.float32)
    mask = np.ones_like(Dbig, dtype=bool)
    mask[:4, 1:4] = False
    assert np.all(np.isnan(Dbig[mask]))     # nothing outside the sub-tensor was written


def test_repeated_label_equals_merged_stride_tensor():
    # Note 6: A[k,i,k] is the tensor A'[k,i] whose k-stride is the sum of both k-strides
    rng = np.random.default_rng(24)
    A, B = rnd(rng, (4, 3, 4), np.float64), rnd(rng, (4, 5), np.float64)
    D1, scale = run(A, "kik", B, "kj", None, "ij")
    it = A.itemsize
    Am = np.lib.stride_tricks.as_strided(A, shape=(4, 3), strides=(A.strides[0] + A.strides[2], A.strides[1]))
    D2, _ = run(Am, "ki", B, "kj", None, "ij")
    assert np.array_equal(D1, D2)
    assert close(D1, np.einsum("kik,kj->ij", A, B), scale, np.float64)


# ---------------------------------------------------------------- conjugation
@pytest.mark.parametrize("dtype", [np.complex64, np.complex128])
def test_conj_flag_equals_conjugated_copy(dtype):
    rng = np.random.default_rng(25)
    A, B, C = rnd(rng, (3, 4), dtype), rnd(rng, (4, 5), dtype), rnd(rng, (3, 5), dtype)
    al, be = dtype(0.5 - 0.25j), dtype(1 + 2j)
    for ca, cb, cc in itertools.product([False, True], repeat=3):
        D1, scale = run(A, "ik", B, "kj", C, "ij", al, be, conjA=ca, conjB=cb, conjC=cc)
        D2, _ = run(np.conj(A) if ca else A, "ik", np.conj(B) if cb else B, "kj",
                    np.conj(C) if cc else C, "ij", al, be)
        assert np.array_equal(D1, D2)
        want = al * ((np.conj(A) if ca else A).astype(np.complex128) @ (np.conj(B) if cb else B)) \
            + be * (np.conj(C) if cc else C)
        assert close(D1, want, scale, dtype)


def test_gram_matrix_is_hermitian_with_column_norms():
    rng = np.random.default_rng(26)
    A = rnd(rng, (6, 4), np.complex128)
    D, scale = run(A, "ki", A, "kj", None, "ij", conjA=True)
    assert close(D, np.conj(D.T), scale, np.complex128)
    assert np.allclose(np.diag(D).imag, 0, atol=1e-15)
    assert np.allclose(np.diag(D).real, np.sum(np.abs(A) ** 2, axis=0), rtol=1e-14)


def test_conj_is_noop_for_real():
    rng = np.random.default_rng(27)
    A, B = rnd(rng, (3, 4), np.float64), rnd(rng, (4, 5), np.float64)
    D1, _ = run(A, "ik", B, "kj", None, "ij")
    D2, _ = run(A, "ik", B, "kj", None, "ij", conjA=True, conjB=True)
    assert np.array_equal(D1, D2)


# ---------------------------------------------------------------- error handling (test items 26-28, Case 5)
def _err(code, *a, **kw):
    with pytest.raises(oracle.OracleError) as ei:
        oracle.contract(*a, **kw)
    assert ei.value.code == code


def test_errors():
    A, B = np.zeros((3, 4), order="F"), np.zeros((4, 5), order="F")
    D, C = np.zeros((3, 5), order="F"), np.zeros((3, 5), order="F")
    _err(oracle.ERR_EXTENT_MISMATCH, A, "ik", np.zeros((5, 5), order="F"), "kj", None, "ij", D, "ij")
    _err(oracle.ERR_EXTENT_MISMATCH, np.zeros((3, 4), order="F"), "kk", B, "kj", None, "j", np.zeros(5), "j")
    _err(oracle.ERR_C_D_MISMATCH, A, "ik", B, "kj", np.zeros((5, 3), order="F"), "ji", D, "ij", 1.0, 1.0)
    _err(oracle.ERR_C_D_MISMATCH, A, "ik", B, "kj", np.zeros((3, 5), order="C"), "ij", D, "ij", 1.0, 1.0)
    _err(oracle.ERR_C_D_MISMATCH, A, "ik", B, "kj", np.zeros((3,)), "i", D, "ij", 1.0, 1.0)
    oracle.contract(A, "ik", B, "kj", np.zeros((5, 3)), "ji", D, "ij", 1.0, 0.0)   # beta == 0: C ignored
    _err(oracle.ERR_D_ALIASING, A, "ik", B, "kj", None, "ij", D, "ij", layouts={"D": ((3, 5), (1, 2))})
    _err(oracle.ERR_D_ALIASING, A, "ik", B, "kj", None, "ij", D, "ij", layouts={"D": ((3, 5), (0, 1))})
    _err(oracle.ERR_LABEL_ONLY_IN_D, A, "ik", B, "kj", None, "ijx", np.zeros((3, 5, 2), order="F"), "ijx")
    _err(oracle.ERR_NOT_SUPPORTED, A, "ik", B, "ki", None, "ii", np.zeros((3, 3), order="F"), "ii")
    _err(oracle.ERR_INVALID_EXTENT, A, "ik", B, "kj", None, "ij", D, "ij", layouts={"A": ((0, 4), (1, 3))})


def test_aliasing_rule_against_address_enumeration():
    """Whenever the rule accepts a D layout, enumerating every address shows no collision."""
    rng = np.random.default_rng(28)
    accepted = 0
    for _ in range(300):
        rank = int(rng.integers(1, 4))
        ext = [int(x) for x in rng.integers(1, 4, rank)]
        strides = [int(x) for x in rng.integers(-7, 8, rank)]
        A = np.zeros(ext, order="F")
        B = np.zeros(())
        lab = "ijk"[:rank]
        D = np.zeros(1)
        try:
            # evaluate no element (empty want list): only the checks run
            oracle.contract(A, lab, B, "", None, lab, D, lab, layouts={"D": (ext, strides)}, want=[])
        except oracle.OracleError as e:
            assert e.code == oracle.ERR_D_ALIASING
            continue
        accepted += 1
        addrs = [sum(i * s for i, s in zip(idx, strides)) for idx in itertools.product(*[range(e) for e in ext])]
        assert len(set(addrs)) == len(addrs), (ext, strides)
    assert accepted > 20


# ---------------------------------------------------------------- input generators
def test_generator_matches_published_splitmix64_vectors():
    import os
    import torch
    from paper_2601_07827_b200 import inputs
    path = os.path.join(os.path.dirname(__file__), "golden", "splitmix64_vectors.txt")
    vec = [int(l, 16) for l in open(path) if l.strip() and not l.startswith("#")]
    gamma = 0x9E3779B97F4A7C15
    state = [(i * gamma) & (2**64 - 1) for i in range(3)]      # generator state before each output
    assert [inputs.splitmix64_int(s) for s in state] == vec
    t = torch.tensor([inputs._s64(s) for s in state], dtype=torch.int64)
    assert [int(v) & (2**64 - 1) for v in inputs.splitmix64(t)] == vec


def test_generator_is_layout_independent_and_seeded():
    import torch
    from paper_2601_07827_b200 import inputs
    flat = inputs.logical_values(5, (3, 4, 2), torch.float64, "uniform", 1.0)
    assert flat.abs().max() <= 1.0 and flat.unique().numel() == 24
    t1 = inputs.place(flat, (3, 4, 2), None, torch.float64)
    t2 = inputs.place(flat, (3, 4, 2), (8, 2, 1), torch.float64)
    t3 = inputs.place(flat, (3, 4, 2), (-1, 3, 20), torch.float64)
    assert np.array_equal(t1.numpy(), t2.numpy()) and np.array_equal(t1.numpy(), t3.numpy())
    assert torch.equal(t3.get_logical(), flat)
    again = inputs.logical_values(5, (3, 4, 2), torch.float64, "uniform", 1.0, chunk=5)
    assert torch.equal(flat, again)
    other = inputs.logical_values(6, (3, 4, 2), torch.float64, "uniform", 1.0)
    assert not torch.equal(flat, other)
    nrm = inputs.logical_values(7, (200, 200), torch.float64, "normal", 0.1)
    assert abs(float(nrm.mean())) < 2e-3 and abs(float(nrm.std()) - 0.1) < 2e-3


def test_workload_symmetry_and_sizes():
    import dataclasses
    from paper_2601_07827_b200 import inputs
    W = inputs.workloads()
    assert W["cfg2_f64_ccsd_ladder"].groups() == (1, 16384, 1024, 16384)
    assert W["cfg3_f32_batched_permuted"].groups() == (64, 96, 9216, 576)
    assert W["cfg4_c64_conj"].groups() == (1, 256, 16384, 2304)
    assert W["cfg5_f32_tensor_network"].groups() == (1, 1024, 1024, 64)
    small = inputs.scaled_down(W["cfg2_f64_ccsd_ladder"], {**{x: 6 for x in "abcd"}, "i": 3, "j": 3})
    A, B, C, D = inputs.make_workload_tensors(small)
    V = A.numpy()
    assert np.array_equal(V, V.transpose(1, 0, 3, 2)) and C is D
    s3 = inputs.scaled_down(W["cfg3_f32_batched_permuted"], {"z": 2, "a": 5, "b": 6, "j": 7, "k": 3, "l": 2})
    assert s3.stridesD == (1, 15, 90, 180)


# ---------------------------------------------------------------- mixed element types
def run_mixed(A, la, B, lb, C, ld, dtypeD, alpha=1.0, beta=0.0, **kw):
    ext = {}
    for t, l in ((A, la), (B, lb)):
        for e, ch in zip(t.shape, l):
            ext[ch] = e
    D = np.full([ext[ch] for ch in ld], np.nan, dtype=dtypeD, order="F")
    scale = oracle.contract_mixed(A, la, B, lb, C, ld, D, ld, alpha, beta, **kw)
    return D, scale


@pytest.mark.parametrize("dtype", DTYPES)
def test_mixed_entry_point_with_one_type_equals_the_plain_oracle(dtype):
    """The mixed-type loop nest must be the same function when every tensor has the same type: identical
    bits for the 64-bit types (both accumulate in long double, in the same order), one rounding apart
    for the 32-bit types (double against long double accumulators)."""
    rng = np.random.default_rng(71)
    A, B, C = rnd(rng, (5, 6, 3), dtype), rnd(rng, (3, 6, 4), dtype), rnd(rng, (4, 5), dtype)
    cplx = np.issubdtype(dtype, np.complexfloating)
    alpha, beta = (0.5 - 0.25j, 1.5 + 2j) if cplx else (0.5, 1.5)
    want, scale = run(A, "ikl", B, "lkj", C, "ji", alpha, beta, conjA=cplx, conjC=cplx)
    got, scale2 = run_mixed(A, "ikl", B, "lkj", C, "ji", dtype, alpha, beta, conjA=cplx, conjC=cplx)
    if dtype in (np.float64, np.complex128):
        assert np.array_equal(got, want)
    else:
        assert np.all(np.abs(got.astype(np.complex128) - want.astype(np.complex128)) <= 2.0 ** -22 * np.abs(want))
    assert np.allclose(scale, scale2, rtol=1e-6)


@pytest.mark.parametrize("real,cplx", [(np.float64, np.complex128), (np.float32, np.complex64)])
@pytest.mark.parametrize("which", ["A", "B", "C", "AB"])
def test_real_operand_among_complex_ones_equals_its_promoted_copy(real, cplx, which):
    """A real tensor is the complex tensor with zero imaginary parts: mixing it in must give what the
    plain oracle gives on the explicitly promoted copy (bit-identical in 64-bit; conj of a real operand
    is a no-op)."""
    rng = np.random.default_rng(72)
    tA = real if "A" in which else cplx
    tB = real if "B" in which else cplx
    tC = real if "C" in which else cplx
    A, B, C = rnd(rng, (4, 7), tA), rnd(rng, (7, 5), tB), rnd(rng, (4, 5), tC)
    alpha, beta = 0.75 - 0.5j, -0.25 + 1.0j
    got, scale = run_mixed(A, "ik", B, "kj", C, "ij", cplx, alpha, beta, conjA=True, conjB=True, conjC=True)
    want, _ = run(A.astype(cplx), "ik", B.astype(cplx), "kj", C.astype(cplx), "ij", alpha, beta, conjA=True, conjB=True, conjC=True)
    if cplx is np.complex128:
        assert np.array_equal(got, want)
    else:
        assert close(got, want, scale, cplx, factor=0.1)


def test_mixed_types_against_explicit_loops_and_einsum():
    """Hand loops in Python complex arithmetic on a tiny case with three different element types, and numpy
    einsum on promoted copies, pin products, conjugation and the alpha / beta step of the mixed loop nest."""
    rng = np.random.default_rng(73)
    A = rnd(rng, (3, 2, 4), np.float32)                  # A[i,k,l] real, 32-bit
    B = rnd(rng, (4, 2, 3), np.complex64)                # B[l,k,j]
    C = rnd(rng, (3, 3), np.float64)                     # C[j,i] real, 64-bit
    alpha, beta = 1.25 + 0.5j, 0.5 - 1.5j
    got, scale = run_mixed(A, "ikl", B, "lkj", C, "ji", np.complex128, alpha, beta, conjB=True)
    want = np.zeros((3, 3), dtype=np.complex128)
    for j in range(3):
        for i in range(3):
            acc = 0j
            for k in range(2):
                for l in range(4):
                    acc += complex(A[i, k, l]) * complex(B[l, k, j]).conjugate()
            want[j, i] = alpha * acc + beta * complex(C[j, i])
    assert np.allclose(got, want, rtol=1e-13, atol=1e-13)
    ein = alpha * np.einsum("ikl,lkj->ji", A.astype(np.complex128), np.conj(B).astype(np.complex128)) + beta * C
    assert np.allclose(got, ein, rtol=1e-13, atol=1e-13)
    # scale = |alpha| sum |a||b| + |beta||c|
    s = abs(alpha) * np.einsum("ikl,lkj->ji", np.abs(A).astype(np.float64), np.abs(B).astype(np.float64)) + abs(beta) * np.abs(C)
    assert np.allclose(scale.reshape(3, 3, order="F"), s, rtol=1e-6)


def test_float32_storage_is_accumulated_wider_than_float32():
    """fp32 tensors through the mixed entry point: the sum is formed wider than fp32 and rounded once, so on
    a long ill-conditioned sum it is far closer to the exact value than fp32 accumulation is."""
    n = 20000
    a = np.asarray(np.full((1, n), 1.0), dtype=np.float32, order="F")
    b = np.asarray(np.full((n, 1), 1e-4), dtype=np.float32, order="F")
    b[0, 0] = 1e4                                         # large first term swallows small ones in fp32
    got, _ = run_mixed(a, "ik", b, "kj", None, "ij", np.float32)
    exact = float(np.sum(b.astype(np.float64)))
    assert abs(float(got[0, 0]) - exact) <= 2.0 ** -23 * exact
    naive = np.float32(0)
    for x in b[:, 0]:
        naive = np.float32(naive + x)
    assert abs(float(naive) - exact) > 100 * abs(float(got[0, 0]) - exact)


def test_mixed_types_reject_a_real_result_of_complex_inputs():
    rng = np.random.default_rng(74)
    A, B = rnd(rng, (3, 4), np.complex128), rnd(rng, (4, 2), np.float64)
    D = np.zeros((3, 2), dtype=np.float64, order="F")
    with pytest.raises(oracle.OracleError) as ei:
        oracle.contract_mixed(A, "ik", B, "kj", None, "ij", D, "ij")
    assert ei.value.code == oracle.ERR_NOT_SUPPORTED
    with pytest.raises(oracle.OracleError):                # a complex alpha cannot scale a real result
        oracle.contract_mixed(B, "ik", B.T.copy(order="F"), "kj", None, "ij", np.zeros((4, 4), order="F"), "ij", alpha=1j)
