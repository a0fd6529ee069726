"""Host-side checks that need no GPU: the shared library loads and exports every symbol the
header declares, descriptors validate, error codes follow the paper's test list (items 26-28,
Case 5), and the planner classifies / fuses / orders labels as designed."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def api():
    from paper_2601_07827_b200 import build
    build.build()
    from paper_2601_07827_b200 import api as _api
    return _api


@pytest.fixture(scope="module")
def handle(api):
    return api.Handle()


def test_every_declared_symbol_is_exported(api):
    header = open(os.path.join(ROOT, "include", "btc.h")).read()
    declared = set(re.findall(r"btc_error_t\s+(btc_\w+)\s*\(", header))
    assert declared == set(api.EXPORTED)
    lib = ctypes.CDLL(api.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name


def test_error_text(api):
    for code in range(0, 14):
        assert len(api.explain_error(code)) > 3
    assert "success" in api.explain_error(0)
    assert "unknown" in api.explain_error(999)


def _op(api, h, eA, la, eB, lb, eD, ld, dtype=None, sA=None, sB=None, sD=None, C=None, **kw):
    dtype = api.F64 if dtype is None else dtype
    tA = api.TensorInfo(h, dtype, eA, sA)
    tB = api.TensorInfo(h, dtype, eB, sB)
    tD = api.TensorInfo(h, dtype, eD, sD)
    tC, lc = None, None
    if C is not None:
        tC = api.TensorInfo(h, C.get("dtype", dtype), C["extents"], C.get("strides"))
        lc = C.get("labels", ld)
    return api.Contraction(h, tA, la, tB, lb, tC, lc, tD, ld, **kw)


def _code(api, fn):
    with pytest.raises(api.BtcError) as ei:
        fn()
    return ei.value.code


def test_descriptor_validation(api, handle):
    assert _code(api, lambda: api.TensorInfo(handle, api.F64, (3, 0))) == api.ERR_INVALID_EXTENT
    assert _code(api, lambda: api.TensorInfo(handle, api.F64, tuple([2] * 33))) == api.ERR_INVALID_ARGUMENT
    assert _code(api, lambda: api.TensorInfo(handle, 9, (2,))) == api.ERR_INVALID_ARGUMENT
    api.TensorInfo(handle, api.C32, ())            # zero-mode tensors are legal
    api.TensorInfo(handle, api.F32, (4, 5), (-1, 0))   # negative and zero strides are legal


def test_error_codes_of_the_paper_test_list(api, h=None):
    h = api.Handle()
    E = api
    assert _code(api, lambda: _op(api, h, (3, 4), "ik", (5, 6), "kj", (3, 6), "ij")) == E.ERR_EXTENT_MISMATCH
    assert _code(api, lambda: _op(api, h, (3, 4), "kk", (3, 5), "kj", (5,), "j")) == E.ERR_EXTENT_MISMATCH
    c_bad = [dict(extents=(5, 3), labels="ji"), dict(extents=(3, 5), strides=(5, 1)), dict(extents=(3,), labels="i"),
             dict(extents=(3, 5), labels="ix")]
    for C in c_bad:
        assert _code(api, lambda: _op(api, h, (3, 4), "ik", (4, 5), "kj", (3, 5), "ij", C=C, beta=1.0)) == E.ERR_C_D_MISMATCH
    assert _code(api, lambda: _op(api, h, (3, 4), "ik", (4, 5), "kj", (3, 5), "ij", sD=(1, 2))) == E.ERR_D_ALIASING
    assert _code(api, lambda: _op(api, h, (3, 4), "ik", (4, 5), "kj", (3, 5), "ij", sD=(0, 1))) == E.ERR_D_ALIASING
    assert _code(api, lambda: _op(api, h, (3, 4), "ik", (4, 5), "kj", (3, 5, 2), "ijx")) == E.ERR_LABEL_ONLY_IN_D
    assert _code(api, lambda: _op(api, h, (3, 4), "ik", (4, 3), "ki", (3, 3), "ii")) == E.ERR_NOT_SUPPORTED
    assert _code(api, lambda: _op(api, h, (3, 4), "ik", (4, 5), "kj", (3, 5), "ij",
                                  C=dict(extents=(3, 5), dtype=api.F32), beta=1.0)) == E.ERR_NOT_SUPPORTED
    # beta != 0 without a C descriptor
    assert _code(api, lambda: _op(api, h, (3, 4), "ik", (4, 5), "kj", (3, 5), "ij", beta=0.5)) == E.ERR_INVALID_ARGUMENT
    # legal: padded D, negative strides in D that do not alias
    _op(api, h, (3, 4), "ik", (4, 5), "kj", (3, 5), "ij", sD=(-1, 4))
    _op(api, h, (3, 4), "ik", (4, 5), "kj", (3, 5), "ij", sD=(7, 1))


def test_aliasing_rule_matches_oracle_rule(api):
    """Both sides state the same sufficient condition; compare decisions on random layouts."""
    import numpy as np
    import oracle
    h = api.Handle()
    rng = np.random.default_rng(5)
    seen = {True: 0, False: 0}
    for _ in range(200):
        rank = int(rng.integers(1, 4))
        ext = [int(x) for x in rng.integers(1, 4, rank)]
        strides = [int(x) for x in rng.integers(-7, 8, rank)]
        lab = "ijk"[:rank]
        try:
            _op(api, h, ext, lab, (), "", ext, lab, sD=strides)
            lib_ok = True
        except api.BtcError as e:
            assert e.code == api.ERR_D_ALIASING
            lib_ok = False
        try:
            oracle.contract(np.zeros(ext, order="F"), lab, np.zeros(()), "", None, lab, np.zeros(1), lab,
                            layouts={"D": (ext, strides)}, want=[])
            orc_ok = True
        except oracle.OracleError:
            orc_ok = False
        assert lib_ok == orc_ok
        seen[lib_ok] += 1
    assert seen[True] > 10 and seen[False] > 10


def test_planner_groups_fusion_and_roles(api, handle):
    from paper_2601_07827_b200 import inputs
    W = inputs.workloads()
    expect = {
        "cfg1_f64_small": ((1, 256, 256, 256), (0, 2, 2, 2), False),
        "cfg2_f64_ccsd_ladder": ((1, 16384, 1024, 16384), (0, 1, 1, 1), False),   # a plain GEMM after fusion
        "cfg3_f32_batched_permuted": ((64, 9216, 96, 576), (1, 4, 1, 2), True),   # j is in B: roles swap; j and b are blocked
        "cfg4_c64_conj": ((1, 256, 16384, 2304), (0, 1, 2, 4), False),            # s and t are split
        "cfg5_f32_tensor_network": ((1, 1024, 1024, 64), (0, 5, 5, 3), False),
        "cfg5b_f32_tensor_network_rev": ((1, 1024, 1024, 64), (0, 5, 5, 3), True),
    }
    for name, (groups, modes, swapped) in expect.items():
        w = W[name]
        dt = {"f32": api.F32, "f64": api.F64, "c32": api.C32, "c64": api.C64}[w.dtype]
        C = dict(extents=w.ext(w.labelsD), strides=w.stridesD) if w.beta != 0 else None
        op = _op(api, handle, w.ext(w.labelsA), w.labelsA, w.ext(w.labelsB), w.labelsB, w.ext(w.labelsD), w.labelsD,
                 dtype=dt, sA=w.stridesA, sB=w.stridesB, sD=w.stridesD, C=C, alpha=w.alpha, beta=w.beta,
                 conjA=w.conjA)
        assert op.groups == groups, name
        assert op.num_modes == modes, name
        assert op.swapped == swapped, name


def test_planner_kernel_choice_and_split_k(api, handle):
    op = _op(api, handle, (16, 16, 16, 16), "acid", (16, 16, 16, 16), "dbcj", (16, 16, 16, 16), "abij")
    assert op.kernel == api.KERNEL_TILED and op.tile == (64, 64, 16)
    assert op.split_k > 1 and op.workspace_size() == 16 * op.split_k * 64 * 64 * 8
    op.set_attr(api.ATTR_SPLIT_K, 1)
    assert op.split_k == 1 and op.workspace_size() == 0
    op.set_attr(api.ATTR_KERNEL, api.KERNEL_GENERIC)
    assert op.kernel == api.KERNEL_GENERIC
    tiny = _op(api, handle, (2, 5), "ik", (5, 2), "kj", (2, 2), "ij")
    assert tiny.kernel == api.KERNEL_GENERIC
    # at most four contracted indices: the streaming kernel, whatever the size
    tiny = _op(api, handle, (2, 3), "ik", (3, 2), "kj", (2, 2), "ij")
    assert tiny.kernel == api.KERNEL_TILED and tiny.variant == 100
    # Case 4, isolated label x: by default A is first summed over x into the workspace and the tiled
    # kernel contracts the result; with the pre-reduction off the generic kernel sums x itself
    case4 = _op(api, handle, (64, 64, 5), "ikx", (64, 64), "kj", (64, 64), "ij")
    assert case4.kernel == api.KERNEL_TILED and case4.pre_reduce == 1
    assert case4.groups == (1, 64, 64, 64)
    assert case4.workspace_size() >= 64 * 64 * 8
    case4.set_attr(api.ATTR_PRE_REDUCE, 0)
    assert case4.kernel == api.KERNEL_GENERIC and case4.pre_reduce == 0
    assert case4.groups == (1, 64, 64, 64 * 5)
    assert _code(api, lambda: case4.set_attr(api.ATTR_KERNEL, api.KERNEL_TILED)) == api.ERR_NOT_SUPPORTED
    assert case4.kernel == api.KERNEL_GENERIC
    case4.set_attr(api.ATTR_PRE_REDUCE, 1)
    assert case4.kernel == api.KERNEL_TILED
    both = _op(api, handle, (7, 64, 64), "xik", (64, 64, 3, 3), "kjyy", (64, 64), "ij")   # x in A; y twice in B
    assert both.pre_reduce == 3 and both.groups == (1, 64, 64, 64)


def test_execute_without_device_fails_loudly(api, handle):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    op = _op(api, handle, (2, 3), "ik", (3, 2), "kj", (2, 2), "ij")
    buf = (ctypes.c_double * 16)()
    p = ctypes.addressof(buf)
    assert _code(api, lambda: op.execute(0, p, p, 0, p)) == api.ERR_CUDA
    assert _code(api, lambda: op.execute_host(0, p, p, 0, p)) == api.ERR_CUDA
    assert _code(api, lambda: api.selftest_bounded_wait(handle)) == api.ERR_CUDA


def test_elementwise_planning_without_a_device(api, handle):
    """Validation, merging and kernel choice of C := alpha op(A) + beta op(B) are host work."""
    t = lambda e, s=None: api.TensorInfo(handle, api.F32, e, s)
    same = api.Elementwise(handle, t((64, 32, 16)), "abc", t((64, 32, 16)), t((64, 32, 16)), "abc", 1.0, 1.0)
    assert same.kernel == api.EW_KERNEL_DIRECT and same.num_modes == (1, 0)       # everything chains into one loop
    perm = api.Elementwise(handle, t((64, 32, 16)), "abc", None, t((16, 64, 32)), "cab")
    assert perm.kernel == api.EW_KERNEL_TRANSPOSING and perm.num_modes == (2, 0)   # (a, b) chain in both tensors
    red = api.Elementwise(handle, t((64, 5, 32)), "axb", None, t((64, 32)), "ab")
    assert red.kernel == api.EW_KERNEL_DIRECT and red.num_modes == (2, 1)
    assert _code(api, lambda: api.Elementwise(handle, t((3, 4)), "ij", None, t((4, 5)), "ji")) == api.ERR_EXTENT_MISMATCH
    assert _code(api, lambda: api.Elementwise(handle, t((3, 4)), "ij", None, t((4, 3), (1, 2)), "ji")) == api.ERR_D_ALIASING
    if not __import__("torch").cuda.is_available():
        buf = (ctypes.c_float * 64 * 32 * 16)()
        p = ctypes.addressof(buf)
        assert _code(api, lambda: same.execute(0, p, p, p)) == api.ERR_CUDA


def test_element_type_mixes(api, handle):
    """Real among complex operands of one part width plan (on the per-element kernel); 32- with 64-bit parts and
    a real result of a complex input are refused (Sec. "Challenge: Datatypes": an implementation may support
    fewer mixes than the reference one)."""
    t = lambda dt, ext: api.TensorInfo(handle, dt, ext)
    op = api.Contraction(handle, t(api.F64, (4, 5)), "ik", t(api.C64, (5, 3)), "kj", None, "ij", t(api.C64, (4, 3)), "ij")
    assert op.kernel == api.KERNEL_GENERIC
    for a, b, d in ((api.F32, api.F64, api.F64), (api.C64, api.F64, api.F64), (api.C32, api.C64, api.C64)):
        with pytest.raises(api.BtcError) as ei:
            api.Contraction(handle, t(a, (4, 5)), "ik", t(b, (5, 3)), "kj", None, "ij", t(d, (4, 3)), "ij")
        assert ei.value.code == api.ERR_NOT_SUPPORTED
