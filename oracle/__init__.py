"""CPU oracle for D = alpha * op(A) * op(B) + beta * op(C)  --  TEST INFRASTRUCTURE ONLY.

A thin ctypes wrapper around ``contract_oracle.c`` (the plain loop nest written from the
paper's definition, Eq. (case2) with Cases 3 and 4).  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this package; the GPU library never does, and the two
share no code.

Tensors are numpy arrays; any strides numpy can express are honoured (negative, zero, padded),
because the C code receives the address of element (0,...,0) and the strides in elements.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "contract_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_contract.so")
_SRC_EW = os.path.join(_HERE, "elementwise_oracle.c")
_LIB_EW = os.path.join(_HERE, "liboracle_elementwise.so")
ERR_B_C_MISMATCH = 4      # elementwise oracle: B does not have C's rank / extents / labels
ERR_C_ALIASING = 5        # elementwise oracle: elements of C alias

OK = 0
ERR_INVALID_ARGUMENT = 1
ERR_INVALID_EXTENT = 2
ERR_EXTENT_MISMATCH = 3
ERR_C_D_MISMATCH = 4
ERR_D_ALIASING = 5
ERR_LABEL_ONLY_IN_D = 6
ERR_NOT_SUPPORTED = 7

_DTYPE_CODE = {
    np.dtype(np.float32): 0,
    np.dtype(np.float64): 1,
    np.dtype(np.complex64): 2,
    np.dtype(np.complex128): 3,
}


class OracleError(Exception):
    def __init__(self, code: int):
        super().__init__(f"oracle error code {code}")
        self.code = code


class _Tensor(ctypes.Structure):
    _fields_ = [
        ("rank", ctypes.c_int32),
        ("extent", ctypes.POINTER(ctypes.c_int64)),
        ("stride", ctypes.POINTER(ctypes.c_int64)),
        ("label", ctypes.POINTER(ctypes.c_int64)),
        ("conj", ctypes.c_int32),
        ("data", ctypes.c_void_p),
    ]


def _compile(src: str, lib: str, force: bool) -> str:
    if force or not os.path.exists(lib) or os.path.getmtime(lib) < os.path.getmtime(src):
        tmp = lib + f".tmp{os.getpid()}"
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, src, "-lm"],
            check=True,
        )
        os.replace(tmp, lib)
    return lib


def build(force: bool = False) -> str:
    """Compile the C oracles into shared libraries next to their sources (gcc, OpenMP)."""
    _compile(_SRC_EW, _LIB_EW, force)
    return _compile(_SRC, _LIB, force)


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.orc_contract.restype = ctypes.c_int
        lib.orc_contract.argtypes = [
            ctypes.c_int,
            ctypes.POINTER(_Tensor), ctypes.POINTER(_Tensor), ctypes.POINTER(_Tensor),
            ctypes.POINTER(_Tensor),
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
            ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
        ]
        lib.orc_long_double_mant_dig.restype = ctypes.c_int
        lib.orc_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def labels_to_ints(labels) -> list:
    """Labels are arbitrary integers; a string stands for the code points of its characters."""
    if isinstance(labels, str):
        return [ord(ch) for ch in labels]
    return [ord(x) if isinstance(x, str) else int(x) for x in labels]


def _describe(arr: Optional[np.ndarray], labels, conj: bool, keep: list,
              extents=None, strides=None):
    """Build the C descriptor of one operand; extents/strides override the array's own."""
    if arr is None:
        return None
    lab = labels_to_ints(labels)
    ext = list(arr.shape) if extents is None else list(extents)
    if strides is None:
        if any(s % arr.itemsize for s in arr.strides):
            raise ValueError("strides must be whole elements")
        strides = [s // arr.itemsize for s in arr.strides]
    strides = list(strides)
    if not (len(lab) == len(ext) == len(strides)):
        raise ValueError("labels, extents and strides must have the same length")
    n = len(lab)
    e = (ctypes.c_int64 * max(n, 1))(*ext)
    s = (ctypes.c_int64 * max(n, 1))(*strides)
    l = (ctypes.c_int64 * max(n, 1))(*lab)
    keep += [e, s, l, arr]
    return _Tensor(n, e, s, l, int(bool(conj)), arr.ctypes.data)


def contract(A: np.ndarray, labelsA, B: np.ndarray, labelsB,
             C: Optional[np.ndarray], labelsC, D: np.ndarray, labelsD,
             alpha=1.0, beta=0.0, *, conjA=False, conjB=False, conjC=False,
             native_acc=False, want: Optional[Sequence[int]] = None,
             with_scale=True, layouts: Optional[dict] = None):
    """Evaluate the contraction.

    Without ``want``: D (a numpy array whose strides are honoured) is overwritten in place and
    the per-element error scale is returned as a flat array in column-major order over D's
    labels (None when ``with_scale`` is false).

    With ``want`` (column-major linear indices over D's labels): D's memory is left alone and
    ``(values, scale)`` for exactly those elements is returned.

    ``layouts`` optionally maps "A"/"B"/"C"/"D" to ``(extents, strides)`` replacing the numpy
    array's own shape and strides (used by the error-handling tests to state inconsistent
    descriptors without creating such arrays).
    """
    lib = _load()
    dt = np.dtype(D.dtype)
    if dt not in _DTYPE_CODE:
        raise OracleError(ERR_NOT_SUPPORTED)
    for t in (A, B, C):
        if t is not None and t.dtype != dt:
            raise OracleError(ERR_NOT_SUPPORTED)
    layouts = layouts or {}
    keep: list = []
    tA = _describe(A, labelsA, conjA, keep, *layouts.get("A", (None, None)))
    tB = _describe(B, labelsB, conjB, keep, *layouts.get("B", (None, None)))
    tC = _describe(C, labelsC, conjC, keep, *layouts.get("C", (None, None)))
    tD = _describe(D, labelsD, False, keep, *layouts.get("D", (None, None)))
    al = np.array([alpha], dtype=dt)
    be = np.array([beta], dtype=dt)

    n_eval = 1
    for e in (layouts["D"][0] if "D" in layouts else D.shape):
        n_eval *= int(e)
    want_arr = None
    out_val = None
    if want is not None:
        want_arr = np.ascontiguousarray(np.asarray(want, dtype=np.int64)).reshape(-1)
        n_eval = want_arr.size
        if n_eval == 0:  # keep the pointer non-NULL: an empty list means "checks only"
            want_arr = np.zeros(1, dtype=np.int64)
        out_val = np.empty(max(n_eval, 1), dtype=dt)[:n_eval]
    scale = np.empty(max(n_eval, 1), dtype=np.float64)[:n_eval] if with_scale else None

    rc = lib.orc_contract(
        _DTYPE_CODE[dt],
        ctypes.byref(tA) if tA is not None else None,
        ctypes.byref(tB) if tB is not None else None,
        ctypes.byref(tC) if tC is not None else None,
        ctypes.byref(tD),
        al.ctypes.data, be.ctypes.data, int(bool(native_acc)),
        n_eval if want_arr is not None else 0,
        want_arr.ctypes.data if want_arr is not None else None,
        out_val.ctypes.data if out_val is not None else None,
        scale.ctypes.data if scale is not None else None,
    )
    if rc != OK:
        raise OracleError(rc)
    if want_arr is not None:
        return out_val, scale
    return scale


def contract_mixed(A: np.ndarray, labelsA, B: np.ndarray, labelsB,
                   C: Optional[np.ndarray], labelsC, D: np.ndarray, labelsD,
                   alpha=1.0, beta=0.0, *, conjA=False, conjB=False, conjC=False,
                   want: Optional[Sequence[int]] = None, layouts: Optional[dict] = None):
    """The contraction with an element type per tensor (float32 / float64 / complex64 / complex128 in any
    mix whose result type can hold the result: D must be complex when an input is).  Same calling
    conventions and return values as ``contract`` (scale always returned)."""
    lib = _load()
    for t in (A, B, C, D):
        if t is not None and np.dtype(t.dtype) not in _DTYPE_CODE:
            raise OracleError(ERR_NOT_SUPPORTED)
    layouts = layouts or {}
    keep: list = []
    tA = _describe(A, labelsA, conjA, keep, *layouts.get("A", (None, None)))
    tB = _describe(B, labelsB, conjB, keep, *layouts.get("B", (None, None)))
    tC = _describe(C, labelsC, conjC, keep, *layouts.get("C", (None, None)))
    tD = _describe(D, labelsD, False, keep, *layouts.get("D", (None, None)))
    al = np.array([complex(alpha).real, complex(alpha).imag], dtype=np.float64)
    be = np.array([complex(beta).real, complex(beta).imag], dtype=np.float64)
    n_eval = 1
    for e in (layouts["D"][0] if "D" in layouts else D.shape):
        n_eval *= int(e)
    want_arr = out_val = None
    if want is not None:
        want_arr = np.ascontiguousarray(np.asarray(want, dtype=np.int64)).reshape(-1)
        n_eval = want_arr.size
        if n_eval == 0:
            want_arr = np.zeros(1, dtype=np.int64)
        out_val = np.empty(max(n_eval, 1), dtype=D.dtype)[:n_eval]
    scale = np.empty(max(n_eval, 1), dtype=np.float64)[:n_eval]
    code = lambda t: _DTYPE_CODE[np.dtype(t.dtype)] if t is not None else _DTYPE_CODE[np.dtype(D.dtype)]
    lib.orc_contract_mixed.restype = ctypes.c_int
    lib.orc_contract_mixed.argtypes = [ctypes.c_int] * 4 + [ctypes.POINTER(_Tensor)] * 4 + [
        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    rc = lib.orc_contract_mixed(
        code(A), code(B), code(C), code(D),
        ctypes.byref(tA) if tA is not None else None, ctypes.byref(tB) if tB is not None else None,
        ctypes.byref(tC) if tC is not None else None, ctypes.byref(tD),
        al.ctypes.data, be.ctypes.data,
        n_eval if want_arr is not None else 0,
        want_arr.ctypes.data if want_arr is not None else None,
        out_val.ctypes.data if out_val is not None else None, scale.ctypes.data)
    if rc != OK:
        raise OracleError(rc)
    if want_arr is not None:
        return out_val, scale
    return scale


_lib_ew = None


def _load_ew():
    global _lib_ew
    if _lib_ew is None:
        build()
        lib = ctypes.CDLL(_LIB_EW)
        lib.ore_elementwise.restype = ctypes.c_int
        lib.ore_elementwise.argtypes = [
            ctypes.c_int, ctypes.POINTER(_Tensor), ctypes.POINTER(_Tensor), ctypes.POINTER(_Tensor),
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
            ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
        ]
        _lib_ew = lib
    return _lib_ew


def elementwise(A: np.ndarray, labelsA, B: Optional[np.ndarray], C: np.ndarray, labelsC,
                alpha=1.0, beta=0.0, *, conjA=False, conjB=False, native_acc=False,
                want: Optional[Sequence[int]] = None, with_scale=True, layouts: Optional[dict] = None):
    """Evaluate C := alpha * op(A) + beta * op(B) (Sec. "Unary and Binary Operations"): labels
    only in A are summed over, A is broadcast along labels only in C, B carries C's labels.

    Same conventions as ``contract``: without ``want`` C is overwritten in place and the flat
    per-element error scale is returned; with ``want`` ``(values, scale)`` of those elements is
    returned and C's memory is left alone."""
    lib = _load_ew()
    dt = np.dtype(C.dtype)
    if dt not in _DTYPE_CODE:
        raise OracleError(ERR_NOT_SUPPORTED)
    for t in (A, B):
        if t is not None and t.dtype != dt:
            raise OracleError(ERR_NOT_SUPPORTED)
    layouts = layouts or {}
    keep: list = []
    tA = _describe(A, labelsA, conjA, keep, *layouts.get("A", (None, None)))
    tB = _describe(B, labelsC, conjB, keep, *layouts.get("B", (None, None)))
    tC = _describe(C, labelsC, False, keep, *layouts.get("C", (None, None)))
    al = np.array([alpha], dtype=dt)
    be = np.array([beta], dtype=dt)
    n_eval = 1
    for e in (layouts["C"][0] if "C" in layouts else C.shape):
        n_eval *= int(e)
    want_arr = None
    out_val = None
    if want is not None:
        want_arr = np.ascontiguousarray(np.asarray(want, dtype=np.int64)).reshape(-1)
        n_eval = want_arr.size
        if n_eval == 0:
            want_arr = np.zeros(1, dtype=np.int64)
        out_val = np.empty(max(n_eval, 1), dtype=dt)[:n_eval]
    scale = np.empty(max(n_eval, 1), dtype=np.float64)[:n_eval] if with_scale else None
    rc = lib.ore_elementwise(
        _DTYPE_CODE[dt], ctypes.byref(tA), ctypes.byref(tB) if tB is not None else None, ctypes.byref(tC),
        al.ctypes.data, be.ctypes.data, int(bool(native_acc)),
        n_eval if want_arr is not None else 0,
        want_arr.ctypes.data if want_arr is not None else None,
        out_val.ctypes.data if out_val is not None else None,
        scale.ctypes.data if scale is not None else None,
    )
    if rc != OK:
        raise OracleError(rc)
    if want_arr is not None:
        return out_val, scale
    return scale


def long_double_mant_dig() -> int:
    return _load().orc_long_double_mant_dig()


def num_threads() -> int:
    return _load().orc_num_threads()
