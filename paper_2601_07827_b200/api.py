"""ctypes binding of the C-ABI contraction library (include/btc.h).

Argument marshalling only: every step of a contraction runs in the CUDA kernels of libbtc.so.
Importing this module loads the shared library and raises if it is missing; there is no other
code path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("BTC_LIB_PATH") or os.path.join(_HERE, "libbtc.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} not found: build the CUDA library first "
        "(python -m paper_2601_07827_b200.build, or __graft_entry__.build())")
_lib = ctypes.CDLL(LIB_PATH)

SUCCESS = 0
ERR_INVALID_ARGUMENT = 1
ERR_INVALID_EXTENT = 2
ERR_EXTENT_MISMATCH = 3
ERR_C_D_MISMATCH = 4
ERR_D_ALIASING = 5
ERR_LABEL_ONLY_IN_D = 6
ERR_NOT_SUPPORTED = 7
ERR_WORKSPACE_TOO_SMALL = 8
ERR_MISALIGNED = 9
ERR_CUDA = 10
ERR_DEVICE_TIMEOUT = 11
ERR_OUT_OF_MEMORY = 12
ERR_SCRATCH_LIMIT = 13

F32, F64, C32, C64 = 0, 1, 2, 3
DTYPE_SIZE = {F32: 4, F64: 8, C32: 8, C64: 16}

ATTR_KERNEL, ATTR_SPLIT_K, ATTR_TILE, ATTR_GROUPS, ATTR_GRID, ATTR_NUM_MODES, ATTR_SWAPPED = 1, 2, 3, 4, 5, 6, 7
ATTR_DEVICE_ERROR = 8
ATTR_VARIANT = 9
ATTR_PRE_REDUCE = 10
ATTR_BATCH_HINT = 11
ATTR_COMPUTE_PRECISION = 12
ATTR_POLL_LIMIT = 13
PRECISION_DEFAULT, PRECISION_STRICT, PRECISION_FP64_SUMS = 0, 1, 2
KERNEL_AUTO, KERNEL_GENERIC, KERNEL_TILED = 0, 1, 2
STATUS_KERNEL, STATUS_LAUNCHES, STATUS_GRID, STATUS_SPLIT_K, STATUS_VARIANT = 1, 2, 3, 4, 5

EXPORTED = [
    "btc_create_handle", "btc_destroy_handle", "btc_create_tensor_info", "btc_destroy_tensor_info",
    "btc_create_contraction", "btc_destroy_contraction", "btc_contraction_workspace_size",
    "btc_set_attr", "btc_get_attr", "btc_execute", "btc_execute_host", "btc_execute_static_scratch",
    "btc_execute_batched", "btc_contraction_batched_workspace_size",
    "btc_status_get",
    "btc_destroy_status", "btc_explain_error", "btc_selftest_bounded_wait", "btc_measure_peak",
    "btc_create_elementwise", "btc_destroy_elementwise", "btc_elementwise_execute", "btc_elementwise_get_attr",
]

_vp = ctypes.c_void_p
_i64p = ctypes.POINTER(ctypes.c_int64)
_lib.btc_create_handle.argtypes = [ctypes.POINTER(_vp)]
_lib.btc_destroy_handle.argtypes = [ctypes.POINTER(_vp)]
_lib.btc_create_tensor_info.argtypes = [_vp, ctypes.c_int, ctypes.c_int32, _i64p, _i64p, ctypes.POINTER(_vp)]
_lib.btc_destroy_tensor_info.argtypes = [ctypes.POINTER(_vp)]
_lib.btc_create_contraction.argtypes = [
    _vp, _vp, _i64p, ctypes.c_int, _vp, _i64p, ctypes.c_int, _vp, _i64p, ctypes.c_int, _vp, _i64p,
    _vp, _vp, ctypes.POINTER(_vp)]
_lib.btc_destroy_contraction.argtypes = [ctypes.POINTER(_vp)]
_lib.btc_contraction_workspace_size.argtypes = [_vp, ctypes.POINTER(ctypes.c_size_t)]
_lib.btc_set_attr.argtypes = [_vp, ctypes.c_int32, _vp, ctypes.c_size_t]
_lib.btc_get_attr.argtypes = [_vp, ctypes.c_int32, _vp, ctypes.c_size_t, ctypes.POINTER(ctypes.c_size_t)]
_lib.btc_execute.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, ctypes.c_size_t, ctypes.POINTER(_vp)]
_lib.btc_execute_host.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.btc_contraction_batched_workspace_size.argtypes = [_vp, ctypes.c_int64, ctypes.POINTER(ctypes.c_size_t)]
_lib.btc_execute_batched.argtypes = [_vp, _vp, _vp, ctypes.POINTER(_vp), ctypes.POINTER(_vp), _vp, ctypes.POINTER(_vp),
                                     ctypes.POINTER(_vp), ctypes.c_int64, _vp, ctypes.c_size_t]
_lib.btc_execute_static_scratch.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.btc_status_get.argtypes = [_vp, ctypes.c_int32, _vp, ctypes.c_size_t]
_lib.btc_destroy_status.argtypes = [ctypes.POINTER(_vp)]
_lib.btc_explain_error.argtypes = [ctypes.c_int, ctypes.c_char_p, ctypes.c_size_t, ctypes.POINTER(ctypes.c_size_t)]
_lib.btc_create_elementwise.argtypes = [_vp, _vp, _i64p, ctypes.c_int, _vp, ctypes.c_int, _vp, _i64p, _vp, _vp,
                                        ctypes.POINTER(_vp)]
_lib.btc_destroy_elementwise.argtypes = [ctypes.POINTER(_vp)]
_lib.btc_elementwise_execute.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp]
_lib.btc_elementwise_get_attr.argtypes = [_vp, ctypes.c_int32, _vp, ctypes.c_size_t, ctypes.POINTER(ctypes.c_size_t)]
_lib.btc_selftest_bounded_wait.argtypes = [_vp, _vp, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32),
                                           ctypes.POINTER(ctypes.c_int32)]
_lib.btc_measure_peak.argtypes = [_vp, ctypes.c_int32, _vp, _vp, ctypes.c_size_t, ctypes.c_int32, ctypes.POINTER(ctypes.c_double)]
for _name in EXPORTED:
    getattr(_lib, _name).restype = ctypes.c_int

PEAK_FP64_FMA, PEAK_FP32_FMA, PEAK_FP64_MMA_K16, PEAK_FP64_MMA_K4, PEAK_TF32_MMA_SYNC = 0, 1, 2, 3, 4
PEAK_HBM_READ, PEAK_HBM_WRITE, PEAK_HBM_COPY = 5, 6, 7


def measure_peak(handle, which: int, stream: int = 0, buffer: int = 0, nbytes: int = 0, repeats: int = 3) -> float:
    """flop/s or byte/s this device sustains on one pipe or on its memory (see btc_measure_peak)."""
    out = ctypes.c_double(0.0)
    _check(_lib.btc_measure_peak(handle._h, which, stream or None, buffer or None, nbytes, repeats, ctypes.byref(out)),
           "btc_measure_peak")
    return out.value


def selftest_bounded_wait(handle, stream: int = 0, polls: int = 1000):
    """Runs the device-side bounded-wait self-test; returns (error code recorded, threads that gave up)."""
    code, count = ctypes.c_int32(0), ctypes.c_int32(0)
    _check(_lib.btc_selftest_bounded_wait(handle._h, stream or None, polls, ctypes.byref(code), ctypes.byref(count)),
           "btc_selftest_bounded_wait")
    return code.value, count.value


def explain_error(code: int) -> str:
    need = ctypes.c_size_t(0)
    _lib.btc_explain_error(code, None, 0, ctypes.byref(need))
    buf = ctypes.create_string_buffer(need.value)
    _lib.btc_explain_error(code, buf, need.value, None)
    return buf.value.decode()


class BtcError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: error {code}: {explain_error(code)}")
        self.code = code


def _check(code: int, where: str) -> None:
    if code != SUCCESS:
        raise BtcError(code, where)


def _labels(labels) -> list:
    if isinstance(labels, str):
        return [ord(c) for c in labels]
    return [ord(x) if isinstance(x, str) else int(x) for x in labels]


def _i64_array(values: Optional[Sequence[int]]):
    if values is None:
        return None
    vals = list(values)
    return (ctypes.c_int64 * max(len(vals), 1))(*vals)


def _scalar(dtype: int, value) -> Optional[ctypes.Array]:
    if value is None:
        return None
    z = complex(value)
    if dtype == F32:
        return (ctypes.c_float * 1)(z.real)
    if dtype == F64:
        return (ctypes.c_double * 1)(z.real)
    if dtype == C32:
        return (ctypes.c_float * 2)(z.real, z.imag)
    return (ctypes.c_double * 2)(z.real, z.imag)


class Handle:
    def __init__(self):
        self._h = _vp()
        _check(_lib.btc_create_handle(ctypes.byref(self._h)), "btc_create_handle")

    def close(self):
        if self._h:
            _lib.btc_destroy_handle(ctypes.byref(self._h))

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class TensorInfo:
    def __init__(self, handle: Handle, dtype: int, extents: Sequence[int], strides: Optional[Sequence[int]] = None):
        self.dtype, self.extents = dtype, tuple(extents)
        self.strides = None if strides is None else tuple(strides)
        self._t = _vp()
        _check(_lib.btc_create_tensor_info(handle._h, dtype, len(self.extents), _i64_array(self.extents),
                                           _i64_array(self.strides), ctypes.byref(self._t)),
               "btc_create_tensor_info")

    def close(self):
        if self._t:
            _lib.btc_destroy_tensor_info(ctypes.byref(self._t))

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Contraction:
    """A validated, planned contraction; execute() enqueues it on a CUDA stream."""

    def __init__(self, handle: Handle, A: TensorInfo, labelsA, B: TensorInfo, labelsB,
                 C: Optional[TensorInfo], labelsC, D: TensorInfo, labelsD,
                 alpha=None, beta=None, conjA=False, conjB=False, conjC=False):
        self.dtype = D.dtype
        self._op = _vp()
        _check(_lib.btc_create_contraction(
            handle._h, A._t, _i64_array(_labels(labelsA)), int(conjA), B._t, _i64_array(_labels(labelsB)),
            int(conjB), C._t if C is not None else None,
            _i64_array(_labels(labelsC)) if C is not None else None, int(conjC),
            D._t, _i64_array(_labels(labelsD)), _scalar(self.dtype, alpha), _scalar(self.dtype, beta),
            ctypes.byref(self._op)), "btc_create_contraction")

    def workspace_size(self) -> int:
        n = ctypes.c_size_t(0)
        _check(_lib.btc_contraction_workspace_size(self._op, ctypes.byref(n)), "btc_contraction_workspace_size")
        return n.value

    def _get(self, key, ctype, count):
        buf = (ctype * count)()
        _check(_lib.btc_get_attr(self._op, key, buf, ctypes.sizeof(buf), None), "btc_get_attr")
        return list(buf)

    @property
    def kernel(self) -> int:
        return self._get(ATTR_KERNEL, ctypes.c_int32, 1)[0]

    @property
    def split_k(self) -> int:
        return self._get(ATTR_SPLIT_K, ctypes.c_int32, 1)[0]

    @property
    def tile(self):
        return tuple(self._get(ATTR_TILE, ctypes.c_int32, 3))

    @property
    def groups(self):
        """(batch, M, N, K) sizes after classification."""
        return tuple(self._get(ATTR_GROUPS, ctypes.c_int64, 4))

    @property
    def grid(self):
        return tuple(self._get(ATTR_GRID, ctypes.c_int32, 3))

    @property
    def num_modes(self):
        return tuple(self._get(ATTR_NUM_MODES, ctypes.c_int32, 4))

    @property
    def swapped(self) -> bool:
        return bool(self._get(ATTR_SWAPPED, ctypes.c_int32, 1)[0])

    @property
    def variant(self) -> int:
        return self._get(ATTR_VARIANT, ctypes.c_int32, 1)[0]

    @property
    def pre_reduce(self) -> int:
        """Case 4: bit 0 / bit 1 set when A / B is summed over its isolated labels before the contraction."""
        return self._get(ATTR_PRE_REDUCE, ctypes.c_int32, 1)[0]

    @property
    def device_error(self) -> int:
        """0, or the code of a bounded device-side wait that gave up (waits for the device)."""
        return self._get(ATTR_DEVICE_ERROR, ctypes.c_int32, 1)[0]

    def set_attr(self, key: int, value: int) -> None:
        v = ctypes.c_int32(value)
        _check(_lib.btc_set_attr(self._op, key, ctypes.byref(v), 4), "btc_set_attr")

    def execute(self, stream: int, A: int, B: int, C: Optional[int], D: int, alpha=None, beta=None,
                workspace: int = 0, workspace_bytes: int = 0, want_status: bool = False):
        """Device pointers as integers; stream is a cudaStream_t value (0 = default stream)."""
        st = _vp()
        rc = _lib.btc_execute(self._op, stream or None, _scalar(self.dtype, alpha), A or None, B or None,
                              _scalar(self.dtype, beta), C or None, D or None, workspace or None,
                              workspace_bytes, ctypes.byref(st) if want_status else None)
        _check(rc, "btc_execute")
        if want_status:
            out = {}
            for name, key, n in (("kernel", STATUS_KERNEL, 1), ("launches", STATUS_LAUNCHES, 1),
                                 ("grid", STATUS_GRID, 3), ("split_k", STATUS_SPLIT_K, 1), ("variant", STATUS_VARIANT, 1)):
                buf = (ctypes.c_int32 * n)()
                _check(_lib.btc_status_get(st, key, buf, ctypes.sizeof(buf)), "btc_status_get")
                out[name] = list(buf) if n > 1 else buf[0]
            _lib.btc_destroy_status(ctypes.byref(st))
            return out
        return None

    def batched_workspace_size(self, count: int) -> int:
        n = ctypes.c_size_t(0)
        _check(_lib.btc_contraction_batched_workspace_size(self._op, count, ctypes.byref(n)),
               "btc_contraction_batched_workspace_size")
        return int(n.value)

    def execute_batched(self, stream: int, A: Sequence[int], B: Sequence[int], C: Optional[Sequence[int]], D: Sequence[int],
                        alpha=None, beta=None, workspace: int = 0, workspace_bytes: int = 0) -> None:
        """Pointer arrays (device pointers as integers), one entry per execution; see btc_execute_batched."""
        n = len(D)
        arr = lambda ps: (_vp * n)(*[p or None for p in ps]) if ps is not None else None
        _check(_lib.btc_execute_batched(self._op, stream or None, _scalar(self.dtype, alpha), arr(A), arr(B),
                                        _scalar(self.dtype, beta), arr(C), arr(D), n, workspace or None, workspace_bytes),
               "btc_execute_batched")

    def execute_host(self, stream: int, A: int, B: int, C: Optional[int], D: int, alpha=None, beta=None):
        """Host pointers as integers; copies in, runs, copies D back, synchronises."""
        _check(_lib.btc_execute_host(self._op, stream or None, _scalar(self.dtype, alpha), A or None, B or None,
                                     _scalar(self.dtype, beta), C or None, D or None), "btc_execute_host")

    def execute_static_scratch(self, stream: int, A: int, B: int, C: Optional[int], D: int, alpha=None, beta=None):
        """Like execute() with device pointers, for callers that can neither allocate device
        memory nor bring a workspace: split-K scratch comes from the library's built-in 8 MiB
        device array.  Calls that could overlap on the GPU must be serialised by the caller;
        operations that need more scratch raise ERR_SCRATCH_LIMIT."""
        _check(_lib.btc_execute_static_scratch(self._op, stream or None, _scalar(self.dtype, alpha), A or None,
                                               B or None, _scalar(self.dtype, beta), C or None, D or None),
               "btc_execute_static_scratch")

    def close(self):
        if self._op:
            _lib.btc_destroy_contraction(ctypes.byref(self._op))

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


_TORCH_DTYPE = None


def dtype_code(torch_dtype) -> int:
    global _TORCH_DTYPE
    if _TORCH_DTYPE is None:
        import torch
        _TORCH_DTYPE = {torch.float32: F32, torch.float64: F64, torch.complex64: C32, torch.complex128: C64}
    return _TORCH_DTYPE[torch_dtype]


EW_ATTR_KERNEL, EW_ATTR_NUM_MODES, EW_ATTR_LAST_KERNEL = 1, 2, 3
EW_KERNEL_DIRECT, EW_KERNEL_TRANSPOSING, EW_KERNEL_VECTOR = 1, 2, 3


class Elementwise:
    """C := alpha op(A) + beta op(B); B (a TensorInfo or None) carries C's labels."""

    def __init__(self, handle: Handle, A: "TensorInfo", labelsA, B: Optional["TensorInfo"], C: "TensorInfo", labelsC,
                 alpha=1.0, beta=0.0, conjA=False, conjB=False):
        self.dtype = C.dtype
        la, lc = _labels(labelsA), _labels(labelsC)
        self._op = _vp()
        _check(_lib.btc_create_elementwise(
            handle._h, A._t, (ctypes.c_int64 * max(len(la), 1))(*la), int(conjA), B._t if B is not None else None,
            int(conjB), C._t, (ctypes.c_int64 * max(len(lc), 1))(*lc), _scalar(self.dtype, alpha),
            _scalar(self.dtype, beta), ctypes.byref(self._op)), "btc_create_elementwise")
        self._keepalive = (handle, A, B, C)

    def _get(self, key, n):
        buf = (ctypes.c_int32 * n)()
        _check(_lib.btc_elementwise_get_attr(self._op, key, buf, ctypes.sizeof(buf), None), "btc_elementwise_get_attr")
        return list(buf)

    @property
    def kernel(self) -> int:
        return self._get(EW_ATTR_KERNEL, 1)[0]

    @property
    def kernel_ran(self) -> int:
        """The kernel the last execute launched (0 before the first)."""
        return self._get(EW_ATTR_LAST_KERNEL, 1)[0]

    @property
    def num_modes(self):
        return tuple(self._get(EW_ATTR_NUM_MODES, 2))

    def execute(self, stream: int, A: int, B: Optional[int], C: int, alpha=None, beta=None) -> None:
        _check(_lib.btc_elementwise_execute(self._op, stream or None, _scalar(self.dtype, alpha), A or None,
                                            _scalar(self.dtype, beta), B or None, C or None), "btc_elementwise_execute")

    def close(self):
        if self._op:
            _lib.btc_destroy_elementwise(ctypes.byref(self._op))

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def elementwise(handle: Handle, A, labelsA, B, C, labelsC, alpha=1.0, beta=0.0, conjA=False, conjB=False, stream: int = 0):
    """One-shot helper like ``contract`` for tensors with .dtype, .extents, .strides, .data_ptr()."""
    tA = TensorInfo(handle, dtype_code(A.dtype), A.extents, A.strides)
    tB = TensorInfo(handle, dtype_code(B.dtype), B.extents, B.strides) if B is not None else None
    tC = TensorInfo(handle, dtype_code(C.dtype), C.extents, C.strides)
    op = Elementwise(handle, tA, labelsA, tB, tC, labelsC, alpha, beta, conjA, conjB)
    op.execute(stream, A.data_ptr(), B.data_ptr() if B is not None else 0, C.data_ptr())
    return op


def contract(handle: Handle, A, labelsA, B, labelsB, C, D, labelsD, alpha=1.0, beta=0.0,
             conjA=False, conjB=False, conjC=False, stream: int = 0, kernel: int = KERNEL_AUTO,
             split_k: int = 0, want_status: bool = False, variant: int = -1, pre_reduce: Optional[bool] = None):
    """One-shot helper for tensors described by objects with .dtype, .extents, .strides and
    .data_ptr() (device memory): builds the descriptors and the operation, allocates the
    workspace with torch, executes on `stream`.  Returns (Contraction, status-or-None)."""
    import torch
    dt = dtype_code(D.dtype)
    tA = TensorInfo(handle, dtype_code(A.dtype), A.extents, A.strides)
    tB = TensorInfo(handle, dtype_code(B.dtype), B.extents, B.strides)
    tD = TensorInfo(handle, dt, D.extents, D.strides)
    tC = TensorInfo(handle, dtype_code(C.dtype), C.extents, C.strides) if C is not None else None
    op = Contraction(handle, tA, labelsA, tB, labelsB, tC, labelsD, tD, labelsD, alpha, beta, conjA, conjB, conjC)
    if pre_reduce is not None:
        op.set_attr(ATTR_PRE_REDUCE, int(pre_reduce))
    if kernel != KERNEL_AUTO:
        op.set_attr(ATTR_KERNEL, kernel)
    if split_k:
        op.set_attr(ATTR_SPLIT_K, split_k)
    if variant >= 0:
        op.set_attr(ATTR_VARIANT, variant)
    ws_bytes = op.workspace_size()
    ws = torch.empty(max(ws_bytes, 1), dtype=torch.uint8, device="cuda") if ws_bytes else None
    st = op.execute(stream, A.data_ptr(), B.data_ptr(), C.data_ptr() if C is not None else 0, D.data_ptr(),
                    workspace=ws.data_ptr() if ws is not None else 0, workspace_bytes=ws_bytes,
                    want_status=want_status)
    op._keepalive = (ws, tA, tB, tC, tD)
    return op, st
