"""ctypes binding of libspmm_b200.so: same names as the C ABI, argument marshalling only.

Every step of the SpMM path runs inside the CUDA library; nothing here
computes.  The library is loaded when this module is imported and a missing
library is an ImportError (there is no fallback of any kind).  Device
pointers are plain integers (``tensor.data_ptr()``), streams are the integer
handle of a CUDA stream (``torch.cuda.current_stream().cuda_stream``) or 0.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("SPMM_B200_LIB") or os.path.join(_HERE, "libspmm_b200.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        "%s is missing: build it with `python -m paper_2604_17834_b200.build` "
        "(there is no CPU fallback)" % LIB_PATH)
_lib = ctypes.CDLL(LIB_PATH)

SPMM_BF16, SPMM_FP16, SPMM_TF32, SPMM_FP8_E4M3 = 0, 1, 2, 3
DTYPE_CODE = {"bf16": SPMM_BF16, "fp16": SPMM_FP16, "tf32": SPMM_TF32, "fp8": SPMM_FP8_E4M3}

SPMM_OK = 0
SPMM_ERR_INVALID_ARG = -1
SPMM_ERR_UNSORTED = -2
SPMM_ERR_OUT_OF_RANGE = -3
SPMM_ERR_UNSUPPORTED = -4
SPMM_ERR_ALLOC = -5
SPMM_ERR_CUDA = -6
SPMM_ERR_DEV_TIMEOUT = -7
SPMM_ERR_HOST_ONLY = -8
SPMM_ERR_TOO_LARGE = -9
SPMM_ERR_DEV_BOUNDS = -10
SPMM_ERR_DEV_UNDRAINED = -11

X_BCSR_BLOCK_ROW_PTR, X_BCSR_BLOCK_COL_IDX, X_BCSR_BLOCKS, X_BCSR_ROW_ORDER = 0, 1, 2, 3
X_BCSR_TILE_PTR, X_BCSR_TILES = 4, 5
X_BCSR_STACK_ROWS, X_BCSR_STACK_PTR, X_BCSR_STACK_COL_IDX, X_BCSR_STACK_TILE_PTR, X_BCSR_STACK_TILES = 6, 7, 8, 9, 20
X_BCSR_UNITS = 21
X_WCSR_WINDOW_ROW_PTR, X_WCSR_WINDOW_COL_IDX, X_WCSR_VALUES, X_WCSR_TASKS = 10, 11, 12, 13
X_WCSR_BIN_PTR, X_WCSR_BIN_TASKS, X_WCSR_GROUP_CLASS = 14, 15, 16

EXPORTED_SYMBOLS = (
    "spmm_bcsr_create_csr", "spmm_bcsr_create_csr_device", "spmm_bcsr_create_coo", "spmm_wcsr_create_csr",
    "spmm_wcsr_create_csr_device", "spmm_wcsr_create_coo",
    "spmm_bcsr_plan", "spmm_prepare", "spmm_run", "spmm_wcsr_run_static", "spmm_run_host", "spmm_check", "spmm_get_info", "spmm_export", "spmm_destroy",
    "spmm_status_string", "spmm_set_wait_limit_ns",
)


class SpmmOpts(ctypes.Structure):
    _fields_ = [("b_col", ctypes.c_int32), ("split_cols", ctypes.c_int32), ("host_only", ctypes.c_int32),
                ("n_ctas", ctypes.c_int32), ("c_type", ctypes.c_int32), ("layout", ctypes.c_int32),
                ("schedule", ctypes.c_int32), ("stack_min_fill", ctypes.c_int32), ("gather", ctypes.c_int32), ("k_split", ctypes.c_int32),
                ("reserved", ctypes.c_int32 * 6)]


class SpmmInfo(ctypes.Structure):
    _fields_ = [
        ("format", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("m", ctypes.c_int64), ("k", ctypes.c_int64), ("nnz", ctypes.c_int64),
        ("block", ctypes.c_int32), ("b_col", ctypes.c_int32),
        ("n_units", ctypes.c_int64), ("stored_values", ctypes.c_int64),
        ("fill_ratio", ctypes.c_double),
        ("n_rows_units", ctypes.c_int64), ("n_empty", ctypes.c_int64),
        ("n_tasks", ctypes.c_int64), ("n_split", ctypes.c_int64), ("n_slots", ctypes.c_int64),
        ("split_cols", ctypes.c_int32), ("n_ctas", ctypes.c_int32),
        ("distinct_b_rows", ctypes.c_int64),
        ("bytes_a", ctypes.c_double), ("bytes_idx", ctypes.c_double),
        ("bytes_b_touched", ctypes.c_double), ("bytes_c", ctypes.c_double),
        ("bytes_gather", ctypes.c_double), ("flops_stored", ctypes.c_double),
        ("workspace_bytes", ctypes.c_int64),
        ("plan_n", ctypes.c_int64), ("plan_token_tile", ctypes.c_int32), ("plan_slab_tiles", ctypes.c_int32),
        ("n_bins", ctypes.c_int32), ("n_stacked_rows", ctypes.c_int32), ("n_stack_blocks", ctypes.c_int64),
    ]

    def as_dict(self):
        return {name: getattr(self, name) for name, _ in self._fields_}


_vp, _i64, _i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
_lib.spmm_bcsr_create_csr.argtypes = [ctypes.POINTER(_vp), _i64, _i64, _vp, _vp, _vp, _i32, _i32, ctypes.POINTER(SpmmOpts)]
_lib.spmm_wcsr_create_csr.argtypes = _lib.spmm_bcsr_create_csr.argtypes
_lib.spmm_bcsr_create_csr_device.argtypes = [ctypes.POINTER(_vp), _i64, _i64, _vp, _vp, _vp, _i32, _i32, ctypes.POINTER(SpmmOpts), _vp]
_lib.spmm_wcsr_create_csr_device.argtypes = _lib.spmm_bcsr_create_csr_device.argtypes
_lib.spmm_bcsr_create_coo.argtypes = [ctypes.POINTER(_vp), _i64, _i64, _i64, _vp, _vp, _vp, _i32, _i32, ctypes.POINTER(SpmmOpts)]
_lib.spmm_wcsr_create_coo.argtypes = _lib.spmm_bcsr_create_coo.argtypes
_lib.spmm_run.argtypes = [_vp, _vp, _vp, _i64, _vp]
_lib.spmm_bcsr_plan.argtypes = [_vp, _i64]
_lib.spmm_prepare.argtypes = [_vp, _i64]
_lib.spmm_run_host.argtypes = [_vp, _vp, _vp, _i64, _vp]
_lib.spmm_wcsr_run_static.argtypes = [_vp, _vp, _vp, _i64, _vp]
_lib.spmm_check.argtypes = [_vp]
_lib.spmm_get_info.argtypes = [_vp, _i64, ctypes.POINTER(SpmmInfo)]
_lib.spmm_export.argtypes = [_vp, _i32, _vp, ctypes.c_size_t, ctypes.POINTER(ctypes.c_size_t)]
_lib.spmm_destroy.argtypes = [_vp]
_lib.spmm_status_string.argtypes = [_i32]
_lib.spmm_status_string.restype = ctypes.c_char_p
_lib.spmm_set_wait_limit_ns.argtypes = [ctypes.c_uint64]
for _n in EXPORTED_SYMBOLS:
    if _n != "spmm_status_string":
        getattr(_lib, _n).restype = ctypes.c_int


class SpmmError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__("%s: %s (%d)" % (where, spmm_status_string(code), code))


def spmm_status_string(code):
    return _lib.spmm_status_string(int(code)).decode()


C_FP32, C_SAME_AS_INPUT = 0, 1
ROWMAJOR, COLMAJOR = 0, 1


SCHED_STATIC, SCHED_DYNAMIC = 0, 1
GATHER_TMA, GATHER_LSU = 0, 1


def _opts(b_col=0, split_cols=0, host_only=False, n_ctas=0, c_type=C_FP32, layout=ROWMAJOR, schedule=SCHED_STATIC,
          stack_min_fill=0, gather=GATHER_TMA, k_split=0):
    """Keyword options of the create functions -> spmm_opts_t (zero = the library's default; the
    header documents every field).  stack_min_fill: BCSR row groups, 0 = default threshold,
    -1 = off, 1..100 = minimum percentage of stored sub-blocks for a group to be formed."""
    o = SpmmOpts()
    o.stack_min_fill = int(stack_min_fill)
    o.gather = int(gather)
    o.k_split = int(k_split)
    o.b_col, o.split_cols, o.host_only, o.n_ctas = b_col, split_cols, int(bool(host_only)), n_ctas
    o.c_type, o.layout, o.schedule = int(c_type), int(layout), int(schedule)
    return o


def _vals_buffer(vals, dtype):
    want = {"bf16": np.uint16, "fp16": np.float16, "tf32": np.float32, "fp8": np.uint8}[dtype]
    v = np.ascontiguousarray(vals)
    if v.dtype != want:
        raise TypeError("vals for %s must be %s (raw storage), got %s" % (dtype, want.__name__, v.dtype))
    return v


def _create_csr(fn, name, m, k, row_ptr, col_idx, vals, dtype, size, opts):
    rp = np.ascontiguousarray(row_ptr, dtype=np.int64)
    ci = np.ascontiguousarray(col_idx, dtype=np.int32)
    v = _vals_buffer(vals, dtype)
    if rp.shape[0] != m + 1 or (m >= 0 and rp.shape[0] and ci.shape[0] != v.shape[0]):
        raise ValueError("array lengths do not match m / nnz")
    h = _vp()
    rc = fn(ctypes.byref(h), m, k, rp.ctypes.data, ci.ctypes.data, v.ctypes.data, DTYPE_CODE[dtype], size,
            ctypes.byref(opts))
    if rc != SPMM_OK:
        raise SpmmError(rc, name)
    return h


def spmm_bcsr_create_csr(m, k, row_ptr, col_idx, vals, dtype, block, **opt):
    """-> handle.  Host CSR arrays (vals in raw storage dtype) -> BCSR with block x block tiles."""
    return _create_csr(_lib.spmm_bcsr_create_csr, "spmm_bcsr_create_csr", m, k, row_ptr, col_idx, vals, dtype, block,
                       _opts(**opt))


def spmm_bcsr_create_csr_device(m, k, row_ptr_dev, col_idx_dev, vals_dev, dtype, block, stream=0, **opt):
    """-> handle.  CSR arrays in device memory (integer addresses: int64 row_ptr, int32 col_idx, values in
    raw storage dtype) -> BCSR built by GPU kernels."""
    h = _vp()
    o = _opts(**opt)
    rc = _lib.spmm_bcsr_create_csr_device(ctypes.byref(h), m, k, _vp(int(row_ptr_dev)), _vp(int(col_idx_dev)),
                                          _vp(int(vals_dev)), DTYPE_CODE[dtype], block, ctypes.byref(o), _vp(stream))
    if rc != SPMM_OK:
        raise SpmmError(rc, "spmm_bcsr_create_csr_device")
    return h


def spmm_wcsr_create_csr_device(m, k, row_ptr_dev, col_idx_dev, vals_dev, dtype, window_height=16, stream=0, **opt):
    """-> handle.  CSR arrays in device memory -> WCSR built by GPU kernels."""
    h = _vp()
    o = _opts(**opt)
    rc = _lib.spmm_wcsr_create_csr_device(ctypes.byref(h), m, k, _vp(int(row_ptr_dev)), _vp(int(col_idx_dev)),
                                          _vp(int(vals_dev)), DTYPE_CODE[dtype], window_height, ctypes.byref(o), _vp(stream))
    if rc != SPMM_OK:
        raise SpmmError(rc, "spmm_wcsr_create_csr_device")
    return h


def spmm_wcsr_create_csr(m, k, row_ptr, col_idx, vals, dtype, window_height=16, **opt):
    """-> handle.  Host CSR arrays -> WCSR with the given window height."""
    return _create_csr(_lib.spmm_wcsr_create_csr, "spmm_wcsr_create_csr", m, k, row_ptr, col_idx, vals, dtype,
                       window_height, _opts(**opt))


def _create_coo(fn, name, m, k, rows, cols, vals, dtype, size, opts):
    r = np.ascontiguousarray(rows, dtype=np.int32)
    c = np.ascontiguousarray(cols, dtype=np.int32)
    v = _vals_buffer(vals, dtype)
    if not (r.shape[0] == c.shape[0] == v.shape[0]):
        raise ValueError("COO arrays differ in length")
    h = _vp()
    rc = fn(ctypes.byref(h), m, k, r.shape[0], r.ctypes.data, c.ctypes.data, v.ctypes.data, DTYPE_CODE[dtype], size,
            ctypes.byref(opts))
    if rc != SPMM_OK:
        raise SpmmError(rc, name)
    return h


def spmm_bcsr_create_coo(m, k, rows, cols, vals, dtype, block, **opt):
    return _create_coo(_lib.spmm_bcsr_create_coo, "spmm_bcsr_create_coo", m, k, rows, cols, vals, dtype, block,
                       _opts(**opt))


def spmm_wcsr_create_coo(m, k, rows, cols, vals, dtype, window_height=16, **opt):
    return _create_coo(_lib.spmm_wcsr_create_coo, "spmm_wcsr_create_coo", m, k, rows, cols, vals, dtype,
                       window_height, _opts(**opt))


def spmm_bcsr_plan(h, N):
    """BCSR: build and keep the tile schedule spmm_run would use for dense width N."""
    rc = _lib.spmm_bcsr_plan(h, N)
    if rc != SPMM_OK:
        raise SpmmError(rc, "spmm_bcsr_plan")


def spmm_prepare(h, N):
    """Both formats: allocate and plan now what the first spmm_run at dense width N would."""
    rc = _lib.spmm_prepare(h, N)
    if rc != SPMM_OK:
        raise SpmmError(rc, "spmm_prepare")


def spmm_run(h, B_dev_ptr, C_dev_ptr, N, stream=0):
    """Asynchronous C = A x B on device pointers (integers)."""
    rc = _lib.spmm_run(h, _vp(B_dev_ptr), _vp(C_dev_ptr), N, _vp(stream))
    if rc != SPMM_OK:
        raise SpmmError(rc, "spmm_run")


def spmm_wcsr_run_static(h, B_dev_ptr, C_dev_ptr, N, stream=0):
    """WCSR only: like spmm_run, but allocates nothing -- the partial tiles of split windows
    use the 8 MiB scratch array built into the library.  For callers that may not allocate
    device memory when they call (a framework's pool owns the device, or an allocation's
    synchronisation is not acceptable).  Raises SpmmError(SPMM_ERR_TOO_LARGE) when the
    partial tiles do not fit; calls that overlap on the GPU race on the shared array."""
    rc = _lib.spmm_wcsr_run_static(h, _vp(B_dev_ptr), _vp(C_dev_ptr), N, _vp(stream))
    if rc != SPMM_OK:
        raise SpmmError(rc, "spmm_wcsr_run_static")


def spmm_run_host(h, B_host, C_host, N, stream=0):
    """C = A x B with host buffers (numpy arrays or integer addresses); returns after the copy back."""
    bp = B_host.ctypes.data if isinstance(B_host, np.ndarray) else int(B_host)
    cp = C_host.ctypes.data if isinstance(C_host, np.ndarray) else int(C_host)
    rc = _lib.spmm_run_host(h, _vp(bp), _vp(cp), N, _vp(stream))
    if rc != SPMM_OK:
        raise SpmmError(rc, "spmm_run_host")


def spmm_check(h):
    rc = _lib.spmm_check(h)
    if rc != SPMM_OK:
        raise SpmmError(rc, "spmm_check")


def spmm_get_info(h, N=0):
    info = SpmmInfo()
    rc = _lib.spmm_get_info(h, N, ctypes.byref(info))
    if rc != SPMM_OK:
        raise SpmmError(rc, "spmm_get_info")
    return info.as_dict()


def spmm_export(h, which, np_dtype):
    """Canonical array `which` as a flat numpy array of np_dtype."""
    need = ctypes.c_size_t(0)
    rc = _lib.spmm_export(h, which, None, 0, ctypes.byref(need))
    if rc != SPMM_OK:
        raise SpmmError(rc, "spmm_export")
    out = np.empty(need.value // np.dtype(np_dtype).itemsize, dtype=np_dtype)
    if need.value:
        rc = _lib.spmm_export(h, which, out.ctypes.data, need.value, ctypes.byref(need))
        if rc != SPMM_OK:
            raise SpmmError(rc, "spmm_export")
    return out


def spmm_destroy(h):
    _lib.spmm_destroy(h)


def spmm_set_wait_limit_ns(ns):
    _lib.spmm_set_wait_limit_ns(int(ns))
