"""ctypes front-end of ``conv_oracle.c`` and ``stencil_oracle.c`` (TEST INFRASTRUCTURE ONLY).

Compiles the C files with gcc on first use (``-O2 -fopenmp``) into
``oracle/_build/liboracle.so`` and exposes numpy-in / numpy-out functions.
Argument checking and array allocation only; every sum is formed in the C file.
"""
import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRCS = [os.path.join(_HERE, "conv_oracle.c"), os.path.join(_HERE, "stencil_oracle.c")]
_OUT_DIR = os.path.join(_HERE, "_build")
_LIB_PATH = os.path.join(_OUT_DIR, "liboracle.so")
_lock = threading.Lock()
_lib = None

_c_ll = ctypes.c_longlong
_c_int = ctypes.c_int
_vp = ctypes.c_void_p


def build_oracle(force: bool = False) -> str:
    """Compile the C oracle if the shared object is missing or stale."""
    os.makedirs(_OUT_DIR, exist_ok=True)
    stale = (not os.path.exists(_LIB_PATH)
             or os.path.getmtime(_LIB_PATH) < max(os.path.getmtime(p) for p in _SRCS))
    if force or stale:
        tmp = _LIB_PATH + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
               "-o", tmp] + _SRCS + ["-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build_oracle())
            lib.oracle_num_threads.restype = _c_int
            lib.oracle_set_num_threads.argtypes = [_c_int]
            lib.oracle_conv1d_f32.argtypes = [_vp, _c_ll, _vp, _c_int, _vp, _vp]
            lib.oracle_conv1d_f32_taps_outer.argtypes = [_vp, _c_ll, _vp, _c_int, _vp]
            lib.oracle_conv1d_f32_at.argtypes = [_vp, _c_ll, _vp, _c_int, _vp, _c_ll, _vp, _vp]
            lib.oracle_conv2d_f32.argtypes = [_vp, _c_int, _c_int, _c_ll, _vp, _c_int, _c_int,
                                              _vp, _vp, _c_ll]
            lib.oracle_conv1d_f32_strided.argtypes = [_vp, _c_ll, _vp, _c_int, _c_int, _vp, _vp]
            lib.oracle_conv2d_f32_strided.argtypes = [_vp, _c_int, _c_int, _c_ll, _vp, _c_int, _c_int,
                                                      _c_int, _c_int, _vp, _vp, _c_ll]
            lib.oracle_conv2d_f32_taps_outer.argtypes = [_vp, _c_int, _c_int, _c_ll, _vp, _c_int,
                                                         _c_int, _vp, _c_ll]
            lib.oracle_conv2d_f32_at.argtypes = [_vp, _c_int, _c_int, _c_ll, _vp, _c_int, _c_int,
                                                 _vp, _vp, _c_ll, _vp, _vp]
            lib.oracle_conv1d_u8s8_s32.argtypes = [_vp, _c_ll, _vp, _c_int, _vp]
            lib.oracle_conv2d_u8s8_s32.argtypes = [_vp, _c_int, _c_int, _c_ll, _vp, _c_int, _c_int,
                                                   _vp, _c_ll]
            lib.oracle_conv2d_u8s8_i64.argtypes = [_vp, _c_int, _c_int, _c_ll, _vp, _c_int, _c_int,
                                                   _vp, _c_ll]
            lib.oracle_stencil2d_f32.argtypes = [_vp, _c_int, _c_int, _c_ll, _vp, _c_int, _vp, _vp]
            lib.oracle_stencil2d_f32.restype = _c_int
            for name in ("oracle_set_num_threads", "oracle_conv1d_f32",
                         "oracle_conv1d_f32_taps_outer", "oracle_conv1d_f32_at",
                         "oracle_conv2d_f32", "oracle_conv2d_f32_taps_outer",
                         "oracle_conv2d_f32_at", "oracle_conv1d_u8s8_s32",
                         "oracle_conv2d_u8s8_s32", "oracle_conv2d_u8s8_i64",
                         "oracle_conv1d_f32_strided", "oracle_conv2d_f32_strided"):
                getattr(lib, name).restype = None
            _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(_vp)


def _as(a, dtype, ndim):
    a = np.ascontiguousarray(a, dtype=dtype)
    if a.ndim != ndim:
        raise ValueError("expected %d-D array, got %d-D" % (ndim, a.ndim))
    return a


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(int(n))


def conv1d_f32(x, w, want_scale=True):
    """Eq. 2 in fp64. Returns (y, S) with S = sum |w||x| per output (or None)."""
    x = _as(x, np.float32, 1)
    w = _as(w, np.float32, 1)
    n, q = x.shape[0], w.shape[0]
    if q < 1 or n < q:
        raise ValueError("need 1 <= Q <= N")
    y = np.empty(n - q + 1, dtype=np.float64)
    s = np.empty(n - q + 1, dtype=np.float64) if want_scale else None
    _load().oracle_conv1d_f32(_ptr(x), n, _ptr(w), q, _ptr(y), _ptr(s) if want_scale else None)
    return y, s


def conv1d_f32_strided(x, w, stride, want_scale=True):
    """Strided Eq. 2, y[c] = sum_q w[q] x[stride*c+q] (Table 2, stride-2 FBS cell) in fp64. Returns (y, S)."""
    x = _as(x, np.float32, 1)
    w = _as(w, np.float32, 1)
    n, q = x.shape[0], w.shape[0]
    if q < 1 or n < q or stride < 1:
        raise ValueError("need 1 <= Q <= N and stride >= 1")
    c = (n - q) // stride + 1
    y = np.empty(c, dtype=np.float64)
    s = np.empty(c, dtype=np.float64) if want_scale else None
    _load().oracle_conv1d_f32_strided(_ptr(x), n, _ptr(w), q, int(stride), _ptr(y),
                                      _ptr(s) if want_scale else None)
    return y, s


def conv2d_f32_strided(x, w, stride, want_scale=True):
    """Strided Eq. 3, y[r][c] = sum w[p][q] x[sr*r+p][sc*c+q]; stride = (sr, sc) or one int. Returns (y, S)."""
    x = _as(x, np.float32, 2)
    w = _as(w, np.float32, 2)
    sr, sc = (stride, stride) if np.isscalar(stride) else stride
    (h, wd), (p, q) = x.shape, w.shape
    if p < 1 or q < 1 or h < p or wd < q or sr < 1 or sc < 1:
        raise ValueError("need 1 <= P <= H, 1 <= Q <= W and strides >= 1")
    oh, ow = (h - p) // sr + 1, (wd - q) // sc + 1
    y = np.empty((oh, ow), dtype=np.float64)
    s = np.empty((oh, ow), dtype=np.float64) if want_scale else None
    _load().oracle_conv2d_f32_strided(_ptr(x), wd, h, wd, _ptr(w), p, q, int(sr), int(sc), _ptr(y),
                                      _ptr(s) if want_scale else None, ow)
    return y, s


def conv1d_f32_taps_outer(x, w):
    x = _as(x, np.float32, 1)
    w = _as(w, np.float32, 1)
    n, q = x.shape[0], w.shape[0]
    if q < 1 or n < q:
        raise ValueError("need 1 <= Q <= N")
    y = np.empty(n - q + 1, dtype=np.float64)
    _load().oracle_conv1d_f32_taps_outer(_ptr(x), n, _ptr(w), q, _ptr(y))
    return y


def conv1d_f32_at(x, w, pos):
    """Eq. 2 at the output positions ``pos`` only. Returns (y, S)."""
    x = _as(x, np.float32, 1)
    w = _as(w, np.float32, 1)
    pos = _as(pos, np.int64, 1)
    n, q = x.shape[0], w.shape[0]
    if pos.size and (pos.min() < 0 or pos.max() > n - q):
        raise ValueError("position outside the valid output range")
    y = np.empty(pos.size, dtype=np.float64)
    s = np.empty(pos.size, dtype=np.float64)
    _load().oracle_conv1d_f32_at(_ptr(x), n, _ptr(w), q, _ptr(pos), pos.size, _ptr(y), _ptr(s))
    return y, s


def conv2d_f32(x, w, want_scale=True):
    """Eq. 3 in fp64 on one image x[H][W] with filter w[P][Q]. Returns (y, S)."""
    x = _as(x, np.float32, 2)
    w = _as(w, np.float32, 2)
    h, wd = x.shape
    p, q = w.shape
    if p < 1 or q < 1 or h < p or wd < q:
        raise ValueError("filter larger than image")
    y = np.empty((h - p + 1, wd - q + 1), dtype=np.float64)
    s = np.empty_like(y) if want_scale else None
    _load().oracle_conv2d_f32(_ptr(x), wd, h, wd, _ptr(w), q, p, _ptr(y),
                              _ptr(s) if want_scale else None, wd - q + 1)
    return y, s


def conv2d_f32_taps_outer(x, w):
    x = _as(x, np.float32, 2)
    w = _as(w, np.float32, 2)
    h, wd = x.shape
    p, q = w.shape
    if p < 1 or q < 1 or h < p or wd < q:
        raise ValueError("filter larger than image")
    y = np.empty((h - p + 1, wd - q + 1), dtype=np.float64)
    _load().oracle_conv2d_f32_taps_outer(_ptr(x), wd, h, wd, _ptr(w), q, p, _ptr(y), wd - q + 1)
    return y


def conv2d_f32_at(x, w, rows, cols):
    """Eq. 3 at output positions (rows[i], cols[i]) only. Returns (y, S)."""
    x = _as(x, np.float32, 2)
    w = _as(w, np.float32, 2)
    rows = _as(rows, np.int64, 1)
    cols = _as(cols, np.int64, 1)
    h, wd = x.shape
    p, q = w.shape
    if rows.shape != cols.shape:
        raise ValueError("rows and cols differ in length")
    if rows.size and (rows.min() < 0 or rows.max() > h - p or cols.min() < 0 or cols.max() > wd - q):
        raise ValueError("position outside the valid output range")
    y = np.empty(rows.size, dtype=np.float64)
    s = np.empty(rows.size, dtype=np.float64)
    _load().oracle_conv2d_f32_at(_ptr(x), wd, h, wd, _ptr(w), q, p, _ptr(rows), _ptr(cols),
                                 rows.size, _ptr(y), _ptr(s))
    return y, s


def conv1d_u8s8_s32(x, w):
    x = _as(x, np.uint8, 1)
    w = _as(w, np.int8, 1)
    n, q = x.shape[0], w.shape[0]
    if q < 1 or n < q:
        raise ValueError("need 1 <= Q <= N")
    y = np.empty(n - q + 1, dtype=np.int32)
    _load().oracle_conv1d_u8s8_s32(_ptr(x), n, _ptr(w), q, _ptr(y))
    return y


def conv2d_u8s8_s32(x, w):
    x = _as(x, np.uint8, 2)
    w = _as(w, np.int8, 2)
    h, wd = x.shape
    p, q = w.shape
    if p < 1 or q < 1 or h < p or wd < q:
        raise ValueError("filter larger than image")
    y = np.empty((h - p + 1, wd - q + 1), dtype=np.int32)
    _load().oracle_conv2d_u8s8_s32(_ptr(x), wd, h, wd, _ptr(w), q, p, _ptr(y), wd - q + 1)
    return y


def conv2d_u8s8_i64(x, w):
    x = _as(x, np.uint8, 2)
    w = _as(w, np.int8, 2)
    h, wd = x.shape
    p, q = w.shape
    if p < 1 or q < 1 or h < p or wd < q:
        raise ValueError("filter larger than image")
    y = np.empty((h - p + 1, wd - q + 1), dtype=np.int64)
    _load().oracle_conv2d_u8s8_i64(_ptr(x), wd, h, wd, _ptr(w), q, p, _ptr(y), wd - q + 1)
    return y


def stencil2d_f32(u, k, sweeps, want_scale=True):
    """``sweeps`` Jacobi sweeps of the 3x3 stencil k (k[dr+1][dc+1]) over the grid u with its outermost ring held
    fixed, in fp64.  Returns (y, S): S = the same sweeps of |k| over |u| (the tolerance scale), or None."""
    u = _as(u, np.float32, 2)
    k = _as(k, np.float32, 2)
    if k.shape != (3, 3):
        raise ValueError("the stencil is 3 x 3")
    if sweeps < 0:
        raise ValueError("sweeps >= 0")
    h, w = u.shape
    y = np.empty((h, w), dtype=np.float64)
    s = np.empty((h, w), dtype=np.float64) if want_scale else None
    rc = _load().oracle_stencil2d_f32(_ptr(u), w, h, w, _ptr(k), int(sweeps), _ptr(y), _ptr(s) if want_scale else None)
    if rc != 0:
        raise MemoryError("oracle_stencil2d_f32")
    return y, s
