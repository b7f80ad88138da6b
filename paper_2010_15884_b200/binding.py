"""Thin ctypes binding of libsysconv.so (see include/sysconv.h).

Argument marshalling only: every step of the computation runs in the CUDA
library.  There is no CPU fallback; if the library cannot be loaded every call
raises.  PyTorch is used for device memory and streams.
"""
import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_NAME = "libsysconv.so"

WS, OS, IS = 0, 1, 2
FSM, BFS, FFS = 3, 4, 5          # the paper's other three 1-D designs (1-D fp32 only)
F32, U8S8_S32 = 0, 1
DESIGN_NAMES = {WS: "WS", OS: "OS", IS: "IS", FSM: "FSM", BFS: "BFS", FFS: "FFS"}
_DESIGN_BY_NAME = {"WS": WS, "BSM": WS, "OS": OS, "FBS": OS, "IS": IS, "SBM": IS, "FSM": FSM, "BFS": BFS, "FFS": FFS}

_c_ll = ctypes.c_longlong
_c_int = ctypes.c_int
_vp = ctypes.c_void_p

_lib = None


class SysconvError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        super().__init__("%s failed: status %d (%s)" % (where, status, status_string(status)))


def library_path():
    return os.path.join(_HERE, _LIB_NAME)


def load_library():
    """Load libsysconv.so (built in-tree by paper_2010_15884_b200.build). Raises if missing."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise SysconvError(-1, "loading %s (not built: run python -m paper_2010_15884_b200.build)" % path)
    lib = ctypes.CDLL(path)
    lib.sysconv1d.restype = _c_int
    lib.sysconv1d.argtypes = [_vp, _c_ll, _c_ll, _vp, _c_int, _vp, _c_ll, _c_int, _c_int, _c_int, _vp]
    lib.sysconv2d.restype = _c_int
    lib.sysconv2d.argtypes = [_vp, _c_int, _c_int, _c_ll, _c_ll, _vp, _c_int, _c_int, _vp, _c_ll, _c_ll,
                              _c_int, _c_int, _c_int, _vp]
    lib.sysconv1d_strided.restype = _c_int
    lib.sysconv1d_strided.argtypes = [_vp, _c_ll, _c_ll, _vp, _c_int, _c_int, _vp, _c_ll, _c_int, _c_int, _c_int, _vp]
    lib.sysconv2d_strided.restype = _c_int
    lib.sysconv2d_strided.argtypes = [_vp, _c_int, _c_int, _c_ll, _c_ll, _vp, _c_int, _c_int, _c_int, _c_int, _vp,
                                      _c_ll, _c_ll, _c_int, _c_int, _c_int, _vp]
    lib.sysconv2d_separable.restype = _c_int
    lib.sysconv2d_separable.argtypes = [_vp, _c_int, _c_int, _c_ll, _c_ll, _vp, _c_int, _vp, _c_int, _vp, _c_ll, _c_ll,
                                        _c_int, _vp]
    lib.sysstencil2d.restype = _c_int
    lib.sysstencil2d.argtypes = [_vp, _c_int, _c_int, _c_ll, _c_ll, _vp, _c_int, _vp, _c_ll, _c_ll, _c_int, _vp, _vp]
    lib.sysconv_spacetime_describe.restype = _c_int
    lib.sysconv_spacetime_describe.argtypes = [_c_int, _c_int, _c_int, _c_int, _c_int, _vp, _vp]
    lib.sysconv1d_spacetime.restype = _c_int
    lib.sysconv1d_spacetime.argtypes = [_vp, _c_ll, _vp, _c_int, _vp, _c_int, _c_int, _c_int, _c_int, _vp]
    lib.sysconv1d_host_workspace_bytes.restype = _c_ll
    lib.sysconv1d_host_workspace_bytes.argtypes = [_c_ll, _c_int, _c_int, _c_int]
    lib.sysconv2d_host_workspace_bytes.restype = _c_ll
    lib.sysconv2d_host_workspace_bytes.argtypes = [_c_int, _c_int, _c_int, _c_int, _c_int, _c_int]
    lib.sysconv1d_host.restype = _c_int
    lib.sysconv1d_host.argtypes = [_vp, _c_ll, _vp, _c_int, _vp, _c_int, _c_int, _c_int, _vp, _c_ll, _vp]
    lib.sysconv2d_host.restype = _c_int
    lib.sysconv2d_host.argtypes = [_vp, _c_int, _c_int, _vp, _c_int, _c_int, _vp, _c_int, _c_int, _c_int,
                                   _vp, _c_ll, _vp]
    lib.sysconv1d_host_multi_workspace_bytes.restype = _c_ll
    lib.sysconv1d_host_multi_workspace_bytes.argtypes = [_c_ll, _vp, _c_int, _c_int]
    lib.sysconv1d_host_multi.restype = _c_int
    lib.sysconv1d_host_multi.argtypes = [_vp, _c_ll, _c_int, _vp, _vp, _vp, _vp, _c_int, _vp, _c_ll, _vp]
    lib.sysconv1d_host_static.restype = _c_int
    lib.sysconv1d_host_static.argtypes = [_vp, _c_ll, _vp, _c_int, _vp, _c_int, _c_int, _c_int, _vp]
    lib.sysconv_static_scratch_bytes.restype = _c_ll
    lib.sysconv_status_string.restype = ctypes.c_char_p
    lib.sysconv_status_string.argtypes = [_c_int]
    lib.sysconv_design_name.restype = ctypes.c_char_p
    lib.sysconv_design_name.argtypes = [_c_int]
    lib.sysconv_version.restype = _c_int
    lib.sysconv_device_status.restype = _c_int
    lib.sysconv_measure_peaks.restype = _c_int
    lib.sysconv_measure_peaks.argtypes = [_vp, _c_ll, _vp, _c_int]
    lib.sysconv_floor_copy.restype = _c_int
    lib.sysconv_floor_copy.argtypes = [_vp, _vp, _c_ll, _c_int, _vp]
    lib.sysconv_selftest_wait_timeout.restype = _c_int
    lib.sysconv_selftest_wait_timeout.argtypes = [_vp]
    lib.sysconv_launch_count.restype = _c_ll
    _lib = lib
    return lib


def status_string(status):
    if _lib is None:
        return "library not loaded"
    return _lib.sysconv_status_string(int(status)).decode()


def design_name(design):
    return load_library().sysconv_design_name(int(design)).decode()


def version():
    return int(load_library().sysconv_version())


def device_status():
    """0 if no kernel gave up a bounded wait on the current device since the last call, else 4 (time-out)."""
    return int(load_library().sysconv_device_status())


def selftest_wait_timeout(stream=None):
    """Enqueue the one-block self-test whose bounded wait runs out; the next device_status() reports 4."""
    st = int(load_library().sysconv_selftest_wait_timeout(_vp(_stream_ptr(stream))))
    if st != 0:
        raise SysconvError(st, "sysconv_selftest_wait_timeout")


PEAK_NAMES = ("ffma_per_clk_sm", "ffma2_mac_per_clk_sm", "imad_per_clk_sm", "dp4a_per_clk_sm", "shfl_per_clk_sm",
              "copy_gbs", "sm_count")


def measure_peaks(scratch):
    """Issue rates of the plain datapaths and the streaming-copy bandwidth of the current device, as a dict.
    scratch: a CUDA uint8 tensor of at least 64 MiB (overwritten)."""
    out = (ctypes.c_double * len(PEAK_NAMES))()
    st = int(load_library().sysconv_measure_peaks(_vp(scratch.data_ptr()), scratch.numel() * scratch.element_size(),
                                                   ctypes.cast(out, _vp), len(PEAK_NAMES)))
    if st != 0:
        raise SysconvError(st, "sysconv_measure_peaks")
    return dict(zip(PEAK_NAMES, [float(v) for v in out]))


def floor_copy(src, dst, bytes_in, widen=False, stream=None):
    """One plain streaming kernel that moves the bytes of a convolution of that size (see sysconv.h)."""
    st = int(load_library().sysconv_floor_copy(_vp(src.data_ptr()), _vp(dst.data_ptr()), int(bytes_in), 1 if widen else 0,
                                                _vp(_stream_ptr(stream))))
    if st != 0:
        raise SysconvError(st, "sysconv_floor_copy")


def launch_count():
    """Kernels launched by the library in this process so far."""
    return int(load_library().sysconv_launch_count())


def _design(design):
    if isinstance(design, str):
        return _DESIGN_BY_NAME[design.upper()]
    return int(design)


def _host_taps(w, dtype, ndim):
    w = np.ascontiguousarray(w.detach().cpu().numpy() if hasattr(w, "detach") else w,
                             dtype=np.float32 if dtype == F32 else np.int8)
    if w.ndim != ndim:
        raise ValueError("filter must be %d-D" % ndim)
    return w


def _stream_ptr(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return int(getattr(stream, "cuda_stream", stream))


# ------------------------------------------------------------------ raw C-ABI calls


def sysconv1d(x_ptr, n, x_batch_stride, w_host, q, y_ptr, y_batch_stride, batch, dtype, design, stream_ptr):
    """Raw call: pointers are integers (device x/y, numpy array for the taps). Returns the status."""
    lib = load_library()
    return int(lib.sysconv1d(_vp(x_ptr), n, x_batch_stride, w_host.ctypes.data_as(_vp), q, _vp(y_ptr),
                             y_batch_stride, batch, dtype, design, _vp(stream_ptr)))


def sysconv2d(x_ptr, width, height, x_pitch, x_batch_stride, w_host, q, p, y_ptr, y_pitch, y_batch_stride,
              batch, dtype, design, stream_ptr):
    lib = load_library()
    return int(lib.sysconv2d(_vp(x_ptr), width, height, x_pitch, x_batch_stride, w_host.ctypes.data_as(_vp),
                             q, p, _vp(y_ptr), y_pitch, y_batch_stride, batch, dtype, design,
                             _vp(stream_ptr)))


def sysconv1d_strided(x_ptr, n, x_batch_stride, w_host, q, stride, y_ptr, y_batch_stride, batch, dtype, design,
                      stream_ptr):
    lib = load_library()
    return int(lib.sysconv1d_strided(_vp(x_ptr), n, x_batch_stride, w_host.ctypes.data_as(_vp), q, stride,
                                     _vp(y_ptr), y_batch_stride, batch, dtype, design, _vp(stream_ptr)))


def sysconv2d_strided(x_ptr, width, height, x_pitch, x_batch_stride, w_host, q, p, stride_c, stride_r, y_ptr,
                      y_pitch, y_batch_stride, batch, dtype, design, stream_ptr):
    lib = load_library()
    return int(lib.sysconv2d_strided(_vp(x_ptr), width, height, x_pitch, x_batch_stride,
                                     w_host.ctypes.data_as(_vp), q, p, stride_c, stride_r, _vp(y_ptr), y_pitch,
                                     y_batch_stride, batch, dtype, design, _vp(stream_ptr)))


def sysconv2d_separable(x_ptr, width, height, x_pitch, x_batch_stride, u_host, v_host, y_ptr, y_pitch, y_batch_stride,
                        batch, stream_ptr):
    """Raw call: u_host = vertical taps (filter rows), v_host = horizontal taps, float32 numpy arrays."""
    lib = load_library()
    return int(lib.sysconv2d_separable(_vp(x_ptr), width, height, x_pitch, x_batch_stride,
                                       u_host.ctypes.data_as(_vp), int(u_host.shape[0]), v_host.ctypes.data_as(_vp),
                                       int(v_host.shape[0]), _vp(y_ptr), y_pitch, y_batch_stride, batch,
                                       _vp(stream_ptr)))


def conv2d_separable(x, u, v, out=None, stream=None):
    """y[b, r, c] = sum_i sum_k u[i] v[k] x[b, r+i, c+k] on float32 CUDA tensors. x: (h, w) or (batch, h, w)."""
    import torch
    if not x.is_cuda:
        raise SysconvError(-1, "conv2d_separable (x is not a CUDA tensor; there is no CPU path)")
    squeeze = x.dim() == 2
    x3 = x.unsqueeze(0) if squeeze else x
    if x3.dim() != 3 or x3.stride(2) != 1 or x3.dtype != torch.float32:
        raise ValueError("x must be float32, (h, w) or (batch, h, w) with contiguous rows")
    u = np.ascontiguousarray(u, dtype=np.float32).reshape(-1)
    v = np.ascontiguousarray(v, dtype=np.float32).reshape(-1)
    batch, h, wd = x3.shape
    if out is None:
        ow = max(wd - len(v) + 1, 0)             # rows padded to 16 bytes, as in conv2d
        out = torch.empty((batch, max(h - len(u) + 1, 0), (ow + 3) // 4 * 4), dtype=torch.float32, device=x.device)[:, :, :ow]
    y3 = out.unsqueeze(0) if out.dim() == 2 else out
    st = sysconv2d_separable(x3.data_ptr(), wd, h, x3.stride(1), x3.stride(0) if batch > 1 else 0, u, v, y3.data_ptr(),
                             y3.stride(1), y3.stride(0) if batch > 1 else 0, batch, _stream_ptr(stream))
    if st != 0:
        raise SysconvError(st, "sysconv2d_separable")
    return out.squeeze(0) if (squeeze and out.dim() == 3) else out


def spacetime_describe(P, s, q):
    """Plan of the generic executor for allocation row P = (p_c, p_q) and schedule row s = (s_c, s_q).

    Returns (status, dict or None); the dict holds the design letters and, per dependence, PE distance and delay.
    """
    lib = load_library()
    info = (ctypes.c_int * 10)()
    name = ctypes.create_string_buffer(4)
    st = int(lib.sysconv_spacetime_describe(int(P[0]), int(P[1]), int(s[0]), int(s[1]), int(q), info, name))
    if st != 0:
        return st, None
    v = list(info)
    return 0, {"name": name.value.decode(), "input": (v[0], v[1]), "weight": (v[2], v[3]), "sum": (v[4], v[5]),
               "outputs_per_array": v[6], "pes": v[7], "steps": v[8], "det": v[9]}


def sysconv1d_spacetime(x_ptr, n, w_host, q, y_ptr, P, s, stream_ptr):
    lib = load_library()
    return int(lib.sysconv1d_spacetime(_vp(x_ptr), n, w_host.ctypes.data_as(_vp), q, _vp(y_ptr), int(P[0]), int(P[1]),
                                       int(s[0]), int(s[1]), _vp(stream_ptr)))


def host_workspace_bytes(shape, filt, dtype=F32):
    """Device workspace the *_host entry points need. shape = (n,) | (batch, n) | (h, w) handled by caller."""
    lib = load_library()
    if len(filt) == 1:
        batch, n = (1, shape[0]) if len(shape) == 1 else shape
        return int(lib.sysconv1d_host_workspace_bytes(n, filt[0], batch, dtype))
    batch, h, w = (1,) + tuple(shape) if len(shape) == 2 else shape
    return int(lib.sysconv2d_host_workspace_bytes(w, h, filt[1], filt[0], batch, dtype))


def sysconv1d_host(x_host, w_host, y_host, design, workspace, stream=None, dtype=F32):
    """x_host: (batch, n) or (n,) host array/tensor (pinned for overlap); y_host likewise; workspace: cuda uint8 tensor."""
    lib = load_library()
    xs = tuple(x_host.shape)
    batch, n = (1, xs[0]) if len(xs) == 1 else xs
    w = _host_taps(w_host, dtype, 1)
    st = lib.sysconv1d_host(_vp(_data_ptr(x_host)), n, w.ctypes.data_as(_vp), w.shape[0], _vp(_data_ptr(y_host)),
                            batch, dtype, _design(design), _vp(workspace.data_ptr()), workspace.numel(),
                            _vp(_stream_ptr(stream)))
    if st != 0:
        raise SysconvError(st, "sysconv1d_host")


def host_multi_workspace_bytes(n, qs, dtype=F32):
    lib = load_library()
    arr = (ctypes.c_int * len(qs))(*[int(v) for v in qs])
    return int(lib.sysconv1d_host_multi_workspace_bytes(int(n), arr, len(qs), dtype))


def sysconv1d_host_multi(x_host, jobs, workspace, stream=None, dtype=F32):
    """One host signal through several (taps, design, y_host) jobs; the signal is copied to the device once.

    jobs: sequence of (w_host, design, y_host); x_host and the y_host are host arrays/tensors (pinned for overlap).
    """
    lib = load_library()
    n = int(tuple(x_host.shape)[0])
    taps = [_host_taps(w, dtype, 1) for w, _, _ in jobs]
    count = len(jobs)
    w_ptrs = (ctypes.c_void_p * count)(*[t.ctypes.data for t in taps])
    y_ptrs = (ctypes.c_void_p * count)(*[_data_ptr(y) for _, _, y in jobs])
    qs = (ctypes.c_int * count)(*[int(t.shape[0]) for t in taps])
    ds = (ctypes.c_int * count)(*[_design(d) for _, d, _ in jobs])
    st = lib.sysconv1d_host_multi(_vp(_data_ptr(x_host)), n, count, w_ptrs, qs, ds, y_ptrs, dtype,
                                  _vp(workspace.data_ptr()), workspace.numel(), _vp(_stream_ptr(stream)))
    if st != 0:
        raise SysconvError(st, "sysconv1d_host_multi")


def static_scratch_bytes():
    """Size of the staging area built into the library for sysconv1d_host_static."""
    return int(load_library().sysconv_static_scratch_bytes())


def sysconv1d_host_static(x_host, w_host, y_host, design, stream=None, dtype=F32):
    """sysconv1d_host without a workspace argument, for callers that cannot allocate device memory.

    The data is staged in a fixed 16 MiB array inside the library, so problems are limited to what
    fits there (SysconvError with status 5 otherwise) and calls that overlap on the GPU race on it.
    """
    lib = load_library()
    xs = tuple(x_host.shape)
    batch, n = (1, xs[0]) if len(xs) == 1 else xs
    w = _host_taps(w_host, dtype, 1)
    st = lib.sysconv1d_host_static(_vp(_data_ptr(x_host)), n, w.ctypes.data_as(_vp), w.shape[0],
                                   _vp(_data_ptr(y_host)), batch, dtype, _design(design),
                                   _vp(_stream_ptr(stream)))
    if st != 0:
        raise SysconvError(st, "sysconv1d_host_static")


def sysconv2d_host(x_host, w_host, y_host, design, workspace, stream=None, dtype=F32):
    lib = load_library()
    xs = tuple(x_host.shape)
    batch, h, wd = (1,) + xs if len(xs) == 2 else xs
    w = _host_taps(w_host, dtype, 2)
    st = lib.sysconv2d_host(_vp(_data_ptr(x_host)), wd, h, w.ctypes.data_as(_vp), w.shape[1], w.shape[0],
                            _vp(_data_ptr(y_host)), batch, dtype, _design(design), _vp(workspace.data_ptr()),
                            workspace.numel(), _vp(_stream_ptr(stream)))
    if st != 0:
        raise SysconvError(st, "sysconv2d_host")


def _data_ptr(a):
    if hasattr(a, "data_ptr"):
        return a.data_ptr()
    return a.ctypes.data


# ------------------------------------------------------------------ torch-tensor front end


def _dtype_of(x):
    import torch
    if x.dtype == torch.float32:
        return F32, torch.float32
    if x.dtype == torch.uint8:
        return U8S8_S32, torch.int32
    raise TypeError("x must be float32 or uint8, got %s" % x.dtype)


def conv1d(x, w, design=OS, out=None, stream=None, stride=1):
    """y[b, c] = sum_k w[k] x[b, stride*c+k] on CUDA tensors. x: (n,) or (batch, n), contiguous rows."""
    import torch
    if not x.is_cuda:
        raise SysconvError(-1, "conv1d (x is not a CUDA tensor; there is no CPU path)")
    dtype, out_dtype = _dtype_of(x)
    squeeze = x.dim() == 1
    x2 = x.unsqueeze(0) if squeeze else x
    if x2.dim() != 2 or x2.stride(1) != 1:
        raise ValueError("x must be (n,) or (batch, n) with contiguous rows")
    taps = _host_taps(w, dtype, 1)
    batch, n = x2.shape
    q = taps.shape[0]
    n_out = (n - q) // stride + 1 if n >= q else 0
    if out is None:
        out = torch.empty((batch, n_out), dtype=out_dtype, device=x.device)
        y2 = out
    else:
        y2 = out.unsqueeze(0) if out.dim() == 1 else out
    st = sysconv1d_strided(x2.data_ptr(), n, x2.stride(0) if batch > 1 else n, taps, q, stride, y2.data_ptr(),
                           y2.stride(0) if batch > 1 else n_out, batch, dtype, _design(design),
                           _stream_ptr(stream))
    if st != 0:
        raise SysconvError(st, "sysconv1d" if stride == 1 else "sysconv1d_strided")
    return out.squeeze(0) if (squeeze and out.dim() == 2) else out


def sysstencil2d(u_ptr, width, height, pitch, batch_stride, k_host, sweeps, out_ptr, out_pitch, out_batch_stride, batch,
                 scratch_ptr, stream_ptr):
    """Raw call (pointers are integers, k_host a numpy array of nine floats). Returns the status."""
    k = np.ascontiguousarray(k_host, dtype=np.float32)
    return int(load_library().sysstencil2d(_vp(u_ptr), int(width), int(height), int(pitch), int(batch_stride),
                                            _vp(k.ctypes.data), int(sweeps), _vp(out_ptr), int(out_pitch),
                                            int(out_batch_stride), int(batch), _vp(scratch_ptr), _vp(stream_ptr)))


def stencil2d(u, k, sweeps, out=None, scratch=None, stream=None):
    """`sweeps` Jacobi sweeps of the 3x3 stencil k over u (CUDA fp32, (h, w) or (batch, h, w), contiguous rows), the
    outermost ring of every grid held fixed.  A scratch tensor like the output is allocated when sweeps > 4 and none
    is given."""
    import torch
    if not u.is_cuda:
        raise SysconvError(-1, "stencil2d (u is not a CUDA tensor; there is no CPU path)")
    if u.dtype != torch.float32:
        raise ValueError("stencil2d works on float32 grids")
    squeeze = u.dim() == 2
    u3 = u.unsqueeze(0) if squeeze else u
    if u3.dim() != 3 or u3.stride(2) != 1:
        raise ValueError("u must be (h, w) or (batch, h, w) with contiguous rows")
    k = np.ascontiguousarray(k.detach().cpu().numpy() if hasattr(k, "detach") else k, dtype=np.float32)
    if k.shape != (3, 3):
        raise ValueError("the stencil is 3 x 3")
    batch, h, wd = u3.shape
    if out is None:
        out = torch.empty((batch, h, wd), dtype=torch.float32, device=u.device)
        o3 = out
    else:
        o3 = out.unsqueeze(0) if out.dim() == 2 else out
    if sweeps > 4 and scratch is None:
        scratch = torch.empty_strided(o3.shape, o3.stride(), dtype=torch.float32, device=u.device)
    st = sysstencil2d(u3.data_ptr(), wd, h, u3.stride(1), u3.stride(0) if batch > 1 else 0, k, sweeps, o3.data_ptr(),
                      o3.stride(1), o3.stride(0) if batch > 1 else 0, batch,
                      scratch.data_ptr() if scratch is not None else 0, _stream_ptr(stream))
    if st != 0:
        raise SysconvError(st, "sysstencil2d")
    return out.squeeze(0) if (squeeze and out.dim() == 3) else out


def conv2d(x, w, design=OS, out=None, stream=None, stride=1):
    """y[b, r, c] = sum_p sum_q w[p, q] x[b, stride*r+p, stride*c+q] on CUDA tensors. x: (h, w) or (batch, h, w).

    Without `out` the result is a view of a buffer whose rows are padded to 16 bytes (rows that start unaligned
    are stored element by element, about twice as slow for the memory-bound filters)."""
    import torch
    if not x.is_cuda:
        raise SysconvError(-1, "conv2d (x is not a CUDA tensor; there is no CPU path)")
    dtype, out_dtype = _dtype_of(x)
    squeeze = x.dim() == 2
    x3 = x.unsqueeze(0) if squeeze else x
    if x3.dim() != 3 or x3.stride(2) != 1:
        raise ValueError("x must be (h, w) or (batch, h, w) with contiguous rows")
    taps = _host_taps(w, dtype, 2)
    batch, h, wd = x3.shape
    p, q = taps.shape
    if out is None:
        oh = (h - p) // stride + 1 if h >= p else 0
        ow = (wd - q) // stride + 1 if wd >= q else 0
        # rows padded to a multiple of four elements (16 bytes) so that every row leaves as 128-bit stores; the
        # result is the (batch, oh, ow) view of that buffer (call .contiguous() for a packed copy)
        out = torch.empty((batch, oh, (ow + 3) // 4 * 4), dtype=out_dtype, device=x.device)[:, :, :ow]
        y3 = out
    else:
        y3 = out.unsqueeze(0) if out.dim() == 2 else out
    st = sysconv2d_strided(x3.data_ptr(), wd, h, x3.stride(1), x3.stride(0) if batch > 1 else 0, taps, q, p,
                           stride, stride, y3.data_ptr(), y3.stride(1), y3.stride(0) if batch > 1 else 0, batch,
                           dtype, _design(design), _stream_ptr(stream))
    if st != 0:
        raise SysconvError(st, "sysconv2d" if stride == 1 else "sysconv2d_strided")
    return out.squeeze(0) if (squeeze and out.dim() == 3) else out
