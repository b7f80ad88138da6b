"""The C-ABI library loads and exports every symbol include/sysconv.h declares (no GPU, no compute)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "sysconv.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2010_15884_b200 import build, binding
    build.build()
    return binding.load_library()


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(sysconv\w*)\s*\(", text)
    return sorted(set(names))


def test_header_declares_the_expected_entry_points():
    names = _declared_functions()
    for must in ("sysconv1d", "sysconv2d", "sysconv1d_strided", "sysconv2d_strided", "sysconv_spacetime_describe",
                 "sysconv1d_spacetime", "sysconv2d_separable", "sysconv1d_host", "sysconv1d_host_multi", "sysconv2d_host", "sysconv_status_string",
                 "sysconv_design_name", "sysconv_version", "sysconv_launch_count"):
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    for name in _declared_functions():
        assert hasattr(lib, name), "libsysconv.so does not export %s" % name


def test_strings_and_version_without_a_gpu(lib):
    from paper_2010_15884_b200 import binding
    assert binding.version() >= 100
    assert binding.status_string(0) == "ok"
    assert binding.status_string(1) == "invalid argument"
    assert binding.status_string(99) == "?"
    assert binding.design_name(binding.WS) == "WS/BSM"
    assert binding.design_name(binding.OS) == "OS/FBS"
    assert binding.design_name(binding.IS) == "IS/SBM"
    assert [binding.design_name(d) for d in (binding.FSM, binding.BFS, binding.FFS)] == ["FSM", "BFS", "FFS"]
    assert binding.design_name(6) == "?"
    assert binding.launch_count() >= 0


def test_argument_validation_needs_no_gpu(lib):
    # every one of these is rejected before any CUDA call is made
    import numpy as np
    from paper_2010_15884_b200 import binding as b
    w = np.ones(4, np.float32)
    fake_x, fake_y = 0x10000, 0x90000000
    assert b.sysconv1d(0, 100, 100, w, 4, fake_y, 97, 1, b.F32, b.OS, 0) == 1          # null x
    assert b.sysconv1d(fake_x, 3, 3, w, 4, fake_y, 0, 1, b.F32, b.OS, 0) == 1           # n < q
    assert b.sysconv1d(fake_x, 100, 100, w, 4, fake_y, 97, 0, b.F32, b.OS, 0) == 1      # batch < 1
    assert b.sysconv1d(fake_x, 100, 100, w, 4, fake_y, 97, 1, 7, b.OS, 0) == 1          # dtype
    assert b.sysconv1d(fake_x, 100, 100, w, 4, fake_y, 97, 1, b.F32, 6, 0) == 1         # design
    assert b.sysconv1d(fake_x, 100, 50, w, 4, fake_y, 97, 2, b.F32, b.OS, 0) == 1       # batch stride < n
    assert b.sysconv1d(fake_x, 100, 100, w, 4, fake_x + 16, 97, 1, b.F32, b.OS, 0) == 1  # overlap
    w33 = np.ones(33, np.float32)
    assert b.sysconv1d(fake_x, 100, 100, w33, 33, fake_y, 68, 1, b.F32, b.OS, 0) == 2   # Q > 32
    w2 = np.ones((3, 3), np.float32)
    assert b.sysconv2d(fake_x, 2, 10, 2, 20, w2, 3, 3, fake_y, 8, 64, 1, b.F32, b.OS, 0) == 1    # width < q
    assert b.sysconv2d(fake_x, 10, 10, 9, 100, w2, 3, 3, fake_y, 8, 64, 1, b.F32, b.OS, 0) == 1  # pitch < width
    assert b.sysconv2d(fake_x, 10, 10, 10, 100, w2, 3, 3, fake_y, 7, 64, 1, b.F32, b.OS, 0) == 1  # y pitch
    w16 = np.ones((16, 3), np.float32)
    assert b.sysconv2d(fake_x, 40, 40, 40, 1600, w16, 3, 16, fake_y, 38, 950, 1, b.F32, b.OS, 0) == 2  # P > 15
    assert lib.sysconv1d_host_workspace_bytes(100, 4, 2, b.F32) == 1024 + 1024
    assert lib.sysconv1d_host_workspace_bytes(3, 4, 1, b.F32) == -1
    assert lib.sysconv2d_host_workspace_bytes(10, 10, 3, 3, 1, b.U8S8_S32) == 256 + 256


def test_strided_argument_validation_needs_no_gpu(lib):
    import numpy as np
    from paper_2010_15884_b200 import binding as b
    w = np.ones(4, np.float32)
    w2 = np.ones((3, 3), np.float32)
    wi = np.ones((3, 3), np.int8)
    x, y = 0x10000, 0x90000000
    assert b.sysconv1d_strided(x, 100, 100, w, 4, 0, y, 49, 1, b.F32, b.OS, 0) == 1        # stride < 1
    assert b.sysconv1d_strided(0, 100, 100, w, 4, 2, y, 49, 1, b.F32, b.OS, 0) == 1        # null x
    assert b.sysconv1d_strided(x, 3, 3, w, 4, 2, y, 1, 1, b.F32, b.OS, 0) == 1             # n < q
    assert b.sysconv1d_strided(x, 100, 100, w, 4, 2, y, 40, 2, b.F32, b.OS, 0) == 1        # y batch stride < n_out
    assert b.sysconv1d_strided(x, 100, 100, w, 4, 3, y, 33, 1, b.F32, b.IS, 0) == 2        # stride 3: output-stationary only
    assert b.sysconv1d_strided(x, 100, 100, w, 4, 2, y, 49, 1, b.F32, b.WS, 0) == 2        # WS: not built
    assert b.sysconv1d_strided(x, 100, 100, w, 4, 2, y, 49, 1, b.U8S8_S32, b.OS, 0) == 2   # integer: not built
    assert b.sysconv2d_strided(x, 64, 64, 64, 0, w2, 3, 3, 2, 0, y, 31, 0, 1, b.F32, b.OS, 0) == 1     # stride_r < 1
    assert b.sysconv2d_strided(x, 64, 64, 64, 0, w2, 3, 3, 2, 2, y, 30, 0, 1, b.F32, b.OS, 0) == 1     # y_pitch < out_w
    assert b.sysconv2d_strided(x, 64, 64, 64, 0, w2, 3, 3, 2, 1, y, 31, 0, 1, b.F32, b.IS, 0) == 2     # mixed strides: output-stationary only
    assert b.sysconv2d_strided(x, 64, 64, 64, 0, w2, 3, 3, 2, 2, y, 31, 0, 1, b.F32, b.WS, 0) == 2     # WS: not built
    assert b.sysconv2d_strided(x, 64, 64, 64, 0, wi, 3, 3, 2, 2, y, 31, 0, 1, b.U8S8_S32, b.IS, 0) == 2
    w9 = np.ones((9, 9), np.float32)
    assert b.sysconv2d_strided(x, 64, 64, 64, 0, w9, 9, 9, 2, 2, y, 28, 0, 1, b.F32, b.IS, 0) == 2     # beyond 7 x 7: output-stationary only


def test_host_multi_argument_validation_needs_no_gpu(lib):
    import ctypes
    import numpy as np
    from paper_2010_15884_b200 import binding as b
    assert b.host_multi_workspace_bytes(1000, [4, 16]) == 4096 + 4096 + 4096
    assert b.host_multi_workspace_bytes(10, [4, 16]) == -1                       # a filter longer than the signal
    assert b.host_multi_workspace_bytes(1000, [4], b.U8S8_S32) == -1             # fp32 only
    w = np.ones(4, np.float32)
    y = np.zeros(997, np.float32)
    x = np.zeros(1000, np.float32)
    q = (ctypes.c_int * 1)(4)
    d = (ctypes.c_int * 1)(b.OS)
    wp = (ctypes.c_void_p * 1)(w.ctypes.data)
    yp = (ctypes.c_void_p * 1)(y.ctypes.data)
    call = lib.sysconv1d_host_multi
    vp = ctypes.c_void_p
    assert call(vp(0), 1000, 1, wp, q, d, yp, b.F32, vp(0x7f0000000000), 1 << 20, vp(0)) == 1          # null x
    assert call(vp(x.ctypes.data), 1000, 0, wp, q, d, yp, b.F32, vp(0x7f0000000000), 1 << 20, vp(0)) == 1   # no jobs
    assert call(vp(x.ctypes.data), 1000, 1, wp, q, d, yp, b.F32, vp(0x7f0000000000), 100, vp(0)) == 1       # workspace too small
    assert call(vp(x.ctypes.data), 1000, 1, wp, q, d, yp, b.F32, vp(0x7f0000000010), 1 << 20, vp(0)) == 1   # misaligned workspace
    assert call(vp(x.ctypes.data), 1000, 1, wp, q, d, yp, b.U8S8_S32, vp(0x7f0000000000), 1 << 20, vp(0)) == 2


def test_separable_argument_validation_needs_no_gpu(lib):
    import numpy as np
    from paper_2010_15884_b200 import binding as b
    u, v = np.ones(3, np.float32), np.ones(5, np.float32)
    x, y = 0x10000, 0x90000000
    assert b.sysconv2d_separable(0, 64, 64, 64, 0, u, v, y, 60, 0, 1, 0) == 1           # null x
    assert b.sysconv2d_separable(x, 4, 64, 4, 0, u, v, y, 1, 0, 1, 0) == 1              # image narrower than v
    assert b.sysconv2d_separable(x, 64, 64, 64, 0, u, v, y, 59, 0, 1, 0) == 1           # y_pitch < out_w
    assert b.sysconv2d_separable(x, 64, 64, 64, 0, u, v, y, 60, 0, 0, 0) == 1           # batch < 1
    assert b.sysconv2d_separable(x, 64, 64, 64, 0, np.ones(16, np.float32), v, y, 60, 0, 1, 0) == 2   # 16 vertical taps
    assert b.sysconv2d_separable(x, 64, 64, 64, 64 * 64, u, v, y, 60, 62 * 60, 70000, 0) == 2         # batch beyond 65535


def test_size_queries_reject_products_beyond_the_index_type(lib):
    # n * batch * 4 would wrap a signed 64-bit product to a small positive number: the queries must say -1 and the
    # entry point that allocates nothing must answer "invalid argument" before anything is enqueued
    import numpy as np
    from paper_2010_15884_b200 import binding as b
    n = (1 << 60) + 1024
    assert lib.sysconv1d_host_workspace_bytes(ctypes.c_longlong(n), 4, 4, b.F32) == -1
    assert lib.sysconv1d_host_workspace_bytes(ctypes.c_longlong(1 << 62), 4, 1, b.F32) == -1
    assert lib.sysconv2d_host_workspace_bytes(1 << 30, 1 << 30, 3, 3, 1 << 20, b.F32) == -1
    assert b.host_multi_workspace_bytes(1 << 61, [4, 16]) == -1
    w = np.ones(4, np.float32)
    before = b.launch_count()
    vp = ctypes.c_void_p
    st = lib.sysconv1d_host_static(vp(0x10000), ctypes.c_longlong(n), vp(w.ctypes.data), 4, vp(0x90000000), 4, b.F32, b.OS,
                                   vp(0))
    assert st == 1
    assert b.launch_count() == before


def test_peak_measurement_argument_validation_needs_no_gpu(lib):
    vp = ctypes.c_void_p
    out = (ctypes.c_double * 8)()
    assert lib.sysconv_measure_peaks(vp(0), ctypes.c_longlong(1 << 30), ctypes.cast(out, vp), 8) == 1          # null scratch
    assert lib.sysconv_measure_peaks(vp(0x7f0000000000), ctypes.c_longlong(1 << 20), ctypes.cast(out, vp), 8) == 1   # too small
    assert lib.sysconv_measure_peaks(vp(0x7f0000000010), ctypes.c_longlong(1 << 30), ctypes.cast(out, vp), 8) == 1   # misaligned
    assert lib.sysconv_measure_peaks(vp(0x7f0000000000), ctypes.c_longlong(1 << 30), ctypes.cast(out, vp), 3) == 1   # too few results
    assert lib.sysconv_floor_copy(vp(0), vp(0x7f0000000000), ctypes.c_longlong(1024), 0, vp(0)) == 1
    assert lib.sysconv_floor_copy(vp(0x7f0000000000), vp(0x7f0000100000), ctypes.c_longlong(1000), 0, vp(0)) == 1    # not x16
    assert lib.sysconv_floor_copy(vp(0x7f0000000004), vp(0x7f0000100000), ctypes.c_longlong(1024), 0, vp(0)) == 1    # misaligned
    assert lib.sysconv_floor_copy(vp(0x7f0000000000), vp(0x7f0000100000), ctypes.c_longlong(1024), 2, vp(0)) == 1    # widen flag


def test_stencil_argument_validation_needs_no_gpu(lib):
    import numpy as np
    from paper_2010_15884_b200 import binding as b
    k = np.ones((3, 3), np.float32)
    u, o, sc = 0x10000, 0x90000000, 0xa0000000
    assert b.sysstencil2d(0, 64, 64, 64, 0, k, 1, o, 64, 0, 1, 0, 0) == 1          # null grid
    assert b.sysstencil2d(u, 64, 64, 63, 0, k, 1, o, 64, 0, 1, 0, 0) == 1          # pitch < width
    assert b.sysstencil2d(u, 64, 64, 64, 0, k, 0, o, 64, 0, 1, 0, 0) == 1          # no sweeps
    assert b.sysstencil2d(u, 64, 64, 64, 0, k, 1, u + 64, 64, 0, 1, 0, 0) == 1     # output overlaps the input
    assert b.sysstencil2d(u, 64, 64, 64, 0, k, 5, o, 64, 0, 1, 0, 0) == 1          # five sweeps need a scratch buffer
    assert b.sysstencil2d(u, 64, 64, 64, 0, k, 5, o, 64, 0, 1, o + 128, 0) == 1    # scratch overlaps the output
    assert b.sysstencil2d(u, 64, 64, 64, 64 * 64, k, 2, o, 64, 64 * 63, 2, sc, 0) == 1    # output batch stride too small
    assert b.sysstencil2d(u, 8, 8, 8, 64, k, 2, o, 8, 64, 70000, sc, 0) == 2       # batch beyond 65535
