"""Parity of the CUDA library (through the C ABI) against the CPU oracle, element by element.

fp32: |y_gpu - y_oracle| <= 1e-5 * S with S = sum |w||x| of the same output (the bound stated for
this build; the oracle accumulates in fp64).  Integer: every int32 equal.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_15884_b200 import binding as B
from paper_2010_15884_b200 import inputs

pytestmark = pytest.mark.gpu

DESIGNS = [B.WS, B.OS, B.IS]
STRIDED_1D = [B.OS, B.IS]
OTHER_DESIGNS = [B.FSM, B.BFS, B.FFS]        # the paper's other three 1-D designs (1-D fp32 only)
TOL = 1e-5
CANARY = 12345.0


def _ids(d):
    return B.DESIGN_NAMES[d]


def assert_close_f32(y_gpu, y_ref, s_ref, what=""):
    y_gpu = np.asarray(y_gpu, dtype=np.float64)
    assert y_gpu.shape == y_ref.shape, (y_gpu.shape, y_ref.shape)
    err = np.abs(y_gpu - y_ref)
    bound = TOL * s_ref
    bad = err > bound
    # outputs whose taps are all zero have S = 0 and must be exactly equal
    if bad.any():
        i = np.argmax(err - bound)
        raise AssertionError("%s: %d outputs beyond 1e-5*S; worst at flat index %d: gpu %r ref %r S %r"
                             % (what, int(bad.sum()), i, y_gpu.flat[i], y_ref.flat[i], s_ref.flat[i]))
    assert np.isfinite(y_gpu).all()


def _assert_same_where_finite(y_gpu, y_ref, s_ref, what):
    """Outputs whose window holds no non-finite input must be finite and within tolerance; the others must be
    non-finite on both sides."""
    y_gpu = np.asarray(y_gpu, np.float64)
    fin = np.isfinite(y_ref)
    assert (np.isfinite(y_gpu) == fin).all(), "%s: non-finite outputs differ (%d vs %d)" % (
        what, int((~np.isfinite(y_gpu)).sum()), int((~fin).sum()))
    assert (np.abs(y_gpu[fin] - y_ref[fin]) <= TOL * s_ref[fin]).all(), what


# ------------------------------------------------------------------------ 1-D fp32


def run_1d(x_np, w_np, design, device, batch_stride=None, offset=0):
    """x_np: (n,) or (batch, n). Returns y as numpy, checks canaries around the output."""
    x2 = x_np.reshape(1, -1) if x_np.ndim == 1 else x_np
    batch, n = x2.shape
    q = w_np.shape[0]
    n_out = n - q + 1
    xs = batch_stride or n
    ys = (batch_stride or n_out)
    xh = np.zeros(offset + batch * xs + 8, dtype=np.float32)
    np.lib.stride_tricks.as_strided(xh[offset:], shape=(batch, n), strides=(4 * xs, 4))[...] = x2
    xbuf = torch.from_numpy(xh).to(device)
    ybuf = torch.full((offset + batch * ys + 64,), CANARY, dtype=torch.float32, device=device)
    st = B.sysconv1d(xbuf.data_ptr() + 4 * offset, n, xs, np.ascontiguousarray(w_np), q,
                     ybuf.data_ptr() + 4 * offset, ys, batch, B.F32, design,
                     torch.cuda.current_stream().cuda_stream)
    assert st == 0, B.status_string(st)
    torch.cuda.synchronize()
    yh = ybuf.cpu().numpy()
    out = np.lib.stride_tricks.as_strided(yh[offset:], shape=(batch, n_out), strides=(4 * ys, 4)).copy()
    mask = np.ones(yh.shape, bool)
    np.lib.stride_tricks.as_strided(mask[offset:], shape=(batch, n_out), strides=(ys, 1))[...] = False
    assert (yh[mask] == CANARY).all(), "write outside the output range"
    return out[0] if x_np.ndim == 1 else out


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
def test_config1_1d_n4096_q8(cuda_device, design):
    x, ws = inputs.make_config(1)
    w = ws[8]
    y_ref, s_ref = oracle.conv1d_f32(x, w)
    assert y_ref.shape == (4089,)
    assert_close_f32(run_1d(x, w, design, cuda_device), y_ref, s_ref, "config 1")


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("q", list(range(1, 33)))
def test_1d_every_filter_length(cuda_device, design, q):
    x, ws = inputs.gen_1d_f32(11000, [q], seed=40 + q)
    y_ref, s_ref = oracle.conv1d_f32(x, ws[q])
    assert_close_f32(run_1d(x, ws[q], design, cuda_device), y_ref, s_ref, "q=%d" % q)


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("q", [1, 4, 5, 16, 31, 32])
@pytest.mark.parametrize("extra", [0, 1, 2, 3, 75, 76, 77, 607, 608, 609, 4863, 4864, 4865, 9731])
def test_1d_ragged_sizes(cuda_device, design, q, extra):
    n = q + extra           # n_out = extra + 1: single output, tile and warp-tile edges, ragged tails
    x, ws = inputs.gen_1d_f32(n, [q], seed=1000 + n)
    y_ref, s_ref = oracle.conv1d_f32(x, ws[q])
    assert_close_f32(run_1d(x, ws[q], design, cuda_device), y_ref, s_ref, "n=%d q=%d" % (n, q))


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("offset", [1, 2, 3])
def test_1d_unaligned_pointers_and_batch_strides(cuda_device, design, offset):
    rng = np.random.default_rng(7)
    x = (rng.random((3, 7001), dtype=np.float32) * 2 - 1).astype(np.float32)
    w = (rng.random(9, dtype=np.float32) * 2 - 1).astype(np.float32)
    y = run_1d(x, w, design, cuda_device, batch_stride=7013, offset=offset)
    for b in range(3):
        y_ref, s_ref = oracle.conv1d_f32(x[b], w)
        assert_close_f32(y[b], y_ref, s_ref, "batch %d" % b)


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("q", [1, 4, 13, 16, 32])
@pytest.mark.parametrize("n_out", [4 * 4864, 4 * 4864 + 1, 7 * 4864 - 1, 100003, 300 * 4864 + 77])
def test_1d_many_tiles_sizes(cuda_device, design, q, n_out):
    """Aligned signals of many tiles (bulk-copy staging): whole tiles, ragged last tile, more tiles than
    CTAs resident at once."""
    n = n_out + q - 1
    x, ws = inputs.gen_1d_f32(n, [q], seed=2000 + q)
    y_ref, s_ref = oracle.conv1d_f32(x, ws[q])
    assert_close_f32(run_1d(x, ws[q], design, cuda_device), y_ref, s_ref, "n_out=%d q=%d" % (n_out, q))
    assert B.device_status() == 0


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("q", [5, 8, 17, 32])
@pytest.mark.parametrize("tiles", [1, 2, 3, 4, 5, 8])
def test_1d_output_count_a_whole_number_of_tiles(cuda_device, design, q, tiles):
    """n_out an exact multiple of the 1216-output tile: the tile after the last one has no outputs, yet the signal's
    last q-1 inputs lie in it.  One signal, and a batch (a block then walks on to the next signal)."""
    n_out = 1216 * tiles
    n = n_out + q - 1
    x, ws = inputs.gen_1d_f32(n, [q], seed=2500 + q + tiles)
    y_ref, s_ref = oracle.conv1d_f32(x, ws[q])
    assert_close_f32(run_1d(x, ws[q], design, cuda_device), y_ref, s_ref, "n_out=%d q=%d" % (n_out, q))
    rng = np.random.default_rng(2600 + q + tiles)
    xb = (rng.random((70000 // n + 3, n), dtype=np.float32) * 2 - 1).astype(np.float32)
    yb = run_1d(xb, ws[q], design, cuda_device, batch_stride=(n + 3) // 4 * 4)
    for b in range(xb.shape[0]):
        y_ref, s_ref = oracle.conv1d_f32(xb[b], ws[q])
        assert_close_f32(yb[b], y_ref, s_ref, "batch %d" % b)
    assert B.device_status() == 0


@pytest.mark.parametrize("design", STRIDED_1D, ids=_ids)
@pytest.mark.parametrize("q", [5, 8, 32])
@pytest.mark.parametrize("tiles", [1, 2, 3, 4])
def test_1d_stride2_output_count_a_whole_number_of_tiles(cuda_device, design, q, tiles):
    n_out = 608 * tiles
    for n in (2 * (n_out - 1) + q, 2 * (n_out - 1) + q + 1):
        x, ws = inputs.gen_1d_f32(n, [q], seed=2700 + q + tiles)
        y_ref, s_ref = oracle.conv1d_f32_strided(x, ws[q], 2)
        assert y_ref.size == n_out
        y = B.conv1d(torch.from_numpy(x).to(cuda_device), ws[q], design, stride=2)
        torch.cuda.synchronize()
        assert_close_f32(y.cpu().numpy(), y_ref, s_ref, "n=%d q=%d" % (n, q))
        xb = np.stack([x, x[::-1].copy(), -x])
        yd = B.conv1d(torch.from_numpy(xb).to(cuda_device), ws[q], design, stride=2)
        torch.cuda.synchronize()
        for b in range(3):
            y_ref, s_ref = oracle.conv1d_f32_strided(xb[b], ws[q], 2)
            assert_close_f32(yd[b].cpu().numpy(), y_ref, s_ref, "batch %d" % b)
    assert B.device_status() == 0


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
def test_1d_many_tiles_batch(cuda_device, design):
    # aligned batch strides: the last tile of every signal is ragged and sits in the middle of a CTA's work list
    rng = np.random.default_rng(9)
    x = (rng.random((5, 50001), dtype=np.float32) * 2 - 1).astype(np.float32)
    w = (rng.random(16, dtype=np.float32) * 2 - 1).astype(np.float32)
    y = run_1d(x, w, design, cuda_device, batch_stride=50004)
    for b in range(5):
        y_ref, s_ref = oracle.conv1d_f32(x[b], w)
        assert_close_f32(y[b], y_ref, s_ref, "batch %d" % b)
    assert B.device_status() == 0


# ---- batches of tiny signals: the paper's own experiment shape (Section 6), small unfolded arrays side by side
ALL_DESIGNS = DESIGNS + OTHER_DESIGNS


def tiles_reference(x2, w):
    """Oracle for a batch of short signals in ONE call: laid end to end they form one long signal whose valid
    convolution holds, at position b*n + c (c < n-q+1), exactly output c of signal b."""
    batch, n = x2.shape
    q = w.shape[0]
    y, s = oracle.conv1d_f32(x2.reshape(-1), w)
    idx = (np.arange(batch)[:, None] * n + np.arange(n - q + 1)[None, :])
    return y[idx], s[idx]


@pytest.mark.parametrize("design", ALL_DESIGNS, ids=_ids)
@pytest.mark.parametrize("q", [1, 2, 5, 8])
@pytest.mark.parametrize("c_out", [1, 2, 4, 15, 16, 17, 25, 32])
def test_1d_tiny_signals_all_designs(cuda_device, design, q, c_out):
    n = c_out + q - 1
    rng = np.random.default_rng(2900 + 64 * q + c_out)
    w = (rng.random(q, dtype=np.float32) * 2 - 1).astype(np.float32)
    for batch, stride in ((2, None), (7, n + 3), (1000, None), (4099, n + 1)):
        x = (rng.random((batch, n), dtype=np.float32) * 2 - 1).astype(np.float32)
        y = run_1d(x, w, design, cuda_device, batch_stride=stride)
        y_ref, s_ref = tiles_reference(x, w)
        assert_close_f32(y, y_ref, s_ref, "%s q=%d C=%d batch=%d" % (_ids(design), q, c_out, batch))


@pytest.mark.parametrize("design", ALL_DESIGNS, ids=_ids)
@pytest.mark.parametrize("q,c_out", [(5, 16), (2, 16), (8, 9), (3, 30)])
def test_1d_tiny_signals_dense_and_shifted_layouts(cuda_device, design, q, c_out):
    """The tiny-signal kernels move densely packed batches as whole 128-bit words and fall back to a gather for any
    other layout: packed batches of several sizes (whole passes, a ragged last pass, fewer signals than one pass),
    the same batches starting 1, 2 and 3 elements off a 16-byte boundary, and a stride one element longer."""
    n = c_out + q - 1
    rng = np.random.default_rng(4000 + 10 * q + c_out)
    w = (rng.random(q, dtype=np.float32) * 2 - 1).astype(np.float32)
    for batch in (3, 64, 257, 1536, 5001):
        x = (rng.random((batch, n), dtype=np.float32) * 2 - 1).astype(np.float32)
        y_ref, s_ref = tiles_reference(x, w)
        for offset, stride in ((0, None), (1, None), (2, None), (3, None), (0, n + 1)):
            y = run_1d(x, w, design, cuda_device, batch_stride=stride, offset=offset)
            assert_close_f32(y, y_ref, s_ref, "%s q=%d C=%d batch=%d offset=%d stride=%s"
                             % (_ids(design), q, c_out, batch, offset, stride))
    assert B.device_status() == 0


@pytest.mark.parametrize("design", ALL_DESIGNS, ids=_ids)
def test_1d_tiny_signals_exact_integers_and_non_finite(cuda_device, design):
    rng = np.random.default_rng(2950)
    x = rng.integers(-50, 51, (3000, 20)).astype(np.float32)
    w = rng.integers(-9, 10, 5).astype(np.float32)
    y_ref, _ = tiles_reference(x, w)
    np.testing.assert_array_equal(run_1d(x, w, design, cuda_device).astype(np.float64), y_ref)
    xf = (rng.random((500, 20), dtype=np.float32) * 2 - 1).astype(np.float32)
    xf[3, 0], xf[3, 19], xf[100, 7], xf[499, 15] = np.inf, np.nan, -np.inf, np.nan
    wf = (rng.random(5, dtype=np.float32) * 2 - 1).astype(np.float32)
    with np.errstate(invalid="ignore"):
        refs = [oracle.conv1d_f32(row, wf) for row in xf]
    y = run_1d(xf, wf, design, cuda_device)
    _assert_same_where_finite(y, np.stack([r[0] for r in refs]), np.stack([r[1] for r in refs]), "non-finite")


@pytest.mark.parametrize("q", [2, 5])
def test_1d_paper_experiment_shape_full_size(cuda_device, q):
    """More than ten million independent convolutions of 16 outputs each (Section 6), filter sizes 2 and 5, all six
    designs: EVERY output against the oracle."""
    tiles, c_out = 10 * (1 << 20), 16
    n = c_out + q - 1
    x, ws = inputs.gen_1d_f32(tiles * n, [q], seed=60 + q)
    x = x.reshape(tiles, n)
    y_ref, s_ref = tiles_reference(x, ws[q])
    xd = torch.from_numpy(x).to(cuda_device)
    yd = torch.empty((tiles, c_out), dtype=torch.float32, device=cuda_device)
    for design in ALL_DESIGNS:
        yd.fill_(CANARY)
        B.conv1d(xd, ws[q], design, out=yd)
        torch.cuda.synchronize()
        y = yd.cpu().numpy()
        for lo in range(0, tiles, 1 << 21):
            assert_close_f32(y[lo:lo + (1 << 21)], y_ref[lo:lo + (1 << 21)], s_ref[lo:lo + (1 << 21)],
                             "%s q=%d tiles %d.." % (_ids(design), q, lo))
    assert B.device_status() == 0


@pytest.mark.parametrize("design", OTHER_DESIGNS, ids=_ids)
@pytest.mark.parametrize("q", [1, 2, 3, 5, 8, 13, 16, 17, 31, 32])
def test_1d_other_designs_filter_lengths(cuda_device, design, q):
    x, ws = inputs.gen_1d_f32(21000, [q], seed=500 + q)
    y_ref, s_ref = oracle.conv1d_f32(x, ws[q])
    assert_close_f32(run_1d(x, ws[q], design, cuda_device), y_ref, s_ref, "q=%d" % q)


@pytest.mark.parametrize("design", OTHER_DESIGNS, ids=_ids)
@pytest.mark.parametrize("extra", [0, 1, 18, 19, 31, 32, 607, 608, 1215, 1216, 2431, 2432, 2433])
def test_1d_other_designs_ragged_sizes_and_config1(cuda_device, design, extra):
    q = 5
    x, ws = inputs.gen_1d_f32(q + extra, [q], seed=600 + extra)
    y_ref, s_ref = oracle.conv1d_f32(x, ws[q])
    assert_close_f32(run_1d(x, ws[q], design, cuda_device), y_ref, s_ref, "n_out=%d" % (extra + 1))
    if extra == 0:
        x1, ws1 = inputs.make_config(1)
        y_ref, s_ref = oracle.conv1d_f32(x1, ws1[8])
        assert_close_f32(run_1d(x1, ws1[8], design, cuda_device), y_ref, s_ref, "config 1")
        xb = np.stack([x1[:3000], x1[1000:4000]])
        yb = run_1d(xb, ws1[8], design, cuda_device, batch_stride=3001, offset=1)
        for b in range(2):
            y_ref, s_ref = oracle.conv1d_f32(xb[b], ws1[8])
            assert_close_f32(yb[b], y_ref, s_ref, "batch %d" % b)


@pytest.mark.parametrize("design", OTHER_DESIGNS, ids=_ids)
def test_1d_other_designs_exact_integers_and_non_finite(cuda_device, design):
    rng = np.random.default_rng(18)
    x = rng.integers(-50, 51, 9000).astype(np.float32)
    w = rng.integers(-9, 10, 7).astype(np.float32)
    y_ref, _ = oracle.conv1d_f32(x, w)
    np.testing.assert_array_equal(run_1d(x, w, design, cuda_device).astype(np.float64), y_ref)
    x, ws = inputs.gen_1d_f32(9000, [6], seed=19)
    x[[3, 607, 608, 4000, 8999]] = [np.inf, np.nan, -np.inf, np.inf, np.nan]
    with np.errstate(invalid="ignore"):
        y_ref, s_ref = oracle.conv1d_f32(x, ws[6])
    _assert_same_where_finite(run_1d(x, ws[6], design, cuda_device), y_ref, s_ref, "non-finite")


def test_other_designs_are_1d_fp32_only(cuda_device):
    x2 = torch.zeros((1, 40, 40), device=cuda_device)
    for design in OTHER_DESIGNS:
        with pytest.raises(B.SysconvError) as e:
            B.conv2d(x2, np.ones((3, 3), np.float32), design)
        assert e.value.status == 2
        with pytest.raises(B.SysconvError) as e:
            B.conv1d(torch.zeros(100, dtype=torch.uint8, device=cuda_device), np.ones(3, np.int8), design)
        assert e.value.status == 2


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
def test_1d_exact_on_small_integers(cuda_device, design):
    # integer-valued data: every design must reproduce the sums exactly, whatever its order
    rng = np.random.default_rng(8)
    x = rng.integers(-50, 51, 30000).astype(np.float32)
    w = rng.integers(-9, 10, 13).astype(np.float32)
    y_ref, _ = oracle.conv1d_f32(x, w)
    np.testing.assert_array_equal(run_1d(x, w, design, cuda_device).astype(np.float64), y_ref)


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("q", [4, 16, 32])
def test_config2_1d_full_size(cuda_device, design, q):
    """N = 2^26, compared on every output, in the launch configuration bench.py times."""
    x, ws = inputs.make_config(2)
    w = ws[q]
    xd = torch.from_numpy(x).to(cuda_device)
    yd = B.conv1d(xd, w, design)
    torch.cuda.synchronize()
    y_gpu = yd.cpu().numpy()
    del xd, yd
    y_ref, s_ref = oracle.conv1d_f32(x, w)
    assert y_gpu.shape == y_ref.shape == ((1 << 26) - q + 1,)
    chunk = 1 << 23
    for lo in range(0, y_ref.size, chunk):
        hi = min(lo + chunk, y_ref.size)
        assert_close_f32(y_gpu[lo:hi], y_ref[lo:hi], s_ref[lo:hi], "config 2 q=%d [%d,%d)" % (q, lo, hi))


# ------------------------------------------------------------------------ 2-D


def run_2d(x_np, w_np, design, device, x_pitch=None, y_pitch=None, x_off=0, y_off=0):
    """x_np: (batch, h, w) float32 or uint8; returns y (batch, oh, ow); checks canaries."""
    batch, h, wd = x_np.shape
    p, q = w_np.shape
    oh, ow = h - p + 1, wd - q + 1
    is_f = x_np.dtype == np.float32
    x_pitch = x_pitch or wd
    y_pitch = y_pitch or ow
    xb = torch.zeros(x_off + batch * h * x_pitch + 16, dtype=torch.float32 if is_f else torch.uint8, device=device)
    canary = CANARY if is_f else 123456789
    yb = torch.full((y_off + batch * oh * y_pitch + 64,), canary, dtype=torch.float32 if is_f else torch.int32,
                    device=device)
    xv = xb[x_off: x_off + batch * h * x_pitch].view(batch, h, x_pitch)
    xv[:, :, :wd] = torch.from_numpy(x_np).to(device)
    st = B.sysconv2d(xb.data_ptr() + x_off * xb.element_size(), wd, h, x_pitch, h * x_pitch,
                     np.ascontiguousarray(w_np), q, p, yb.data_ptr() + y_off * 4, y_pitch, oh * y_pitch, batch,
                     B.F32 if is_f else B.U8S8_S32, design, torch.cuda.current_stream().cuda_stream)
    assert st == 0, B.status_string(st)
    torch.cuda.synchronize()
    yh = yb.cpu().numpy()
    body = yh[y_off: y_off + batch * oh * y_pitch].reshape(batch, oh, y_pitch)
    out = body[:, :, :ow].copy()
    assert (body[:, :, ow:] == canary).all(), "write into the pitch padding"
    assert (yh[:y_off] == canary).all() and (yh[y_off + batch * oh * y_pitch:] == canary).all()
    return out


def check_2d(x_np, w_np, design, device, **kw):
    y = run_2d(x_np, w_np, design, device, **kw)
    for b in range(x_np.shape[0]):
        if x_np.dtype == np.float32:
            y_ref, s_ref = oracle.conv2d_f32(x_np[b], w_np)
            assert_close_f32(y[b], y_ref, s_ref, "image %d" % b)
        else:
            np.testing.assert_array_equal(y[b], oracle.conv2d_u8s8_s32(x_np[b], w_np))


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
def test_config3_2d_1920x1080_5x5(cuda_device, design):
    x, ws = inputs.make_config(3)
    check_2d(x, ws[(5, 5)], design, cuda_device)


FILTERS_2D = [(1, 1), (1, 5), (5, 1), (2, 2), (3, 3), (5, 5), (7, 7), (9, 9), (15, 15), (2, 11), (13, 4), (15, 1),
              (1, 15), (8, 6)]


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("pq", FILTERS_2D, ids=lambda f: "%dx%d" % f)
def test_2d_f32_filter_shapes(cuda_device, design, pq):
    p, q = pq
    x, ws = inputs.gen_2d_f32(300, 75, [pq], seed=50 + p * 16 + q, batch=2)
    check_2d(x, ws[pq], design, cuda_device)


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("hw", [(0, 0), (1, 0), (0, 1), (2, 3), (31, 127), (32, 128), (33, 129), (40, 255), (7, 513)])
@pytest.mark.parametrize("pq", [(3, 3), (5, 7), (15, 15)], ids=lambda f: "%dx%d" % f)
def test_2d_f32_ragged_image_sizes(cuda_device, design, hw, pq):
    # output sizes (hw[0]+1) x (hw[1]+1): single output, strip/band edges, ragged tails
    p, q = pq
    x, ws = inputs.gen_2d_f32(q + hw[1], p + hw[0], [pq], seed=77 + hw[0] + hw[1])
    check_2d(x, ws[pq], design, cuda_device)


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("pitches", [(203, 199, 1, 1), (204, 198, 0, 2), (201, 200, 3, 0), (208, 196, 4, 4)])
def test_2d_f32_pitches_and_alignment(cuda_device, design, pitches):
    xp, yp, xo, yo = pitches
    x, ws = inputs.gen_2d_f32(200, 41, [(5, 5)], seed=91, batch=2)
    check_2d(x, ws[(5, 5)], design, cuda_device, x_pitch=xp, y_pitch=yp, x_off=xo, y_off=yo)


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("k", [3, 9, 15])
def test_config5_reduced_and_exact_integers(cuda_device, design, k):
    x, ws = inputs.make_config(5, scale=dict(width=520, height=300, batch=2, filters=[k]))
    check_2d(x, ws[(k, k)], design, cuda_device)
    rng = np.random.default_rng(k)
    xi = rng.integers(0, 16, (1, 100, 260)).astype(np.float32)
    wi = rng.integers(-4, 5, (k, k)).astype(np.float32)
    y = run_2d(xi, wi, design, cuda_device)
    np.testing.assert_array_equal(y[0].astype(np.float64), oracle.conv2d_f32(xi[0], wi)[0])


@pytest.mark.parametrize("k", [3, 9, 15])
def test_config5_full_size_every_output(cuda_device, k):
    """16 x 4096 x 4096 in the bench's launch configuration: EVERY output of every image, for the three designs,
    against the oracle (one oracle pass per image, the three designs compared with it in turn)."""
    x, ws = inputs.make_config(5, scale=dict(filters=[k]))
    w = ws[(k, k)]
    xd = torch.from_numpy(x).to(cuda_device)
    oh = ow = 4096 - k + 1
    outs = {}
    for design in DESIGNS:
        # pitch rounded up to 4 elements, as bench.py allocates its outputs; the padding keeps its canary
        yd = torch.full((16, oh, (ow + 3) // 4 * 4), CANARY, dtype=torch.float32, device=cuda_device)
        B.conv2d(xd, w, design, out=yd[:, :, :ow])
        outs[design] = yd
    torch.cuda.synchronize()
    del xd
    for b in range(16):
        y_ref, s_ref = oracle.conv2d_f32(x[b], w)
        for design in DESIGNS:
            got = outs[design][b].cpu().numpy()
            assert (got[:, ow:] == CANARY).all(), "write into the pitch padding"
            assert_close_f32(got[:, :ow], y_ref, s_ref, "config 5 k=%d design %s image %d" % (k, _ids(design), b))


# Problems of a few waves of blocks get short bands chosen by the number of waves they give: ragged right edges
# (width not a multiple of the 16-byte unit, inside an aligned pitch), ragged last bands, several images, and the
# same data once more from unaligned rows.
@pytest.mark.parametrize("design", [B.OS, B.IS], ids=_ids)
@pytest.mark.parametrize("pq", [(5, 5), (3, 3), (1, 1), (2, 11), (5, 4), (1, 15), (4, 6)], ids=lambda f: "%dx%d" % f)
@pytest.mark.parametrize("size", [(517, 83, 3), (1001, 241, 1), (1920, 131, 2), (130, 40, 1), (16, 16, 5)],
                         ids=lambda t: "%dx%dx%d" % t)
def test_2d_f32_small_problems(cuda_device, design, pq, size):
    wd, h, batch = size
    p, q = pq
    if wd < q or h < p:
        pytest.skip("image smaller than the filter")
    x, ws = inputs.gen_2d_f32(wd, h, [pq], seed=1300 + 16 * p + q + wd, batch=batch)
    xp = (wd + 3) // 4 * 4
    y_al = run_2d(x, ws[pq], design, cuda_device, x_pitch=xp, y_pitch=wd)
    for b in range(batch):
        y_ref, s_ref = oracle.conv2d_f32(x[b], ws[pq])
        assert_close_f32(y_al[b], y_ref, s_ref, "image %d" % b)
    y_un = run_2d(x, ws[pq], design, cuda_device, x_pitch=xp + 1, y_pitch=wd)
    for b in range(batch):
        y_ref, s_ref = oracle.conv2d_f32(x[b], ws[pq])
        assert_close_f32(y_un[b], y_ref, s_ref, "image %d, unaligned rows" % b)
    assert B.device_status() == 0


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("pq", [(3, 3), (7, 7), (1, 1), (5, 13), (7, 15), (2, 4), (15, 15), (11, 9)], ids=lambda f: "%dx%d" % f)
@pytest.mark.parametrize("size", [(1101, 83, 2), (3840, 140, 1), (1000, 41, 1), (4097, 64, 1), (64, 20, 3), (496, 35, 1), (497, 36, 2)],
                         ids=lambda t: "%dx%dx%d" % t)
def test_2d_u8_small_problems(cuda_device, design, pq, size):
    wd, h, batch = size
    p, q = pq
    x, ws = inputs.gen_2d_u8s8(wd, h, [pq], seed=1400 + 16 * p + q + wd, batch=batch)
    xp = (wd + 15) // 16 * 16
    check_2d(x, ws[pq], design, cuda_device, x_pitch=xp)
    check_2d(x, ws[pq], design, cuda_device, x_pitch=xp + 4, y_off=1)      # rows aligned to 4 bytes only, unaligned outputs
    assert B.device_status() == 0


# The fp32 OS / IS kernels for small filters (P*Q <= 25) have a form with eight PEs per lane that only large
# problems reach (256-column strips x images x 8-row groups >= 4736); these cases are sized for it, with a ragged
# right edge and a ragged last band.
@pytest.mark.parametrize("design", [B.OS, B.IS], ids=_ids)
@pytest.mark.parametrize("pq", [(5, 5), (2, 11), (1, 15), (4, 6), (3, 8), (5, 4), (1, 1), (2, 2), (3, 3), (12, 2), (15, 1)],
                         ids=lambda f: "%dx%d" % f)
def test_2d_f32_small_filters_eight_pes_per_lane(cuda_device, design, pq):
    p, q = pq
    wd, h, batch = 1301, 803, 8
    assert ((wd - q + 1 + 255) // 256) * batch * ((h - p + 1 + 7) // 8) >= 4736
    x, ws = inputs.gen_2d_f32(wd, h, [pq], seed=1200 + 16 * p + q, batch=batch)
    check_2d(x, ws[pq], design, cuda_device)
    check_2d(x[:6, :, :1290], ws[pq], design, cuda_device, x_pitch=1292, y_pitch=1292, x_off=4, y_off=4)


# ------------------------------------------------------------------------ non-finite inputs


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("q", [3, 5, 13, 16, 31, 32])
def test_1d_non_finite_inputs_stay_inside_their_windows(cuda_device, design, q):
    x, ws = inputs.gen_1d_f32(30000, [q], seed=3000 + q)
    x[[17, 4863, 4864, 9000, 9001, 20000, 29990]] = [np.inf, -np.inf, np.nan, np.inf, np.inf, np.nan, np.inf]
    with np.errstate(invalid="ignore"):
        y_ref, s_ref = oracle.conv1d_f32(x, ws[q])
    _assert_same_where_finite(run_1d(x, ws[q], design, cuda_device), y_ref, s_ref, "1-D q=%d" % q)


BAD_PIXELS = ((0, 0, np.inf), (40, 127, np.nan), (41, 128, -np.inf), (63, 255, np.inf), (64, 256, np.nan),
              (119, 299, np.inf), (100, 5, np.inf))


@pytest.mark.parametrize("pq", [(6, 5), (7, 8), (8, 7), (9, 8), (9, 5), (15, 4), (14, 3), (11, 4), (13, 2), (1, 9), (1, 15), (2, 12),
                                (2, 15), (1, 14)],
                         ids=lambda f: "%dx%d" % f)
def test_2d_ws_register_form_taller_filters(cuda_device, pq):
    """The all-register weight-stationary form takes every filter of at most 8 columns whose window of P+3 rows fits
    96 registers: several slices of 31 segments, a ragged last slice, bands that end inside a four-row pass, a batch,
    and rows that do not start 16-byte aligned."""
    p, q = pq
    x, ws = inputs.gen_2d_f32(1030, 90, [pq], seed=700 + 16 * p + q, batch=2)
    check_2d(x, ws[pq], B.WS, cuda_device)
    check_2d(x[:, :67, :517], ws[pq], B.WS, cuda_device, x_pitch=519, y_pitch=517)
    assert B.device_status() == 0


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("pq", [(3, 3), (5, 5), (8, 6), (9, 9), (10, 7), (15, 15), (4, 8), (12, 12)],
                         ids=lambda f: "%dx%d" % f)
def test_2d_non_finite_inputs_stay_inside_their_windows(cuda_device, design, pq):
    """A non-finite pixel affects exactly the outputs whose window holds it -- except for the two documented
    zero-tap paddings (OS with P >= 12: one more row above and below; WS with Q % 4 != 0: up to three more columns
    to the left), where those extra outputs may be NaN and everything else must still be exact."""
    p, q = pq
    x, ws = inputs.gen_2d_f32(300, 120, [pq], seed=3100 + p)
    for r, c, v in BAD_PIXELS:
        x[0, r, c] = v
    with np.errstate(invalid="ignore"):
        y_ref, s_ref = oracle.conv2d_f32(x[0], ws[pq])
    y = run_2d(x, ws[pq], design, cuda_device)[0].astype(np.float64)
    oh, ow = y_ref.shape
    may_differ = np.zeros((oh, ow), bool)
    for rb, cb, _ in BAD_PIXELS:
        c_lo, c_hi = max(cb - q + 1, 0), min(cb, ow - 1)
        if design == B.OS and p >= 12:
            for r in (rb - p, rb + 1):
                if 0 <= r < oh and c_lo <= c_hi:
                    may_differ[r, c_lo:c_hi + 1] = True
        if design == B.WS and q % 4:
            qp = (q + 3) // 4 * 4
            r_lo, r_hi = max(rb - p + 1, 0), min(rb, oh - 1)
            cc_lo, cc_hi = max(cb - qp + 1, 0), min(cb - q, ow - 1)
            if r_lo <= r_hi and cc_lo <= cc_hi:
                may_differ[r_lo:r_hi + 1, cc_lo:cc_hi + 1] = True
    strict = ~may_differ
    fin = np.isfinite(y_ref)
    assert (np.isfinite(y[strict]) == fin[strict]).all(), "non-finite outputs differ outside the documented cells"
    ok = strict & fin
    assert (np.abs(y[ok] - y_ref[ok]) <= TOL * s_ref[ok]).all()
    loose = may_differ & fin & np.isfinite(y)
    assert (np.abs(y[loose] - y_ref[loose]) <= TOL * s_ref[loose]).all()


# The fp32 weight-stationary 2-D kernel with one array per lane runs when the problem gives its one-warp CTAs
# enough work (bands of 128 rows x segments of >= 128 columns x images >= 592); these cases are sized for it.
WS_LANE_BATCH = 150


@pytest.mark.parametrize("pq", [(1, 1), (3, 3), (5, 5), (2, 11), (13, 4), (9, 9), (15, 15), (7, 10), (15, 1), (1, 15),
                                (4, 9), (6, 2)], ids=lambda f: "%dx%d" % f)
def test_2d_ws_one_array_per_lane_kernel(cuda_device, pq):
    p, q = pq
    x, ws = inputs.gen_2d_f32(261, 150, [pq], seed=900 + 16 * p + q, batch=WS_LANE_BATCH)
    assert ((150 - p + 1 + 127) // 128) * ((261 - q + 1 + 127) // 128) * WS_LANE_BATCH >= 592
    check_2d(x, ws[pq], B.WS, cuda_device)


def test_2d_ws_one_array_per_lane_kernel_layouts_and_non_finite(cuda_device):
    pq = (5, 7)
    x, ws = inputs.gen_2d_f32(300, 150, [pq], seed=77, batch=WS_LANE_BATCH)
    assert ((150 - 5 + 1 + 127) // 128) * ((300 - 7 + 1 + 127) // 128) * WS_LANE_BATCH >= 592
    check_2d(x, ws[pq], B.WS, cuda_device, x_pitch=307, y_pitch=299, x_off=1, y_off=3)
    check_2d(x, ws[pq], B.WS, cuda_device, x_pitch=304, y_pitch=296, x_off=4, y_off=4)
    # this kernel applies no zero taps: a non-finite pixel must affect exactly the outputs whose window holds it
    for r, c, v in BAD_PIXELS:
        x[3, r, c] = v
    with np.errstate(invalid="ignore"):
        y_ref, s_ref = oracle.conv2d_f32(x[3], ws[pq])
    y = run_2d(x, ws[pq], B.WS, cuda_device)[3].astype(np.float64)
    fin = np.isfinite(y_ref)
    assert (np.isfinite(y) == fin).all()
    assert (np.abs(y[fin] - y_ref[fin]) <= TOL * s_ref[fin]).all()


# ------------------------------------------------------------------------ stride 2 (Table 2, cell 6)

STRIDED_DESIGNS = [B.OS, B.IS]


@pytest.mark.parametrize("design", STRIDED_DESIGNS, ids=_ids)
@pytest.mark.parametrize("q", [1, 2, 3, 4, 5, 7, 8, 15, 16, 31, 32])
def test_1d_stride2_filter_sizes(cuda_device, design, q):
    n = 3 * 2432 + 1216 + 37          # several CTA tiles, one ragged
    x, ws = inputs.gen_1d_f32(n, [q], seed=300 + q)
    y = B.conv1d(torch.from_numpy(x).to(cuda_device), ws[q], design, stride=2)
    torch.cuda.synchronize()
    y_ref, s_ref = oracle.conv1d_f32_strided(x, ws[q], 2)
    assert y.shape == y_ref.shape
    assert_close_f32(y.cpu().numpy(), y_ref, s_ref, "stride 2, q=%d" % q)


@pytest.mark.parametrize("design", STRIDED_DESIGNS, ids=_ids)
@pytest.mark.parametrize("n", [5, 6, 7, 8, 303, 304, 305, 607, 608, 609, 639, 640, 641, 1216, 1217, 1247, 1248, 1249,
                               2431, 2432, 2433, 2463, 2464, 2465, 4864 + 33])
def test_1d_stride2_lengths_around_tile_edges(cuda_device, design, n):
    q = 5
    x, ws = inputs.gen_1d_f32(n, [q], seed=400 + n % 97)
    y = B.conv1d(torch.from_numpy(x).to(cuda_device), ws[q], design, stride=2)
    torch.cuda.synchronize()
    y_ref, s_ref = oracle.conv1d_f32_strided(x, ws[q], 2)
    assert y.shape == y_ref.shape
    assert_close_f32(y.cpu().numpy(), y_ref, s_ref, "stride 2, n=%d" % n)


@pytest.mark.parametrize("design", STRIDED_DESIGNS, ids=_ids)
def test_1d_stride2_batch_unaligned_and_canaries(cuda_device, design):
    q, n, batch = 9, 7001, 3
    x, ws = inputs.gen_1d_f32(n * batch, [q], seed=77)
    x = x.reshape(batch, n)
    n_out = (n - q) // 2 + 1
    for x_off, y_off, xs, ys in [(0, 0, n, n_out), (1, 3, n + 3, n_out + 5), (4, 4, n + 4, n_out + 4)]:
        xb = torch.zeros(x_off + batch * xs + 8, dtype=torch.float32, device=cuda_device)
        yb = torch.full((y_off + batch * ys + 8,), CANARY, dtype=torch.float32, device=cuda_device)
        xb[x_off: x_off + batch * xs].view(batch, xs)[:, :n] = torch.from_numpy(x).to(cuda_device)
        st = B.sysconv1d_strided(xb.data_ptr() + 4 * x_off, n, xs, ws[q], q, 2, yb.data_ptr() + 4 * y_off, ys, batch,
                                 B.F32, design, torch.cuda.current_stream().cuda_stream)
        assert st == 0, B.status_string(st)
        torch.cuda.synchronize()
        yh = yb.cpu().numpy()
        body = yh[y_off: y_off + batch * ys].reshape(batch, ys)
        assert (body[:, n_out:] == CANARY).all() and (yh[:y_off] == CANARY).all()
        assert (yh[y_off + batch * ys:] == CANARY).all()
        for b in range(batch):
            y_ref, s_ref = oracle.conv1d_f32_strided(x[b], ws[q], 2)
            assert_close_f32(body[b, :n_out], y_ref, s_ref, "signal %d" % b)


def test_1d_stride2_large_sampled(cuda_device):
    n, q = (1 << 24) + 3, 16
    x, ws = inputs.gen_1d_f32(n, [q], seed=9)
    xd = torch.from_numpy(x).to(cuda_device)
    rng = np.random.default_rng(5)
    n_out = (n - q) // 2 + 1
    pos = np.unique(np.concatenate([rng.integers(0, n_out, 4000), np.arange(64), np.arange(n_out - 64, n_out)]))
    y_ref, s_ref = oracle.conv1d_f32_at(x, ws[q], 2 * pos)
    for design in STRIDED_DESIGNS:
        y = B.conv1d(xd, ws[q], design, stride=2)
        torch.cuda.synchronize()
        assert y.numel() == n_out
        assert_close_f32(y.cpu().numpy()[pos], y_ref, s_ref, "sampled, %s" % B.DESIGN_NAMES[design])


def run_2d_s2(x_np, w_np, design, device, x_pitch=None, y_pitch=None, x_off=0, y_off=0):
    batch, h, wd = x_np.shape
    p, q = w_np.shape
    oh, ow = (h - p) // 2 + 1, (wd - q) // 2 + 1
    x_pitch = x_pitch or wd
    y_pitch = y_pitch or ow
    xb = torch.zeros(x_off + batch * h * x_pitch + 16, dtype=torch.float32, device=device)
    yb = torch.full((y_off + batch * oh * y_pitch + 64,), CANARY, dtype=torch.float32, device=device)
    xb[x_off: x_off + batch * h * x_pitch].view(batch, h, x_pitch)[:, :, :wd] = torch.from_numpy(x_np).to(device)
    st = B.sysconv2d_strided(xb.data_ptr() + 4 * x_off, wd, h, x_pitch, h * x_pitch, np.ascontiguousarray(w_np), q, p,
                             2, 2, yb.data_ptr() + 4 * y_off, y_pitch, oh * y_pitch, batch, B.F32, design,
                             torch.cuda.current_stream().cuda_stream)
    assert st == 0, B.status_string(st)
    torch.cuda.synchronize()
    yh = yb.cpu().numpy()
    body = yh[y_off: y_off + batch * oh * y_pitch].reshape(batch, oh, y_pitch)
    assert (body[:, :, ow:] == CANARY).all(), "write into the pitch padding"
    assert (yh[:y_off] == CANARY).all() and (yh[y_off + batch * oh * y_pitch:] == CANARY).all()
    return body[:, :, :ow].copy()


def check_2d_s2(x_np, w_np, design, device, **kw):
    y = run_2d_s2(x_np, w_np, design, device, **kw)
    for b in range(x_np.shape[0]):
        y_ref, s_ref = oracle.conv2d_f32_strided(x_np[b], w_np, 2)
        assert y[b].shape == y_ref.shape
        assert_close_f32(y[b], y_ref, s_ref, "image %d" % b)


@pytest.mark.parametrize("design", STRIDED_DESIGNS, ids=_ids)
@pytest.mark.parametrize("pq", [(p, q) for p in range(1, 8) for q in range(1, 8)], ids=lambda f: "%dx%d" % f)
def test_2d_stride2_all_filter_shapes(cuda_device, design, pq):
    x, ws = inputs.gen_2d_f32(533, 61, [pq], seed=500 + 8 * pq[0] + pq[1], batch=2)
    check_2d_s2(x, ws[pq], design, cuda_device)


@pytest.mark.parametrize("design", STRIDED_DESIGNS, ids=_ids)
@pytest.mark.parametrize("hw", [(0, 0), (1, 0), (0, 1), (1, 1), (2, 3), (9, 239), (10, 240), (11, 241), (12, 247),
                                (13, 248), (14, 249), (5, 255), (6, 256), (7, 257), (8, 1000)])
@pytest.mark.parametrize("pq", [(3, 3), (2, 5), (7, 7)], ids=lambda f: "%dx%d" % f)
def test_2d_stride2_sizes_around_strip_and_band_edges(cuda_device, design, pq, hw):
    p, q = pq
    h, wd = p + hw[0], q + hw[1]
    x, ws = inputs.gen_2d_f32(wd, h, [pq], seed=600 + h + wd, batch=1)
    check_2d_s2(x, ws[pq], design, cuda_device)


@pytest.mark.parametrize("design", STRIDED_DESIGNS, ids=_ids)
def test_2d_stride2_pitch_offsets_and_tall_image(cuda_device, design):
    x, ws = inputs.gen_2d_f32(301, 75, [(3, 3), (5, 4)], seed=71, batch=2)
    for pq in [(3, 3), (5, 4)]:
        check_2d_s2(x, ws[pq], design, cuda_device, x_pitch=307, y_pitch=155, x_off=1, y_off=1)
        check_2d_s2(x, ws[pq], design, cuda_device, x_pitch=304, y_pitch=152, x_off=4, y_off=4)
    x, ws = inputs.gen_2d_f32(70, 2100, [(7, 3)], seed=72, batch=1)
    check_2d_s2(x, ws[(7, 3)], design, cuda_device)


def test_2d_stride2_full_hd_sampled(cuda_device):
    x, ws = inputs.gen_2d_f32(1920, 1080, [(5, 5)], seed=73, batch=1)
    xd = torch.from_numpy(x).to(cuda_device)
    rng = np.random.default_rng(6)
    oh, ow = (1080 - 5) // 2 + 1, (1920 - 5) // 2 + 1
    rows = np.concatenate([rng.integers(0, oh, 3000), [0, 0, oh - 1, oh - 1]])
    cols = np.concatenate([rng.integers(0, ow, 3000), [0, ow - 1, 0, ow - 1]])
    y_ref, s_ref = oracle.conv2d_f32_at(x[0], ws[(5, 5)], 2 * rows, 2 * cols)
    for design in STRIDED_DESIGNS:
        y = B.conv2d(xd, ws[(5, 5)], design, stride=2)
        torch.cuda.synchronize()
        assert tuple(y.shape) == (1, oh, ow)
        assert_close_f32(y.cpu().numpy()[0][rows, cols], y_ref, s_ref, "sampled, %s" % B.DESIGN_NAMES[design])


# ------------------------------------------------------------------------ any strides (output-stationary array)


@pytest.mark.parametrize("stride", [3, 4, 5, 7, 16, 40])
@pytest.mark.parametrize("q", [1, 2, 3, 5, 8, 16, 31, 32])
def test_1d_any_stride(cuda_device, stride, q):
    for n in (q, q + 1, 777, 3 * 128 * stride + q + 5):
        x, ws = inputs.gen_1d_f32(n, [q], seed=3300 + q + stride)
        y = B.conv1d(torch.from_numpy(x).to(cuda_device), ws[q], B.OS, stride=stride)
        torch.cuda.synchronize()
        y_ref, s_ref = oracle.conv1d_f32_strided(x, ws[q], stride)
        assert y.shape == y_ref.shape
        assert_close_f32(y.cpu().numpy(), y_ref, s_ref, "stride %d, q=%d, n=%d" % (stride, q, n))


def test_1d_any_stride_batch_strides_and_canaries(cuda_device):
    q, n, batch, stride = 9, 7001, 3, 3
    x, ws = inputs.gen_1d_f32(n * batch, [q], seed=78)
    x = x.reshape(batch, n)
    n_out = (n - q) // stride + 1
    for x_off, y_off, xs, ys in [(0, 0, n, n_out), (1, 3, n + 3, n_out + 5)]:
        xb = torch.zeros(x_off + batch * xs + 8, dtype=torch.float32, device=cuda_device)
        yb = torch.full((y_off + batch * ys + 8,), CANARY, dtype=torch.float32, device=cuda_device)
        xb[x_off: x_off + batch * xs].view(batch, xs)[:, :n] = torch.from_numpy(x).to(cuda_device)
        st = B.sysconv1d_strided(xb.data_ptr() + 4 * x_off, n, xs, ws[q], q, stride, yb.data_ptr() + 4 * y_off, ys, batch,
                                 B.F32, B.OS, torch.cuda.current_stream().cuda_stream)
        assert st == 0, B.status_string(st)
        torch.cuda.synchronize()
        yh = yb.cpu().numpy()
        body = yh[y_off: y_off + batch * ys].reshape(batch, ys)
        assert (body[:, n_out:] == CANARY).all() and (yh[:y_off] == CANARY).all()
        assert (yh[y_off + batch * ys:] == CANARY).all()
        for b in range(batch):
            y_ref, s_ref = oracle.conv1d_f32_strided(x[b], ws[q], stride)
            assert_close_f32(body[b, :n_out], y_ref, s_ref, "signal %d" % b)


def run_2d_strided(x_np, w_np, sr, sc, device, x_pitch=None, y_pitch=None, x_off=0, y_off=0):
    batch, h, wd = x_np.shape
    p, q = w_np.shape
    oh, ow = (h - p) // sr + 1, (wd - q) // sc + 1
    x_pitch = x_pitch or wd
    y_pitch = y_pitch or ow
    xb = torch.zeros(x_off + batch * h * x_pitch + 16, dtype=torch.float32, device=device)
    yb = torch.full((y_off + batch * oh * y_pitch + 64,), CANARY, dtype=torch.float32, device=device)
    xb[x_off: x_off + batch * h * x_pitch].view(batch, h, x_pitch)[:, :, :wd] = torch.from_numpy(x_np).to(device)
    st = B.sysconv2d_strided(xb.data_ptr() + 4 * x_off, wd, h, x_pitch, h * x_pitch, np.ascontiguousarray(w_np), q, p,
                             sc, sr, yb.data_ptr() + 4 * y_off, y_pitch, oh * y_pitch, batch, B.F32, B.OS,
                             torch.cuda.current_stream().cuda_stream)
    assert st == 0, B.status_string(st)
    torch.cuda.synchronize()
    yh = yb.cpu().numpy()
    body = yh[y_off: y_off + batch * oh * y_pitch].reshape(batch, oh, y_pitch)
    assert (body[:, :, ow:] == CANARY).all(), "write into the pitch padding"
    assert (yh[:y_off] == CANARY).all() and (yh[y_off + batch * oh * y_pitch:] == CANARY).all()
    for b in range(batch):
        y_ref, s_ref = oracle.conv2d_f32_strided(x_np[b], w_np, (sr, sc))
        assert body[b, :, :ow].shape == y_ref.shape
        assert_close_f32(body[b, :, :ow], y_ref, s_ref, "image %d, strides (%d, %d)" % (b, sr, sc))


@pytest.mark.parametrize("strides", [(3, 3), (2, 1), (1, 2), (2, 3), (3, 2), (4, 4), (5, 1), (1, 7), (9, 9)],
                         ids=lambda t: "r%dc%d" % t)
@pytest.mark.parametrize("pq", [(1, 1), (3, 3), (5, 5), (7, 7), (9, 9), (15, 15), (2, 11), (13, 4)], ids=lambda f: "%dx%d" % f)
def test_2d_any_strides(cuda_device, strides, pq):
    sr, sc = strides
    x, ws = inputs.gen_2d_f32(533, 61, [pq], seed=3400 + 16 * pq[0] + pq[1] + sr, batch=2)
    run_2d_strided(x, ws[pq], sr, sc, cuda_device)
    run_2d_strided(x[:, :, :301], ws[pq], sr, sc, cuda_device, x_pitch=307, y_pitch=310, x_off=1, y_off=3)


def test_2d_stride_two_large_filters_and_full_hd_stride_three(cuda_device):
    # stride 2 beyond 7 x 7 goes to the run-time-stride array too
    x, ws = inputs.gen_2d_f32(300, 120, [(9, 9), (15, 15), (8, 3)], seed=3500, batch=1)
    for pq in ws:
        run_2d_strided(x, ws[pq], 2, 2, cuda_device)
    x, ws = inputs.gen_2d_f32(1920, 1080, [(5, 5)], seed=3501, batch=1)
    run_2d_strided(x, ws[(5, 5)], 3, 3, cuda_device)
    # single-output and degenerate sizes
    x, ws = inputs.gen_2d_f32(5, 5, [(5, 5)], seed=3502, batch=3)
    run_2d_strided(x, ws[(5, 5)], 3, 4, cuda_device)


# ------------------------------------------------------------------------ separable 2-D convolution


def check_separable(x_np, u, v, device, x_pitch=None, y_pitch=None, x_off=0, y_off=0):
    batch, h, wd = x_np.shape
    p, q = len(u), len(v)
    oh, ow = h - p + 1, wd - q + 1
    x_pitch = x_pitch or wd
    y_pitch = y_pitch or ow
    xb = torch.zeros(x_off + batch * h * x_pitch + 16, dtype=torch.float32, device=device)
    yb = torch.full((y_off + batch * oh * y_pitch + 64,), CANARY, dtype=torch.float32, device=device)
    xb[x_off: x_off + batch * h * x_pitch].view(batch, h, x_pitch)[:, :, :wd] = torch.from_numpy(x_np).to(device)
    st = B.sysconv2d_separable(xb.data_ptr() + 4 * x_off, wd, h, x_pitch, h * x_pitch, u, v, yb.data_ptr() + 4 * y_off,
                               y_pitch, oh * y_pitch, batch, torch.cuda.current_stream().cuda_stream)
    assert st == 0, B.status_string(st)
    torch.cuda.synchronize()
    yh = yb.cpu().numpy()
    body = yh[y_off: y_off + batch * oh * y_pitch].reshape(batch, oh, y_pitch)
    assert (body[:, :, ow:] == CANARY).all(), "write into the pitch padding"
    assert (yh[:y_off] == CANARY).all() and (yh[y_off + batch * oh * y_pitch:] == CANARY).all()
    w = np.outer(u.astype(np.float64), v.astype(np.float64)).astype(np.float32)
    for b in range(batch):
        # the definition: Eq. 3 with the rank-one filter u v^T (fp32 product of the taps, as the oracle takes fp32 taps)
        y_ref, s_ref = oracle.conv2d_f32(x_np[b], w)
        assert_close_f32(body[b, :, :ow], y_ref, s_ref, "image %d" % b)


@pytest.mark.parametrize("pq", [(1, 1), (3, 3), (5, 5), (7, 7), (8, 8), (9, 9), (15, 15), (2, 11), (13, 4), (15, 1), (1, 15),
                                (7, 15), (8, 3)], ids=lambda f: "%dx%d" % f)
def test_separable_filter_shapes(cuda_device, pq):
    p, q = pq
    rng = np.random.default_rng(1000 + 16 * p + q)
    x = rng.random((2, 75, 700), dtype=np.float32)
    u = rng.uniform(-1, 1, p).astype(np.float32)
    v = rng.uniform(-1, 1, q).astype(np.float32)
    check_separable(x, u, v, cuda_device)
    check_separable(x[:, :, :301], u, v, cuda_device, x_pitch=307, y_pitch=303, x_off=1, y_off=1)


@pytest.mark.parametrize("hw", [(0, 0), (1, 0), (0, 1), (2, 3), (31, 127), (32, 128), (33, 129), (40, 255), (7, 513), (70, 1030)])
@pytest.mark.parametrize("pq", [(3, 3), (5, 7), (15, 15)], ids=lambda f: "%dx%d" % f)
def test_separable_ragged_image_sizes(cuda_device, pq, hw):
    p, q = pq
    rng = np.random.default_rng(1100 + hw[0] + hw[1])
    x = rng.random((1, p + hw[0], q + hw[1]), dtype=np.float32)
    check_separable(x, rng.uniform(-1, 1, p).astype(np.float32), rng.uniform(-1, 1, q).astype(np.float32), cuda_device)


def test_separable_exact_on_integers_and_equal_to_the_full_convolution(cuda_device):
    # integer-valued data and taps: every order of summation is exact, so the separable result must equal the
    # full 2-D convolution with the outer-product filter bit for bit
    rng = np.random.default_rng(7)
    x = rng.integers(-8, 9, (2, 300, 1200)).astype(np.float32)
    u = rng.integers(-3, 4, 5).astype(np.float32)
    v = rng.integers(-3, 4, 9).astype(np.float32)
    xd = torch.from_numpy(x).to(cuda_device)
    y = B.conv2d_separable(xd, u, v)
    full = B.conv2d(xd, np.outer(u, v).astype(np.float32), B.OS)
    torch.cuda.synchronize()
    assert torch.equal(y, full)
    ref, _ = oracle.conv2d_f32(x[1], np.outer(u, v).astype(np.float32))
    np.testing.assert_array_equal(y[1].cpu().numpy().astype(np.float64), ref)


def test_separable_full_size_sampled(cuda_device):
    x, _ = inputs.make_config(5, dict(filters=[3], batch=2))
    rng = np.random.default_rng(8)
    u = rng.normal(0, 1 / 3, 9).astype(np.float32)
    v = rng.normal(0, 1 / 3, 9).astype(np.float32)
    y = B.conv2d_separable(torch.from_numpy(x).to(cuda_device), u, v)
    torch.cuda.synchronize()
    oh, ow = 4096 - 8, 4096 - 8
    rows = np.concatenate([rng.integers(0, oh, 3000), [0, 0, oh - 1, oh - 1]])
    cols = np.concatenate([rng.integers(0, ow, 3000), [0, ow - 1, 0, ow - 1]])
    y_ref, s_ref = oracle.conv2d_f32_at(x[1], np.outer(u.astype(np.float64), v.astype(np.float64)).astype(np.float32), rows, cols)
    assert_close_f32(y[1].cpu().numpy()[rows, cols], y_ref, s_ref, "sampled")


# ------------------------------------------------------------------------ iterated 3x3 stencil (second workload)

K_FIVE = np.array([[0, 0.2, 0], [0.15, 0.3, 0.25], [0, 0.1, 0]], np.float32)
K_NINE = np.array([[0.05, 0.2, -0.1], [0.15, 0.3, 0.25], [0.07, 0.1, -0.02]], np.float32)


def check_stencil(u_np, k, sweeps, device, pitch=None, out_pitch=None, u_off=0, o_off=0):
    """u_np: (batch, h, w).  Runs sysstencil2d through the C ABI, checks canaries, compares every point of every
    grid with the oracle: |y - y_ref| <= 1e-5 * S, S = the same sweeps of |k| over |u|."""
    batch, h, wd = u_np.shape
    pitch = pitch or wd
    out_pitch = out_pitch or wd
    ub = torch.zeros(u_off + batch * h * pitch + 16, dtype=torch.float32, device=device)
    ob = torch.full((o_off + batch * h * out_pitch + 64,), CANARY, dtype=torch.float32, device=device)
    sb = torch.full((o_off + batch * h * out_pitch + 64,), CANARY, dtype=torch.float32, device=device)
    ub[u_off: u_off + batch * h * pitch].view(batch, h, pitch)[:, :, :wd] = torch.from_numpy(u_np).to(device)
    st = B.sysstencil2d(ub.data_ptr() + 4 * u_off, wd, h, pitch, h * pitch, k, sweeps, ob.data_ptr() + 4 * o_off, out_pitch,
                        h * out_pitch, batch, sb.data_ptr() + 4 * o_off if sweeps > 4 else 0,
                        torch.cuda.current_stream().cuda_stream)
    assert st == 0, B.status_string(st)
    torch.cuda.synchronize()
    for buf in (ob, sb):
        yh = buf.cpu().numpy()
        body = yh[o_off: o_off + batch * h * out_pitch].reshape(batch, h, out_pitch)
        assert (body[:, :, wd:] == CANARY).all(), "write into the pitch padding"
        assert (yh[:o_off] == CANARY).all() and (yh[o_off + batch * h * out_pitch:] == CANARY).all()
    yh = ob.cpu().numpy()
    body = yh[o_off: o_off + batch * h * out_pitch].reshape(batch, h, out_pitch)
    for b in range(batch):
        y_ref, s_ref = oracle.stencil2d_f32(u_np[b], k, sweeps)
        assert_close_f32(body[b, :, :wd], y_ref, s_ref, "grid %d, %d sweeps" % (b, sweeps))


@pytest.mark.parametrize("k", [K_FIVE, K_NINE], ids=["five_point", "nine_point"])
@pytest.mark.parametrize("sweeps", [1, 2, 3, 4, 5, 7, 8, 9, 13])
def test_stencil_sweep_counts(cuda_device, k, sweeps):
    rng = np.random.default_rng(1500 + sweeps)
    u = rng.uniform(-1, 1, (2, 150, 300)).astype(np.float32)
    check_stencil(u, k, sweeps, cuda_device)


@pytest.mark.parametrize("sweeps", [1, 3, 4, 6])
@pytest.mark.parametrize("hw", [(1, 1), (1, 9), (9, 1), (2, 2), (3, 3), (3, 200), (200, 3), (4, 5), (17, 119), (18, 120),
                                (19, 121), (40, 127), (41, 128), (42, 129), (130, 241), (131, 255), (260, 113)])
def test_stencil_ragged_grid_sizes(cuda_device, sweeps, hw):
    # grids without interior, widths around the 120- and 112-column strips, heights around the band edges
    rng = np.random.default_rng(1600 + hw[0] + hw[1])
    u = rng.uniform(0, 1, (1, hw[0], hw[1])).astype(np.float32)
    check_stencil(u, K_NINE, sweeps, cuda_device)


@pytest.mark.parametrize("layout", [(203, 201, 1, 3), (204, 204, 0, 0), (208, 200, 4, 4), (201, 202, 2, 2)])
def test_stencil_pitches_and_alignment(cuda_device, layout):
    pitch, out_pitch, u_off, o_off = layout
    rng = np.random.default_rng(1700)
    u = rng.uniform(-1, 1, (3, 70, 200)).astype(np.float32)
    for sweeps in (2, 6):
        check_stencil(u, K_FIVE, sweeps, cuda_device, pitch=pitch, out_pitch=out_pitch, u_off=u_off, o_off=o_off)


def test_stencil_fixed_points_exact_integers_and_non_finite(cuda_device):
    # a constant field under coefficients that sum to one (dyadic, exact) is a fixed point at every sweep count
    k = np.array([[0.125, 0.0625, 0.0625], [0.25, 0.25, 0.0625], [0.0625, 0.0625, 0.0625]], np.float32)
    u = torch.full((1, 300, 500), 3.0, device=cuda_device)
    for sweeps in (1, 4, 11):
        assert torch.equal(B.stencil2d(u, k, sweeps), u)
    # integer data and dyadic coefficients: exact in fp32 whatever the order, so every bit must match the oracle
    rng = np.random.default_rng(1800)
    ui = rng.integers(-8, 9, (2, 140, 260)).astype(np.float32)
    kd = np.array([[0.25, 0.5, 0.25], [0.5, -1.0, 0.5], [0.25, 0.5, 0.25]], np.float32)
    for sweeps in (1, 4, 6):
        y = B.stencil2d(torch.from_numpy(ui).to(cuda_device), kd, sweeps).cpu().numpy()
        for b in range(2):
            np.testing.assert_array_equal(y[b].astype(np.float64), oracle.stencil2d_f32(ui[b], kd, sweeps)[0])
    # a non-finite value spreads exactly as the definition says: one ring of neighbours per sweep, never through
    # the fixed boundary ring
    uf = rng.uniform(0, 1, (1, 90, 260)).astype(np.float32)
    for r, c, v in ((0, 0, np.nan), (40, 127, np.inf), (41, 128, -np.inf), (89, 130, np.nan), (30, 0, np.inf), (60, 259, np.nan)):
        uf[0, r, c] = v
    for sweeps in (1, 3, 4, 5):
        with np.errstate(invalid="ignore"):
            y_ref, s_ref = oracle.stencil2d_f32(uf[0], K_NINE, sweeps)
        y = B.stencil2d(torch.from_numpy(uf).to(cuda_device), K_NINE, sweeps).cpu().numpy()[0].astype(np.float64)
        _assert_same_where_finite(y, y_ref, s_ref, "%d sweeps" % sweeps)


def test_stencil_many_small_grids_and_the_eigenfunction(cuda_device):
    rng = np.random.default_rng(1900)
    check_stencil(rng.uniform(-1, 1, (40, 33, 47)).astype(np.float32), K_NINE, 4, cuda_device)
    # Dirichlet eigenfunction of the five-point Jacobi sweep: decays by its closed-form factor per sweep
    h, w, a = 129, 257, 0.125
    r, c = np.mgrid[0:h, 0:w]
    u = (np.sin(np.pi * r / (h - 1)) * np.sin(np.pi * c / (w - 1))).astype(np.float32)
    u[0] = u[-1] = 0
    u[:, 0] = u[:, -1] = 0
    k = np.array([[0, a, 0], [a, 1 - 4 * a, a], [0, a, 0]], np.float32)
    lam = 1 - 4 * a + 2 * a * (np.cos(np.pi / (h - 1)) + np.cos(np.pi / (w - 1)))
    y = B.stencil2d(torch.from_numpy(u).to(cuda_device), k, 16).cpu().numpy().astype(np.float64)
    np.testing.assert_allclose(y, lam ** 16 * u.astype(np.float64), rtol=0, atol=5e-6)


@pytest.mark.parametrize("sweeps", [1, 4, 8])
def test_stencil_full_size_every_point(cuda_device, sweeps):
    """16 x 4096 x 4096, the launch configuration bench.py times: every point of every grid against the oracle."""
    x, _ = inputs.make_config(5, scale=dict(filters=[3]))
    xd = torch.from_numpy(x).to(cuda_device)
    y = B.stencil2d(xd, K_NINE if sweeps != 4 else K_FIVE, sweeps)
    torch.cuda.synchronize()
    del xd
    for b in range(16):
        y_ref, s_ref = oracle.stencil2d_f32(x[b], K_NINE if sweeps != 4 else K_FIVE, sweeps)
        assert_close_f32(y[b].cpu().numpy(), y_ref, s_ref, "grid %d" % b)


# ------------------------------------------------------------------------ generic space-time executor

ST_PAPER = {"SBM": ((1, 1), (0, 1)), "BSM": ((0, 1), (1, 1)), "FSM": ((0, 1), (1, -1)), "BFS": ((1, 0), (1, 1)),
            "FFS": ((1, 0), (2, 1)), "FBS": ((1, 0), (0, 1))}
# other valid transforms: mirrored arrays, slower schedules, skewed allocations, a non-unimodular one
ST_OTHER = [((-1, 0), (0, 1)), ((1, 0), (0, -1)), ((1, 0), (1, 2)), ((1, 0), (3, 1)), ((0, 1), (2, 1)),
            ((1, 1), (1, -1)), ((1, -1), (0, 1)), ((1, 1), (-1, 2)), ((2, 1), (0, 1)), ((1, 2), (1, 1)),
            ((0, -1), (1, 1)), ((1, 0), (-1, 1)), ((1, 1), (0, 2)), ((2, 0), (1, 1))]


def run_spacetime(x, w, P, s, device):
    n, q = x.shape[0], w.shape[0]
    xd = torch.from_numpy(x).to(device)
    yd = torch.full((n - q + 1 + 16,), CANARY, dtype=torch.float32, device=device)
    st = B.sysconv1d_spacetime(xd.data_ptr(), n, w, q, yd.data_ptr(), P, s, torch.cuda.current_stream().cuda_stream)
    assert st == 0, (P, s, B.status_string(st))
    torch.cuda.synchronize()
    yh = yd.cpu().numpy()
    assert (yh[n - q + 1:] == CANARY).all()
    return yh[:n - q + 1]


@pytest.mark.parametrize("name", list(ST_PAPER))
@pytest.mark.parametrize("q", [1, 2, 5, 8, 16, 31, 32])
def test_spacetime_executor_runs_the_six_designs(cuda_device, name, q):
    P, s = ST_PAPER[name]
    x, ws = inputs.gen_1d_f32(5000 + q, [q], seed=700 + q)
    y = run_spacetime(x, ws[q], P, s, cuda_device)
    y_ref, s_ref = oracle.conv1d_f32(x, ws[q])
    assert_close_f32(y, y_ref, s_ref, "%s q=%d" % (name, q))
    st, info = B.spacetime_describe(P, s, q)
    assert st == 0 and info["name"] == name


@pytest.mark.parametrize("Ps", ST_OTHER, ids=lambda t: "P%d,%d_s%d,%d" % (t[0] + t[1]))
def test_spacetime_executor_runs_other_valid_transforms(cuda_device, Ps):
    P, s = Ps
    for q, n in [(5, 777), (12, 4099), (1, 40), (3, 3)]:
        st, info = B.spacetime_describe(P, s, q)
        if st == 2:
            continue                      # valid but not covered at this filter length (array too long)
        assert st == 0
        x, ws = inputs.gen_1d_f32(n, [q], seed=800 + q)
        y = run_spacetime(x, ws[q], P, s, cuda_device)
        y_ref, s_ref = oracle.conv1d_f32(x, ws[q])
        assert_close_f32(y, y_ref, s_ref, "%s q=%d" % (Ps, q))


def test_spacetime_executor_matches_the_folded_kernels_on_integers(cuda_device):
    # integer-valued data: every order of summation is exact, so all designs must agree bit for bit
    rng = np.random.default_rng(8)
    x = rng.integers(-8, 9, 20000).astype(np.float32)
    w = rng.integers(-4, 5, 7).astype(np.float32)
    ref = B.conv1d(torch.from_numpy(x).to(cuda_device), w, B.OS).cpu().numpy()
    for P, s in list(ST_PAPER.values()) + ST_OTHER[:6]:
        np.testing.assert_array_equal(run_spacetime(x, w, P, s, cuda_device), ref)


def test_spacetime_executor_rejects_invalid_transforms(cuda_device):
    x = torch.zeros(100, device=cuda_device)
    y = torch.zeros(96, device=cuda_device)
    w = np.ones(5, np.float32)
    s0 = torch.cuda.current_stream().cuda_stream
    assert B.sysconv1d_spacetime(x.data_ptr(), 100, w, 5, y.data_ptr(), (1, 1), (1, 1), s0) == 1
    assert B.sysconv1d_spacetime(x.data_ptr(), 100, w, 5, y.data_ptr(), (0, 1), (1, 0), s0) == 1
    assert B.sysconv1d_spacetime(x.data_ptr(), 100, w, 5, y.data_ptr(), (1, 0), (5, 1), s0) == 2
    assert B.sysconv1d_spacetime(x.data_ptr(), 100, w, 5, x.data_ptr(), (1, 0), (0, 1), s0) == 1     # x and y overlap


def test_host_multi_entry_point(cuda_device):
    """One host signal, several (filter, design) jobs in one call: every job's result equals the oracle's."""
    for n in (3_000_001, 5000, 33):
        qs = [4, 16, 32, 7, 1]
        x, ws = inputs.gen_1d_f32(n, qs, seed=123)
        designs = [B.WS, B.OS, B.IS, B.FSM, B.OS]
        xh = torch.from_numpy(x).pin_memory()
        jobs = [(ws[q], d, torch.full((n - q + 1,), CANARY, dtype=torch.float32).pin_memory())
                for q, d in zip(qs, designs)]
        work = torch.empty(B.host_multi_workspace_bytes(n, qs), dtype=torch.uint8, device=cuda_device)
        B.sysconv1d_host_multi(xh, jobs, work)
        torch.cuda.synchronize()
        for (w, d, yh), q in zip(jobs, qs):
            y_ref, s_ref = oracle.conv1d_f32(x, w)
            assert_close_f32(yh.numpy(), y_ref, s_ref, "n=%d q=%d %s" % (n, q, B.DESIGN_NAMES[d]))
    assert B.device_status() == 0


# ------------------------------------------------------------------------ measured peaks and yardstick kernels


def test_measured_peaks_are_plausible_and_floor_kernels_move_the_bytes(cuda_device):
    scratch = torch.empty(512 << 20, dtype=torch.uint8, device=cuda_device)
    pk = B.measure_peaks(scratch)
    assert pk["sm_count"] == torch.cuda.get_device_properties(cuda_device).multi_processor_count
    # an SM has 128 fp32 lanes; nothing can exceed them and a healthy device gets most of the way there
    assert 90 <= pk["ffma_per_clk_sm"] <= 129
    assert 90 <= pk["ffma2_mac_per_clk_sm"] <= 257
    assert 30 <= pk["imad_per_clk_sm"] <= 129
    assert 30 <= pk["dp4a_per_clk_sm"] <= 129
    assert 16 <= pk["shfl_per_clk_sm"] <= 129
    assert 2000 <= pk["copy_gbs"] <= 9000
    del scratch
    src = torch.randint(0, 256, (1 << 20,), dtype=torch.uint8, device=cuda_device)
    dst = torch.zeros(1 << 20, dtype=torch.uint8, device=cuda_device)
    B.floor_copy(src, dst, src.numel())
    wide = torch.full((1 << 20,), -1, dtype=torch.int32, device=cuda_device)
    B.floor_copy(src, wide, src.numel(), widen=True)
    torch.cuda.synchronize()
    assert torch.equal(src, dst)
    assert torch.equal(src.to(torch.int32), wide)


# ------------------------------------------------------------------------ bounded device-side waits


def test_a_bounded_wait_that_runs_out_is_reported_once(cuda_device):
    """The pipelined kernels poll for their asynchronous copies a bounded number of times; a block whose limit runs
    out raises a flag and returns.  The self-test block waits for bytes that are never sent (it issues no copy), so
    its limit must run out: the launch completes, the status call reports the time-out once, then the device is
    clean again and ordinary work runs."""
    assert B.device_status() == 0
    B.selftest_wait_timeout()
    torch.cuda.synchronize()                       # the block returned by itself
    assert B.device_status() == 4
    assert B.device_status() == 0
    side = torch.cuda.Stream()                     # a stream the legacy default stream does not wait for
    B.selftest_wait_timeout(stream=side)
    assert B.device_status() == 4                  # the status call synchronises the whole device itself
    assert B.device_status() == 0
    x, ws = inputs.make_config(1)
    y_ref, s_ref = oracle.conv1d_f32(x, ws[8])
    assert_close_f32(run_1d(x, ws[8], B.OS, cuda_device), y_ref, s_ref, "after the self-test")
    assert B.device_status() == 0


# ------------------------------------------------------------------------ launches inside a CUDA graph


def test_device_entry_points_replay_inside_a_cuda_graph(cuda_device):
    """The device-pointer entry points only enqueue kernels on the caller's stream, so a launch-bound loop of
    small problems can be captured once and replayed; the replayed results must equal the direct ones."""
    x1, ws1 = inputs.make_config(1)
    x2, ws2 = inputs.gen_2d_f32(200, 90, [(3, 3)], seed=5)
    xd1, xd2 = torch.from_numpy(x1).to(cuda_device), torch.from_numpy(x2).to(cuda_device)
    w1, w2 = ws1[8], ws2[(3, 3)]
    direct = [B.conv1d(xd1, w1, d) for d in DESIGNS] + [B.conv2d(xd2, w2, d) for d in DESIGNS]   # also first-call set-up
    outs = [torch.zeros_like(t) for t in direct]
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for i, d in enumerate(DESIGNS):
                B.conv1d(xd1, w1, d, out=outs[i], stream=side)
                B.conv2d(xd2, w2, d, out=outs[3 + i], stream=side)
    for o in outs:
        o.zero_()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    for got, want in zip(outs, direct):
        assert torch.equal(got, want)
    assert B.device_status() == 0


# ------------------------------------------------------------------------ integer


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("k", [3, 7])
def test_config4_2d_u8_full(cuda_device, design, k):
    x, ws = inputs.make_config(4, scale=dict(filters=[k]))
    check_2d(x, ws[(k, k)], design, cuda_device)


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("pq", [(1, 1), (3, 3), (7, 7), (2, 5), (15, 15), (4, 13)], ids=lambda f: "%dx%d" % f)
def test_2d_u8_shapes_and_extremes(cuda_device, design, pq):
    p, q = pq
    x, ws = inputs.gen_2d_u8s8(301, 67, [pq], seed=60 + p + q, batch=2)
    check_2d(x, ws[pq], design, cuda_device)
    check_2d(x, ws[pq], design, cuda_device, x_pitch=307, y_pitch=303, x_off=1, y_off=1)
    xm = np.full((1, 40, 150), 255, np.uint8)
    for v in (8, -8):
        check_2d(xm, np.full(pq, v, np.int8), design, cuda_device)


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("pq", [(1, 1), (3, 3), (5, 5), (7, 7), (7, 15), (8, 15), (15, 15), (9, 2), (4, 13), (12, 8),
                                (1, 4), (2, 5), (6, 9), (7, 12), (3, 8)], ids=lambda f: "%dx%d" % f)
def test_2d_u8_packed_rows(cuda_device, design, pq):
    """Rows that start 4-byte aligned take the packed four-taps-per-step kernels (OS and IS: every filter size, IS in
    two forms by filter height; WS: rows aligned to 16 bytes): several strips, a ragged right edge, pitch padding, unaligned
    outputs, and the extreme pixel/tap values."""
    p, q = pq
    x, ws = inputs.gen_2d_u8s8(1101, 41, [pq], seed=90 + p + q, batch=2)
    check_2d(x, ws[pq], design, cuda_device, x_pitch=1104)
    check_2d(x, ws[pq], design, cuda_device, x_pitch=1120, y_pitch=1103, y_off=3)
    check_2d(x[:, :, :1040], ws[pq], design, cuda_device)
    check_2d(x[:, :, :528], ws[pq], design, cuda_device, x_pitch=528)
    xm = np.full((1, 33, 160), 255, np.uint8)
    for v in (127, -128):
        check_2d(xm, np.full(pq, v, np.int8), design, cuda_device)
    wmix = np.where((np.arange(p * q).reshape(p, q) % 2) == 0, 127, -128).astype(np.int8)
    check_2d(x[:1, :, :512], wmix, design, cuda_device)


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
def test_1d_u8(cuda_device, design):
    x, ws = inputs.gen_1d_u8s8(5000, [7], seed=3)
    xd = torch.from_numpy(x).to(cuda_device)
    y = B.conv1d(xd, ws[7], design)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(y.cpu().numpy(), oracle.conv1d_u8s8_s32(x, ws[7]))


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
def test_1d_u8_batches(cuda_device, design):
    """Integer signals run as images with one signal per row: a batch of short signals, packed and with a longer
    stride, canaries between the outputs."""
    rng = np.random.default_rng(77)
    for n, batch, q, stride in ((300, 40, 7, None), (300, 40, 7, 304), (33, 1000, 4, 36), (5000, 3, 15, 5003)):
        x = rng.integers(0, 256, (batch, n), dtype=np.uint8)
        w = rng.integers(-128, 128, q, dtype=np.int8)
        xs = stride or n
        n_out = n - q + 1
        ys = stride or n_out
        xh = np.zeros(batch * xs + 16, np.uint8)
        np.lib.stride_tricks.as_strided(xh, shape=(batch, n), strides=(xs, 1))[...] = x
        xd = torch.from_numpy(xh).to(cuda_device)
        yd = torch.full((batch * ys + 16,), 123456789, dtype=torch.int32, device=cuda_device)
        st = B.sysconv1d(xd.data_ptr(), n, xs, w, q, yd.data_ptr(), ys, batch, B.U8S8_S32, design,
                         torch.cuda.current_stream().cuda_stream)
        assert st == 0, B.status_string(st)
        torch.cuda.synchronize()
        yh = yd.cpu().numpy()
        got = np.lib.stride_tricks.as_strided(yh, shape=(batch, n_out), strides=(4 * ys, 4))
        for b in range(0, batch, max(batch // 7, 1)):
            np.testing.assert_array_equal(got[b], oracle.conv1d_u8s8_s32(x[b], w))
        mask = np.ones(yh.shape, bool)
        np.lib.stride_tricks.as_strided(mask, shape=(batch, n_out), strides=(ys, 1))[...] = False
        assert (yh[mask] == 123456789).all(), "write outside the output range"
    assert B.device_status() == 0


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
@pytest.mark.parametrize("q", [1, 4, 9, 15, 16, 23, 32])
def test_1d_short_signal_batches(cuda_device, design, q):
    """Batches of short signals (more than 32 and at most 512 outputs) run as images with one signal per row (filters
    of more than 15 taps: output- and input-stationary only); longer signals and single signals stay on the 1-D kernels.  Both sides of each
    limit, packed and padded strides (rows 16-byte aligned or not), element offsets, canaries around every output."""
    rng = np.random.default_rng(8100 + q)
    w = (rng.random(q, dtype=np.float32) * 2 - 1).astype(np.float32)
    for n_out, batch in ((33, 700), (100, 257), (255, 64), (512, 9), (513, 9), (300, 1), (300, 2)):
        n = n_out + q - 1
        x = (rng.random((batch, n), dtype=np.float32) * 2 - 1).astype(np.float32)
        y_ref, s_ref = tiles_reference(x, w)
        for offset, stride in ((0, None), (0, (n + 3) // 4 * 4), (1, n + 1), (3, None)):
            y = run_1d(x, w, design, cuda_device, batch_stride=stride, offset=offset).reshape(batch, n_out)
            assert_close_f32(y, y_ref, s_ref, "%s q=%d n_out=%d batch=%d offset=%d stride=%s"
                             % (_ids(design), q, n_out, batch, offset, stride))
    assert B.device_status() == 0


# ------------------------------------------------------------------------ host-buffer entry points


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
def test_host_entry_points(cuda_device, design):
    x, ws = inputs.gen_1d_f32(100000, [16], seed=21)
    xh = torch.from_numpy(x).pin_memory()
    yh = torch.empty(100000 - 15, dtype=torch.float32).pin_memory()
    wsz = B.host_workspace_bytes((100000,), (16,))
    work = torch.empty(wsz, dtype=torch.uint8, device=cuda_device)
    B.sysconv1d_host(xh, ws[16], yh, design, work)
    torch.cuda.synchronize()
    y_ref, s_ref = oracle.conv1d_f32(x, ws[16])
    assert_close_f32(yh.numpy(), y_ref, s_ref, "1-D host")
    small = torch.empty(wsz - 256, dtype=torch.uint8, device=cuda_device)
    with pytest.raises(B.SysconvError):
        B.sysconv1d_host(xh, ws[16], yh, design, small)

    x2, ws2 = inputs.gen_2d_u8s8(333, 222, [(3, 3)], seed=22, batch=2)
    xh2 = torch.from_numpy(x2).pin_memory()
    yh2 = torch.empty((2, 220, 331), dtype=torch.int32).pin_memory()
    work2 = torch.empty(B.host_workspace_bytes((2, 222, 333), (3, 3), B.U8S8_S32), dtype=torch.uint8,
                        device=cuda_device)
    B.sysconv2d_host(xh2, ws2[(3, 3)], yh2, design, work2, dtype=B.U8S8_S32)
    torch.cuda.synchronize()
    for b in range(2):
        np.testing.assert_array_equal(yh2[b].numpy(), oracle.conv2d_u8s8_s32(x2[b], ws2[(3, 3)]))


@pytest.mark.parametrize("design", DESIGNS, ids=_ids)
def test_host_entry_points_chunked_overlap(cuda_device, design):
    """Problems large enough for the chunked (copy/compute overlapped) form of the host-buffer calls."""
    n, q = 5_000_003, 16
    x, ws = inputs.gen_1d_f32(n, [q], seed=31)
    xh = torch.from_numpy(x).pin_memory()
    yh = torch.full((n - q + 1,), float("nan"), dtype=torch.float32).pin_memory()
    work = torch.empty(B.host_workspace_bytes((n,), (q,)), dtype=torch.uint8, device=cuda_device)
    B.sysconv1d_host(xh, ws[q], yh, design, work)
    torch.cuda.synchronize()
    y_ref, s_ref = oracle.conv1d_f32(x, ws[q])
    assert_close_f32(yh.numpy(), y_ref, s_ref, "1-D host, chunked")

    # one large image: bands of rows; three images: one chunk per image
    for shape in ((1, 1500, 1400), (3, 300, 500)):
        x2, ws2 = inputs.gen_2d_f32(shape[2], shape[1], [(5, 3)], seed=32, batch=shape[0])
        xh2 = torch.from_numpy(x2).pin_memory()
        yh2 = torch.full((shape[0], shape[1] - 4, shape[2] - 2), float("nan"), dtype=torch.float32).pin_memory()
        work2 = torch.empty(B.host_workspace_bytes(shape, (5, 3)), dtype=torch.uint8, device=cuda_device)
        B.sysconv2d_host(xh2, ws2[(5, 3)], yh2, design, work2)
        torch.cuda.synchronize()
        for b in range(shape[0]):
            y_ref, s_ref = oracle.conv2d_f32(x2[b], ws2[(5, 3)])
            assert_close_f32(yh2[b].numpy(), y_ref, s_ref, "2-D host, chunked %s image %d" % (shape, b))


def test_unsupported_and_invalid_on_device(cuda_device):
    x = torch.zeros(1000, device=cuda_device)
    with pytest.raises(B.SysconvError) as e:
        B.conv1d(x, np.ones(33, np.float32))
    assert e.value.status == 2
    with pytest.raises(B.SysconvError) as e:
        B.conv1d(x[:5], np.ones(8, np.float32), out=torch.zeros(8, device=cuda_device))
    assert e.value.status == 1
    with pytest.raises(B.SysconvError):
        B.conv1d(torch.zeros(10), np.ones(3, np.float32))     # CPU tensor: no fallback
    before = B.launch_count()
    B.conv1d(x, np.ones(8, np.float32))
    assert B.launch_count() == before + 1


def test_2d_batches_beyond_one_grid(cuda_device):
    """More images than one launch can index (65535): the call goes out in slices."""
    batch = 65535 + 4097
    rng = np.random.default_rng(12)
    picks = [0, 1, 65534, 65535, 65536, batch - 1]
    x = rng.random((batch, 6, 9), dtype=np.float32)
    w = rng.uniform(-1, 1, (3, 2)).astype(np.float32)
    xu = rng.integers(0, 256, (batch, 6, 12)).astype(np.uint8)
    wu = rng.integers(-128, 128, (2, 5)).astype(np.int8)
    for design in DESIGNS:
        y = B.conv2d(torch.from_numpy(x).to(cuda_device), w, design).cpu().numpy()
        yu = B.conv2d(torch.from_numpy(xu).to(cuda_device), wu, design).cpu().numpy()
        for b in picks:
            y_ref, s_ref = oracle.conv2d_f32(x[b], w)
            assert_close_f32(y[b], y_ref, s_ref, "image %d" % b)
            np.testing.assert_array_equal(yu[b], oracle.conv2d_u8s8_s32(xu[b], wu))
    st = B.sysconv2d_strided(1 << 20, 9, 6, 9, 54, w, 2, 3, 2, 2, 1 << 30, 4, 8, batch, B.F32, B.OS, 0)
    assert st == 2


# ------------------------------------------------------------------------ randomized shapes


def test_randomized_1d_shapes(cuda_device):
    """Seeded random lengths, filter lengths, designs, strides, batches and pointer offsets."""
    rng = np.random.default_rng(2024)
    for case in range(160):
        q = int(rng.integers(1, 33))
        n = q + int(rng.choice([0, 1, 2, 5, 100, 607, 608, 609, 1215, 1216, 1217, 2431, 2432, 2433, 4000, 9000]))
        n += int(rng.integers(0, 40))
        batch = int(rng.choice([1, 1, 2, 3]))
        stride = int(rng.choice([1, 1, 2]))
        design = int(rng.choice([B.OS, B.IS] if stride == 2 else [B.WS, B.OS, B.IS, B.FSM, B.BFS, B.FFS]))
        x_off, y_off = int(rng.integers(0, 4)), int(rng.integers(0, 4))
        xs = n + int(rng.integers(0, 5)) * (batch > 1)
        n_out = (n - q) // stride + 1
        ys = n_out + int(rng.integers(0, 5)) * (batch > 1)
        x = rng.uniform(-1, 1, (batch, n)).astype(np.float32)
        w = rng.uniform(-1, 1, q).astype(np.float32)
        xb = torch.zeros(x_off + batch * xs + 8, dtype=torch.float32, device=cuda_device)
        yb = torch.full((y_off + batch * ys + 8,), CANARY, dtype=torch.float32, device=cuda_device)
        xb[x_off: x_off + batch * xs].view(batch, xs)[:, :n] = torch.from_numpy(x).to(cuda_device)
        st = B.sysconv1d_strided(xb.data_ptr() + 4 * x_off, n, xs, w, q, stride, yb.data_ptr() + 4 * y_off, ys, batch,
                                 B.F32, design, torch.cuda.current_stream().cuda_stream)
        what = "case %d: n=%d q=%d batch=%d stride=%d design=%d offs=%d,%d" % (case, n, q, batch, stride, design, x_off, y_off)
        assert st == 0, what
        torch.cuda.synchronize()
        yh = yb.cpu().numpy()
        body = yh[y_off: y_off + batch * ys].reshape(batch, ys)
        assert (body[:, n_out:] == CANARY).all() and (yh[:y_off] == CANARY).all(), what
        assert (yh[y_off + batch * ys:] == CANARY).all(), what
        for b in range(batch):
            y_ref, s_ref = oracle.conv1d_f32_strided(x[b], w, stride)
            assert_close_f32(body[b, :n_out], y_ref, s_ref, what)
    assert B.device_status() == 0


def test_randomized_2d_shapes(cuda_device):
    """Seeded random image sizes (around the strip widths of every kernel), filters, designs, data types,
    strides, pitches and offsets."""
    rng = np.random.default_rng(2025)
    edges = [1, 2, 3, 4, 5, 31, 32, 33, 119, 120, 121, 124, 125, 127, 128, 129, 236, 240, 244, 248, 249, 252, 253,
             255, 256, 257, 480, 496, 504, 511, 512, 513, 600, 1000]
    for case in range(220):
        p, q = int(rng.integers(1, 16)), int(rng.integers(1, 16))
        is_u8 = bool(rng.integers(0, 3) == 0)
        stride = 1 if is_u8 else int(rng.choice([1, 1, 2]))
        if stride == 2:
            p, q = min(p, 7), min(q, 7)
        design = int(rng.choice([B.OS, B.IS] if stride == 2 else [B.WS, B.OS, B.IS]))
        ow = int(rng.choice(edges)) + int(rng.integers(0, 3))
        oh = int(rng.choice([1, 2, 7, 8, 9, 15, 16, 17, 31, 33, 64, 70]))
        wd, h = stride * (ow - 1) + q + int(rng.integers(0, stride)), stride * (oh - 1) + p + int(rng.integers(0, stride))
        batch = int(rng.choice([1, 1, 2]))
        aligned = bool(rng.integers(0, 2))
        x_pitch = (wd + 3) // 4 * 4 if aligned else wd + int(rng.integers(0, 4))
        x_off = 0 if aligned else int(rng.integers(0, 4))
        y_pitch = ow + int(rng.integers(0, 4))
        y_off = int(rng.integers(0, 4))
        what = "case %d: %dx%d image, %dx%d filter, batch %d, %s, stride %d, design %d, pitches %d/%d, offs %d/%d" % (
            case, wd, h, p, q, batch, "u8" if is_u8 else "f32", stride, design, x_pitch, y_pitch, x_off, y_off)
        if is_u8:
            x = rng.integers(0, 256, (batch, h, wd)).astype(np.uint8)
            w = rng.integers(-128, 128, (p, q)).astype(np.int8)
            check_2d(x, w, design, cuda_device, x_pitch=x_pitch, y_pitch=y_pitch, x_off=x_off, y_off=y_off)
        else:
            x = rng.random((batch, h, wd), dtype=np.float32)
            w = rng.uniform(-1, 1, (p, q)).astype(np.float32)
            try:
                if stride == 2:
                    check_2d_s2(x, w, design, cuda_device, x_pitch=x_pitch, y_pitch=y_pitch, x_off=x_off, y_off=y_off)
                else:
                    check_2d(x, w, design, cuda_device, x_pitch=x_pitch, y_pitch=y_pitch, x_off=x_off, y_off=y_off)
            except AssertionError as e:
                raise AssertionError(what + ": " + str(e))
    assert B.device_status() == 0
