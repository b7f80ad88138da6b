"""Pins of the CPU oracle against what the mathematics fixes (no GPU).

The oracle is the plain definition (Eq. 2 / Eq. 3); these tests tie it to
closed forms, invariants, special cases, a textbook library routine and brute
force, chosen so that a dropped term, a flipped filter, a transposed operand or
a wrong index fails at least one of them.
"""
import numpy as np
import pytest

import oracle


def _ints(rng, lo, hi, shape):
    return rng.integers(lo, hi + 1, size=shape).astype(np.float32)


# ----------------------------------------------------------------- 1-D, fp32


@pytest.mark.parametrize("q,k", [(1, 0), (5, 0), (5, 3), (8, 7), (32, 17)])
def test_1d_impulse_reproduces_shifted_input(q, k):
    rng = np.random.default_rng(10)
    x = rng.standard_normal(200).astype(np.float32)
    w = np.zeros(q, np.float32)
    w[k] = 1.0
    y, s = oracle.conv1d_f32(x, w)
    assert y.shape == (200 - q + 1,)
    # no filter flip: tap k picks x[i + k]
    np.testing.assert_array_equal(y, x[k:k + y.size].astype(np.float64))
    np.testing.assert_array_equal(s, np.abs(x[k:k + y.size]).astype(np.float64))


def test_1d_constant_input_gives_tap_sum():
    w = np.array([1, -2, 3, 4, -5, 6, 7], np.float32)
    y, s = oracle.conv1d_f32(np.full(50, 3.0, np.float32), w)
    np.testing.assert_array_equal(y, np.full(44, 3.0 * w.sum()))
    np.testing.assert_array_equal(s, np.full(44, 3.0 * np.abs(w).sum()))


@pytest.mark.parametrize("q", [1, 2, 5, 16, 32])
def test_1d_ramp_box_closed_form(q):
    n = 300
    x = np.arange(n, dtype=np.float32)
    y, _ = oracle.conv1d_f32(x, np.ones(q, np.float32))
    i = np.arange(n - q + 1, dtype=np.float64)
    np.testing.assert_array_equal(y, q * i + q * (q - 1) / 2.0)


def test_1d_ramp_weights_closed_form():
    # w[k] = k+1, x[i] = i:  y[i] = sum_k (k+1)(i+k) = i*Q(Q+1)/2 + sum_k k(k+1)
    q, n = 6, 40
    x = np.arange(n, dtype=np.float32)
    w = np.arange(1, q + 1, dtype=np.float32)
    y, _ = oracle.conv1d_f32(x, w)
    i = np.arange(n - q + 1, dtype=np.float64)
    const = sum(k * (k + 1) for k in range(q))
    np.testing.assert_array_equal(y, i * q * (q + 1) / 2.0 + const)


def test_1d_linearity_and_shift_invariance_exact_on_integers():
    rng = np.random.default_rng(11)
    x1, x2 = _ints(rng, -50, 50, 120), _ints(rng, -50, 50, 120)
    w = _ints(rng, -9, 9, 7)
    y1, _ = oracle.conv1d_f32(x1, w)
    y2, _ = oracle.conv1d_f32(x2, w)
    y12, _ = oracle.conv1d_f32(3 * x1 - 2 * x2, w)
    np.testing.assert_array_equal(y12, 3 * y1 - 2 * y2)
    d = 13
    ys, _ = oracle.conv1d_f32(x1[d:], w)
    np.testing.assert_array_equal(ys, y1[d:])


def test_1d_q1_scales_and_n_equals_q_is_one_dot_product():
    rng = np.random.default_rng(12)
    x = rng.standard_normal(33).astype(np.float32)
    y, _ = oracle.conv1d_f32(x, np.array([2.5], np.float32))
    np.testing.assert_array_equal(y, x.astype(np.float64) * 2.5)
    w = rng.standard_normal(33).astype(np.float32)
    y, s = oracle.conv1d_f32(x, w)
    assert y.shape == (1,)
    assert y[0] == pytest.approx(float(np.dot(x.astype(np.float64), w.astype(np.float64))), rel=1e-14)
    assert s[0] == pytest.approx(float(np.dot(np.abs(x).astype(np.float64), np.abs(w).astype(np.float64))),
                                 rel=1e-14)


def test_1d_matches_numpy_correlate_and_brute_force():
    rng = np.random.default_rng(13)
    x = rng.uniform(-1, 1, 257).astype(np.float32)
    w = rng.uniform(-1, 1, 9).astype(np.float32)
    y, s = oracle.conv1d_f32(x, w)
    ref = np.correlate(x.astype(np.float64), w.astype(np.float64), mode="valid")
    np.testing.assert_allclose(y, ref, rtol=0, atol=1e-14)
    # pure-Python nested loops in exact rational-free float64 arithmetic
    brute = [sum(float(w[k]) * float(x[i + k]) for k in range(9)) for i in range(249)]
    np.testing.assert_allclose(y, brute, rtol=0, atol=1e-14)
    np.testing.assert_allclose(s, np.correlate(np.abs(x).astype(np.float64),
                                               np.abs(w).astype(np.float64), "valid"), atol=1e-14)
    np.testing.assert_allclose(oracle.conv1d_f32_taps_outer(x, w), y, rtol=0, atol=1e-14)


def test_1d_sampled_form_equals_full_form():
    rng = np.random.default_rng(14)
    x = rng.uniform(-1, 1, 1000).astype(np.float32)
    w = rng.uniform(-1, 1, 16).astype(np.float32)
    y, s = oracle.conv1d_f32(x, w)
    pos = np.array([0, 1, 17, 500, 984], np.int64)
    ya, sa = oracle.conv1d_f32_at(x, w, pos)
    np.testing.assert_array_equal(ya, y[pos])
    np.testing.assert_array_equal(sa, s[pos])
    with pytest.raises(ValueError):
        oracle.conv1d_f32_at(x, w, np.array([985], np.int64))


def test_1d_rejects_filter_longer_than_signal():
    with pytest.raises(ValueError):
        oracle.conv1d_f32(np.zeros(3, np.float32), np.zeros(4, np.float32))


# ----------------------------------------------------------------- 2-D, fp32


@pytest.mark.parametrize("p,q,p0,q0", [(3, 5, 2, 1), (5, 3, 0, 2), (1, 4, 0, 3), (4, 1, 3, 0)])
def test_2d_impulse_gives_shifted_crop(p, q, p0, q0):
    rng = np.random.default_rng(20)
    x = rng.standard_normal((17, 23)).astype(np.float32)
    w = np.zeros((p, q), np.float32)
    w[p0, q0] = 1.0
    y, _ = oracle.conv2d_f32(x, w)
    assert y.shape == (17 - p + 1, 23 - q + 1)
    # w[p][q]: p is the filter ROW (pairs with image rows), q the column
    np.testing.assert_array_equal(y, x[p0:p0 + y.shape[0], q0:q0 + y.shape[1]].astype(np.float64))


def test_2d_ramp_box_closed_form():
    p, q, h, wd = 3, 5, 20, 31
    r_idx, c_idx = np.meshgrid(np.arange(h), np.arange(wd), indexing="ij")
    x = (c_idx + 1000 * r_idx).astype(np.float32)
    y, _ = oracle.conv2d_f32(x, np.ones((p, q), np.float32))
    r, c = np.meshgrid(np.arange(h - p + 1), np.arange(wd - q + 1), indexing="ij")
    expect = p * q * (c + 1000.0 * r) + p * q * (q - 1) / 2.0 + 1000.0 * q * p * (p - 1) / 2.0
    np.testing.assert_array_equal(y, expect)


def test_2d_constant_and_linearity():
    rng = np.random.default_rng(21)
    w = _ints(rng, -9, 9, (4, 3))
    y, s = oracle.conv2d_f32(np.full((9, 8), 2.0, np.float32), w)
    np.testing.assert_array_equal(y, np.full((6, 6), 2.0 * w.sum()))
    np.testing.assert_array_equal(s, np.full((6, 6), 2.0 * np.abs(w).sum()))
    x1, x2 = _ints(rng, -20, 20, (12, 14)), _ints(rng, -20, 20, (12, 14))
    y1, _ = oracle.conv2d_f32(x1, w)
    y2, _ = oracle.conv2d_f32(x2, w)
    y12, _ = oracle.conv2d_f32(2 * x1 + 5 * x2, w)
    np.testing.assert_array_equal(y12, 2 * y1 + 5 * y2)
    # shift invariance in both directions
    ys, _ = oracle.conv2d_f32(x1[2:, 3:], w)
    np.testing.assert_array_equal(ys, y1[2:, 3:])


def test_2d_separable_filter_is_row_pass_then_column_pass():
    rng = np.random.default_rng(22)
    x = _ints(rng, -9, 9, (15, 18))
    u = _ints(rng, -4, 4, 4)      # along rows (p)
    v = _ints(rng, -4, 4, 5)      # along columns (q)
    y, _ = oracle.conv2d_f32(x, np.outer(u, v).astype(np.float32))
    rows = np.stack([oracle.conv1d_f32(x[r], v)[0] for r in range(15)])          # 15 x 14
    cols = np.stack([oracle.conv1d_f32(rows[:, c].astype(np.float32), u)[0] for c in range(14)], 1)
    np.testing.assert_array_equal(y, cols)


def test_2d_height_one_reduces_to_1d_and_brute_force():
    rng = np.random.default_rng(23)
    x = rng.uniform(0, 1, (1, 64)).astype(np.float32)
    w = rng.uniform(-1, 1, (1, 7)).astype(np.float32)
    y2, s2 = oracle.conv2d_f32(x, w)
    y1, s1 = oracle.conv1d_f32(x[0], w[0])
    np.testing.assert_array_equal(y2[0], y1)
    np.testing.assert_array_equal(s2[0], s1)
    x = rng.uniform(0, 1, (9, 11)).astype(np.float32)
    w = rng.uniform(-1, 1, (3, 4)).astype(np.float32)
    y, s = oracle.conv2d_f32(x, w)
    for r in range(7):
        for c in range(8):
            acc = sum(float(w[p, q]) * float(x[r + p, c + q]) for p in range(3) for q in range(4))
            assert y[r, c] == pytest.approx(acc, abs=1e-14)
    np.testing.assert_allclose(oracle.conv2d_f32_taps_outer(x, w), y, rtol=0, atol=1e-14)
    rows = np.array([0, 6, 3], np.int64)
    cols = np.array([7, 0, 2], np.int64)
    ya, sa = oracle.conv2d_f32_at(x, w, rows, cols)
    np.testing.assert_array_equal(ya, y[rows, cols])
    np.testing.assert_array_equal(sa, s[rows, cols])


def test_2d_matches_scipy_correlate2d():
    from scipy.signal import correlate2d
    rng = np.random.default_rng(24)
    x = rng.uniform(0, 1, (21, 19)).astype(np.float32)
    w = rng.uniform(-1, 1, (5, 3)).astype(np.float32)
    y, _ = oracle.conv2d_f32(x, w)
    ref = correlate2d(x.astype(np.float64), w.astype(np.float64), mode="valid")
    np.testing.assert_allclose(y, ref, rtol=0, atol=1e-13)


# ----------------------------------------------------------------- strided forms


@pytest.mark.parametrize("stride", [1, 2, 3])
def test_1d_strided_is_the_subsampled_numpy_correlation(stride):
    rng = np.random.default_rng(31)
    for n, q in [(200, 7), (201, 7), (64, 32), (33, 32), (9, 9)]:
        x = rng.uniform(-1, 1, n).astype(np.float32)
        w = rng.uniform(-1, 1, q).astype(np.float32)
        y, s = oracle.conv1d_f32_strided(x, w, stride)
        ref = np.correlate(x.astype(np.float64), w.astype(np.float64), mode="valid")[::stride]
        assert y.shape == ref.shape == ((n - q) // stride + 1,)
        np.testing.assert_allclose(y, ref, rtol=0, atol=1e-14)
        ref_s = np.correlate(np.abs(x).astype(np.float64), np.abs(w).astype(np.float64), "valid")[::stride]
        np.testing.assert_allclose(s, ref_s, rtol=0, atol=1e-14)


def test_1d_stride_two_closed_forms():
    # ramp through a box of Q ones: y[c] = Q*(2c) + Q(Q-1)/2; impulse at tap k: y[c] = x[2c+k]
    n, q = 101, 6
    x = np.arange(n, dtype=np.float32)
    y, _ = oracle.conv1d_f32_strided(x, np.ones(q, np.float32), 2)
    c = np.arange((n - q) // 2 + 1)
    np.testing.assert_array_equal(y, q * 2.0 * c + q * (q - 1) / 2)
    for k in range(q):
        w = np.zeros(q, np.float32)
        w[k] = 1
        y, _ = oracle.conv1d_f32_strided(x, w, 2)
        np.testing.assert_array_equal(y, x[k::2][:len(c)])


def test_1d_stride_two_equals_the_stride_two_fbs_array_of_table_2():
    from oracle import systolic_sim as sim
    rng = np.random.default_rng(32)
    x = _ints(rng, -8, 8, 41)
    w = _ints(rng, -4, 4, 5)
    y, _ = oracle.conv1d_f32_strided(x, w, 2)
    ys, _ = sim.simulate_1d("FBS", x, w, stride=2)
    np.testing.assert_array_equal(y, np.asarray(ys, dtype=np.float64))


@pytest.mark.parametrize("stride", [(1, 1), (2, 2), (2, 1), (1, 2), (3, 2)])
def test_2d_strided_is_the_subsampled_scipy_correlation(stride):
    from scipy.signal import correlate2d
    rng = np.random.default_rng(33)
    for (h, wd), (p, q) in [((21, 19), (5, 3)), ((20, 18), (3, 5)), ((15, 15), (15, 15)), ((9, 40), (1, 4))]:
        x = rng.uniform(0, 1, (h, wd)).astype(np.float32)
        w = rng.uniform(-1, 1, (p, q)).astype(np.float32)
        y, s = oracle.conv2d_f32_strided(x, w, stride)
        ref = correlate2d(x.astype(np.float64), w.astype(np.float64), mode="valid")[::stride[0], ::stride[1]]
        assert y.shape == ref.shape
        np.testing.assert_allclose(y, ref, rtol=0, atol=1e-13)
        ref_s = correlate2d(np.abs(x).astype(np.float64), np.abs(w).astype(np.float64), mode="valid")
        np.testing.assert_allclose(s, ref_s[::stride[0], ::stride[1]], rtol=0, atol=1e-13)


def test_2d_stride_two_impulse_and_asymmetry():
    # an impulse tap at (p0, q0) picks x[2r+p0][2c+q0]: catches a row/column stride swap on a non-square image
    x = np.arange(11 * 17, dtype=np.float32).reshape(11, 17)
    w = np.zeros((3, 4), np.float32)
    w[2, 1] = 1
    y, _ = oracle.conv2d_f32_strided(x, w, (2, 3))
    np.testing.assert_array_equal(y, x[2::2, 1::3][:y.shape[0], :y.shape[1]])
    assert y.shape == ((11 - 3) // 2 + 1, (17 - 4) // 3 + 1)


# ----------------------------------------------------------------- integer


def test_int_2d_equals_int64_and_python_loops():
    rng = np.random.default_rng(30)
    x = rng.integers(0, 256, (13, 17), dtype=np.uint8)
    w = rng.integers(-8, 9, (3, 7), dtype=np.int8)
    y = oracle.conv2d_u8s8_s32(x, w)
    assert y.dtype == np.int32 and y.shape == (11, 11)
    np.testing.assert_array_equal(y.astype(np.int64), oracle.conv2d_u8s8_i64(x, w))
    for r in (0, 5, 10):
        for c in (0, 4, 10):
            acc = sum(int(w[p, q]) * int(x[r + p, c + q]) for p in range(3) for q in range(7))
            assert int(y[r, c]) == acc


def test_int_extremes_sign_and_zero_extension():
    # pixels are zero-extended (255 stays +255), taps are sign-extended (-8 stays -8)
    x = np.full((7, 7), 255, np.uint8)
    assert int(oracle.conv2d_u8s8_s32(x, np.full((7, 7), 8, np.int8))[0, 0]) == 49 * 255 * 8
    assert int(oracle.conv2d_u8s8_s32(x, np.full((7, 7), -8, np.int8))[0, 0]) == -49 * 255 * 8
    x1 = np.array([200, 100, 255, 0, 7], np.uint8)
    w1 = np.array([-8, 8, -1], np.int8)
    np.testing.assert_array_equal(oracle.conv1d_u8s8_s32(x1, w1),
                                  [-200 * 8 + 100 * 8 - 255, -100 * 8 + 255 * 8 - 0, -255 * 8 + 0 - 7])


def test_int_impulse_and_1d_vs_2d():
    rng = np.random.default_rng(31)
    x = rng.integers(0, 256, (10, 12), dtype=np.uint8)
    w = np.zeros((3, 3), np.int8)
    w[1, 2] = 1
    np.testing.assert_array_equal(oracle.conv2d_u8s8_s32(x, w), x[1:9, 2:12].astype(np.int32))
    w1 = rng.integers(-8, 9, 5, dtype=np.int8)
    np.testing.assert_array_equal(oracle.conv1d_u8s8_s32(x[0], w1),
                                  oracle.conv2d_u8s8_s32(x[:1], w1[None, :])[0])
    np.testing.assert_array_equal(oracle.conv1d_u8s8_s32(x[0], w1),
                                  np.correlate(x[0].astype(np.int64), w1.astype(np.int64), "valid"))


def test_thread_count_is_reported():
    assert oracle.num_threads() >= 1
