"""Pins of the stencil oracle (oracle/stencil_oracle.c) to what the mathematics fixes: fixed points, a closed-form
eigenfunction decay, the impulse response (orientation of the coefficients), library correlations, brute force."""
import numpy as np
import pytest
import scipy.signal

import oracle

FIVE_POINT = np.array([[0, 0.2, 0], [0.15, 0.3, 0.25], [0, 0.1, 0]], np.float32)     # asymmetric on purpose
AVERAGING = np.array([[0.05, 0.1, 0.05], [0.1, 0.4, 0.1], [0.05, 0.1, 0.05]], np.float32)


def test_constant_field_is_a_fixed_point_when_the_coefficients_sum_to_one():
    k = np.array([[0.125, 0.0625, 0.0625], [0.25, 0.25, 0.0625], [0.0625, 0.0625, 0.0625]], np.float32)   # dyadic: exact
    assert float(k.astype(np.float64).sum()) == 1.0
    u = np.full((9, 13), 3.0, np.float32)
    for t in (0, 1, 2, 5):
        y, s = oracle.stencil2d_f32(u, k, t)
        assert np.array_equal(y, np.full((9, 13), 3.0))
        assert np.array_equal(s, y)


def test_linear_field_is_preserved_by_a_symmetric_averaging_stencil():
    # k symmetric under (dr, dc) -> (-dr, -dc) with sum 1 reproduces a*r + b*c + d at interior points; the ring is fixed
    k = np.array([[0.0625, 0.125, 0.0625], [0.125, 0.25, 0.125], [0.0625, 0.125, 0.0625]], np.float32)
    r, c = np.mgrid[0:17, 0:23]
    u = (2.0 * r - 3.0 * c + 5.0).astype(np.float32)
    for t in (1, 3, 8):
        y, _ = oracle.stencil2d_f32(u, k, t)
        assert np.array_equal(y, u.astype(np.float64))


def test_impulse_response_pins_the_orientation_of_the_coefficients():
    u = np.zeros((9, 11), np.float32)
    u[4, 5] = 1.0
    y, _ = oracle.stencil2d_f32(u, FIVE_POINT, 1)
    # v(r, c) = sum k(dr, dc) u(r+dr, c+dc): the impulse at (4, 5) reaches v(4-dr, 5-dc) with weight k(dr, dc)
    for dr in (-1, 0, 1):
        for dc in (-1, 0, 1):
            assert y[4 - dr, 5 - dc] == np.float64(FIVE_POINT[dr + 1, dc + 1])
    assert np.count_nonzero(y) == np.count_nonzero(FIVE_POINT)
    assert y[3, 5] == np.float64(np.float32(0.1)) and y[5, 5] == np.float64(np.float32(0.2))      # spelled out once
    assert y[4, 4] == np.float64(np.float32(0.25)) and y[4, 6] == np.float64(np.float32(0.15))


def test_ring_is_fixed_and_interior_equals_a_valid_correlation():
    rng = np.random.default_rng(3)
    u = rng.uniform(-1, 1, (12, 19)).astype(np.float32)
    k = rng.uniform(-1, 1, (3, 3)).astype(np.float32)
    y, s = oracle.stencil2d_f32(u, k, 1)
    ref = scipy.signal.correlate2d(u.astype(np.float64), k.astype(np.float64), mode="valid")
    np.testing.assert_allclose(y[1:-1, 1:-1], ref, rtol=0, atol=1e-14)
    assert np.array_equal(y[0], u[0].astype(np.float64)) and np.array_equal(y[-1], u[-1].astype(np.float64))
    assert np.array_equal(y[:, 0], u[:, 0].astype(np.float64)) and np.array_equal(y[:, -1], u[:, -1].astype(np.float64))
    ref_s = scipy.signal.correlate2d(np.abs(u).astype(np.float64), np.abs(k).astype(np.float64), mode="valid")
    np.testing.assert_allclose(s[1:-1, 1:-1], ref_s, rtol=0, atol=1e-14)


def test_two_sweeps_far_from_the_ring_equal_the_composite_5x5_operator():
    rng = np.random.default_rng(4)
    u = rng.uniform(-1, 1, (20, 24)).astype(np.float32)
    k = rng.uniform(-1, 1, (3, 3)).astype(np.float64)
    y, _ = oracle.stencil2d_f32(u, k.astype(np.float32), 2)
    k32 = k.astype(np.float32).astype(np.float64)
    composite = scipy.signal.convolve2d(k32, k32, mode="full")           # correlation kernels compose by convolution
    ref = scipy.signal.correlate2d(u.astype(np.float64), composite, mode="valid")      # points at least 2 from the ring
    np.testing.assert_allclose(y[2:-2, 2:-2], ref, rtol=0, atol=1e-13)


def test_dirichlet_eigenfunction_decays_by_its_closed_form_factor():
    # u = sin(pi r/(H-1)) sin(pi c/(W-1)) vanishes on the ring and is an eigenfunction of the five-point Jacobi sweep
    # k = [centre 1-4a, four neighbours a]: factor 1 - 4a + 2a (cos(pi/(H-1)) + cos(pi/(W-1))) per sweep
    h, w, a = 33, 41, 0.125
    r, c = np.mgrid[0:h, 0:w]
    u64 = np.sin(np.pi * r / (h - 1)) * np.sin(np.pi * c / (w - 1))
    u = u64.astype(np.float32)
    u[0] = u[-1] = 0
    u[:, 0] = u[:, -1] = 0
    k = np.array([[0, a, 0], [a, 1 - 4 * a, a], [0, a, 0]], np.float32)
    lam = 1 - 4 * a + 2 * a * (np.cos(np.pi / (h - 1)) + np.cos(np.pi / (w - 1)))
    for t in (1, 4, 8):
        y, _ = oracle.stencil2d_f32(u, k, t)
        np.testing.assert_allclose(y, lam ** t * u.astype(np.float64), rtol=0, atol=2e-7)    # fp32 rounding of u only


def test_sweeps_compose_and_zero_sweeps_is_the_identity():
    rng = np.random.default_rng(5)
    u = rng.uniform(0, 1, (10, 14)).astype(np.float32)
    y0, s0 = oracle.stencil2d_f32(u, AVERAGING, 0)
    assert np.array_equal(y0, u.astype(np.float64)) and np.array_equal(s0, np.abs(u).astype(np.float64))
    # dyadic data and coefficients: every intermediate is exact in fp32 too, so sweeps can be chained through fp32
    ud = rng.integers(-8, 9, (10, 14)).astype(np.float32)
    kd = np.array([[0.25, 0.5, 0.25], [0.5, -1.0, 0.5], [0.25, 0.5, 0.25]], np.float32)
    y3, _ = oracle.stencil2d_f32(ud, kd, 3)
    step = ud
    for _ in range(3):
        step = oracle.stencil2d_f32(step, kd, 1)[0].astype(np.float32)
    assert np.array_equal(y3, step.astype(np.float64))


def test_brute_force_on_a_tiny_grid():
    rng = np.random.default_rng(6)
    u = rng.uniform(-1, 1, (5, 6)).astype(np.float32)
    k = rng.uniform(-1, 1, (3, 3)).astype(np.float32)
    cur = [[float(v) for v in row] for row in u]
    for _ in range(3):
        nxt = [row[:] for row in cur]
        for r in range(1, 4):
            for c in range(1, 5):
                nxt[r][c] = sum(float(k[dr + 1][dc + 1]) * cur[r + dr][c + dc] for dr in (-1, 0, 1) for dc in (-1, 0, 1))
        cur = nxt
    y, _ = oracle.stencil2d_f32(u, k, 3)
    np.testing.assert_allclose(y, np.array(cur), rtol=0, atol=1e-15)


def test_degenerate_grids_have_no_interior():
    k = FIVE_POINT
    for shape in ((1, 7), (2, 7), (7, 1), (7, 2), (1, 1), (2, 2)):
        u = np.arange(shape[0] * shape[1], dtype=np.float32).reshape(shape)
        y, _ = oracle.stencil2d_f32(u, k, 4)
        assert np.array_equal(y, u.astype(np.float64))
    with pytest.raises(ValueError):
        oracle.stencil2d_f32(np.zeros((4, 4), np.float32), np.zeros((3, 2), np.float32), 1)
