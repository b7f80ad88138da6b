"""Pins of the design-faithful systolic simulator (no GPU).

* against the paper: the analytical model of Table 4 (time steps, PE counts,
  lane utilisation) read from tests/golden/table4_model.txt; the validity
  conditions of Section 2.2; the register depths s.e implied by Code 2;
* against the oracle (plain definition) on small integer-valued inputs, where
  every design must give exactly the same sums;
* the URE interpreter (no schedule) against both.
"""
import os

import numpy as np
import pytest

import oracle
from oracle import systolic_sim as sim

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table4_model.txt")


def _table4():
    rows = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, outturn, util = line.split()
            rows[name] = (float(outturn), int(util))
    return rows


def _ints(rng, lo, hi, n):
    return [int(v) for v in rng.integers(lo, hi + 1, n)]


@pytest.mark.parametrize("design", sim.DESIGNS_1D)
def test_table4_outturn_and_utilisation(design):
    outturn, util = _table4()[design]
    rng = np.random.default_rng(1)
    x, w = _ints(rng, -9, 9, 20), _ints(rng, -5, 5, 5)     # 16 outputs, filter size 5
    y, res = sim.simulate_1d(design, x, w)
    assert len(y) == 16
    # outturn = 16 / #steps, printed with two significant digits
    assert abs(16.0 / res.n_steps - outturn) < 0.01 + 1e-9
    # utilisation = 16 * 5 / (#lanes * #steps), printed as a whole percentage
    assert abs(100.0 * 16 * 5 / (res.n_pe * res.n_steps) - util) < 0.5
    assert abs(res.utilisation * 100 - util) < 0.5


@pytest.mark.parametrize("design,n_pe,n_steps", [
    ("SBM", 20, 5), ("BSM", 5, 20), ("FSM", 5, 20), ("BFS", 16, 20), ("FFS", 16, 35), ("FBS", 16, 5)])
def test_pe_and_step_counts_closed_forms(design, n_pe, n_steps):
    rng = np.random.default_rng(2)
    _, res = sim.simulate_1d(design, _ints(rng, -9, 9, 20), _ints(rng, -5, 5, 5))
    assert (res.n_pe, res.n_steps) == (n_pe, n_steps)
    assert res.max_neighbour <= 1          # linear array: neighbour-only transfers


@pytest.mark.parametrize("design", sim.DESIGNS_1D)
@pytest.mark.parametrize("n,q", [(5, 5), (6, 5), (12, 1), (17, 2), (40, 8), (33, 32)])
def test_1d_designs_equal_oracle(design, n, q):
    rng = np.random.default_rng(100 + n + q)
    x, w = _ints(rng, -20, 20, n), _ints(rng, -9, 9, q)
    ref, _ = oracle.conv1d_f32(np.array(x, np.float32), np.array(w, np.float32))
    y, _ = sim.simulate_1d(design, x, w)
    np.testing.assert_array_equal(np.array(y, np.float64), ref)
    np.testing.assert_array_equal(np.array(sim.interpret_1d(design, x, w), np.float64), ref)


@pytest.mark.parametrize("design", sim.DESIGNS_1D)
def test_1d_validity_conditions(design):
    rng = np.random.default_rng(3)
    x, w = _ints(rng, -9, 9, 14), _ints(rng, -5, 5, 4)
    P, s = sim.TRANSFORM_1D[design]
    assert sim.validity(sim.ure_1d(design, x, w), P, s) == []


def test_invalid_transforms_are_caught():
    rng = np.random.default_rng(4)
    x, w = _ints(rng, -9, 9, 14), _ints(rng, -5, 5, 4)
    # FBS UREs with time = c only: two taps of one output at the same PE and time
    assert any("processor" in m for m in sim.validity(sim.ure_1d("FBS", x, w), (1, 0), (1, 0)))
    # time running against the partial-sum dependence
    assert any("s.e" in m for m in sim.validity(sim.ure_1d("FBS", x, w), (1, 0), (0, -1)))


def test_register_depths_follow_s_dot_e():
    rng = np.random.default_rng(5)
    x, w = _ints(rng, -9, 9, 20), _ints(rng, -5, 5, 5)
    depth = {d: sim.simulate_1d(d, x, w)[1].reg_depth for d in sim.DESIGNS_1D}
    # the two designs with a two-step-delay dependence are exactly FSM (inputs) and FFS (weights)
    assert depth["FSM"]["X"] == 2 and depth["FFS"]["W"] == 2
    for d in ("SBM", "BSM", "BFS", "FBS"):
        assert max(depth[d].values()) == 1
    # broadcast data has no register history
    assert depth["SBM"]["W"] == 0 and depth["FBS"]["W"] == 0 and depth["BSM"]["X"] == 0


def test_worked_sbm_example_direction():
    # Section 3.1: s = ccc + q, t = q; Z(s) takes Z(s-1); results sit in PEs Q-1 .. Q+C-2
    x, w = [1, 2, 3, 4, 5, 6], [1, 10, 100]
    _, res = sim.simulate_1d("SBM", x, w)
    assert res.pe_range == (0, 4 + 3 - 2) and res.t_range == (0, 2)


def test_fbs_stride_two():
    rng = np.random.default_rng(6)
    x, w = _ints(rng, -9, 9, 21), _ints(rng, -5, 5, 5)
    y, res = sim.simulate_1d("FBS", x, w, stride=2)
    assert y == [sum(w[k] * x[2 * c + k] for k in range(5)) for c in range(9)]
    assert res.reg_depth["X"] == 2 and res.n_steps == 5


@pytest.mark.parametrize("design", ["SBM", "FBS", "BSM"])
@pytest.mark.parametrize("h,wd,p,q", [(6, 9, 3, 4), (5, 5, 5, 5), (4, 7, 1, 3), (7, 4, 3, 1), (8, 8, 2, 2)])
def test_2d_designs_equal_oracle(design, h, wd, p, q):
    rng = np.random.default_rng(200 + h * wd + p * q)
    img = [[int(v) for v in row] for row in rng.integers(0, 10, (h, wd))]
    w = [[int(v) for v in row] for row in rng.integers(-5, 6, (p, q))]
    ref, _ = oracle.conv2d_f32(np.array(img, np.float32), np.array(w, np.float32))
    y, results = sim.simulate_2d(design, img, w)
    np.testing.assert_array_equal(np.array(y, np.float64), ref)
    np.testing.assert_array_equal(np.array(sim.interpret_2d(design, img, w), np.float64), ref)
    alloc, sched = sim.transform_2d(design, p, q)
    assert sim.validity(sim.ure_2d(design, img, w, 0), alloc, sched) == []
    assert results[0].max_neighbour <= 1


def test_2d_sbm_two_projection_shape():
    # Section 5: PE = c + q, t = p + P*q; the stationary input is a P-deep register
    img = [[r * 10 + c for c in range(9)] for r in range(6)]
    w = [[1, 2, 3, 4], [5, 6, 7, 8], [9, 10, 11, 12]]
    _, results = sim.simulate_2d("SBM", img, w)
    res = results[0]
    assert res.n_pe == 6 + 4 - 1 and res.n_steps == 3 * 4
    assert res.reg_depth["X"] == 3 and res.reg_depth["Z"] == 1


def test_2d_ws_derived_shape():
    img = [[r * 10 + c for c in range(9)] for r in range(6)]
    w = [[1, 2, 3, 4], [5, 6, 7, 8], [9, 10, 11, 12]]
    _, results = sim.simulate_2d("BSM", img, w)
    res = results[0]
    # PE = q holds the P taps of filter column q; C + Q - 1 macro-steps of P sub-steps
    assert res.n_pe == 4 and res.n_steps == 3 * (6 + 4 - 1)
    assert res.reg_depth["W"] == 3 and res.reg_depth["X"] == 0


# ------------------------------------------------------------ folded warp model


@pytest.mark.parametrize("R,q", [(4, 1), (4, 7), (8, 16), (20, 32), (20, 5)])
def test_warp_os_matches_oracle_on_valid_prefix(R, q):
    rng = np.random.default_rng(300 + R + q)
    xs = rng.integers(-9, 10, 32 * R).astype(np.float32)
    w = rng.integers(-5, 6, q).astype(np.float32)
    ref, _ = oracle.conv1d_f32(xs, w)
    z = sim.warp_os_1d(xs, w, R)
    np.testing.assert_array_equal(z[:ref.size], ref)


@pytest.mark.parametrize("R,q,drain", [(4, 1, 0), (4, 7, 2), (8, 16, 1), (20, 32, 1), (20, 5, 0)])
def test_warp_is_matches_oracle_after_offset(R, q, drain):
    rng = np.random.default_rng(400 + R + q)
    xs = rng.integers(-9, 10, 32 * R).astype(np.float32)
    w = rng.integers(-5, 6, q).astype(np.float32)
    ref, _ = oracle.conv1d_f32(xs, w)
    z = sim.warp_is_1d(xs, w, R, drain)
    off = q - 1 + drain
    np.testing.assert_array_equal(z[off:], ref[:32 * R - off])


@pytest.mark.parametrize("lanes,R,q,seg", [(4, 1, 3, 76), (4, 4, 16, 76), (4, 8, 32, 76), (8, 2, 13, 20),
                                           (2, 1, 2, 9)])
def test_warp_ws_matches_oracle(lanes, R, q, seg):
    rng = np.random.default_rng(500 + lanes + R + q)
    n_arr = 32 // lanes
    xs = rng.integers(-9, 10, n_arr * seg + q - 1).astype(np.float32)
    w = rng.integers(-5, 6, q).astype(np.float32)
    ref, _ = oracle.conv1d_f32(xs, w)
    y = sim.warp_ws_1d(xs, w, lanes, R, seg)
    np.testing.assert_array_equal(y.reshape(-1), ref[:n_arr * seg])


# ---- the forms the kernels ship beyond the plain folded passes: paired sums, one-lane arrays with hand-over,
# run-time strides; integer-valued data, so every order of summation is exact


@pytest.mark.parametrize("R", [2, 4, 20])
@pytest.mark.parametrize("q", [1, 2, 5, 12, 13, 32])
def test_paired_output_stationary_pass_matches_oracle(R, q):
    rng = np.random.default_rng(100 + q)
    xs = rng.integers(-8, 9, 32 * R).astype(np.float32)
    w = rng.integers(-4, 5, q).astype(np.float32)
    z = sim.warp_os_1d_paired(xs, w, R)
    y, _ = oracle.conv1d_f32(xs, w)
    valid = 32 * R - (q - 1)
    np.testing.assert_array_equal(z[:valid], y[:valid])
    np.testing.assert_array_equal(z[:valid], sim.warp_os_1d(xs, w, R)[:valid])


@pytest.mark.parametrize("q", [1, 2, 5, 12, 13, 32])
def test_paired_input_stationary_pass_matches_oracle(q):
    rng = np.random.default_rng(110 + q)
    xs = rng.integers(-8, 9, 640).astype(np.float32)
    w = rng.integers(-4, 5, q).astype(np.float32)
    y_pairs = sim.warp_is_1d_paired(xs, w, 20)
    y, _ = oracle.conv1d_f32(xs, w)
    np.testing.assert_array_equal(y_pairs, y[:y_pairs.size])
    assert y_pairs.size >= 640 - q - 1


@pytest.mark.parametrize("q", [1, 2, 3, 8, 31, 32])
@pytest.mark.parametrize("seg,arrays", [(76, 32), (40, 4), (33, 2), (76, 1)])
def test_one_lane_weight_stationary_arrays_hand_their_sums_over(q, seg, arrays):
    if q > seg:
        pytest.skip("array longer than a segment")
    rng = np.random.default_rng(120 + q + seg)
    xs = rng.integers(-8, 9, arrays * seg + q - 1).astype(np.float32)
    w = rng.integers(-4, 5, q).astype(np.float32)
    y = sim.warp_ws_1d_one_lane(xs, w, seg, arrays)
    ref, _ = oracle.conv1d_f32(xs, w)
    np.testing.assert_array_equal(y, ref)


@pytest.mark.parametrize("stride", [1, 2, 3, 4, 7])
@pytest.mark.parametrize("q", [1, 2, 5, 8, 32])
def test_strided_output_stationary_array_by_residue_classes(stride, q):
    rng = np.random.default_rng(130 + q + stride)
    n_pes = 37
    xs = rng.integers(-8, 9, stride * (n_pes - 1) + q + stride * 40).astype(np.float32)
    w = rng.integers(-4, 5, q).astype(np.float32)
    z = sim.warp_os_1d_strided(xs, w, stride, n_pes)
    ref, _ = oracle.conv1d_f32_strided(xs, w, stride)
    np.testing.assert_array_equal(z, ref[:n_pes])
    if stride == 2:
        ys, _ = sim.simulate_1d("FBS", xs[: 2 * (n_pes - 1) + q], w, stride=2)       # Table 2's own stride-2 cell
        np.testing.assert_array_equal(z, np.asarray(ys, dtype=np.float64))
