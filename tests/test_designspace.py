"""Host logic of the generic space-time executor: planner, design letters, enumerator (no GPU).

Pinned to the paper: the transforms of Section 3.1 / Table 2 must come out with the names the paper gives
them, and the enumerator's analytical model must print the figures of Table 4 (tests/golden/table4_model.txt).
"""
import os

import pytest

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table4_model.txt")


@pytest.fixture(scope="module")
def ds():
    from paper_2010_15884_b200 import build, designspace
    build.build()
    return designspace


def _table4():
    rows = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        name, outturn, util = line.split()
        rows[name] = (float(outturn), float(util))
    return rows


def test_paper_transforms_get_the_papers_names(ds):
    for name, (P, s) in ds.PAPER_DESIGNS.items():
        info = ds.classify(P, s, 5)
        assert info is not None, name
        assert info["name"] == name
        assert abs(info["det"]) == 1


def test_dependence_geometry_of_the_six_designs(ds):
    # (PE distance, delay) of input, weight, partial sum as Section 3.1 / Table 2 describe them
    want = {
        "SBM": ((0, 1), (1, 0), (1, 1)),      # inputs stay, weights broadcast, sums move one PE per step
        "BSM": ((1, 0), (0, 1), (1, 1)),      # inputs broadcast, weights stay
        "FSM": ((-1, 2), (0, 1), (-1, 1)),    # inputs forwarded with a two-step delay
        "BFS": ((-1, 0), (1, 1), (0, 1)),     # weights forwarded, sums stay
        "FFS": ((1, 1), (1, 2), (0, 1)),      # weights forwarded with a two-step delay
        "FBS": ((-1, 1), (1, 0), (0, 1)),     # inputs forwarded from the next PE, weights broadcast
    }
    for name, (P, s) in ds.PAPER_DESIGNS.items():
        info = ds.classify(P, s, 5)
        got = (info["input"], info["weight"], info["sum"])
        for g, w in zip(got, want[name]):
            assert g[1] == w[1], (name, got)                       # delays
            assert (g[0] == 0) == (w[0] == 0), (name, got)         # stays or moves
            if w[1] > 0:
                assert g[0] == w[0], (name, got)                   # direction of a forwarded value


def test_model_prints_table_4(ds):
    for name, (outturn, util) in _table4().items():
        P, s = ds.PAPER_DESIGNS[name]
        m = ds.model(P, s, outputs=16, q=5)
        digits = 2 if name == "FFS" else 1
        assert round(m["outturn"], digits) == outturn, (name, m)
        assert round(100 * m["utilisation"]) == util, (name, m)


def test_invalid_and_unsupported_transforms(ds):
    from paper_2010_15884_b200 import binding as b
    assert b.spacetime_describe((1, 1), (1, 1), 5)[0] == 1       # P parallel to s: two points share a PE and a step
    assert b.spacetime_describe((0, 0), (0, 1), 5)[0] == 1
    assert b.spacetime_describe((0, 1), (1, 0), 5)[0] == 1       # s_q = 0: a sum would accumulate within one step
    assert b.spacetime_describe((1, 0), (0, 1), 33)[0] == 1      # filter length outside 1..32
    assert b.spacetime_describe((1, 0), (5, 1), 5)[0] == 2       # weight delay 5 > 4: valid, not covered
    assert b.spacetime_describe((3, 2), (0, 1), 32)[0] == 2      # more than 32 PEs for one output
    assert b.spacetime_describe((1, 0), (0, 1), 5)[0] == 0


def test_enumerator_finds_the_six_designs_and_ranks_fbs_first(ds):
    rows = ds.enumerate_designs(q=5, outputs=16)
    by_transform = {(r["P"], r["s"]): r for r in rows}
    for name, (P, s) in ds.PAPER_DESIGNS.items():
        assert (P, s) in by_transform and by_transform[(P, s)]["name"] == name
    assert rows[0]["utilisation"] == 1.0
    assert any(r["name"] == "FBS" and r["utilisation"] == 1.0 for r in rows)
    for r in rows:                                   # the model can never exceed full use of the lanes
        assert 0 < r["utilisation"] <= 1.0
        assert r["pes"] * r["steps"] >= 16 * 5
    assert len({(r["P"], r["s"]) for r in rows}) == len(rows)
