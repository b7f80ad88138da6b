"""Design-space enumerator for the 1-D convolution UREs (the tool the paper leaves as future work).

Every pair of an allocation row P = (p_c, p_q) and a schedule row s = (s_c, s_q) over the iteration space
(c, q) is a candidate systolic design (Section 2.2).  ``enumerate_designs`` walks the small integer
transforms, keeps those the library's planner accepts (validity conditions: P and s linearly independent,
every dependence available in time), names each with the paper's letters (input / weight: Broadcast,
Forwarded, Stays; partial sum: Migrates, Stays) and scores it with the analytical model of Table 4:

    outturn     = outputs / time steps
    utilisation = outputs * filter size / (PEs * time steps)

for ONE array producing ``outputs`` results with a filter of ``q`` taps.  The planning itself is done by
``sysconv_spacetime_describe`` in the CUDA library's host code (the same planner the generic executor
runs), so the table always describes what ``sysconv1d_spacetime`` would execute.  Host-only: no GPU needed.
"""
from . import binding

# (P; s) of the six designs the paper discusses (Section 3.1 and Table 2)
PAPER_DESIGNS = {
    "SBM": ((1, 1), (0, 1)),
    "BSM": ((0, 1), (1, 1)),
    "FSM": ((0, 1), (1, -1)),
    "BFS": ((1, 0), (1, 1)),
    "FFS": ((1, 0), (2, 1)),
    "FBS": ((1, 0), (0, 1)),
}


def _span(a, n):
    """Extent of a*i over i in [0, n): (min, max)."""
    return (a * (n - 1), 0) if a < 0 else (0, a * (n - 1))


def model(P, s, outputs, q):
    """Time steps, PEs, outturn and lane utilisation of one array (Table 4's footnotes a and b)."""
    steps = sum(hi - lo for lo, hi in (_span(s[0], outputs), _span(s[1], q))) + 1
    pes = sum(hi - lo for lo, hi in (_span(P[0], outputs), _span(P[1], q))) + 1
    return {"steps": steps, "pes": pes, "outturn": outputs / steps,
            "utilisation": outputs * q / (pes * steps)}


def classify(P, s, q=5):
    """Design letters and dependence geometry of (P; s), or None if the transform is not a valid design."""
    st, info = binding.spacetime_describe(P, s, q)
    return info if st == 0 else None


def enumerate_designs(q=5, outputs=16, lo=-1, hi=2):
    """All valid designs with transform entries in [lo, hi], best utilisation first.

    Transforms that differ only by the sign of P (a mirrored array) are listed once.
    """
    rows = []
    rng = range(lo, hi + 1)
    for pc in rng:
        for pq in rng:
            lead = pc if pc != 0 else pq
            if lead <= 0:                     # (0, 0) is no allocation; -P is P mirrored
                continue
            for sc in rng:
                for sq in rng:
                    info = classify((pc, pq), (sc, sq), q)
                    if info is None:
                        continue
                    row = {"P": (pc, pq), "s": (sc, sq), "name": info["name"], "input": info["input"],
                           "weight": info["weight"], "sum": info["sum"]}
                    row.update(model((pc, pq), (sc, sq), outputs, q))
                    rows.append(row)
    rows.sort(key=lambda r: (-r["utilisation"], r["steps"], r["P"], r["s"]))
    return rows


def main():
    import argparse
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--q", type=int, default=5)
    ap.add_argument("--outputs", type=int, default=16)
    args = ap.parse_args()
    known = {v: k for k, v in PAPER_DESIGNS.items()}
    print("P        s        name  steps  PEs  outturn  utilisation")
    for r in enumerate_designs(args.q, args.outputs):
        tag = known.get((r["P"], r["s"]), "")
        print("%-8s %-8s %-5s %5d %4d %8.2f %11.0f%%  %s" % (r["P"], r["s"], r["name"], r["steps"], r["pes"],
                                                          r["outturn"], 100 * r["utilisation"], tag))


if __name__ == "__main__":
    main()
