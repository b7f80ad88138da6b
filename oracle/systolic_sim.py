"""Design-faithful CPU model of the paper's linear systolic arrays.

TEST INFRASTRUCTURE ONLY -- never imported by the product package, shares no
code with the CUDA kernels.  It pins the *method* (the results themselves are
pinned by the plain definition in ``conv_oracle.c``).

Three layers, each written from the paper:

* ``UreSystem`` -- a system of uniform recurrence equations (Section 2.1,
  Eq. 1) for convolution: variables X (inputs), W (weights), Z (partial sums),
  each either loaded from outside (broadcast / boundary) or read from the point
  ``z - e`` at a constant distance ``e``.  ``interpret()`` evaluates the
  equations as the pure functions they are (each value computed once, on
  demand), with no schedule and no PEs.
* ``run_space_time()`` -- the space-time transformed execution (Section 2.2 and
  Section 4.1, Code 2): point ``z`` runs on PE ``P.z`` at time ``s.z``; every
  recurrent variable lives in a per-PE register file of depth ``s.e + 1``; at
  each time step a PE shifts its own history, then reads its operand from the
  PE ``P.e`` away as written ``s.e`` steps ago.  Idle PEs do nothing (the
  CheckTime behaviour of Table 1), which is what the utilisation figures of
  Table 4 count.  The source PE is ``x - P.e`` (the worked SBM example reads
  ``Z(s-1)`` for ``e = (0,1)``, ``P = (1 1)``; the ``+`` printed in Code 2-4 is
  taken to be a misprint).
* ``ure_1d()`` / ``ure_2d()`` with ``TRANSFORM_1D`` / ``transform_2d()`` -- the six 1-D designs (SBM of Section 3.1
  and the cells of Table 2: BSM, FSM, BFS, FFS, FBS), FBS with a stride, and
  the 2-D designs: SBM 2-D (Section 5, two projections, allocation (1 0 1),
  schedule (0 1 P)), FBS 2-D ("multiple FBS 1-D convolutions"), and a
  weight-stationary 2-D design that the paper does not give and that is
  derived here from BSM plus the 2-D partial-sum chain: PE = q, time
  = P*(c+q) + p.

``validity()`` checks the two conditions of Section 2.2 (data availability
``s.e >= 0`` and ``!= 0`` for non-broadcast data; processor availability: no
two points on one PE at one time).

Finally the ``warp_*`` functions restate, on numpy arrays shaped
[32 lanes][R registers], the *folded* form in which R consecutive PEs share one
lane and the PE-to-PE transfer is a warp shuffle with CUDA's out-of-range rule
(a lane whose source is outside the warp keeps its own value).  Every PE always
runs (no CheckTime); PEs whose result is invalid are simply not drained.
"""
from itertools import product

import numpy as np

# ----------------------------------------------------------------------------
# URE systems
# ----------------------------------------------------------------------------


class Var:
    """One recurrent variable of a URE system.

    ``dep(z)`` returns the dependence distance ``e`` (a tuple) when the value at
    point ``z`` comes from point ``z - e``, or ``None`` when it is loaded from
    outside at ``z`` (a boundary point or broadcast data); ``load(z)`` gives the
    outside value.  ``deps`` lists every distance ``dep`` can return.
    """

    def __init__(self, name, deps, dep, load):
        self.name, self.deps, self.dep, self.load = name, list(deps), dep, load


class UreSystem:
    """Convolution as UREs: Z(z) = (Zinit(z) ? 0 : Z(z - eZ)) + X(z) * W(z)."""

    def __init__(self, extents, X, W, Z, is_out, out_index, names):
        self.extents = tuple(extents)      # loop extents, outermost first
        self.X, self.W, self.Z = X, W, Z
        self.is_out = is_out               # z -> bool: Out(.) takes Z(z)
        self.out_index = out_index         # z -> index into the output
        self.names = names                 # loop names, outermost first

    def points(self):
        return product(*[range(e) for e in self.extents])

    def interpret(self):
        """Evaluate the UREs as the pure functions they are (dynamic single
        assignment): each value is computed once, on demand, from the values it
        names -- no schedule, no PEs."""
        memo = {"X": {}, "W": {}, "Z": {}}

        def value(v, z):
            got = memo[v.name].get(z)
            if got is None:
                e = v.dep(z)
                got = v.load(z) if e is None else value(v, _sub(z, e))
                if v is self.Z:
                    got = got + value(self.X, z) * value(self.W, z)
                memo[v.name][z] = got
            return got

        out = {}
        for z in self.points():
            if self.is_out(z):
                out[self.out_index(z)] = value(self.Z, z)
        return out


def _sub(z, e):
    return tuple(a - b for a, b in zip(z, e))


def _dot(a, b):
    return sum(x * y for x, y in zip(a, b))


# ----------------------------------------------------------------------------
# Space-time transformed execution (Code 2)
# ----------------------------------------------------------------------------


class SpaceTimeResult:
    def __init__(self):
        self.out = {}
        self.n_pe = 0
        self.n_steps = 0
        self.n_points = 0
        self.max_neighbour = 0
        self.reg_depth = {}
        self.pe_range = (0, 0)
        self.t_range = (0, 0)

    @property
    def utilisation(self):
        return self.n_points / float(self.n_pe * self.n_steps)


def validity(ure, P, s):
    """The two conditions of Section 2.2; returns a list of violations."""
    bad = []
    for v in (ure.X, ure.W, ure.Z):
        for e in v.deps:
            se = _dot(s, e)
            if se < 0:
                bad.append("%s: s.e = %d < 0 for e=%s" % (v.name, se, (e,)))
            if se == 0:
                bad.append("%s: s.e = 0 for a forwarded value, e=%s" % (v.name, (e,)))
    seen = {}
    for z in ure.points():
        key = (_dot(P, z), _dot(s, z))
        if key in seen:
            bad.append("processor availability: %s and %s both at PE %d, time %d"
                       % (seen[key], z, key[0], key[1]))
            break
        seen[key] = z
    return bad


def run_space_time(ure, P, s):
    """Run ``ure`` on a linear array: PE = P.z, time = s.z (Code 2 pattern)."""
    res = SpaceTimeResult()
    sched = {}
    for z in ure.points():
        key = (_dot(P, z), _dot(s, z))
        if key in sched:
            raise ValueError("two points share PE %d at time %d" % key)
        sched[key] = z
    pes = [k[0] for k in sched]
    ts = [k[1] for k in sched]
    pe_lo, pe_hi, t_lo, t_hi = min(pes), max(pes), min(ts), max(ts)
    res.n_pe, res.n_steps = pe_hi - pe_lo + 1, t_hi - t_lo + 1
    res.n_points = len(sched)
    res.pe_range, res.t_range = (pe_lo, pe_hi), (t_lo, t_hi)

    variables = (ure.X, ure.W, ure.Z)
    depth = {}
    for v in variables:
        d = 0
        for e in v.deps:
            se = _dot(s, e)
            if se < 0:
                raise ValueError("%s: data availability violated" % v.name)
            d = max(d, se)
            res.max_neighbour = max(res.max_neighbour, abs(_dot(P, e)))
        depth[v.name] = d
    res.reg_depth = dict(depth)
    # V[PE][0 .. s.e]: slot k holds what this PE wrote k steps ago
    reg = {v.name: {pe: [None] * (depth[v.name] + 1) for pe in range(pe_lo, pe_hi + 1)}
           for v in variables}

    def read(v, pe, z, e):
        src_pe, ago = pe - _dot(P, e), _dot(s, e)
        if not (pe_lo <= src_pe <= pe_hi):
            raise ValueError("%s at %s reads outside the array" % (v.name, (z,)))
        got = reg[v.name][src_pe][ago] if ago > 0 else None
        if got is None:
            raise ValueError("%s at %s: operand not available" % (v.name, (z,)))
        return got

    for t in range(t_lo, t_hi + 1):
        # every PE shifts its own history first (line 5 of Code 2)
        for v in variables:
            for pe in range(pe_lo, pe_hi + 1):
                h = reg[v.name][pe]
                h[1:] = h[:-1]
                h[0] = None
        # then every PE with a point scheduled now computes (vectorised loop);
        # all operands read were written in earlier steps (slots >= 1)
        for pe in range(pe_lo, pe_hi + 1):
            z = sched.get((pe, t))
            if z is None:
                continue                      # CheckTime: idle PE
            cur = {}
            for v in (ure.X, ure.W):
                e = v.dep(z)
                cur[v.name] = v.load(z) if e is None else read(v, pe, z, e)
                reg[v.name][pe][0] = cur[v.name]
            e = ure.Z.dep(z)
            prev = ure.Z.load(z) if e is None else read(ure.Z, pe, z, e)
            zval = prev + cur["X"] * cur["W"]
            reg["Z"][pe][0] = zval
            if ure.is_out(z):
                res.out[ure.out_index(z)] = zval
    return res


# ----------------------------------------------------------------------------
# The 1-D designs.  Iteration space (c, q), c outer.
# ----------------------------------------------------------------------------


def _ure_1d(x, w, C, Q, x_dep, w_dep, z_desc, stride=1):
    """Build a 1-D URE system.  x_dep/w_dep: z -> e or None; z_desc: run q down."""
    xin = lambda z: x[stride * z[0] + z[1]]
    win = lambda z: w[z[1]]
    X = Var("X", [e for e in x_dep.deps], x_dep, xin)
    W = Var("W", [e for e in w_dep.deps], w_dep, win)
    if z_desc:   # partial sum runs from q = Q-1 down to 0
        zdep = lambda z: None if z[1] == Q - 1 else (0, -1)
        Z = Var("Z", [(0, -1)], zdep, lambda z: 0)
        is_out = lambda z: z[1] == 0
    else:
        zdep = lambda z: None if z[1] == 0 else (0, 1)
        Z = Var("Z", [(0, 1)], zdep, lambda z: 0)
        is_out = lambda z: z[1] == Q - 1
    return UreSystem((C, Q), X, W, Z, is_out, lambda z: z[0], ("c", "q"))


class _Dep:
    def __init__(self, fn, deps):
        self.fn, self.deps = fn, deps

    def __call__(self, z):
        return self.fn(z)


def ure_1d(design, x, w, C=None, stride=1):
    """URE system of one of the paper's 1-D designs for inputs x and taps w."""
    Q = len(w)
    if C is None:
        C = (len(x) - Q) // stride + 1
    bcast = _Dep(lambda z: None, [])
    if design in ("SBM", "FBS"):
        # X(c,q) = select(q < stride || c == C-1, x(stride*c+q), X(c+1, q-stride))
        xd = _Dep(lambda z: None if (z[1] < stride or z[0] == C - 1) else (-1, stride),
                  [(-1, stride)])
        return _ure_1d(x, w, C, Q, xd, bcast, False, stride)
    if stride != 1:
        raise ValueError("stride is given for SBM/FBS only")
    # W(c,q) = select(c == 0, w(q), W(c-1, q))
    wd = _Dep(lambda z: None if z[0] == 0 else (1, 0), [(1, 0)])
    # X(c,q) = select(c == 0 || q == Q-1, x(c+q), X(c-1, q+1))
    xf = _Dep(lambda z: None if (z[0] == 0 or z[1] == Q - 1) else (1, -1), [(1, -1)])
    if design == "BSM":
        return _ure_1d(x, w, C, Q, bcast, wd, False)
    if design == "FSM":
        return _ure_1d(x, w, C, Q, xf, wd, True)
    if design == "BFS":
        return _ure_1d(x, w, C, Q, bcast, wd, False)
    if design == "FFS":
        return _ure_1d(x, w, C, Q, xf, wd, False)
    raise ValueError("unknown design %r" % design)


# (allocation P, schedule s) on the loop vector (c, q)
TRANSFORM_1D = {
    "SBM": ((1, 1), (0, 1)),    # s = c + q, t = q        inputs stay
    "BSM": ((0, 1), (1, 1)),    # s = q,     t = c + q    weights stay
    "FSM": ((0, 1), (1, -1)),   # s = q,     t = c - q    weights stay
    "BFS": ((1, 0), (1, 1)),    # s = c,     t = c + q    sums sediment
    "FFS": ((1, 0), (2, 1)),    # s = c,     t = 2c + q   sums sediment
    "FBS": ((1, 0), (0, 1)),    # s = c,     t = q        sums sediment
}
DESIGNS_1D = tuple(TRANSFORM_1D)


def simulate_1d(design, x, w, stride=1):
    """Run one 1-D design; returns (y as list, SpaceTimeResult)."""
    ure = ure_1d(design, x, w, stride=stride)
    P, s = TRANSFORM_1D[design]
    res = run_space_time(ure, P, s)
    C = ure.extents[0]
    return [res.out[c] for c in range(C)], res


def interpret_1d(design, x, w, stride=1):
    ure = ure_1d(design, x, w, stride=stride)
    out = ure.interpret()
    return [out[c] for c in range(ure.extents[0])]


# ----------------------------------------------------------------------------
# The 2-D designs.  One output row r at a time; iteration space (c, p, q).
# ----------------------------------------------------------------------------


def ure_2d(design, img, w, r):
    """URE system over (c, p, q) for output row r of image img[H][W], taps w[P][Q]."""
    Pn, Q = len(w), len(w[0])
    C = len(img[0]) - Q + 1
    xin = lambda z: img[r + z[1]][z[0] + z[2]]
    win = lambda z: w[z[1]][z[2]]
    bcast = _Dep(lambda z: None, [])
    if design == "SBM":
        # X(c,p,q,r) = select(c == C-1 || q == 0, x(c+q, r+p), X(c+1, p, q-1, r))
        xd = _Dep(lambda z: None if (z[0] == C - 1 or z[2] == 0) else (-1, 0, 1), [(-1, 0, 1)])
        wd = bcast
        extents, order = (C, Q, Pn), "cqp"   # loop order of the schedule: q major, p minor
    elif design == "FBS":
        # each filter row p is one FBS 1-D pass over input row r+p
        xd = _Dep(lambda z: None if (z[0] == C - 1 or z[2] == 0) else (-1, 0, 1), [(-1, 0, 1)])
        wd = bcast
        extents, order = (C, Pn, Q), "cpq"
    elif design == "BSM":
        xd = bcast
        # W(c,p,q) = select(c == 0, w(q,p), W(c-1, p, q))
        wd = _Dep(lambda z: None if z[0] == 0 else (1, 0, 0), [(1, 0, 0)])
        extents, order = (C, Q, Pn), "cqp"
    else:
        raise ValueError("unknown 2-D design %r" % design)
    X = Var("X", xd.deps, xd, xin)
    W = Var("W", wd.deps, wd, win)
    if order == "cqp":
        # Z(c,p,q) = select(p==0 && q==0, 0,
        #              select(p==0, Z(c, p+P-1, q-1), Z(c, p-1, q))) + X*W
        def zdep(z):
            c, p, q = z
            if p == 0 and q == 0:
                return None
            return (0, -(Pn - 1), 1) if p == 0 else (0, 1, 0)
        zdeps = [(0, 1, 0)] + ([(0, -(Pn - 1), 1)] if Q > 1 else [])
    else:
        def zdep(z):
            c, p, q = z
            if p == 0 and q == 0:
                return None
            return (0, 1, -(Q - 1)) if q == 0 else (0, 0, 1)
        zdeps = [(0, 0, 1)] + ([(0, 1, -(Q - 1))] if Pn > 1 else [])
    Z = Var("Z", zdeps, zdep, lambda z: 0)
    is_out = lambda z: z[1] == Pn - 1 and z[2] == Q - 1
    ure = UreSystem((C, Pn, Q), X, W, Z, is_out, lambda z: z[0], ("c", "p", "q"))
    return ure


def transform_2d(design, Pn, Q):
    """(allocation, schedule) on the loop vector (c, p, q)."""
    if design == "SBM":
        return (1, 0, 1), (0, 1, Pn)        # PE = c + q, t = p + P*q   (Section 5)
    if design == "FBS":
        return (1, 0, 0), (0, Q, 1)         # PE = c,     t = q + Q*p   (row passes)
    if design == "BSM":
        return (0, 0, 1), (Pn, 1, Pn)       # PE = q,     t = P*(c+q) + p   (derived)
    raise ValueError(design)


def simulate_2d(design, img, w):
    """Run a 2-D design row by row; returns (y[R][C] as lists, list of results)."""
    Pn, Q = len(w), len(w[0])
    R = len(img) - Pn + 1
    C = len(img[0]) - Q + 1
    alloc, sched = transform_2d(design, Pn, Q)
    rows, results = [], []
    for r in range(R):
        res = run_space_time(ure_2d(design, img, w, r), alloc, sched)
        rows.append([res.out[c] for c in range(C)])
        results.append(res)
    return rows, results


def interpret_2d(design, img, w):
    Pn, Q = len(w), len(w[0])
    R = len(img) - Pn + 1
    C = len(img[0]) - Q + 1
    rows = []
    for r in range(R):
        out = ure_2d(design, img, w, r).interpret()
        rows.append([out[c] for c in range(C)])
    return rows


# ----------------------------------------------------------------------------
# Folded warp model: 32 lanes x R registers, shuffles as the PE-to-PE transfer.
# PE index = lane * R + j.  No CheckTime: every PE runs at every step.
# ----------------------------------------------------------------------------

LANES = 32


def _shfl_down1(v):
    """Lane l takes lane l+1's value; lane 31 keeps its own."""
    out = v.copy()
    out[:-1] = v[1:]
    return out


def _shfl_up1(v, width=LANES):
    """Lane l takes lane l-1's value inside segments of ``width``; first lane keeps its own."""
    out = v.copy()
    out[1:] = v[:-1]
    first = np.arange(v.shape[0]) % width == 0
    out[first] = v[first]
    return out


def warp_os_1d(xs, w, R):
    """Output-stationary (FBS) step sequence on one warp tile.

    xs: 32*R inputs of the tile.  PE c keeps Z(c); inputs move one PE down per
    step.  Returns all 32*R sums; only the first 32*R-(Q-1) are complete.
    """
    Q = len(w)
    X = np.asarray(xs, dtype=np.float64).reshape(LANES, R).copy()
    Z = np.zeros((LANES, R))
    for t in range(Q):
        Z += X * w[t]
        if t < Q - 1:
            incoming = _shfl_down1(X[:, 0])
            X[:, :-1] = X[:, 1:]
            X[:, -1] = incoming
    return Z.reshape(-1)


def warp_is_1d(xs, w, R, drain=0):
    """Input-stationary (SBM) step sequence on one warp tile.

    PE s keeps x(s); partial sums move one PE up per step; ``drain`` further
    moves without arithmetic.  After the last step PE s holds y(s-(Q-1)-drain);
    the first Q-1+drain PEs hold incomplete sums.
    """
    Q = len(w)
    X = np.asarray(xs, dtype=np.float64).reshape(LANES, R)
    Z = X * w[0]
    for t in range(1, Q + drain):
        incoming = _shfl_up1(Z[:, -1])
        Zn = np.empty_like(Z)
        Zn[:, 1:] = Z[:, :-1]
        Zn[:, 0] = incoming
        if t < Q:
            Zn += X * w[t]
        Z = Zn
    return Z.reshape(-1)


def warp_ws_1d(xs, w, lanes_per_array, R, seg_len):
    """Weight-stationary (BSM) step sequence on one warp tile.

    The warp holds 32/lanes_per_array independent arrays; array a streams the
    segment xs[a*seg_len : a*seg_len + seg_len + Qp - 1] (Qp = lanes_per_array*R
    PEs, taps beyond Q are zero).  PE s keeps w(s); x(t) is broadcast; partial
    sums move one PE up per step; the last PE emits y(t-(Qp-1)) at step t.
    Returns y[array][seg_len].
    """
    Q = len(w)
    Qp = lanes_per_array * R
    assert Qp >= Q and LANES % lanes_per_array == 0
    n_arr = LANES // lanes_per_array
    wp = np.zeros(Qp)
    wp[:Q] = w
    Wreg = np.tile(wp.reshape(lanes_per_array, R), (n_arr, 1))       # [32][R]
    xs = np.asarray(xs, dtype=np.float64)
    Z = np.zeros((LANES, R))
    first = np.arange(LANES) % lanes_per_array == 0
    last = np.arange(LANES) % lanes_per_array == lanes_per_array - 1
    y = np.zeros((n_arr, seg_len))
    for t in range(seg_len + Qp - 1):
        idx = np.arange(n_arr) * seg_len + t
        xb = np.repeat(np.where(idx < xs.size, xs[np.minimum(idx, xs.size - 1)], 0.0),
                       lanes_per_array)                              # broadcast in each array
        incoming = _shfl_up1(Z[:, -1], lanes_per_array)
        incoming[first] = 0.0                                        # PE 0 starts a new sum
        Zn = np.empty_like(Z)
        Zn[:, 1:] = Z[:, :-1]
        Zn[:, 0] = incoming
        Zn += xb[:, None] * Wreg
        Z = Zn
        c = t - (Qp - 1)
        if c >= 0:
            y[:, c] = Z[last, -1]
    return y


# ----------------------------------------------------------------------------
# The forms the CUDA kernels actually ship beyond the plain folded passes above: the same dataflows with a
# different choice of WHICH sums a PE-step updates together (pairs), with a whole array folded into one lane
# (weight-stationary), and with run-time strides.  Modelled step by step so that the method, not only the
# result, is pinned on the CPU.
# ----------------------------------------------------------------------------


def warp_os_1d_paired(xs, w, R):
    """Output-stationary, PE-paired: the sums of PEs 2m and 2m+1 form a pair that ONE operation updates with
    the same forwarded input x and the tap pair (w(t), w(t-1)): the odd PE lags one step behind the even one.
    Q+1 steps; the first and the last touch only one sum of each pair.  Returns all 32*R sums (valid prefix
    as for warp_os_1d)."""
    Q = len(w)
    assert R % 2 == 0
    D = np.asarray(xs, dtype=np.float64).reshape(-1).copy()          # forwarded inputs, PE-major
    n = D.size
    Z = np.zeros(n)
    even = np.arange(0, n, 2)
    for t in range(Q + 1):
        x = D[even]                                                  # the input the even PE of each pair holds
        if t == 0:
            Z[even] = x * w[0]
            Z[even + 1] = 0.0
        elif t == Q:
            Z[even + 1] += x * w[Q - 1]
        else:
            Z[even] += x * w[t]
            Z[even + 1] += x * w[t - 1]
        if t < Q:
            # inputs move one PE down: inside a lane by renaming, across lanes by one shuffle (lane 31 keeps its own)
            Dn = D.copy()
            Dn[:-1] = D[1:]
            D = Dn
    return Z


def warp_is_1d_paired(xs, w, R):
    """Input-stationary, paired: the sums of two neighbouring outputs o (even) and o+1 travel together; in PE
    s = o + t the pair takes x(s) * (w(t), w(t-1)).  Q+1 steps.  Returns y[o] for the outputs whose whole chain
    lies inside the tile (the first 32*R - Q of them, counted from output 0)."""
    Q = len(w)
    X = np.asarray(xs, dtype=np.float64).reshape(-1)
    n = X.size
    # pair[o/2] = (sum of output o, sum of output o+1), sitting in PE o + t after step t
    n_pairs = (n - Q) // 2
    first = np.zeros(n_pairs)
    second = np.zeros(n_pairs)
    for t in range(Q + 1):
        for m in range(n_pairs):
            s = 2 * m + t                                            # the PE the pair sits in at this step
            if t == 0:
                first[m] = X[s] * w[0]
            elif t == Q:
                second[m] += X[s] * w[Q - 1]
            else:
                first[m] += X[s] * w[t]
                second[m] += X[s] * w[t - 1]
    y = np.empty(2 * n_pairs)
    y[0::2], y[1::2] = first, second
    return y


def warp_ws_1d_one_lane(xs, w, seg_len, n_arrays):
    """Weight-stationary with a whole array (Q PEs) folded into ONE lane and the arrays handing their sums over
    instead of filling and draining.  Array a streams exactly the seg_len inputs of segment a.  PE s keeps w(s);
    at step t PE s adds x(t) * w(s) to the sum it took from PE s-1 (PE 0 opens a new sum); PE Q-1 emits.  The
    sum of output o = t - (Q-1) of the segment is emitted at step t; for o < 0 it is the part of an output of
    segment a-1's tail that array a's inputs contribute, and is stored there; when array a stops, the sums still
    in flight in its PEs 1 .. Q-1 are the parts its own inputs contribute to those tail outputs, and are added.
    The slice's last array has no successor: its tail takes the missing taps from a direct sum over the halo.
    xs holds n_arrays*seg_len + Q - 1 inputs; returns the n_arrays*seg_len outputs."""
    Q = len(w)
    xs = np.asarray(xs, dtype=np.float64)
    total = n_arrays * seg_len
    y = np.zeros(total)
    in_flight = np.zeros((n_arrays, Q))
    for a in range(n_arrays):
        Z = np.zeros(Q)
        for t in range(seg_len):
            x = xs[a * seg_len + t]
            Zn = np.empty(Q)
            Zn[0] = x * w[0]
            Zn[1:] = Z[:-1] + x * w[1:]
            Z = Zn
            o = a * seg_len + t - (Q - 1)
            if o >= 0:
                # t >= Q-1: a complete output of this segment; t < Q-1: array a's share of a tail output of
                # segment a-1, which array a-1 never emitted (the first array of the slice has no predecessor)
                y[o] = Z[Q - 1]
        in_flight[a] = Z
    for a in range(n_arrays):
        # PE s stopped while holding the part of output (a+1)*seg_len - 1 - s that array a's own inputs give
        for s in range(Q - 1):
            o = (a + 1) * seg_len - 1 - s
            y[o] += in_flight[a][s]
    # the last array's tail: no successor, the missing taps summed directly over the halo
    for j in range(Q - 1):
        o = total - 1 - j
        for k in range(j + 1, Q):
            y[o] += w[k] * xs[o + k]
    return y


def warp_os_1d_strided(xs, w, stride, n_pes):
    """Output-stationary with any stride, residue class by residue class: for b < stride the inputs x(stride*c + b)
    enter the PEs and move one PE down per step a, meeting the taps w(stride*a + b); the sums stay.  The last PE
    takes its inputs from memory.  Returns the n_pes sums."""
    Q = len(w)
    xs = np.asarray(xs, dtype=np.float64)
    Z = np.zeros(n_pes)
    c = np.arange(n_pes)
    for b in range(min(stride, Q)):
        X = xs[stride * c + b].copy()
        steps = (Q - b + stride - 1) // stride
        for a in range(steps):
            Z += X * w[stride * a + b]
            if a + 1 < steps:
                Xn = np.empty_like(X)
                Xn[:-1] = X[1:]
                Xn[-1] = xs[stride * (n_pes + a) + b]               # the array's last PE loads from memory
                X = Xn
    return Z
