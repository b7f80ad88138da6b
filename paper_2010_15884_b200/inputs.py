"""Seeded synthetic inputs for the benchmark configurations.

This module only draws random numbers (numpy ``default_rng`` = PCG64, the same
stream on every platform) and shapes them; it holds none of the method's
arithmetic.  The same arrays are handed to the CPU oracle and, copied to the
device, to the CUDA library.

Draw order inside one generator: the signal / image first, then one filter per
listed filter size, in the listed order.

The paper measured synthetic work as well (millions of independent small
convolutions, Section 6); there is no public dataset behind these inputs.
"""
from collections import OrderedDict

import numpy as np

# id -> description of the five benchmark configurations
CONFIGS = OrderedDict([
    (1, dict(kind="1d_f32", n=4096, filters=[8], seed=0,
             note="1-D fp32, N=4096, Q=8, x,w ~ U[-1,1)")),
    (2, dict(kind="1d_f32", n=1 << 26, filters=[4, 16, 32], seed=1,
             note="1-D fp32, N=2^26, Q in {4,16,32}, x,w ~ U[-1,1)")),
    (3, dict(kind="2d_f32", width=1920, height=1080, batch=1, filters=[5], seed=2, taps="uniform",
             note="2-D fp32 1920x1080, 5x5, pixels U[0,1), taps U[-1,1)")),
    (4, dict(kind="2d_u8s8", width=3840, height=2160, batch=1, filters=[3, 7], seed=3,
             note="2-D u8 x s8 -> s32, 3840x2160, 3x3 and 7x7, pixels 0..255, taps -8..8")),
    (5, dict(kind="2d_f32", width=4096, height=4096, batch=16, filters=[3, 9, 15], seed=4,
             taps="normal",
             note="2-D fp32 16 x 4096x4096, 3x3/9x9/15x15, pixels U[0,1), taps N(0, (1/k)^2)")),
])


def _uniform_pm1(rng, shape):
    """U[-1, 1) in fp32."""
    return (rng.random(shape, dtype=np.float32) * np.float32(2.0) - np.float32(1.0)).astype(np.float32)


def gen_1d_f32(n, filters, seed):
    """Signal x[n] ~ U[-1,1) and one filter w[q] ~ U[-1,1) per q in ``filters``."""
    rng = np.random.default_rng(seed)
    x = _uniform_pm1(rng, n)
    ws = OrderedDict((int(q), _uniform_pm1(rng, int(q))) for q in filters)
    return x, ws


def gen_2d_f32(width, height, filters, seed, batch=1, taps="uniform"):
    """Images x[batch][height][width] ~ U[0,1); one k x k filter per k in ``filters``.

    taps="uniform": U[-1,1).  taps="normal": N(0, sigma=1/k), so that the
    outputs stay O(1) whatever the filter size.
    ``filters`` entries may be ints (k x k) or (p, q) pairs (p rows, q columns).
    """
    rng = np.random.default_rng(seed)
    x = rng.random((batch, height, width), dtype=np.float32)
    ws = OrderedDict()
    for f in filters:
        p, q = (f, f) if np.isscalar(f) else f
        if taps == "uniform":
            w = _uniform_pm1(rng, (p, q))
        elif taps == "normal":
            w = (rng.standard_normal((p, q)) / float(max(p, q))).astype(np.float32)
        else:
            raise ValueError(taps)
        ws[(int(p), int(q))] = w
    return x, ws


def gen_2d_u8s8(width, height, filters, seed, batch=1):
    """Images uint8 uniform in 0..255; int8 taps uniform on the 17 integers -8..8."""
    rng = np.random.default_rng(seed)
    x = rng.integers(0, 256, size=(batch, height, width), dtype=np.uint8)
    ws = OrderedDict()
    for f in filters:
        p, q = (f, f) if np.isscalar(f) else f
        ws[(int(p), int(q))] = rng.integers(-8, 9, size=(p, q), dtype=np.int8)
    return x, ws


def gen_1d_u8s8(n, filters, seed):
    rng = np.random.default_rng(seed)
    x = rng.integers(0, 256, size=n, dtype=np.uint8)
    ws = OrderedDict((int(q), rng.integers(-8, 9, size=int(q), dtype=np.int8)) for q in filters)
    return x, ws


def make_config(cfg_id, scale=None):
    """Inputs of benchmark configuration ``cfg_id`` (1..5).

    ``scale`` optionally overrides sizes with a dict (e.g. ``{"n": 100000}`` or
    ``{"width": 512, "height": 300, "batch": 2}``) to get a reduced case with
    the same distributions and seed.  Returns (x, filters) as from ``gen_*``.
    """
    c = dict(CONFIGS[cfg_id])
    if scale:
        c.update(scale)
    if c["kind"] == "1d_f32":
        return gen_1d_f32(c["n"], c["filters"], c["seed"])
    if c["kind"] == "2d_f32":
        return gen_2d_f32(c["width"], c["height"], c["filters"], c["seed"], c["batch"], c["taps"])
    if c["kind"] == "2d_u8s8":
        return gen_2d_u8s8(c["width"], c["height"], c["filters"], c["seed"], c["batch"])
    raise ValueError(c["kind"])
