#!/usr/bin/env python
"""Benchmark of the warp-systolic convolution library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfgN]

Prints ONE JSON line.  A "step" is one pass of the whole hot path over the
workload: every filter size of the configuration through every systolic design
(weight-, output-, input-stationary), one kernel launch each.  The default
workload is configuration 2 (1-D fp32, N = 2^26, Q in {4, 16, 32}: nine
launches per step); the metric is output elements per second.

* value      device-resident inputs, CUDA-event time around K steps
* e2e        the same step through the host-buffer C-ABI entry points (pinned
             host memory, host<->device copies inside the timed region); 1-D:
             one sysconv1d_host_multi call per step (signal copied in once)
* roofline   the kernel with the largest share of the step, algorithmic bytes /
             its average launch time (per-launch CUDA events) vs the measured
             HBM copy bandwidth of this machine (MEASURED_PEAKS.json)
* cpu_baseline  the CPU oracle timed on this machine's cores on a bounded sample
* detail     per (configuration, filter, design): time, Gpix/s, GB/s, roofline
             fraction (all five configurations unless --no-detail).  The
             configurations that fit the L2 cache (1, 3, 4) are timed three
             ways: launches back to back over a rotating set of buffer pairs
             larger than L2 inside one event pair (directly launched and
             replayed from a CUDA graph; every launch L2-cold), one launch at a
             time after an L2 flush, and warm (the same buffers again)
* target     best design per configuration and filter against the 0.70 bar
* peaks      issue rates of the plain datapaths measured on this device by the
             library (sysconv_measure_peaks): the ALU roofline denominators

--impl reference times the CPU oracle (the only reference there is: the paper
ships no code and its comparison system is Intel fixed-function hardware).
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

HBM_FALLBACK_GBS = 6650.0
HBM_NOMINAL_GBS = 8000.0
SM_COUNT = 148
# Plain-datapath rates in multiply-adds per clock per SM.  These are the architectural figures; run_ours() replaces
# them with what the library measures on the device (sysconv_measure_peaks) before any roofline is computed.
FP32_LANES_PER_SM = 128
# dp4a issues on 64 lanes per clock per SM on B200 and does four 8-bit multiply-adds per lane
INT8_DOT_MACS_PER_SM = 256
NAMES = {0: "WS", 1: "OS", 2: "IS"}
TARGET_FRAC = 0.70
ROTATING_BYTES = 160e6          # a rotating set of buffer pairs is at least this large (L2 holds 126 MB)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured", float(d.get("sm_max_mhz", 1965.0))
    except Exception:
        return HBM_FALLBACK_GBS, "fallback", 1965.0


# --------------------------------------------------------------------------- clocks


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); pw.append(float(r[2]))
            except ValueError:
                continue
            for name, flag in zip(names, r[3:7]):
                if flag.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------- workloads


class Case:
    """One kernel launch of a workload: a (filter, design) pair on resident device buffers.

    launchers[i](stream) enqueues the launch on buffer pair i; pair 0 is the one the step uses, the others hold
    the same data and exist only so that back-to-back launches never find their data in L2."""

    def __init__(self, cfg, label, design, launchers, n_out, alg_bytes, macs, mac_lanes=None, floor=None):
        self.cfg, self.label, self.design, self.launchers = cfg, label, design, launchers
        self.n_out, self.alg_bytes, self.macs = n_out, alg_bytes, macs
        # multiply-adds per clock per SM of the plain (non-tensor) datapath this case runs on
        self.mac_lanes = mac_lanes or FP32_LANES_PER_SM
        self.floor = floor              # launchers of the plain streaming kernel that moves the same bytes
        self.times_ms = []

    def launch(self, stream=None):
        self.launchers[0](stream)


def build_cases(cfg_id, device, designs=(0, 1, 2), scale=None, rotate=False):
    """Generate the configuration's inputs, copy them to the device, return (cases, keepalive).

    rotate: allocate at least 16 copies of the input and output buffers, and enough that one pass over all copies
    touches more than ROTATING_BYTES (for the configurations that would otherwise sit in L2)."""
    import torch
    from paper_2010_15884_b200 import binding as B
    from paper_2010_15884_b200 import inputs
    x, ws = inputs.make_config(cfg_id, scale)
    kind = inputs.CONFIGS[cfg_id]["kind"]
    dtype = B.U8S8_S32 if kind == "2d_u8s8" else B.F32
    out_dtype = torch.int32 if kind == "2d_u8s8" else torch.float32
    per_pair = x.size * x.itemsize * 5 if kind == "2d_u8s8" else x.size * x.itemsize * 2
    copies = max(16, min(64, int(-(-ROTATING_BYTES // per_pair)))) if rotate else 1
    xds = [torch.from_numpy(x).to(device) for _ in range(copies)]
    cases, keep = [], list(xds)

    def stream_ptr(stream):
        return (stream if stream is not None else torch.cuda.current_stream()).cuda_stream

    def checked(call, *cargs):
        def run(stream=None):
            st = call(*cargs, stream_ptr(stream))
            if st != 0:
                raise B.SysconvError(st, call.__name__)
        return run

    for key, w in ws.items():
        w = np.ascontiguousarray(w)
        keep.append(w)
        if kind == "1d_f32":
            q = key
            n = x.shape[0]
            n_out = n - q + 1
            yds = [torch.empty(n_out, dtype=out_dtype, device=device) for _ in range(copies)]
            alg = 4 * n + 4 * n_out
            macs = n_out * q
            label = "Q=%d" % q

            def mk(d, w=w, q=q, n=n, n_out=n_out, yds=yds):
                return [checked(B.sysconv1d, xd.data_ptr(), n, n, w, q, yd.data_ptr(), n_out, 1, dtype, d)
                        for xd, yd in zip(xds, yds)]
            in_bytes = 4 * n
        else:
            p, q = key
            batch, h, wd = x.shape
            oh, ow = h - p + 1, wd - q + 1
            # output rows padded to a 16-byte multiple so that every row starts aligned
            y_pitch = (ow + 3) // 4 * 4
            yds = [torch.empty((batch, oh, y_pitch), dtype=out_dtype, device=device) for _ in range(copies)]
            n_out = batch * oh * ow
            alg = x.size * x.itemsize + 4 * n_out
            macs = n_out * p * q
            label = "%dx%d" % (p, q)

            def mk(d, w=w, p=p, q=q, h=h, wd=wd, oh=oh, y_pitch=y_pitch, batch=batch, yds=yds):
                return [checked(B.sysconv2d, xd.data_ptr(), wd, h, wd, h * wd, w, q, p, yd.data_ptr(), y_pitch,
                                oh * y_pitch, batch, dtype, d) for xd, yd in zip(xds, yds)]
            in_bytes = x.size * x.itemsize
        keep += yds
        floor = None
        if rotate:
            # the yardstick: one plain streaming kernel that reads the input bytes and writes as many bytes as the
            # convolution writes (uint8: widened to int32), on the same rotating buffers
            widen = kind == "2d_u8s8"
            out_bytes = yds[0].numel() * 4
            nb = min(in_bytes, out_bytes // 4 if widen else out_bytes) // 16 * 16
            floor = [checked(B.load_library().sysconv_floor_copy, xd.data_ptr(), yd.data_ptr(), nb, 1 if widen else 0)
                     for xd, yd in zip(xds, yds)]
        for d in designs:
            cases.append(Case(cfg_id, label, d, mk(d), n_out, alg, macs,
                              INT8_DOT_MACS_PER_SM if kind == "2d_u8s8" else None, floor))
    return cases, keep


def build_strided_cases(device):
    """Stride-2 forms (Table 2, cell 6) at the sizes of configurations 2 and 5 (OS and IS designs), and separable
    filters on the images of configuration 5."""
    import torch
    from paper_2010_15884_b200 import binding as B
    from paper_2010_15884_b200 import inputs
    cases, keep = [], []

    def checked(call, *cargs):
        def run(stream=None):
            st = call(*cargs, (stream if stream is not None else torch.cuda.current_stream()).cuda_stream)
            if st != 0:
                raise B.SysconvError(st, call.__name__)
        return run

    x, ws = inputs.make_config(2)
    xd = torch.from_numpy(x).to(device)
    keep.append(xd)
    n = x.shape[0]
    for q, w in ws.items():
        n_out = (n - q) // 2 + 1
        yd = torch.empty(n_out, dtype=torch.float32, device=device)
        keep += [w, yd]
        for d in (B.OS, B.IS):
            cases.append(Case("2/stride2", "Q=%d" % q, d,
                              [checked(B.sysconv1d_strided, xd.data_ptr(), n, n, w, q, 2, yd.data_ptr(), n_out, 1,
                                       B.F32, d)], n_out, 4 * n + 4 * n_out, n_out * q))
    x, ws = inputs.make_config(5, dict(filters=[3]))
    x2 = torch.from_numpy(x).to(device)
    keep.append(x2)
    batch, h, wd = x.shape
    rng = np.random.default_rng(11)
    for k in (3, 7):
        w = rng.normal(0, 1.0 / k, (k, k)).astype(np.float32)
        oh, ow = (h - k) // 2 + 1, (wd - k) // 2 + 1
        y_pitch = (ow + 3) // 4 * 4
        yd = torch.empty((batch, oh, y_pitch), dtype=torch.float32, device=device)
        keep += [w, yd]
        n_out = batch * oh * ow
        for d in (B.OS, B.IS):
            cases.append(Case("5/stride2", "%dx%d" % (k, k), d,
                              [checked(B.sysconv2d_strided, x2.data_ptr(), wd, h, wd, h * wd, w, k, k, 2, 2,
                                       yd.data_ptr(), y_pitch, oh * y_pitch, batch, B.F32, d)],
                              n_out, x.size * 4 + 4 * n_out, n_out * k * k))
    # separable filters (rank-one u v^T) on the same images: P + Q multiply-adds per output
    for k in (3, 9, 15):
        u = rng.normal(0, 1.0 / np.sqrt(k), k).astype(np.float32)
        v = rng.normal(0, 1.0 / np.sqrt(k), k).astype(np.float32)
        oh, ow = h - k + 1, wd - k + 1
        y_pitch = (ow + 3) // 4 * 4
        yd = torch.empty((batch, oh, y_pitch), dtype=torch.float32, device=device)
        keep += [u, v, yd]
        n_out = batch * oh * ow
        cases.append(Case("5/separable", "%d+%d" % (k, k), B.OS,
                          [checked(B.sysconv2d_separable, x2.data_ptr(), wd, h, wd, h * wd, u, v, yd.data_ptr(), y_pitch,
                                   oh * y_pitch, batch)], n_out, x.size * 4 + 4 * n_out, n_out * 2 * k))
    # the second workload: Jacobi sweeps of a 3x3 stencil over the same 16 grids, up to four sweeps fused per pass
    # (algorithmic bytes: the grid read and written once per pass of up to four sweeps)
    five = np.array([[0, 0.125, 0], [0.125, 0.5, 0.125], [0, 0.125, 0]], np.float32)
    nine = np.array([[0.0625, 0.125, 0.0625], [0.125, 0.25, 0.125], [0.0625, 0.125, 0.0625]], np.float32)
    out = torch.empty((batch, h, wd), dtype=torch.float32, device=device)
    scratch = torch.empty((batch, h, wd), dtype=torch.float32, device=device)
    keep += [five, nine, out, scratch]
    for name, k in (("5pt", five), ("9pt", nine)):
        for sweeps in (1, 4, 8):
            passes = -(-sweeps // 4)
            cases.append(Case("5/stencil", "%s x%d" % (name, sweeps), B.OS,
                              [checked(B.sysstencil2d, x2.data_ptr(), wd, h, wd, h * wd, k, sweeps, out.data_ptr(), wd, h * wd,
                                       batch, scratch.data_ptr())], batch * h * wd * sweeps, 8 * x.size * passes,
                              batch * (h - 2) * (wd - 2) * sweeps * (5 if name == "5pt" else 9)))
    return cases, keep


def roofline_time_s(case, hbm_gbs, sm_mhz):
    """max(bytes / HBM bandwidth, MACs / plain-ALU MAC rate) for one launch."""
    t_mem = case.alg_bytes / (hbm_gbs * 1e9)
    mac_rate = SM_COUNT * case.mac_lanes * sm_mhz * 1e6
    t_alu = case.macs / mac_rate
    return max(t_mem, t_alu), ("hbm" if t_mem >= t_alu else "alu")


def time_cases_individually(cases, warmup, reps, flush):
    """Per-launch CUDA-event timing, each launch bracketed by its own event pair."""
    import torch
    for c in cases:
        for _ in range(warmup):
            c.launch()
    torch.cuda.synchronize()
    for c in cases:
        c.times_ms = []
        for _ in range(reps):
            if flush is not None:
                flush.add_(1.0)          # > L2 write between iterations
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            c.launch()
            e1.record()
            e1.synchronize()
            c.times_ms.append(e0.elapsed_time(e1))


def time_back_to_back(launchers, rounds=10):
    """Microseconds per launch of a chain of launches over rotating buffer pairs, all inside ONE event pair on one
    stream: (directly launched, replayed from a CUDA graph that holds one launch per buffer pair).  With more than
    L2 of distinct data in the set every launch starts L2-cold; neither per-launch events nor a flush kernel sit
    between the launches."""
    import torch
    side = torch.cuda.Stream()
    n = len(launchers)
    with torch.cuda.stream(side):
        for f in launchers:
            f(side)
        side.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(side)
        for _ in range(rounds):
            for f in launchers:
                f(side)
        e1.record(side)
        e1.synchronize()
        direct_us = e0.elapsed_time(e1) * 1e3 / (rounds * n)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for f in launchers:
                f(side)
        graph.replay()
        side.synchronize()
        e0.record(side)
        for _ in range(rounds):
            graph.replay()
        e1.record(side)
        e1.synchronize()
        graph_us = e0.elapsed_time(e1) * 1e3 / (rounds * n)
    del graph
    return direct_us, graph_us


def detail_rows(cases, hbm_gbs, peak_kind, sm_max):
    rows = []
    for c in cases:
        med = statistics.median(c.times_ms)
        t_roof, bound = roofline_time_s(c, hbm_gbs, sm_max)
        rows.append({
            "config": c.cfg, "filter": c.label, "design": NAMES[c.design],
            "ms_median": round(med, 5), "ms_min": round(min(c.times_ms), 5),
            "gpix_s": round(c.n_out / (med * 1e-3) / 1e9, 3),
            "gb_s": round(c.alg_bytes / (med * 1e-3) / 1e9, 1),
            "roofline_bound": bound,
            "roofline_us": round(t_roof * 1e6, 3),
            "roofline_frac": round(t_roof / (med * 1e-3), 4),
            "hbm_frac": round(c.alg_bytes / (med * 1e-3) / 1e9 / hbm_gbs, 4),
            "hbm_frac_of_nominal_8tbs": round(c.alg_bytes / (med * 1e-3) / 1e9 / HBM_NOMINAL_GBS, 4),
        })
    return rows


def l2_sized_rows(cfg_id, device, hbm_gbs, peak_kind, sm_max, reps, flush):
    """Detail rows of a configuration whose data fit the L2 cache: the launch is timed L2-cold back to back over
    rotating buffers (direct and graph-replayed), one at a time after a flush, and warm; the roofline fraction
    quoted is that of the graph-replayed chain (device time per launch, no host launch cost between launches)."""
    import torch
    cases, keep = build_cases(cfg_id, device, rotate=True)
    time_cases_individually(cases, 3, reps, flush)
    rows = detail_rows(cases, hbm_gbs, peak_kind, sm_max)
    floors = {}
    for c, row in zip(cases, rows):
        t_roof, _ = roofline_time_s(c, hbm_gbs, sm_max)
        direct_us, graph_us = time_back_to_back(c.launchers)
        row["timing"] = "back to back over %d rotating buffer pairs (%.0f MB), one event pair" % (
            len(c.launchers), len(c.launchers) * c.alg_bytes / 1e6)
        row["us_back_to_back"] = round(direct_us, 3)
        row["us_back_to_back_graph"] = round(graph_us, 3)
        row["us_flushed_single"] = round(row.pop("ms_median") * 1e3, 3)
        row["us_flushed_single_min"] = round(row.pop("ms_min") * 1e3, 3)
        # warm: the same buffer pair again and again (graph-replayed, like the cold chain)
        row["us_warm_l2_graph"] = round(time_back_to_back([c.launchers[0]] * 8)[1], 3)
        best_us = min(direct_us, graph_us)
        row["gpix_s"] = round(c.n_out / best_us / 1e3, 3)
        row["gb_s"] = round(c.alg_bytes / best_us / 1e3, 1)
        row["roofline_frac"] = round(t_roof * 1e6 / best_us, 4)
        row["hbm_frac"] = round(c.alg_bytes / best_us / 1e3 / hbm_gbs, 4)
        row["hbm_frac_of_nominal_8tbs"] = round(c.alg_bytes / best_us / 1e3 / HBM_NOMINAL_GBS, 4)
        if c.label not in floors:
            floors[c.label] = time_back_to_back(c.floor)
        f_direct, f_graph = floors[c.label]
        row["plain_streaming_kernel_same_bytes_us"] = round(min(f_direct, f_graph), 3)
        row["frac_of_plain_streaming_kernel"] = round(min(f_direct, f_graph) / best_us, 3)
    del cases, keep
    torch.cuda.empty_cache()
    return rows


def target_table(rows, cfg_ids):
    """The stated target, row by row: the best design of every (configuration, filter) against TARGET_FRAC of its
    roofline, and the minimum over the configurations."""
    out, worst = [], None
    for cfg in cfg_ids:
        mine = [r for r in rows if r["config"] == cfg]
        for label in sorted({r["filter"] for r in mine}, key=lambda t: [int(v) for v in t.replace("Q=", "").split("x")]):
            best = max((r for r in mine if r["filter"] == label), key=lambda r: r["roofline_frac"])
            entry = {"config": cfg, "filter": label, "best_design": best["design"], "roofline_frac": best["roofline_frac"],
                     "bound": best["roofline_bound"], "roofline_us": best["roofline_us"],
                     "pass_at_%.2f" % TARGET_FRAC: bool(best["roofline_frac"] >= TARGET_FRAC)}
            if "plain_streaming_kernel_same_bytes_us" in best:
                entry["plain_streaming_kernel_frac"] = round(best["roofline_us"] / best["plain_streaming_kernel_same_bytes_us"], 4)
            if cfg == 1:
                entry["note"] = "roofline 5 ns: no launch can approach it; listed, not counted in the minimum"
            elif worst is None or best["roofline_frac"] < worst:
                worst = best["roofline_frac"]
            out.append(entry)
    return {"bar": TARGET_FRAC, "rows": out, "min_over_configs_2_to_5": worst,
            "all_pass": bool(worst is not None and worst >= TARGET_FRAC)}


# --------------------------------------------------------------------------- CPU oracle arm


def oracle_sample(cfg_id):
    """Time the oracle, as it stands, on a bounded sample of the configuration.

    Returns (outputs, seconds, threads, description).  1-D: passes per filter length over the first
    2^24 samples.  2-D: passes per filter size over the first 1024 rows of image 0.  The passes repeat until
    about one second of wall time (10-20 core-seconds on this machine's host cores) has gone by.
    """
    import oracle
    from paper_2010_15884_b200 import inputs
    x, ws = inputs.make_config(cfg_id)
    kind = inputs.CONFIGS[cfg_id]["kind"]
    outs = 0
    if kind == "1d_f32":
        x = x[: 1 << 24]
        oracle.conv1d_f32(x[: 1 << 16], next(iter(ws.values())), want_scale=False)   # load + warm
        t0, reps = time.perf_counter(), 0
        while reps < 50 and time.perf_counter() - t0 < 1.0:
            for w in ws.values():
                outs += oracle.conv1d_f32(x, w, want_scale=False)[0].size
            reps += 1
        what = "%d fp64 passes of Eq. 2 per filter length over the first %d samples" % (reps, x.shape[0])
    else:
        img = np.ascontiguousarray(x[0][:1024])
        f = oracle.conv2d_f32 if kind == "2d_f32" else (lambda a, b, want_scale=False: (oracle.conv2d_u8s8_s32(a, b), None))
        f(img[:32], next(iter(ws.values())), want_scale=False)
        t0, reps = time.perf_counter(), 0
        while reps < 50 and time.perf_counter() - t0 < 1.0:
            for w in ws.values():
                outs += f(img, w, want_scale=False)[0].size
            reps += 1
        what = "%d passes of Eq. 3 per filter size over the first %d rows of image 0" % (reps, img.shape[0])
    return outs, time.perf_counter() - t0, oracle.num_threads(), what


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores, rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    sample_n = 1 << 24
    import oracle
    from paper_2010_15884_b200 import inputs
    x, ws = inputs.make_config(2)
    x = x[:sample_n]
    for _ in range(max(args.warmup, 1)):
        oracle.conv1d_f32(x[: 1 << 18], ws[4], want_scale=False)
    outs, t0 = 0, time.perf_counter()
    for _ in range(args.steps):
        for q, w in ws.items():
            y, _ = oracle.conv1d_f32(x, w, want_scale=False)
            outs += 3 * y.size                          # the three designs share this one definition
    dt = time.perf_counter() - t0
    value = outs / dt / 1e9
    sample = ("per step: one fp64 pass of Eq. 2 per filter length (4, 16, 32) over the first 2^24 samples of "
              "configuration 2, counted once per design")
    line = {
        "impl": "reference", "metric": "output elements/s", "value": round(value, 4), "unit": "Gpix/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": round(dt / args.steps * 1e3, 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "cfg2: 1-D fp32 N=2^26, Q in {4,16,32}, designs WS/OS/IS", "sample": sample},
        "cpu_baseline": {"value": round(value, 4), "unit": "Gpix/s", "cores": oracle.num_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": round(value, 4), "unit": "Gpix/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- our arm


def run_ours(args):
    global FP32_LANES_PER_SM, INT8_DOT_MACS_PER_SM
    import torch
    import torch.distributed as dist
    from paper_2010_15884_b200 import binding as B
    from paper_2010_15884_b200 import inputs, shard

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    B.load_library()
    hbm_gbs, peak_kind, sm_max = measured_peaks()

    # ---- the plain-datapath rates of this device, measured by the library: the ALU roofline denominators
    scratch = torch.empty(1 << 30, dtype=torch.uint8, device=device)
    peaks = B.measure_peaks(scratch)
    del scratch
    torch.cuda.empty_cache()
    FP32_LANES_PER_SM = peaks["ffma_per_clk_sm"]
    INT8_DOT_MACS_PER_SM = 4.0 * peaks["dp4a_per_clk_sm"]

    cfg_id = int(args.workload.replace("cfg", ""))
    scale = None
    if args.profile_n and cfg_id in (1, 2):
        scale = {"n": args.profile_n}                  # reduced case for ncu captures only
    if args.profile_batch and cfg_id == 5:
        scale = {"batch": args.profile_batch}
    if args.profile_filter and cfg_id in (4, 5):
        scale = dict(scale or {}, filters=[args.profile_filter])   # ncu captures only: one filter's buffers on the device
    split = args.split_images and cfg_id == 5 and world > 1
    if split:
        # strong scaling: the 16 independent images are dealt out to the ranks (no collective on the data path)
        lo, hi = shard.split_range(inputs.CONFIGS[5]["batch"], rank, world)
        scale = dict(scale or {}, batch=max(hi - lo, 1))
    cases, keep = build_cases(cfg_id, device, scale=scale)   # every rank holds its own copy: weak scaling
    outputs_per_step = sum(c.n_out for c in cases)

    # ---- device-resident timing: W warm-up steps, then exactly K timed steps
    small = max(c.alg_bytes for c in cases) < 256e6     # fits L2: flush between steps
    flush = torch.zeros(64 << 20, dtype=torch.float32, device=device) if small else None
    for _ in range(args.warmup):
        for c in cases:
            c.launch()
    launches0 = B.launch_count()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    torch.cuda.synchronize()
    shard.barrier(world)
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in cases]
          for _ in range(args.steps)]
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    flush_ms = 0.0
    start.record()
    for k in range(args.steps):
        if flush is not None:
            f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            f0.record(); flush.add_(1.0); f1.record()
            ev[k].append((f0, f1))
        for i, c in enumerate(cases):
            ev[k][i][0].record()
            c.launch()
            ev[k][i][1].record()
    stop.record()
    torch.cuda.synchronize()
    shard.barrier(world)
    clocks = sampler.stop() if rank == 0 else None
    launches = B.launch_count() - launches0
    total_ms = start.elapsed_time(stop)
    if flush is not None:
        flush_ms = sum(ev[k][-1][0].elapsed_time(ev[k][-1][1]) for k in range(args.steps))
        total_ms -= flush_ms
    for i, c in enumerate(cases):
        c.times_ms = [ev[k][i][0].elapsed_time(ev[k][i][1]) for k in range(args.steps)]
    # whole-job throughput: the outputs of all ranks over the slowest rank's time
    value = shard.aggregate_throughput(outputs_per_step * args.steps, total_ms * 1e-3, world, device) / 1e9
    total_ms = shard.max_over_ranks(total_ms, world, device)

    # ---- roofline of the kernel with the largest share of the step
    top = max(cases, key=lambda c: sum(c.times_ms))
    avg_s = statistics.mean(top.times_ms) * 1e-3
    t_roof, bound = roofline_time_s(top, hbm_gbs, sm_max)
    if bound == "hbm":
        roofline = {
            "kernel": "%s %s" % (NAMES[top.design], top.label), "bound": "hbm",
            "achieved": round(top.alg_bytes / avg_s / 1e9, 1), "peak": hbm_gbs, "unit": "GB/s",
            "frac": round(top.alg_bytes / avg_s / 1e9 / hbm_gbs, 4), "peak_source": "of " + peak_kind,
        }
    else:
        # plain FP32/INT32 ALUs (no tensor cores: small-filter stencil): SMs x measured MACs per clock x 2 flops x SM max clock
        peak_tflops = SM_COUNT * top.mac_lanes * 2 * sm_max * 1e6 / 1e12
        roofline = {
            "kernel": "%s %s" % (NAMES[top.design], top.label), "bound": "alu",
            "achieved": round(2 * top.macs / avg_s / 1e12, 2), "peak": round(peak_tflops, 1), "unit": "TFLOP/s",
            "frac": round(2 * top.macs / avg_s / 1e12 / peak_tflops, 4),
            "peak_source": "derived: 148 SMs x %.1f multiply-adds per clock per SM (measured on this device) x 2 x %.0f MHz"
                           % (top.mac_lanes, sm_max),
        }
    sm_mhz = (clocks or {}).get("sm_mhz")
    roofline.update({
        "traffic": ncu_traffic(cfg_id, top),
        "algorithmic_bytes": int(top.alg_bytes),
        "share_of_step": round(sum(top.times_ms) / sum(sum(c.times_ms) for c in cases), 4),
        "hbm_time_frac": round(top.alg_bytes / (hbm_gbs * 1e9) / avg_s, 4),
        "hbm_frac_of_nominal_8tbs": round(top.alg_bytes / avg_s / 1e9 / HBM_NOMINAL_GBS, 4),
        "alu_time_frac": round(top.macs / (SM_COUNT * top.mac_lanes * sm_max * 1e6) / avg_s, 4),
        # the kernel's duration in SM cycles at the clock sampled during the run: comparable between a short run at
        # the boost clock and a long one under the power cap
        "avg_us": round(avg_s * 1e6, 3),
        "avg_kcycles_at_sampled_clock": round(avg_s * sm_mhz * 1e3, 1) if sm_mhz else None,
    })

    # ---- end to end through the host-buffer entry points (rank-local pinned buffers)
    e2e = None if (args.no_e2e or scale) else run_e2e(cfg_id, device, args, world)

    line = {
        "metric": "output elements/s", "value": round(value, 3), "unit": "Gpix/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(total_ms / args.steps, 4),
        "higher_is_better": True, "scaling": "strong" if split else "weak", "vs_baseline": None,
        "dtype": "f32" if inputs.CONFIGS[cfg_id]["kind"] != "2d_u8s8" else "s32", "data": "synthetic",
        "config": {"workload": "cfg%d: %s; every filter x designs WS/OS/IS, one launch each"
                               % (cfg_id, inputs.CONFIGS[cfg_id]["note"]),
                   "launches_per_step": len(cases),
                   "l2": "flushed between steps (256 MiB write, excluded from the time)" if small
                         else "inputs larger than L2 (268 MB signal per launch)",
                   "per_rank": ("the 16 images are dealt out to the ranks (independent problems, no collective)" if split else
                                "each rank convolves its own copy (independent problems, no collective)")},
        "roofline": roofline, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
    }
    if rank == 0:
        if scale:
            line["config"]["reduced_for_profiling"] = scale
        line["peaks"] = dict({k: round(v, 2) for k, v in peaks.items()},
                             hbm_gbs=hbm_gbs, hbm_source=peak_kind, hbm_nominal_gbs=HBM_NOMINAL_GBS, sm_max_mhz=sm_max,
                             fp32_tflops=round(SM_COUNT * FP32_LANES_PER_SM * 2 * sm_max * 1e-6, 1),
                             int8_dot_tmacs=round(SM_COUNT * INT8_DOT_MACS_PER_SM * sm_max * 1e-6, 1))
        if not args.no_cpu:
            outs, secs, cores, what = oracle_sample(cfg_id)
            line["cpu_baseline"] = {
                "value": round(outs / secs / 1e9, 4), "unit": "Gpix/s", "cores": cores, "kind": "oracle",
                "sample": "%s of configuration %d (%.1f s wall on %d threads)" % (what, cfg_id, secs, cores)}
            line["cpu_baseline"]["one_core"] = oracle_one_core(cfg_id)
        line["per_kernel"] = detail_rows(cases, hbm_gbs, peak_kind, sm_max)
        # context only: another machine, another baseline (Intel GEN9.5, fixed-function sampler); not comparable
        line["paper_context"] = ("the paper (abstract, Section 6) reports its best software systolic designs, SBM and "
                                 "FBS, 14-59 % faster than the GEN9.5 GPU's hardware sampler on the same 1-D and "
                                 "small 2-D convolutions; neither that GPU nor a sampler exists here")
        if not args.no_detail and world == 1 and not scale:
            mine = [dict(r) for r in line["per_kernel"]]
            del cases, keep
            torch.cuda.empty_cache()
            line["detail"] = all_config_detail(device, hbm_gbs, peak_kind, sm_max, skip=cfg_id,
                                               reps=args.detail_reps)
            line["target"] = target_table(mine + line["detail"], (1, 2, 3, 4, 5))
            line["six_designs_paper_experiment"] = six_designs_table(device, args.detail_reps, hbm_gbs)
            line["cfg1_step_in_cuda_graph"] = graph_replay_ms(1, device, 200)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def oracle_one_core(cfg_id):
    """The same oracle on ONE host thread, on a smaller sample of the configuration (about a second)."""
    import oracle
    from paper_2010_15884_b200 import inputs
    x, ws = inputs.make_config(cfg_id)
    kind = inputs.CONFIGS[cfg_id]["kind"]
    threads = oracle.num_threads()
    oracle.set_num_threads(1)
    try:
        outs, t0 = 0, time.perf_counter()
        if kind == "1d_f32":
            part = x[: 1 << 21]
            for w in ws.values():
                outs += oracle.conv1d_f32(part, w, want_scale=False)[0].size
            what = "one fp64 pass of Eq. 2 per filter length over the first %d samples" % part.shape[0]
        else:
            img = np.ascontiguousarray(x[0][:128])
            for w in ws.values():
                if kind == "2d_f32":
                    outs += oracle.conv2d_f32(img, w, want_scale=False)[0].size
                else:
                    outs += oracle.conv2d_u8s8_s32(img, w).size
            what = "one pass of Eq. 3 per filter size over the first %d rows of image 0" % img.shape[0]
        secs = time.perf_counter() - t0
    finally:
        oracle.set_num_threads(threads)
    return {"value": round(outs / secs / 1e9, 5), "unit": "Gpix/s", "cores": 1, "sample": what}


def ncu_traffic(cfg_id, case):
    """DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch of this kernel from the ncu captures
    summarised under profiles/ (traffic.json, written from the captures), if one covers it."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            table = json.load(f)["dram_bytes_per_launch"]
    except Exception:
        return None
    return table.get("cfg%d %s %s" % (cfg_id, NAMES[case.design], case.label))


def run_e2e(cfg_id, device, args, world):
    """The same step from pinned HOST buffers through sysconv*_host (copies inside the timed region)."""
    import torch
    from paper_2010_15884_b200 import binding as B
    from paper_2010_15884_b200 import inputs, shard
    x, ws = inputs.make_config(cfg_id)
    kind = inputs.CONFIGS[cfg_id]["kind"]
    dtype = B.U8S8_S32 if kind == "2d_u8s8" else B.F32
    xh = torch.from_numpy(x).pin_memory()
    jobs, h2d, d2h, outputs = [], 0, 0, 0
    for key, w in ws.items():
        if kind == "1d_f32":
            yh = torch.empty(x.shape[0] - key + 1, dtype=torch.float32).pin_memory()
            wbytes = B.host_workspace_bytes(tuple(x.shape), (key,), dtype)
            call = B.sysconv1d_host
        else:
            p, q = key
            yh = torch.empty((x.shape[0], x.shape[1] - p + 1, x.shape[2] - q + 1),
                             dtype=torch.int32 if dtype == B.U8S8_S32 else torch.float32).pin_memory()
            wbytes = B.host_workspace_bytes(tuple(x.shape), (p, q), dtype)
            call = B.sysconv2d_host
        for d in (0, 1, 2):
            jobs.append((call, w, yh, d))
            h2d += xh.numel() * xh.element_size()
            d2h += yh.numel() * yh.element_size()
            outputs += yh.numel()
    steps = max(1, min(args.steps, args.e2e_steps))
    if kind == "1d_f32":
        # one call per step: the signal crosses to the device once, every (filter, design) job copies its result back
        multi = [(w, d, torch.empty_like(yh).pin_memory()) for _, w, yh, d in jobs]
        h2d = xh.numel() * xh.element_size() + sum(4 * len(w) for w, _, _ in multi)
        work = torch.empty(B.host_multi_workspace_bytes(x.shape[0], [len(w) for w, _, _ in multi]), dtype=torch.uint8,
                           device=device)
        path = "sysconv1d_host_multi: pinned host signal -> device once -> 9 kernels per chunk -> 9 pinned host results"

        def one_step():
            B.sysconv1d_host_multi(xh, multi, work)
    else:
        work = torch.empty(max(B.host_workspace_bytes(tuple(x.shape), k, dtype) for k in ws), dtype=torch.uint8,
                           device=device)
        path = "sysconv2d_host per (filter, design): pinned host -> device workspace -> kernel -> pinned host"

        def one_step():
            for call, w, yh, d in jobs:
                call(xh, w, yh, d, work, dtype=dtype)

    one_step()
    torch.cuda.synchronize()
    shard.barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        one_step()
    e1.record()
    torch.cuda.synchronize()
    shard.barrier(world)
    ms = shard.max_over_ranks(e0.elapsed_time(e1), world, device)
    return {"value": round(world * outputs * steps / (ms * 1e-3) / 1e9, 4), "unit": "Gpix/s",
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": steps,
            "ms_per_step": round(ms / steps, 3),
            "path": path}


def graph_replay_ms(cfg_id, device, reps):
    """One step of a launch-bound configuration (every filter x design) captured once in a CUDA graph and replayed:
    ms per step by replay and by direct launches (CUDA events around `reps` back-to-back steps, no L2 flush)."""
    import torch
    cases, keep = build_cases(cfg_id, device)
    for c in cases:
        c.launch()                       # first-call set-up happens outside the capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for c in cases:
                c.launch(side)
    out = {}
    for name, run in (("graph_replay", graph.replay), ("direct_launches", lambda: [c.launch() for c in cases])):
        for _ in range(3):
            run()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            run()
        e1.record(); e1.synchronize()
        out[name + "_ms_per_step"] = round(e0.elapsed_time(e1) / reps, 5)
    out["launches_per_step"] = len(cases)
    del cases, keep
    return out


def six_designs_table(device, reps, hbm_gbs):
    """The paper's own experiment (Section 6, Tables 3 and 4) on B200: more than ten million independent 1-D
    convolutions of 16 outputs each, filter sizes 2 and 5, through all six designs (small unfolded arrays side by
    side in a warp).  Throughput = outputs / kernel time, as in the paper; beside it the analytical model's outturn
    and lane utilisation for 16 outputs, filter size 5 (Table 4), and the paper's own relative performance against
    the GEN9.5 sampler (Table 3; context only: that baseline does not exist here)."""
    import torch
    from paper_2010_15884_b200 import binding as B
    from paper_2010_15884_b200 import inputs
    model = {"SBM": (3.2, 80), "BSM": (0.8, 80), "FSM": (0.8, 80), "BFS": (0.8, 25), "FFS": (0.46, 14), "FBS": (3.2, 100)}
    paper_rel = {"SBM": (157, 147), "BSM": (67, 49), "FSM": (56, 39), "BFS": (56, 48), "FFS": (33, 30), "FBS": (159, 157)}
    enum = {"SBM": B.IS, "BSM": B.WS, "FSM": B.FSM, "BFS": B.BFS, "FFS": B.FFS, "FBS": B.OS}
    tiles, c_out = 10 * (1 << 20), 16
    stream = torch.cuda.current_stream().cuda_stream
    rows = []
    for qi, q in enumerate((2, 5)):
        n = c_out + q - 1
        x, ws = inputs.gen_1d_f32(tiles * n, [q], seed=60 + q)
        xd = torch.from_numpy(x).to(device)
        yd = torch.empty(tiles * c_out, dtype=torch.float32, device=device)
        w = ws[q]
        alg_bytes = 4.0 * tiles * (n + c_out)
        times = {}
        for name, d in enum.items():
            def launch(d=d):
                st = B.sysconv1d(xd.data_ptr(), n, n, w, q, yd.data_ptr(), c_out, tiles, B.F32, d, stream)
                if st != 0:
                    raise B.SysconvError(st, "sysconv1d")
            for _ in range(3):
                launch()
            ts = []
            for _ in range(reps):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); launch(); e1.record(); e1.synchronize()
                ts.append(e0.elapsed_time(e1))
            times[name] = statistics.median(ts)
        for name in enum:
            rows.append({"design": name, "filter": q, "signals": tiles, "outputs_per_signal": c_out,
                         "ms": round(times[name], 5),
                         "gpix_s": round(tiles * c_out / (times[name] * 1e-3) / 1e9, 2),
                         "hbm_frac": round(alg_bytes / (times[name] * 1e-3) / 1e9 / hbm_gbs, 4),
                         "relative_to_FBS": round(times["FBS"] / times[name], 3),
                         "model_outturn_q5": model[name][0], "model_utilisation_pct_q5": model[name][1],
                         "paper_pct_of_gen9_sampler": paper_rel[name][qi]})
        del xd, yd
        torch.cuda.empty_cache()
    return rows


def all_config_detail(device, hbm_gbs, peak_kind, sm_max, skip, reps):
    import torch
    rows = []
    flush = torch.zeros(64 << 20, dtype=torch.float32, device=device)
    for cfg_id in (1, 3, 4, 5):
        if cfg_id == skip:
            continue
        if cfg_id in (1, 3, 4):
            rows += l2_sized_rows(cfg_id, device, hbm_gbs, peak_kind, sm_max, reps, flush)
            continue
        cases, keep = build_cases(cfg_id, device)
        time_cases_individually(cases, 3, reps, None)
        rows += detail_rows(cases, hbm_gbs, peak_kind, sm_max)
        del cases, keep
        torch.cuda.empty_cache()
    cases, keep = build_strided_cases(device)
    time_cases_individually(cases, 3, reps, None)
    rows += detail_rows(cases, hbm_gbs, peak_kind, sm_max)
    del cases, keep
    torch.cuda.empty_cache()
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--no-detail", action="store_true", help="skip the per-kernel table of the other configurations")
    ap.add_argument("--detail-reps", type=int, default=10)
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--split-images", action="store_true",
                    help="cfg5 on several GPUs: deal the 16 images out to the ranks (strong scaling) instead of one copy each")
    ap.add_argument("--profile-n", type=int, default=0,
                    help="ncu captures only: shrink the 1-D signal to this many samples (keep it > L2)")
    ap.add_argument("--profile-batch", type=int, default=0,
                    help="ncu captures only: shrink configuration 5 to this many images")
    ap.add_argument("--profile-filter", type=int, default=0,
                    help="ncu captures only: keep one filter size of configuration 4 or 5 (only its buffers are allocated)")
    ap.add_argument("--paper-experiment", action="store_true",
                    help="only the table of the paper's own experiment (10.5 M signals of 16 outputs, six designs); "
                         "also the command the ncu capture of the tiny-signal kernel runs")
    args = ap.parse_args()
    if args.paper_experiment:
        import torch
        from paper_2010_15884_b200 import binding as B
        B.load_library()
        rows = six_designs_table(torch.device("cuda", 0), args.detail_reps, measured_peaks()[0])
        print(json.dumps({"six_designs_paper_experiment": rows}))
        return
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
