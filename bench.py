#!/usr/bin/env python
"""Benchmark of the BLAS level-1/2 family: achieved HBM GB/s per variant and their geomean.

A "step" is one pass over the whole variant cross-product (every routine x {f32, f64} x
trans/uplo/diag options x inc in {1, 2}), each variant sized to a 256 MiB working set.  Every
variant is timed with its own pair of CUDA events on the launching stream; every working set
is larger than L2 and L2 is additionally swept (256 MiB read-only pass) before each variant,
so no number is an L2-resident one.  Rank 0 prints ONE short JSON line (summary keys only) as
the last line of stdout; the per-variant rows go to a table file (--table).

    python bench.py --gpus 1 --steps 20 --warmup 3
    python bench.py --impl reference        # the CPU oracle on the host cores (bounded sample)
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

MIB = 1 << 20
ROW, COL, NOTR, TR, UP, LO, NONU, UNIT = 101, 102, 111, 112, 121, 122, 131, 132
FALLBACK_PEAK_GBS = 6650.0
NOMINAL_PEAK_GBS = 8000.0  # the vendor's spec-sheet HBM3e figure for this part (second denominator)


def ncu_dram_bytes_per_launch():
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of each kernel template at the
    bench sizes, as recorded beside the ncu summaries (one entry per kernel family; null once a
    kernel has changed and its counters have not been retaken)."""
    try:
        with open(os.path.join(ROOT, "profiles", "ncu_dram_bytes_per_launch.json")) as f:
            return json.load(f)["bytes_per_launch"]
    except Exception:
        return {}


# --------------------------------------------------------------------------- variant table
def variant_specs(scale: int = 1):
    """The cross-product.  `scale` divides the element counts (used by the CPU legs).
    Each spec: name, family (kernel template), routine, dtype, options, sizes, bytes."""
    specs = []
    for dt, s in (("f32", 4), ("f64", 8)):
        for inc in (1, 2):
            n2 = (128 * MIB // s) // inc // scale  # two-vector routines: 2 x 128 MiB spans
            n1 = (256 * MIB // s) // inc // scale  # one-vector routines: one 256 MiB span
            for r, per_elem, nvec in (("axpy", 3, 2), ("scal", 2, 1), ("copy", 2, 2), ("swap", 4, 2), ("rot", 4, 2),
                                      ("dot", 2, 2), ("asum", 1, 1), ("nrm2", 1, 1), ("iamax", 1, 1)):
                n = n2 if nvec == 2 else n1
                fam = "l1_map" if r in ("axpy", "scal", "copy", "swap", "rot") else "l1_reduce"
                specs.append(dict(name=f"{r}_{dt}_inc{inc}", family=fam, routine=r, dtype=dt, inc=inc, n=n,
                                  useful=per_elem * n * s, touched=per_elem * n * s * inc))
        ng = (8192 if s == 4 else 5760) // int(math.isqrt(scale))
        nt = (11520 if s == 4 else 8192) // int(math.isqrt(scale))
        for inc in (1, 2):
            vec = ng * s * inc
            for tr, tn in ((NOTR, "n"), (TR, "t")):
                specs.append(dict(name=f"gemv_{tn}_{dt}_inc{inc}", family="l2_tile", routine="gemv", dtype=dt, inc=inc,
                                  n=ng, trans=tr, useful=(ng * ng + 3 * ng) * s, touched=ng * ng * s + 3 * vec))
            specs.append(dict(name=f"ger_{dt}_inc{inc}", family="ger", routine="ger", dtype=dt, inc=inc, n=ng,
                              useful=(2 * ng * ng + 2 * ng) * s, touched=2 * ng * ng * s + 2 * vec))
            tri = nt * (nt + 1) // 2
            tvec = nt * s * inc
            for ul, un in ((UP, "u"), (LO, "l")):
                specs.append(dict(name=f"symv_{un}_{dt}_inc{inc}", family="l2_tile", routine="symv", dtype=dt, inc=inc,
                                  n=nt, uplo=ul, useful=(tri + 3 * nt) * s, touched=tri * s + 3 * tvec))
                for tr, tn in ((NOTR, "n"), (TR, "t")):
                    for dg, dn in ((NONU, "n"), (UNIT, "u")):
                        t = tri - (nt if dg == UNIT else 0)
                        for r, fam in (("trmv", "l2_tile"), ("trsv", "trsv")):
                            specs.append(dict(name=f"{r}_{un}{tn}{dn}_{dt}_inc{inc}", family=fam, routine=r, dtype=dt,
                                              inc=inc, n=nt, uplo=ul, trans=tr, diag=dg,
                                              useful=(t + 2 * nt) * s, touched=t * s + 2 * tvec))
    return specs


def geomean(vals):
    vals = [v for v in vals if v > 0]
    return math.exp(sum(math.log(v) for v in vals) / len(vals)) if vals else 0.0


def peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_PEAK_GBS, "fallback (no MEASURED_PEAKS.json)"


# --------------------------------------------------------------------------- clocks sampler
class ClockSampler:
    """nvidia-smi polled every 50 ms from before the warm-up; `stop` summarises the samples that
    fall inside the timed region (marked by `mark_start` / `mark_end`), and when the region is too
    short to hold three of them, the samples taken from the warm-up on (the same load)."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        self.lines = []  # (arrival time, text)
        self.t_load = self.t0 = self.t1 = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.monotonic(), line.strip()))

    def wait_first(self, timeout=10.0):
        """Blocks until the first sample has arrived (nvidia-smi takes a moment to start)."""
        t_end = time.monotonic() + timeout
        while self.proc is not None and not self.lines and time.monotonic() < t_end:
            time.sleep(0.02)

    def mark_load(self):
        self.t_load = time.monotonic()

    def mark_start(self):
        self.t0 = time.monotonic()

    def mark_end(self):
        self.t1 = time.monotonic()

    @staticmethod
    def summarise(lines, t_load, t0, t1):
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        parsed = []
        for t, line in lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                parsed.append((t, float(parts[0]), float(parts[1]),
                               [nm for nm, val in zip(names, parts[2:6]) if val.lower().startswith("active")]))
            except ValueError:
                continue
        inside = [r for r in parsed if t0 is not None and t1 is not None and t0 <= r[0] <= t1 + 0.05]
        window = "timed region"
        if len(inside) < 3:
            inside = [r for r in parsed if t_load is None or t1 is None or t_load <= r[0] <= t1 + 0.05]
            window = "warm-up and timed region (the timed region alone is shorter than three samples)"
        sm = sorted(r[1] for r in inside)
        reasons = sorted({nm for r in inside for nm in r[3]})
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": inside[-1][2] if inside else None,
                "reasons": reasons, "samples": len(sm), "window": window}

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        time.sleep(0.06)  # one more sample that still belongs to the region
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        return self.summarise(list(self.lines), self.t_load, self.t0, self.t1)


# --------------------------------------------------------------------------- GPU arm
class GpuWorkload:
    """Device buffers (seeded synthetic data) and one launcher per variant."""

    CALLS = 4  # back-to-back calls inside one event bracket (see `step`)

    def __init__(self, device, name_filter=None):
        import torch
        from paper_2411_07211_b200 import binding as b2
        from paper_2411_07211_b200 import synth
        self.torch, self.b2, self.synth = torch, b2, synth
        self.dev = device
        self.ctx = b2.Context(device)
        self.ctx.reset()
        self.specs = variant_specs()
        if name_filter:
            keys = name_filter.split(",")
            self.specs = [sp for sp in self.specs if any(k in sp["name"] for k in keys)]
        dtypes = {sp["dtype"] for sp in self.specs}
        self.flush = torch.zeros(64 * MIB, dtype=torch.float32, device=device)  # 256 MiB
        self.flush_res = torch.zeros(1, dtype=torch.float32, device=device)
        tdt = {"f32": torch.float32, "f64": torch.float64}
        self.buf = {}
        for dt, s in (("f32", 4), ("f64", 8)):
            if dt not in dtypes:
                continue
            t = tdt[dt]
            nel = 256 * MIB // s
            # level-1 vectors: X is a 256 MiB span, Y a 128 MiB span (+1 so inc=2 spans fit)
            self.buf[dt, "x"] = synth.vector_torch(0, 10, nel, t, device)
            self.buf[dt, "y"] = synth.vector_torch(0, 11, nel // 2, t, device)
            ng = 8192 if s == 4 else 5760
            nt = 11520 if s == 4 else 8192
            self.buf[dt, "ag"] = synth.matrix_torch(0, 12, ng, ng, ng, t, device)
            self.buf[dt, "ager"] = synth.matrix_torch(0, 13, ng, ng, ng, t, device)
            self.buf[dt, "at"] = synth.matrix_torch(0, 14, nt, nt, nt, t, device, tri_n=nt)
            nv = max(ng, nt)
            self.buf[dt, "vx0"] = synth.vector_torch(0, 15, 2 * nv, t, device)  # pristine copies
            self.buf[dt, "vy0"] = synth.vector_torch(0, 16, 2 * nv, t, device)
            self.buf[dt, "vy"] = self.buf[dt, "vy0"].clone()
            # trmv / trsv work in place: every call of a bracket gets its own copy of the vector
            self.buf[dt, "vx0r"] = self.buf[dt, "vx0"].repeat(self.CALLS)
            self.buf[dt, "vxr"] = self.buf[dt, "vx0r"].clone()
            self.buf[dt, "vx"] = self.buf[dt, "vxr"][: 2 * nv]  # (the first copy)
            self.buf[dt, "res"] = torch.zeros(4, dtype=t, device=device)
        self.ires = torch.zeros(1, dtype=torch.int64, device=device)
        torch.cuda.synchronize(device)
        self._prepared = {}

    def sweep_l2(self):
        """Streams a separate 256 MiB buffer through L2 with a read-only kernel, so nothing of the
        next variant's data is resident and L2 holds only CLEAN lines.  (A write sweep would leave
        up to an L2's worth of dirty lines whose write-back is then billed to the timed kernel.)"""
        self.b2.asum(self.ctx, self.flush.numel(), self.flush, 1, self.flush_res)

    def restore(self, sp):
        """Puts back vectors that a previous in-place call changed (tiny; uses the library's own
        copy kernel, outside the variant's event bracket)."""
        if sp["routine"] in ("trmv", "trsv"):
            B, dt = self.buf, sp["dtype"]
            self.b2.copy(self.ctx, B[dt, "vx0r"].numel(), B[dt, "vx0r"], 1, B[dt, "vxr"], 1)

    def launch(self, sp, j=0):
        """One call of the variant; j selects the copy of the in-place vector (trmv / trsv)."""
        b2, ctx, B = self.b2, self.ctx, self.buf
        dt, inc, n, r = sp["dtype"], sp["inc"], sp["n"], sp["routine"]
        x, y, res = B[dt, "x"], B[dt, "y"], B[dt, "res"]
        vlen = B[dt, "vx0"].numel()
        xj = B[dt, "vxr"][j * vlen:(j + 1) * vlen]
        if r == "axpy":
            b2.axpy(ctx, n, 1.5, x, inc, y, inc)
        elif r == "scal":
            b2.scal(ctx, n, -0.75, x, inc)
        elif r == "copy":
            b2.copy(ctx, n, x, inc, y, inc)
        elif r == "swap":
            b2.swap(ctx, n, x, inc, y, inc)
        elif r == "rot":
            b2.rot(ctx, n, x, inc, y, inc, 0.6, 0.8)
        elif r == "dot":
            b2.dot(ctx, n, x, inc, y, inc, res[0:1])
        elif r == "asum":
            b2.asum(ctx, n, x, inc, res[1:2])
        elif r == "nrm2":
            b2.nrm2(ctx, n, x, inc, res[2:3])
        elif r == "iamax":
            b2.iamax(ctx, n, x, inc, self.ires)
        elif r == "gemv":
            b2.gemv(ctx, ROW, sp["trans"], n, n, 1.25, B[dt, "ag"], n, B[dt, "vx"], inc, 0.5, B[dt, "vy"], inc)
        elif r == "ger":
            b2.ger(ctx, ROW, n, n, 1.25, B[dt, "vx0"], inc, B[dt, "vy0"], inc, B[dt, "ager"], n)
        elif r == "symv":
            b2.symv(ctx, ROW, sp["uplo"], n, 1.25, B[dt, "at"], n, B[dt, "vx0"], inc, 0.5, B[dt, "vy"], inc)
        elif r == "trmv":
            b2.trmv(ctx, ROW, sp["uplo"], sp["trans"], sp["diag"], n, B[dt, "at"], n, xj, inc)
        elif r == "trsv":
            b2.trsv(ctx, ROW, sp["uplo"], sp["trans"], sp["diag"], n, B[dt, "at"], n, xj, inc)
        else:
            raise KeyError(r)

    def bracket(self, k):
        """The CALLS back-to-back calls of variant k, marshalled once (a Python wrapper call costs
        about 10 us of host time; the replay keeps the host ahead of the device)."""
        if k not in self._prepared:
            sp = self.specs[k]
            self._prepared[k] = self.b2.prepare(lambda: [self.launch(sp, j) for j in range(self.CALLS)])
        return self._prepared[k]

    def step(self, events=None):
        """One pass over every variant: L2 swept, in-place vectors restored, then CALLS calls of the
        variant back to back inside one event bracket (`events`: list of (start, end) pairs); the
        variant's time is the bracket / CALLS.  A bracket around a single 40-us call bills it 2-3 us
        of event and launch latency that a stream of calls does not pay; the working sets are
        twice the L2 size, so a call finds nothing of its predecessor's data there."""
        for k, sp in enumerate(self.specs):
            run = self.bracket(k)
            self.sweep_l2()
            self.restore(sp)
            if events is not None:
                events[k][0].record()
            run()
            if events is not None:
                events[k][1].record()


def next_rows_leg(wl: GpuWorkload, steps: int, peak: float, only=None):
    """The routines beyond the 14 of the headline metric (built after them: syr, syr2, rotm, dsdot,
    sdsdot), timed the same way (L2 swept, one event bracket around CALLS calls, median) on 256 MiB working
    sets; they are NOT part of `value`.  syr / syr2 update the general matrix of the ger variants in
    place and rotm rotates the level-1 vectors: this leg runs after everything else."""
    torch, b2, ctx, B = wl.torch, wl.b2, wl.ctx, wl.buf
    rows = []

    def timed(name, call, touched):
        if only and not any(k in name for k in only.split(",")):
            return
        ts = []
        run = b2.prepare(lambda: [call() for _ in range(wl.CALLS)])
        for it in range(steps + 3):
            wl.sweep_l2()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            run()
            e1.record()
            torch.cuda.synchronize()
            if it >= 3:
                ts.append(e0.elapsed_time(e1) / wl.CALLS)
        ts.sort()
        ms = ts[len(ts) // 2]
        gbs = touched / (ms * 1e-3) / 1e9
        rows.append({"name": name, "ms": round(ms, 4), "gbs": round(gbs, 1), "frac": round(gbs / peak, 4)})

    dres = torch.zeros(1, dtype=torch.float64, device=wl.dev)
    sres = torch.zeros(1, dtype=torch.float32, device=wl.dev)
    for dt, s in (("f32", 4), ("f64", 8)):
        if (dt, "ager") not in B:
            continue
        n = 8192 if s == 4 else 5760
        tri = n * (n + 1) // 2
        for r in ("syr", "syr2"):
            for ul, un in ((UP, "u"), (LO, "l")):
                for inc in (1, 2):
                    if r == "syr":
                        call = lambda: b2.syr(ctx, ROW, ul, n, 1e-3, B[dt, "vx0"], inc, B[dt, "ager"], n)
                    else:
                        call = lambda: b2.syr2(ctx, ROW, ul, n, 1e-3, B[dt, "vx0"], inc, B[dt, "vy0"], inc,
                                               B[dt, "ager"], n)
                    nvec = 1 if r == "syr" else 2
                    timed(f"{r}_{un}_{dt}_inc{inc}", call, 2 * tri * s + nvec * n * s * inc)
        for inc in (1, 2):
            nv = (128 * MIB // s) // inc  # two vectors, 128 MiB span each
            x, y = B[dt, "x"], B[dt, "y"]
            # a plain rotation written as a full H (flag -1): magnitudes stay put over the repeats
            timed(f"rotm_{dt}_inc{inc}", lambda: b2.rotm(ctx, nv, x, inc, y, inc, [-1.0, 0.6, -0.8, 0.8, 0.6]),
                  4 * nv * s * inc)
            if dt == "f32":
                timed(f"dsdot_inc{inc}", lambda: b2.dsdot(ctx, nv, x, inc, y, inc, dres), 2 * nv * s * inc)
                timed(f"sdsdot_inc{inc}", lambda: b2.sdsdot(ctx, nv, 0.5, x, inc, y, inc, sres), 2 * nv * s * inc)
    # narrow matrices (the paper's second level-2 workload, Section 6.2.2: N = 40, static sizes up
    # to 88 (float) / 44 (double), M a power of 2 or 3), in both storage orders
    tdt = {"f32": torch.float32, "f64": torch.float64}
    for dt, s, shapes in (("f32", 4, ((1 << 20, 40), (1 << 20, 88), (3 ** 13, 40))),
                          ("f64", 8, ((1 << 20, 40), (1 << 20, 44), (3 ** 13, 24)))):
        if (dt, "ager") not in B or (only and "skinny" not in only):
            continue
        amax = max(m * n for m, n in shapes)
        a = wl.synth.vector_torch(0, 17, amax, tdt[dt], wl.dev)
        for m, n in shapes:
            xm, ym = B[dt, "x"], B[dt, "y"]  # length-m vectors
            xn, yn = B[dt, "vx0"], B[dt, "vy"]  # length-n vectors
            for order, on, lda in ((ROW, "rm", n), (COL, "cm", m)):
                tag = f"skinny_{m}x{n}_{on}_{dt}"
                timed(f"gemv_n_{tag}", lambda: b2.gemv(ctx, order, NOTR, m, n, 1.25, a, lda, xn, 1, 0.5, ym, 1),
                      (m * n + 2 * m + n) * s)
                timed(f"gemv_t_{tag}", lambda: b2.gemv(ctx, order, TR, m, n, 1.25, a, lda, xm, 1, 0.5, yn, 1),
                      (m * n + m + 2 * n) * s)
                timed(f"ger_{tag}", lambda: b2.ger(ctx, order, m, n, 1e-3, xm, 1, xn, 1, a, lda),
                      (2 * m * n + m + n) * s)
        del a
    return {"note": "rows built after the headline set; bytes = touched sectors (2 x stored triangle + vectors for "
                    "syr/syr2, spans for the level-1 rows); not part of `value`",
            "geomean_frac": geomean([r["frac"] for r in rows]), "variants": rows}


def configs_leg(device, peak: float, reps: int, only=None):
    """The size sweeps beside the headline set (not part of `value`): the 1 Mi-element float dot
    product; the level-1 routines at n = 2^16 .. 2^28; gemv / ger at 4096^2, 16384^2, 2^20 x 64 and
    64 x 2^20 with beta 0 and 0.5; symv / trmv / trsv at n = 1024, 8192, 32768.  Working sets below
    the L2 size are timed twice and labelled: "hot" (the same buffers every call: L2-resident, NOT
    an HBM figure) and "cold" (calls rotate through enough distinct buffers to exceed twice the L2
    size); larger ones once, behind a sweep of L2 like the headline set.  Small calls are timed in
    batches (one event pair around `reps` calls) because a single call is shorter than the timer's
    resolution."""
    import torch
    from paper_2411_07211_b200 import binding as b2
    from paper_2411_07211_b200 import synth
    ctx = b2.Context(device)
    ctx.reset()
    l2 = int(torch.cuda.get_device_properties(device).L2_cache_size)
    flush = torch.zeros(64 * MIB, dtype=torch.float32, device=device)
    fres = torch.zeros(1, dtype=torch.float32, device=device)
    tdt = {"f32": torch.float32, "f64": torch.float64}
    rows = []

    def batch_ms(call, nbuf, count):
        """Median over 5 batches of `count` calls (buffer k % nbuf), per call.  The calls are
        marshalled once (binding.prepare): a Python wrapper call costs more than a small kernel."""
        fast = [b2.prepare(lambda k=k: call(k)) for k in range(nbuf)]
        order = [fast[k % nbuf] for k in range(count)]
        ts = []
        for it in range(7):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for f in order:
                f()
            e1.record()
            torch.cuda.synchronize()
            if it >= 2:
                ts.append(e0.elapsed_time(e1) / count)
        ts.sort()
        return ts[len(ts) // 2]

    def swept_ms(call, calls=4):
        """L2 swept, then `calls` calls back to back in one event bracket (working sets above the
        L2 size: a call finds nothing of its predecessor's data there); per call."""
        ts = []
        run = b2.prepare(lambda: [call(0) for _ in range(calls)])
        for it in range(reps + 3):
            b2.asum(ctx, flush.numel(), flush, 1, fres)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            run()
            e1.record()
            torch.cuda.synchronize()
            if it >= 3:
                ts.append(e0.elapsed_time(e1) / calls)
        ts.sort()
        return ts[len(ts) // 2]

    def emit(name, ms, touched, label):
        gbs = touched / (ms * 1e-3) / 1e9
        rows.append({"name": name, "l2": label, "us": round(ms * 1e3, 2), "gbs": round(gbs, 1),
                     "frac": round(gbs / peak, 4), "frac_nominal": round(gbs / NOMINAL_PEAK_GBS, 4)})

    def measure(name, make_call, ws_bytes, touched, max_sets=None):
        """make_call(nbuf) -> call(k): the routine on buffer set k of nbuf."""
        if only and not any(k in name for k in only.split(",")):
            return
        if ws_bytes < l2:
            nbuf = max(2, -(-2 * l2 // ws_bytes) + 1)
            if max_sets:
                nbuf = min(nbuf, max_sets)
            call = make_call(nbuf)
            count = max(8, min(256, nbuf))
            emit(name, batch_ms(call, 1, count), touched, "hot (L2-resident)")
            label = "cold (rotating buffers > 2 x L2)" if nbuf * ws_bytes > 2 * l2 else "cold (rotating buffers, < 2 x L2)"
            emit(name, batch_ms(call, nbuf, max(count, nbuf)), touched, label)
        else:
            emit(name, swept_ms(make_call(1)), touched, "cold (working set > L2; L2 swept, then 4 calls back to back)")

    # ---- level 1: config 1 (sdot, 1 Mi floats) is the n = 2^20 row of the sweep
    for dt, s in (("f32", 4), ("f64", 8)):
        pool = synth.vector_torch(0, 20, 1 << 29, tdt[dt], device)  # rotating sets are slices of this (2 GiB / 4 GiB)
        for lg in (16, 20, 24, 28):
            n = 1 << lg
            for inc in (1, 2):
                span = n * inc
                if 2 * span > pool.numel():
                    continue  # (n = 2^28 with increment 2: two spans of 2^29 elements do not fit the pool)
                res = torch.zeros(4, dtype=tdt[dt], device=device)
                ires = torch.zeros(1, dtype=torch.int64, device=device)
                for r, per_elem, nvec in (("axpy", 3, 2), ("scal", 2, 1), ("copy", 2, 2), ("swap", 4, 2),
                                          ("rot", 4, 2), ("dot", 2, 2), ("asum", 1, 1), ("nrm2", 1, 1), ("iamax", 1, 1)):
                    ws = nvec * span * s

                    def make_call(nbuf, r=r, nvec=nvec, span=span, n=n, inc=inc):
                        nbuf = max(1, min(nbuf, pool.numel() // (nvec * span)))
                        def call(k):
                            x = pool[k * nvec * span:(k * nvec + 1) * span]
                            y = pool[(k * nvec + 1) * span:(k * nvec + 2) * span] if nvec == 2 else None
                            if r == "axpy":
                                b2.axpy(ctx, n, 1e-3, x, inc, y, inc)
                            elif r == "scal":
                                b2.scal(ctx, n, -1.0, x, inc)
                            elif r == "copy":
                                b2.copy(ctx, n, x, inc, y, inc)
                            elif r == "swap":
                                b2.swap(ctx, n, x, inc, y, inc)
                            elif r == "rot":
                                b2.rot(ctx, n, x, inc, y, inc, 0.6, 0.8)
                            elif r == "dot":
                                b2.dot(ctx, n, x, inc, y, inc, res[0:1])
                            elif r == "asum":
                                b2.asum(ctx, n, x, inc, res[1:2])
                            elif r == "nrm2":
                                b2.nrm2(ctx, n, x, inc, res[2:3])
                            else:
                                b2.iamax(ctx, n, x, inc, ires)
                        call.nbuf = nbuf
                        return call
                    measure(f"{r}_{dt}_n2^{lg}_inc{inc}", make_call, ws, per_elem * n * s * inc,
                            max_sets=pool.numel() // (nvec * span))
        del pool
        torch.cuda.empty_cache()

    # ---- gemv / ger (row-major, lda = n)
    for dt, s in (("f32", 4), ("f64", 8)):
        for m, n in ((4096, 4096), (16384, 16384), (1 << 20, 64), (64, 1 << 20)):
            ws = m * n * s
            nsets = 1 if ws >= l2 else -(-2 * l2 // ws) + 1
            a = synth.vector_torch(0, 21, nsets * m * n, tdt[dt], device).view(nsets, m * n)
            xv = synth.vector_torch(0, 22, max(m, n), tdt[dt], device)
            yv = synth.vector_torch(0, 23, max(m, n), tdt[dt], device)
            for tr, tn in ((NOTR, "n"), (TR, "t")):
                for beta in (0.0, 0.5):
                    mk = lambda nbuf, tr=tr, beta=beta: (lambda k: b2.gemv(ctx, ROW, tr, m, n, 1.25, a[k % nsets], n, xv, 1,
                                                                           beta, yv, 1))
                    ylen = m if tr == NOTR else n
                    measure(f"gemv_{tn}_{dt}_{m}x{n}_beta{beta}", mk, ws, (m * n + m + n + (ylen if beta else 0)) * s,
                            max_sets=nsets)
            mk = lambda nbuf: (lambda k: b2.ger(ctx, ROW, m, n, 1e-3, xv, 1, yv, 1, a[k % nsets], n))
            measure(f"ger_{dt}_{m}x{n}", mk, ws, (2 * m * n + m + n) * s, max_sets=nsets)
            del a
            torch.cuda.empty_cache()

    # ---- symv / trmv / trsv
    for dt, s in (("f32", 4), ("f64", 8)):
        for n in (1024, 8192, 32768):
            ws = n * n * s  # the buffer holds the full square; the routines touch one triangle of it
            tri = n * (n + 1) // 2
            nsets = 1 if ws // 2 >= l2 else -(-2 * l2 // (ws // 2)) + 1
            a = synth.matrix_torch(0, 24, n, n, n, tdt[dt], device, tri_n=n).unsqueeze(0)
            if nsets > 1:
                a = a.repeat(nsets, 1, 1)
            x0 = synth.vector_torch(0, 25, n, tdt[dt], device)
            xv, yv = x0.clone(), x0.clone()
            for ul, un in ((UP, "u"), (LO, "l")):
                mk = lambda nbuf, ul=ul: (lambda k: b2.symv(ctx, ROW, ul, n, 1.25, a[k % nsets], n, x0, 1, 0.5, yv, 1))
                measure(f"symv_{un}_{dt}_n{n}", mk, ws // 2, (tri + 3 * n) * s, max_sets=nsets)
                for tr, tn in ((NOTR, "n"), (TR, "t")):
                    for dg, dn in ((NONU, "n"), (UNIT, "u")):
                        t = tri - (n if dg == UNIT else 0)
                        # (both work in place: a copy launch inside the bracket restores their vector)
                        def mk_trmv(nbuf, ul=ul, tr=tr, dg=dg):
                            def call(k):
                                b2.copy(ctx, n, x0, 1, xv, 1)
                                b2.trmv(ctx, ROW, ul, tr, dg, n, a[k % nsets], n, xv, 1)
                            return call
                        measure(f"trmv_{un}{tn}{dn}_{dt}_n{n}", mk_trmv, ws // 2, (t + 2 * n) * s, max_sets=nsets)
                        def mk_trsv(nbuf, ul=ul, tr=tr, dg=dg):
                            def call(k):
                                b2.copy(ctx, n, x0, 1, xv, 1)
                                b2.trsv(ctx, ROW, ul, tr, dg, n, a[k % nsets], n, xv, 1)
                            return call
                        measure(f"trsv_{un}{tn}{dn}_{dt}_n{n}", mk_trsv, ws // 2, (t + 2 * n) * s, max_sets=nsets)
            assert ctx.device_status() == 0, "a trsv wait timed out"
            del a
            torch.cuda.empty_cache()
    return {"note": "size sweeps beside the headline set; `l2` says whether a figure is an HBM one; bytes = "
                    "algorithmic bytes of the call (touched sectors for increment 2); trmv / trsv rows include the "
                    "copy launch that restores their vector",
            "l2_bytes": l2, "rows": rows}


def e2e_leg(wl: GpuWorkload, steps: int):
    """Same metric through the C ABI with HOST data: per variant, pinned host -> device copies of
    its inputs, the call, and a device -> host read of its outputs, all inside the timed bracket."""
    torch, B = wl.torch, wl.buf
    pinned = {}

    def pin(key):
        """One pinned host mirror per device buffer (inputs are read from it, outputs land in it)."""
        if key not in pinned:
            t = dev(key)
            pinned[key] = torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t)
        return pinned[key]

    def io(sp):
        dt, r = sp["dtype"], sp["routine"]
        v = ("x", "y") if sp["family"] in ("l1_map", "l1_reduce") else ("vx", "vy")
        ins, outs = [], []
        if r in ("axpy", "swap", "rot", "dot"):
            ins = [v[0], v[1]]
        elif r in ("scal", "copy", "asum", "nrm2", "iamax"):
            ins = [v[0]]
        elif r == "gemv":
            ins = ["ag", "vx", "vy"]
        elif r == "ger":
            ins = ["ager", "vx0", "vy0"]
        elif r == "symv":
            ins = ["at", "vx0", "vy"]
        else:
            ins = ["at", "vx"]
        outs = {"axpy": ["y"], "scal": ["x"], "copy": ["y"], "swap": ["x", "y"], "rot": ["x", "y"], "dot": ["res"],
                "asum": ["res"], "nrm2": ["res"], "iamax": ["ires"], "gemv": ["vy"], "ger": ["ager"],
                "symv": ["vy"], "trmv": ["vx"], "trsv": ["vx"]}[r]
        return [(dt, k) for k in ins], [(dt, k) for k in outs]

    def sl(sp, key, t):
        """The part of a buffer this variant really uses (so copies are not oversized)."""
        if key[1] in ("x", "y"):
            return t[: (sp["n"] - 1) * sp["inc"] + 1]
        if key[1] in ("vx", "vy", "vx0", "vy0"):
            return t[: (sp["n"] - 1) * sp["inc"] + 1]
        return t

    def dev(key):
        return wl.ires if key[1] == "ires" else B[key]

    per_variant = [[] for _ in wl.specs]
    h2d = d2h = 0
    for it in range(steps + 1):  # first pass is warm-up (also pins the host copies)
        h2d = d2h = 0
        for k, sp in enumerate(wl.specs):
            ins, outs = io(sp)
            hin = [(key, sl(sp, key, pin(key))) for key in ins]
            hout = [(key, sl(sp, key, pin(key))) for key in outs]
            wl.sweep_l2()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for key, h in hin:
                sl(sp, key, dev(key)).copy_(h, non_blocking=True)
                h2d += h.numel() * h.element_size()
            wl.launch(sp)
            for key, h in hout:
                h.copy_(sl(sp, key, dev(key)), non_blocking=True)
                d2h += h.numel() * h.element_size()
            e1.record()
            e1.synchronize()
            if it > 0:
                per_variant[k].append(e0.elapsed_time(e1))
    med = [sorted(v)[len(v) // 2] for v in per_variant]
    gbs = [sp["touched"] / (t * 1e-3) / 1e9 for sp, t in zip(wl.specs, med)]
    return {"value": geomean(gbs), "unit": "GB/s (geomean over variants, host buffers in and out)",
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": steps}


# --------------------------------------------------------------------------- CPU oracle legs
def oracle_pass(scale: int, seed: int = 0):
    """Times the CPU oracle, as it stands, over every variant at 1/scale of the bench's element
    counts.  Returns per-variant GB/s (touched bytes of the SAMPLE / oracle seconds)."""
    import numpy as np
    from oracle import blas_oracle as orc
    from paper_2411_07211_b200 import synth
    out = []
    cache = {}

    def vec(dt, stream, n):
        key = (dt, stream, n)
        if key not in cache:
            cache[key] = synth.vector_np(seed, stream, n, np.float32 if dt == "f32" else np.float64)
        return cache[key]

    for sp in variant_specs(scale):
        dt, inc, n, r = sp["dtype"], sp["inc"], sp["n"], sp["routine"]
        npdt = np.float32 if dt == "f32" else np.float64
        if sp["family"] in ("l1_map", "l1_reduce"):
            x = vec(dt, 10, (n - 1) * inc + 1).copy()
            y = vec(dt, 11, (n - 1) * inc + 1).copy()
            fn = {"axpy": lambda: orc.axpy(n, npdt(1.5), x, inc, y, inc), "scal": lambda: orc.scal(n, npdt(-0.75), x, inc),
                  "copy": lambda: orc.copy(n, x, inc, y, inc), "swap": lambda: orc.swap(n, x, inc, y, inc),
                  "rot": lambda: orc.rot(n, x, inc, y, inc, npdt(0.6), npdt(0.8)),
                  "dot": lambda: orc.dot(n, x, inc, y, inc), "asum": lambda: orc.asum(n, x, inc),
                  "nrm2": lambda: orc.nrm2(n, x, inc), "iamax": lambda: orc.iamax(n, x, inc)}[r]
        else:
            key = (dt, "mat", n, r in ("symv", "trmv", "trsv"))
            if key not in cache:
                cache[key] = synth.matrix_np(seed, 14, n, n, n, npdt, tri_n=n if key[3] else None).ravel()
            a = cache[key]
            x = vec(dt, 15, (n - 1) * inc + 1).copy()
            y = vec(dt, 16, (n - 1) * inc + 1).copy()
            if r == "gemv":
                fn = lambda: orc.gemv(ROW, sp["trans"], n, n, npdt(1.25), a, n, x, inc, npdt(0.5), y, inc)
            elif r == "ger":
                a = a.copy()
                fn = lambda: orc.ger(ROW, n, n, npdt(1.25), x, inc, y, inc, a, n, want_absterms=False)
            elif r == "symv":
                fn = lambda: orc.symv(ROW, sp["uplo"], n, npdt(1.25), a, n, x, inc, npdt(0.5), y, inc)
            elif r == "trmv":
                fn = lambda: orc.trmv(ROW, sp["uplo"], sp["trans"], sp["diag"], n, a, n, x, inc)
            else:
                fn = lambda: orc.trsv(ROW, sp["uplo"], sp["trans"], sp["diag"], n, a, n, x, inc)
        t0 = time.perf_counter()
        fn()
        dt_s = time.perf_counter() - t0
        out.append((sp["name"], sp["touched"] / dt_s / 1e9, dt_s))
    return out


def reference_arm(args):
    """`--impl reference`: the oracle, as it stands, on the host cores; each step is one pass over
    every variant at 1/16 of the bench's element counts (bounded so the run ends in minutes)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    scale = 16
    from oracle import blas_oracle as orc
    orc.build()
    for _ in range(args.warmup):
        oracle_pass(scale)
    t0 = time.perf_counter()
    runs = [oracle_pass(scale) for _ in range(args.steps)]
    wall = time.perf_counter() - t0
    per = [geomean([run[k][1] for run in runs]) for k in range(len(runs[0]))]
    value = geomean(per)
    sample = f"every variant at 1/{scale} of the bench element counts (16 MiB working sets), 1 thread"
    print(json.dumps({
        "impl": "reference", "metric": "achieved HBM GB/s per BLAS-1/2 variant, geomean over variants",
        "value": value, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": wall / max(1, args.steps) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32+f64", "data": "synthetic",
        "config": {"workload": "config 5: every routine x {f32,f64} x trans/uplo/diag x inc {1,2}, 256 MiB working "
                               "set per variant, row-major", "variants": len(per), "sample": sample,
                   "bytes": "touched sectors (span bytes)", "parallelism": "one host core"},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (replicas run independently; a
    variant's time for the job is the slowest replica's).  Identity without a process group."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.cpu().tolist()


def aggregate(specs, med_ms, world, peak):
    """Per-variant rows and the whole-job value (N replicas: N x the geomean rate)."""
    rows = []
    for sp, t in zip(specs, med_ms):
        gbs = sp["touched"] / (t * 1e-3) / 1e9
        rows.append({"name": sp["name"], "family": sp["family"], "ms": t, "gbs": gbs,
                     "gbs_useful": sp["useful"] / (t * 1e-3) / 1e9, "frac": gbs / peak,
                     "frac_nominal": gbs / NOMINAL_PEAK_GBS})
    return rows, world * geomean([r["gbs"] for r in rows])


# --------------------------------------------------------------------------- main
def _short(v, digits=4):
    """Floats to `digits` significant digits, recursively (keeps the printed line short)."""
    if isinstance(v, float):
        return float(f"{v:.{digits}g}")
    if isinstance(v, dict):
        return {k: _short(x, digits) for k, x in v.items()}
    if isinstance(v, (list, tuple)):
        return [_short(x, digits) for x in v]
    return v


def final_line(out: dict) -> str:
    """The ONE line printed last: the summary keys only, floats shortened.  Per-variant rows never
    go here (they are written to the table file): a reader that keeps only the end of stdout must
    still see the whole line."""
    keep = {k: v for k, v in out.items() if k not in ("variants", "next_rows")}
    line = json.dumps(_short(keep, 5), separators=(",", ":"))
    assert len(line) < 4096, f"final line too long ({len(line)} bytes)"
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--filter", default=None, help="only variants whose name contains one of these comma-separated "
                                                   "strings (tuning runs; the headline run uses all)")
    ap.add_argument("--next-only", action="store_true", help="time only the rows built after the headline set "
                                                             "(--filter then selects among those)")
    ap.add_argument("--knob", action="append", default=[], metavar="ID=VALUE",
                    help="set a tuning knob of the library before timing (tuning runs; the headline run sets none)")
    ap.add_argument("--configs", action="store_true", help="time the size sweeps beside the headline set (rows go "
                                                           "to the table file; --filter selects among them)")
    ap.add_argument("--table", default=None, help="where the per-variant table (JSON) is written "
                                                  "(default: bench_table.json in the run's output folder)")
    args = ap.parse_args()
    if args.impl == "reference":
        reference_arm(args)
        return

    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    from paper_2411_07211_b200 import binding as b2
    for kv in args.knob:
        kid, val = kv.split("=")
        b2.set_tuning(int(kid), int(val))
    if args.configs:
        if world > 1:
            raise SystemExit("--configs is a single-GPU run")
        peak, peak_src = peak_gbs()
        table = configs_leg(device, peak, max(5, min(args.steps, 10)), args.filter)
        table["peak_gbs"], table["peak_source"] = peak, peak_src
        path = args.table or os.path.join(ROOT, "gpurun_out", "bench_configs_table.json")
        os.makedirs(os.path.dirname(os.path.abspath(path)), exist_ok=True)
        with open(path, "w") as f:
            json.dump(table, f, indent=1)
        hbm = [r["frac"] for r in table["rows"] if r["l2"].startswith("cold")]
        print(json.dumps({"configs_rows": len(table["rows"]), "geomean_frac_cold_rows": round(geomean(hbm), 4),
                          "table": os.path.relpath(path, ROOT)}))
        return
    if args.next_only:
        if world > 1:
            raise SystemExit("--next-only is a single-GPU profiling aid")
        wl = GpuWorkload(device, None)
        print(json.dumps({"next_rows": next_rows_leg(wl, args.steps, peak_gbs()[0], args.filter)}))
        return
    wl = GpuWorkload(device, args.filter)
    nv = len(wl.specs)
    warm = max(3, args.warmup)
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.wait_first()
        sampler.mark_load()
    for _ in range(warm):
        wl.step()
    torch.cuda.synchronize(device)
    events = [[[torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)] for _ in range(nv)]
              for _ in range(args.steps)]
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize(device)
    if sampler:
        sampler.mark_start()
    launches0 = b2.launch_count()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    for s in range(args.steps):
        wl.step(events[s])
    t_end.record()
    torch.cuda.synchronize(device)
    if sampler:
        sampler.mark_end()
    if world > 1:
        dist.barrier()
    launches = b2.launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    total_ms = t_start.elapsed_time(t_end)
    assert wl.ctx.device_status() == 0, "a trsv wait timed out during the bench"

    med = []
    for k in range(nv):
        ts = sorted(events[s][k][0].elapsed_time(events[s][k][1]) / wl.CALLS for s in range(args.steps))
        med.append(ts[len(ts) // 2])
    times = max_over_ranks(med + [total_ms], device)
    med, total_ms = times[:-1], times[-1]
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_src = peak_gbs()
    rows, value = aggregate(wl.specs, med, world, peak)
    fam = {}
    for sp, r in zip(wl.specs, rows):
        f = fam.setdefault(sp["family"], {"ms": 0.0, "bytes": 0, "launches": 0})
        f["ms"] += r["ms"]
        f["bytes"] += sp["touched"]
        f["launches"] += 1
    by_kernel = {k: {"achieved": v["bytes"] / (v["ms"] * 1e-3) / 1e9, "frac": v["bytes"] / (v["ms"] * 1e-3) / 1e9 / peak,
                     "share_of_time": v["ms"] / sum(x["ms"] for x in fam.values()), "variants": v["launches"]}
                 for k, v in fam.items()}
    dom = max(fam, key=lambda k: fam[k]["ms"])
    traffic = ncu_dram_bytes_per_launch().get(dom)
    roofline = {"bound": "hbm", "kernel": dom, "achieved": by_kernel[dom]["achieved"], "peak": peak, "unit": "GB/s",
                "frac": by_kernel[dom]["frac"], "traffic": traffic, "peak_source": peak_src,
                "by_kernel": by_kernel}
    no_trsv = [r for r in rows if r["family"] != "trsv"]
    out = {
        "metric": "achieved HBM GB/s per BLAS-1/2 variant, geomean over variants",
        "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": warm,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32+f64", "data": "synthetic",
        "config": {"workload": "config 5: every routine x {f32,f64} x trans/uplo/diag x inc {1,2}, 256 MiB working "
                               "set per variant, row-major", "variants": nv,
                   "l2": "inputs larger than L2 (256 MiB working sets); in addition a separate 256 MiB buffer is streamed "
                         "through L2 by a read-only kernel before every variant (clean lines only)", "bytes": "touched sectors (span bytes)",
                   "calls_per_event_bracket": wl.CALLS,
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "geomean_frac_of_peak": value / world / peak,
        "geomean_frac_of_nominal_8tbs": value / world / NOMINAL_PEAK_GBS,
        "geomean_frac_of_peak_without_trsv": geomean([r["frac"] for r in no_trsv]),
        "geomean_frac_by_family": {k: geomean([r["frac"] for r in rows if r["family"] == k]) for k in fam},
        "min_variant": min(rows, key=lambda r: r["frac"])["name"],
        "gpu_launches": launches, "clocks": clocks, "roofline": roofline,
    }
    if not args.no_e2e and world == 1:
        out["e2e"] = e2e_leg(wl, min(args.steps, 2))
    else:
        out["e2e"] = None
    if not args.no_cpu and world == 1:
        scale = 16
        t0 = time.perf_counter()
        res = oracle_pass(scale)
        t_one = time.perf_counter() - t0
        out["cpu_baseline"] = {"value": geomean([r[1] for r in res]), "unit": "GB/s", "cores": 1, "kind": "oracle",
                               "sample": f"every variant once at 1/{scale} of the bench element counts "
                                         f"({t_one:.1f} s of CPU work)"}
        # second figure, context only: the same loops with an OpenMP parallel-for over the outer
        # index on every host core (trsv and iamax stay serial)
        try:
            from oracle import blas_oracle as orc
            orc.use_all_cores(True)
            oracle_pass(scale)  # starts the thread pool, touches the pages
            res_all = oracle_pass(scale)
            out["cpu_baseline"]["all_cores"] = {"value": geomean([r[1] for r in res_all]), "unit": "GB/s",
                                                "cores": os.cpu_count(), "kind": "oracle loops + OpenMP parallel-for"}
        except Exception as e:  # no OpenMP on the box: the one-core figure stands alone
            out["cpu_baseline"]["all_cores"] = {"unavailable": str(e)[:80]}
        finally:
            orc.use_all_cores(False)
    else:
        out["cpu_baseline"] = None
    table = dict(out)
    table["variants"] = [{k: (round(v, 4) if isinstance(v, float) else v) for k, v in r.items()} for r in rows]
    if world == 1 and not args.filter:
        table["next_rows"] = next_rows_leg(wl, min(args.steps, 10), peak)
        out["next_rows_geomean_frac"] = table["next_rows"]["geomean_frac"]
    path = args.table or os.path.join(ROOT, "gpurun_out", "bench_table.json")
    os.makedirs(os.path.dirname(os.path.abspath(path)), exist_ok=True)
    with open(path, "w") as f:
        json.dump(table, f, indent=1)
    print(final_line(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
