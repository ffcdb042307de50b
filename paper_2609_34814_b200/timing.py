"""Measurement helpers shared by bench.py and calibrate_guard: an interleaved A/B timer for
two variants of one kernel call, and a clock sampler that keeps only samples taken while a
named phase of the run was on the GPU.

Why interleaved: the two row orders of the same attention kernel differ by a few per cent,
which is less than what the SM clock moves between two back-to-back runs of several launches
(power capping).  Timing A A A ... then B B B ... therefore measures the clock drift, not the
orders.  Here the launches alternate (A B B A A B ...), every launch is bracketed by its own
events, nothing but the launches is enqueued between them, and the result is the median of the
per-pair ratios together with its range.  Next to the times each launch's length in SM cycles
(the kernel's own count, see waveal_bsattn_workspace_bytes) gives a ratio that does not depend
on the clock at all."""
from __future__ import annotations

import datetime
import os
import statistics
import subprocess
import tempfile
import time
from typing import Callable, Dict, List, Optional, Sequence, Tuple


def ab_interleaved(fn_a: Callable[[], None], fn_b: Callable[[], None], pairs: int, stream,
                   cycles_of: Optional[Callable[[], "object"]] = None) -> Dict[str, object]:
    """Times fn_a and fn_b `pairs` times each, alternating which goes first (A B | B A | ...).
    `cycles_of()` returns a 1-element device tensor holding the cycle count of the launch just
    enqueued (it is copied on the stream right after each launch).  Returns medians, the median
    and range of b/a per pair, and the same for cycles when available."""
    import torch
    ev = lambda: torch.cuda.Event(enable_timing=True)
    log = torch.zeros((2 * pairs,), dtype=torch.int32, device="cuda") if cycles_of else None
    marks: List[Tuple[int, object, object]] = []
    fn_a(); fn_b()                       # both variants warm
    torch.cuda.synchronize()
    slot = 0
    for i in range(pairs):
        for which in ((0, 1) if i % 2 == 0 else (1, 0)):
            e0, e1 = ev(), ev()
            e0.record(stream)
            (fn_a if which == 0 else fn_b)()
            e1.record(stream)
            if log is not None:
                log[slot:slot + 1].copy_(cycles_of(), non_blocking=True)
            marks.append((which, e0, e1))
            slot += 1
    torch.cuda.synchronize()
    t = [[], []]
    c = [[], []]
    cyc = log.tolist() if log is not None else None
    for s, (which, e0, e1) in enumerate(marks):
        t[which].append(e0.elapsed_time(e1))
        if cyc is not None:
            c[which].append(cyc[s])
    ratios = [b / a for a, b in zip(t[0], t[1])]
    out = {"a_ms": statistics.median(t[0]), "b_ms": statistics.median(t[1]),
           "b_over_a": statistics.median(ratios), "b_over_a_min": min(ratios), "b_over_a_max": max(ratios),
           "pairs": pairs}
    if cyc is not None and all(x > 0 for x in c[0] + c[1]):
        cr = [b / a for a, b in zip(c[0], c[1])]
        out.update(a_cycles=statistics.median(c[0]), b_cycles=statistics.median(c[1]),
                   b_over_a_cycles=statistics.median(cr), b_over_a_cycles_min=min(cr), b_over_a_cycles_max=max(cr))
    return out


class ClockSampler:
    """nvidia-smi clock / power / throttle-reason samples every 20 ms (reading only).  The caller
    brackets phases of the run with begin()/end() (host wall clock, taken after a device
    synchronisation); summary(name) reports the median SM clock of the samples whose timestamps
    fall inside that phase - samples from before, between or after the phases (an idle GPU
    reads its maximum clock) are not mixed in."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        self.phases: Dict[str, List[float]] = {}
        self.rows: Optional[List[Tuple[float, float, float, float, List[str]]]] = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "20", "-i", str(index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            pass

    def begin(self, name: str):
        self.phases[name] = [time.time(), float("inf")]

    def end(self, name: str):
        self.phases[name][1] = time.time()

    @staticmethod
    def _stamp(s: str) -> Optional[float]:
        for fmt in ("%Y/%m/%d %H:%M:%S.%f", "%Y-%m-%d %H:%M:%S.%f"):
            try:
                return datetime.datetime.strptime(s.strip(), fmt).timestamp()
            except ValueError:
                continue
        return None

    def stop(self):
        if self.p is None or self.rows is not None:
            return
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.rows = []
        for line in open(self.f.name):
            r = [x.strip() for x in line.strip().split(", ")]
            if len(r) < 8:
                continue
            ts = self._stamp(r[0])
            try:
                sm, mx, pw = float(r[1]), float(r[2]), float(r[3])
            except ValueError:
                continue
            if ts is None:
                continue
            self.rows.append((ts, sm, mx, pw, [n for n, v in zip(self.NAMES, r[4:8]) if v.lower().startswith("active")]))
        os.unlink(self.f.name)

    def summary(self, name: str) -> Dict[str, object]:
        """Clocks of one phase.  A sample counts when its timestamp lies inside the phase, 30 ms
        after its start at the earliest (nvidia-smi reports what it read a few ms before)."""
        self.stop()
        if self.p is None or not self.rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        t0, t1 = self.phases[name]
        inside = [r for r in self.rows if t0 + 0.03 <= r[0] <= t1]
        if not inside:                 # a phase shorter than the sampling period: nearest samples in the phase
            inside = [r for r in self.rows if t0 <= r[0] <= t1 + 0.02]
        reasons = sorted({n for r in inside for n in r[4]})
        sm = [r[1] for r in inside]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(r[2] for r in self.rows), "power_w": statistics.median([r[3] for r in inside]) if inside else None,
                "reasons": reasons, "samples": len(sm), "selection": "samples stamped inside the phase"}
