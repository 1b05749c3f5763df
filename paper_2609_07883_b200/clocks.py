"""SM clock, power and throttle reasons during a timed region, sampled with ``nvidia-smi`` (reading only: no setting of the
GPU is touched).  One sampler runs for a whole program; every timed window then picks its own samples by time stamp."""
from __future__ import annotations

import datetime
import os
import subprocess
import tempfile

import numpy as np


class ClockSampler:
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")
    REASONS = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")

    def __init__(self, gpu_index: int, period_ms: int = 50):
        self.gpu_index, self.period_ms = gpu_index, period_ms
        self.proc = self.path = None
        self.rows = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", str(self.period_ms)],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            self.rows = []
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        try:
            for line in open(self.path).read().splitlines():
                f = [x.strip() for x in line.split(",")]
                if len(f) < 8:
                    continue
                try:
                    ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    rows.append((ts, float(f[1]), float(f[2]), float(f[3]),
                                 [name for name, val in zip(self.REASONS, f[4:8]) if val.lower().startswith("active")]))
                except ValueError:
                    continue
            os.unlink(self.path)
        except Exception:
            pass
        self.rows = rows

    def window(self, t0: float, t1: float) -> dict:
        """Median SM clock, maximum power and the throttle reasons seen between two host time stamps."""
        if not self.rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"], "samples": 0}
        rows = [r for r in self.rows if t0 <= r[0] <= t1]
        if not rows:   # a window shorter than the sampling period: the nearest sample
            mid = 0.5 * (t0 + t1)
            rows = [min(self.rows, key=lambda r: abs(r[0] - mid))]
        reasons = sorted({x for r in rows for x in r[4]})
        return {"sm_mhz": float(np.median([r[1] for r in rows])), "sm_max_mhz": float(max(r[2] for r in rows)),
                "power_w_max": float(max(r[3] for r in rows)), "reasons": reasons, "samples": len(rows)}


