"""Read-only sampling of GPU clocks and throttle reasons while a measurement runs.

Only queries (`nvidia-smi --query-gpu`); nothing on the GPU is set or reset.  Every harness that
prints a timing samples the clocks over its timed region and stores the summary next to the number:
median SM clock under load, the maximum, and which slowdown reasons were seen active."""
from __future__ import annotations

import statistics
import subprocess
import threading
import time

FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
          "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
REASONS = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
REJECT = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}     # a number taken under these is re-measured


class ClockSampler:
    def __init__(self, index: int = 0, period_ms: int = 100):
        self.index, self.period_ms, self.proc, self.lines, self.marks = index, period_ms, None, [], []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", str(self.period_ms)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.monotonic(), line.strip()))

    def mark(self):
        """Start of a row group: summary(since=mark) covers the samples taken after it."""
        self.marks.append(time.monotonic())
        return self.marks[-1]

    def summary(self, since: float | None = None) -> dict:
        sm, mx, pw, reasons = [], [], [], set()
        for (t, l) in list(self.lines):
            if since is not None and t < since:
                continue
            parts = [p.strip() for p in l.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            try:
                pw.append(float(parts[2]))
            except ValueError:
                pass
            for name, val in zip(REASONS, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "power_w_max": max(pw) if pw else None,
                "reasons": sorted(reasons), "samples": len(sm), "rejected": bool(reasons & REJECT)}

    def stop(self) -> dict:
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0, "rejected": False}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        return self.summary()
