"""SM clock, power and throttle-reason samples taken with nvidia-smi while a measurement runs.

Read-only: this only queries the GPU (`nvidia-smi --query-gpu ... -lms`), it never sets a clock,
a power limit or any other device state.
"""
from __future__ import annotations

import datetime
import os
import statistics
import subprocess
import tempfile
import time
from pathlib import Path

FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
          "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
          "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
REASONS = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
REJECTING = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown")


def _die_with_parent():
    """Runs in the child before exec: ask the kernel to end it when the parent goes away, so that
    an aborted measurement never leaves an nvidia-smi loop behind."""
    try:
        import ctypes
        import signal
        ctypes.CDLL("libc.so.6", use_errno=True).prctl(1, signal.SIGTERM)   # PR_SET_PDEATHSIG
    except Exception:
        pass


def parse_rows(rows):
    """[(unix time, sm MHz, max sm MHz, watts, {reason: bool})] from nvidia-smi CSV rows."""
    out = []
    for r in rows:
        c = [x.strip() for x in r.split(",")]
        if len(c) < 9:
            continue
        try:
            ts = datetime.datetime.strptime(c[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
            rec = (ts, float(c[1]), float(c[2]), float(c[3]),
                   {name: c[5 + k].lower().startswith("active") for k, name in enumerate(REASONS)})
        except ValueError:
            continue
        out.append(rec)
    return out


def summarise(samples, t_begin: float, t_end: float, slack: float = 0.02) -> dict:
    """Median SM clock, power and the reasons seen between two host times.  Falls back to all
    samples (and says so) when fewer than two fall inside the window."""
    inside = [s for s in samples if t_begin - slack <= s[0] <= t_end + slack]
    use = inside if len(inside) >= 2 else samples
    if not use:
        return {"sm_mhz": None, "sm_max_mhz": None, "power_w": None, "reasons": ["no samples"],
                "samples": 0, "during_timed_region": False}
    reasons = sorted({name for s in use for name, on in s[4].items() if on})
    return {"sm_mhz": statistics.median(s[1] for s in use), "sm_max_mhz": use[0][2],
            "sm_mhz_min": min(s[1] for s in use), "power_w": statistics.median(s[3] for s in use),
            "reasons": reasons, "samples": len(use), "during_timed_region": len(inside) >= 2,
            "rejected": any(r in REJECTING for r in reasons)}


class ClockSampler:
    """Runs nvidia-smi in the background at a fixed period; window() summarises a time span."""

    def __init__(self, device_index: int, period_ms: int = 50):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", str(period_ms), "-i", str(device_index)],
                stdout=self.file, stderr=subprocess.DEVNULL, preexec_fn=_die_with_parent)
        except OSError:
            self.proc = None

    def wait_first_sample(self, timeout: float = 5.0) -> None:
        t0 = time.time()
        while self.proc and time.time() - t0 < timeout:
            if os.path.getsize(self.file.name) > 0:
                return
            time.sleep(0.02)

    def samples(self):
        return parse_rows(Path(self.file.name).read_text().splitlines())

    def window(self, t_begin: float, t_end: float) -> dict:
        return summarise(self.samples(), t_begin, t_end)

    def stop(self) -> None:
        if self.proc:
            self.proc.terminate()        # the exact process started above
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.proc = None
        try:
            os.unlink(self.file.name)
        except OSError:
            pass
