"""Read-only sampling of the SM clock, power draw and clock-event reasons through NVML, for the
benchmarks: a number is only as good as the clocks it was taken at."""
import statistics
import threading
import time


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML (read-only) every 20 ms."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks",
               0x10: "sync_boost", 0x100: "display_clock"}

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.stop_flag, self.ok = index, [], False, False
        self.sm_max = None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        while not self.stop_flag:
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                try:
                    watts = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                except Exception:
                    watts = None
                self.samples.append((time.perf_counter(), mhz, mask, watts))
            except Exception:
                pass
            time.sleep(0.02)

    def summary(self, t0, t1):
        """Median SM clock, reasons seen and peak power over host times [t0, t1]; when fewer than
        three samples fall inside (a region shorter than ~60 ms), over everything sampled."""
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        window = "timed region"
        if len(inside) < 3:
            inside, window = list(self.samples), "warm-up + timed region (timed region < 3 samples)"
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": [], "samples": 0,
                    "window": "NVML unavailable"}
        mask = 0
        for s in inside:
            mask |= s[2]
        reasons = sorted(name for bit, name in self.REASONS.items() if mask & bit)
        watts = [s[3] for s in inside if s[3] is not None]
        return {"sm_mhz": int(statistics.median(s[1] for s in inside)),
                "sm_max_mhz": self.sm_max, "reasons": reasons, "samples": len(inside),
                "power_w_max": max(watts) if watts else None, "window": window}

    def stop(self):
        self.stop_flag = True
        self.join(timeout=2)
