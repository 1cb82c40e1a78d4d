#!/usr/bin/env python
"""Benchmark of the fused norm-test + AdamW step (one JSON line on stdout).

Workload: the GPT-2-small-shaped parameter vector (124,439,808 elements), K=8 bf16 worker
gradient buffers, fp32 master params and AdamW moments, eta=0.1, b_cur=512, one call of
abs_normtest_adamw per step (gbar kept in registers).  Synthetic seeded inputs.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N>1 (under torchrun, one rank per GPU): every rank runs the same step on its own replica
of the workload -- the path needs no data-path collective -- and the reported value is
the bytes all ranks processed divided by the slowest rank's time (weak scaling).
--impl reference times the fp64 CPU oracle on the host cores instead (rank 0 only).
"""
import argparse
import hashlib
import json
import os
import re
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "norm-test+AdamW step: HBM GB/s (% of peak) and ms/step at 124M params, K=8"
K_WORKERS = 8
ETA, B_CUR, STEP0 = 0.1, 512, 100
HP = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)
GRAD_BYTES = 2           # bf16
BYTES_PER_ELEM = K_WORKERS * GRAD_BYTES + 24   # K*s read + p,m,v read and written
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0


def workload_config(d):
    return {"workload": "config2: GPT-2-small-shaped flat vector, fused abs_normtest_adamw",
            "d": d, "K": K_WORKERS, "grad_dtype": "bf16", "state_dtype": "fp32",
            "eta": ETA, "b_cur": B_CUR, "gbar_out": "none (registers only)",
            "bytes_per_step": BYTES_PER_ELEM * d,
            "l2": "inputs (5.0 GB per step) are larger than the 126 MB L2; no flush needed"}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


def kernel_source_hash():
    """Hash of the kernel sources as the compiler sees them: comments, blank lines and
    indentation do not count (no string literal in those files contains a comment marker)."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2412_21124_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        with open(os.path.join(csrc, name), "r", encoding="utf-8") as f:
            text = f.read()
        text = re.sub(r"/\*.*?\*/", " ", text, flags=re.S)
        h.update(name.encode())
        for line in text.splitlines():
            code = " ".join(line.split("//", 1)[0].split())
            if code:
                h.update(code.encode())
                h.update(b"\n")
    return h.hexdigest()[:16]


def recorded_traffic(d):
    """DRAM bytes per launch of the fused kernel from the committed ncu summary, or None
    when the kernel sources changed after the counters were taken."""
    path = os.path.join(ROOT, "profiles", "fused_k8_bf16_dram_traffic.json")
    try:
        with open(path) as f:
            rec = json.load(f)
        if rec.get("kernel_source_hash") != kernel_source_hash():
            return None
        return float(rec["dram_bytes_per_element"]) * d
    except Exception:
        return None


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


# ------------------------------------------------------------------------- CPU oracle
def oracle_sample(d_sample, seed=5):
    """Host copies of a prefix of the workload (same generator, CPU) for the oracle."""
    import numpy as np
    import torch
    from paper_2412_21124_b200 import synth
    sizes = synth.gpt2_small_tensor_sizes()
    sig_all = synth.per_tensor_sigma(sizes, seed + 1)
    # the prefix covers the first tensors of the declaration order (token embedding first)
    pre, sig, left = [], [], d_sample
    for s, sg in zip(sizes, sig_all):
        if left <= 0:
            break
        pre.append(min(s, left))
        sig.append(sg)
        left -= pre[-1]
    grads = synth.worker_grads(pre, K_WORKERS, torch.bfloat16, seed, "cpu", sigma=sig)
    p, m, v = synth.adam_state(d_sample, seed + 2, "cpu", zero_moments=False)
    host = [g.view(torch.int16).numpy().view(np.uint16) for g in grads]
    return host, p.numpy(), m.numpy(), v.numpy()


def oracle_step(orc, host, p, m, v):
    import numpy as np
    f = lambda x: float(np.float32(x))
    r = orc.norm_test(host, ETA, B_CUR)
    orc.adamw(p, m, v, r["gbar"], f(HP["lr"]), f(HP["beta1"]), f(HP["beta2"]), f(HP["eps"]),
              f(HP["weight_decay"]), STEP0)
    return r


def time_oracle(d_sample, reps):
    from oracle import abs_oracle as orc
    host, p, m, v = oracle_sample(d_sample)
    times = []
    for _ in range(reps):
        t0 = time.perf_counter()
        oracle_step(orc, host, p, m, v)
        times.append(time.perf_counter() - t0)
    return times, orc.threads()


def run_reference(args, d):
    """The oracle as it stands, on the host cores.  Each step is the oracle on a prefix of the
    workload sized (from a short calibration pass) so that all steps end within ~2 minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    calib, cores = time_oracle(1 << 20, 2)
    rate = (1 << 20) / min(calib)                       # elements per second
    budget = 120.0 / (args.steps + args.warmup)         # seconds per step
    d_sample = int(max(1 << 16, min(d, 1 << 24, rate * budget)))
    times, cores = time_oracle(d_sample, args.warmup + args.steps)
    timed = times[args.warmup:]
    sec = sum(timed) / len(timed)
    gbs = BYTES_PER_ELEM * d_sample / sec / 1e9
    sample = ("each step = the oracle (norm test + AdamW, fp64) on the first %d of %d elements; "
              "GB/s counts the same %d B/element; ms_per_step is scaled to the full vector"
              % (d_sample, d, BYTES_PER_ELEM))
    line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": sec * 1e3 * (d / d_sample), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(d),
            "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": cores, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------ ours
def run_ours(args, d):
    import torch

    import paper_2412_21124_b200 as absnt
    from paper_2412_21124_b200 import dist as adist
    from paper_2412_21124_b200 import synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    rank, world, local_rank = adist.init_from_env()
    if world != args.gpus:
        raise SystemExit("--gpus %d but WORLD_SIZE=%d: launch with torchrun" % (args.gpus, world))
    torch.cuda.set_device(local_rank)
    dev = "cuda:%d" % local_rank
    absnt.binding.lib()

    sizes = synth.gpt2_small_tensor_sizes()
    sig = synth.per_tensor_sigma(sizes, 6)
    grads = synth.worker_grads(sizes, K_WORKERS, torch.bfloat16, 5 + 100 * rank, dev, sigma=sig)
    p, m, v = synth.adam_state(d, 7 + 100 * rank, dev, zero_moments=False)
    stats = absnt.alloc_stats(d, 1, dev)
    b_next = torch.zeros(1, dtype=torch.int64, device=dev)
    stream = torch.cuda.current_stream()
    launches_per_step = 2  # streaming kernel + finalize kernel

    def step(i):
        absnt.abs_normtest_adamw(grads, ETA, B_CUR, stats, None, b_next, p, m, v, HP, STEP0 + i)

    sampler = ClockSampler(local_rank)
    sampler.start()
    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    adist.barrier(dev)
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    ev0.record(stream)
    for i in range(args.steps):
        step(args.warmup + i)
    ev1.record(stream)
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    adist.barrier(dev)
    torch.cuda.synchronize()
    sampler.stop_flag = True
    sampler.join(timeout=2)
    ms_local = ev0.elapsed_time(ev1) / args.steps
    ms = adist.max_over_ranks(ms_local, dev)
    clocks = sampler.summary(t0, t1)
    final = absnt.read_stats(stats)
    assert final["S"] > 0 and final["n2"] > 0 and int(b_next.item()) >= B_CUR

    bytes_step = BYTES_PER_ELEM * d
    value = world * bytes_step / (ms * 1e-3) / 1e9
    kernel_gbs = bytes_step / (ms_local * 1e-3) / 1e9

    # end to end: pinned host gradients -> device, the fused call, stats + b_next -> host
    e2e_steps = max(1, min(args.steps, 8))
    host_grads = [torch.empty(d, dtype=torch.bfloat16, pin_memory=True) for _ in range(K_WORKERS)]
    for hg, g in zip(host_grads, grads):
        hg.copy_(g)
    host_stats = torch.empty(absnt.binding.ABS_STATS_HEADER, dtype=torch.float64, pin_memory=True)
    host_b = torch.empty(1, dtype=torch.int64, pin_memory=True)
    torch.cuda.synchronize()

    def e2e_step(i):
        for hg, g in zip(host_grads, grads):
            g.copy_(hg, non_blocking=True)
        step(i)
        host_stats.copy_(stats[:absnt.binding.ABS_STATS_HEADER], non_blocking=True)
        host_b.copy_(b_next, non_blocking=True)
        stream.synchronize()  # the caller needs b_next on the host to resize its sampler
        return int(host_b.item())

    e2e_step(0)
    adist.barrier(dev)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(e2e_steps):
        e2e_step(i + 1)
    e1.record(stream)
    torch.cuda.synchronize()
    e2e_ms = adist.max_over_ranks(e0.elapsed_time(e1) / e2e_steps, dev)
    h2d = K_WORKERS * d * GRAD_BYTES
    d2h = absnt.binding.ABS_STATS_HEADER * 8 + 8
    e2e = {"value": world * bytes_step / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s",
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
           "steps": e2e_steps,
           "note": "pinned host gradients copied in, fused call, stats header + b_next read back"}

    if rank != 0:
        return
    peak, peak_src = measured_peak()
    roofline = {"bound": "hbm", "achieved": kernel_gbs, "peak": peak, "unit": "GB/s",
                "frac": kernel_gbs / peak, "peak_source": peak_src,
                "frac_of_nominal_8TBs": kernel_gbs / NOMINAL_HBM_GBS,
                "kernel": "normtest_bulk_kernel<bf16,K=8,fused AdamW> (cp.async.bulk staging; + finalize, same timed call)",
                "algorithmic_bytes_per_launch": bytes_step,
                "traffic": recorded_traffic(d)}
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        d_sample = min(d, 1 << 25)
        times, cores = time_oracle(d_sample, 3)
        sec = min(times)
        cpu = {"value": BYTES_PER_ELEM * d_sample / sec / 1e9, "unit": "GB/s", "cores": cores,
               "kind": "oracle",
               "sample": "first %d of %d elements, best of 3 passes (%.2f s each), same %d "
                         "B/element" % (d_sample, d, sec, BYTES_PER_ELEM)}
    line = {"metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": workload_config(d), "clocks": clocks, "e2e": e2e,
            "gpu_launches": launches_per_step * args.steps, "roofline": roofline,
            "cpu_baseline": cpu,
            "pct_of_nominal_8TBs": 100.0 * value / world / NOMINAL_HBM_GBS,
            "T": final["T"], "b_next": int(b_next.item())}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    from paper_2412_21124_b200 import synth
    d = sum(synth.gpt2_small_tensor_sizes())
    if args.impl == "reference":
        run_reference(args, d)
    else:
        run_ours(args, d)
    import torch.distributed as tdist
    if tdist.is_available() and tdist.is_initialized():
        tdist.destroy_process_group()


if __name__ == "__main__":
    main()
