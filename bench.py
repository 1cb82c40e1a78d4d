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
TIMED_REGION_MS = 1000.0   # the timed blocks together last about this long ...
MIN_BLOCKS, MAX_BLOCKS = 3, 400   # ... but there are at least 3 and at most 400 of them


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


FUSED_KERNEL_SOURCES = ("abs_device.cuh", "normtest_bulk.cuh", "normtest_stream.cuh")


def kernel_source_hash():
    """Hash of the sources the fused kernel is compiled from, as the compiler sees them:
    comments, blank lines and indentation do not count (no string literal in those files
    contains a comment marker)."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2412_21124_b200", "csrc")
    for name in FUSED_KERNEL_SOURCES:
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
    """DRAM bytes per launch of the fused kernel from the committed ncu counters, or None when
    the kernel sources changed after the counters were taken.  The record holds the counters
    of launches at `d_measured` coordinates.  When that is this workload's d they are used as
    they are.  Otherwise the launch is scaled by the rule the counters follow: every
    algorithmic byte crosses DRAM once, except the part of the optimizer state that the
    previous launch left in the L2 -- a fixed number of bytes, not a fraction -- so
    traffic(d) = algorithmic(d) - (algorithmic(d_measured) - measured)."""
    path = os.path.join(ROOT, "profiles", "fused_k8_bf16_dram_traffic.json")
    try:
        with open(path) as f:
            rec = json.load(f)
        if rec.get("kernel_source_hash") != kernel_source_hash():
            return None
        measured = float(rec["dram_bytes_per_launch"])
        d_measured = int(rec["d_measured"])
        if d_measured == d:
            return measured
        residue = BYTES_PER_ELEM * d_measured - measured
        return BYTES_PER_ELEM * d - residue
    except Exception:
        return None


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
    from paper_2412_21124_b200.clocks import ClockSampler

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
    step_no = [0]

    def step():
        absnt.abs_normtest_adamw(grads, ETA, B_CUR, stats, None, b_next, p, m, v, HP,
                                 STEP0 + step_no[0])
        step_no[0] += 1

    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()

    # The timed region is a sequence of blocks of exactly `steps` back-to-back calls, each
    # block bracketed by CUDA events on the launching stream, the whole sequence by a barrier
    # and a synchronize.  One block of a short run (20 steps = 14 ms) is a single sample taken
    # before the board has reached its steady clocks, so the block is repeated until about a
    # second of device time has passed, and the reported time is the median block.
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    ev[0].record(stream)
    for _ in range(args.steps):
        step()
    ev[1].record(stream)
    torch.cuda.synchronize()
    est_ms = max(ev[0].elapsed_time(ev[1]), 1e-3)          # a first, untimed block
    est_ms = adist.max_over_ranks(est_ms, dev)             # every rank must time the same blocks
    n_blocks = int(min(MAX_BLOCKS, max(MIN_BLOCKS, -(-TIMED_REGION_MS // est_ms))))
    events = [torch.cuda.Event(enable_timing=True) for _ in range(n_blocks + 1)]
    adist.barrier(dev)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    events[0].record(stream)
    for blk in range(n_blocks):
        for _ in range(args.steps):
            step()
        events[blk + 1].record(stream)
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    adist.barrier(dev)
    torch.cuda.synchronize()
    sampler.stop()
    block_ms_local = [events[i].elapsed_time(events[i + 1]) / args.steps for i in range(n_blocks)]
    # per block the slowest rank counts; then the median over blocks
    block_ms = adist.max_over_ranks_vec(block_ms_local, dev)
    ms = statistics.median(block_ms)
    ms_local = statistics.median(block_ms_local)
    clocks = sampler.summary(t0, t1)
    blocks = {"n": n_blocks, "steps_per_block": args.steps, "min_ms": min(block_ms),
              "median_ms": ms, "max_ms": max(block_ms),
              "note": "ms per step of each block of `steps` back-to-back calls (max over ranks); "
                      "ms_per_step is the median block; clocks cover all blocks"}
    # time x clock per block, where a block is long enough to hold clock samples of its own
    span = (t1 - t0) / n_blocks
    per_block_mhz = []
    for i in range(n_blocks):
        inside = [s_[1] for s_ in sampler.samples if t0 + i * span <= s_[0] <= t0 + (i + 1) * span]
        per_block_mhz.append(int(statistics.median(inside)) if len(inside) >= 3 else None)
    if all(x is not None for x in per_block_mhz):
        blocks["sm_mhz_per_block"] = per_block_mhz
        blocks["ms_x_ghz_per_block"] = [t * f / 1e3 for t, f in zip(block_ms, per_block_mhz)]
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
        step()
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
            "blocks": blocks,
            "gpu_launches": launches_per_step * args.steps * n_blocks, "roofline": roofline,
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
