"""Per-call micro-benchmark of the library on synthetic inputs (one JSON line per point).

  python -m paper_2412_21124_b200.microbench --call fused --d 33554432 --K 8 --dtype bf16
  python -m paper_2412_21124_b200.microbench --sweep            # the d x K x dtype grid
  python -m paper_2412_21124_b200.microbench --report           # the grid and every other call
  python -m paper_2412_21124_b200.microbench --format out.jsonl # those lines as markdown tables

Every point carries the SM clock (median over the timed region), the clock-event reasons seen
and the peak power draw, read through NVML while the point was timed.

Timing: CUDA events on the launching stream around `steps` back-to-back calls after
`warmup` calls; calls whose first estimate is under ~200 us (where the host's per-call cost of
50-80 us through the Python binding would set the pace) are captured in a CUDA graph and the
replays are timed, so that the figure is device time.  Points whose working set is smaller than twice the L2 rotate over several
independent buffer sets so that every call reads cold data.  GB/s counts algorithmic bytes:
fused (K*s + 24) per coordinate (+4 with --gbar, +2 with --mixed), normtest K*s + 4,
adamw 28 (+2 with --mixed), persample 4 (fp32) or 2 (bf16) per matrix element.
"""
import argparse
import json
import os
import sys
import time

import torch

from . import binding as B
from . import synth
from .clocks import ClockSampler

HP = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)
L2_BYTES = 126 * 1024 * 1024
SWEEP_D = (1_048_576, 16_777_216, 124_439_808, 400_000_000, 1_235_814_400)
SWEEP_K = (2, 4, 8, 16, 32)
MEM_CAP = 160e9


def _sizes(d):
    if d == 124_439_808:
        return synth.gpt2_small_tensor_sizes()
    return synth.pseudo_tensor_sizes(d)


def bytes_per_call(call, d, K, esz, gbar, b):
    if call == "fused":
        return (K * esz + 24 + (4 if gbar else 0)) * d
    if call == "normtest":
        return (K * esz + 4) * d
    if call == "adamw":
        return 28 * d
    if call == "accumulate":  # the K new gradients once, the running mean read and written
        return (K * esz + 8) * d
    if call == "accumulate_adamw":  # the closing call: mean read, p/m/v read and written
        return (K * esz + 4 + 24) * d
    return esz * b * d


def run_point(call, d, K, dtype, n_shards=1, steps=None, warmup=3, gbar=False, b=4096, dev="cuda",
              graph=None, mixed=False, coordwise=False, with_q=False):
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    esz = 2 if dtype == "bf16" else 4
    nbytes = bytes_per_call(call, d, K, esz, gbar, b)
    if mixed:  # the bf16 copy of the parameters: 2 more bytes per coordinate
        if call not in ("fused", "adamw"):
            raise SystemExit("--mixed applies to the fused and adamw calls")
        nbytes += 2 * d
    n_sets = 1 if nbytes >= 2 * L2_BYTES else -(-2 * L2_BYTES // nbytes) + 1
    offs = synth.equal_shard_offsets(d, n_shards) if n_shards > 1 else None
    sets = []
    for i in range(n_sets):
        s = {}
        if call in ("fused", "normtest", "accumulate", "accumulate_adamw"):
            sizes = _sizes(d)
            sig = synth.per_tensor_sigma(sizes, 11)
            s["grads"] = synth.worker_grads(sizes, K, tdt, 100 + i, dev, sigma=sig)
            s["stats"] = B.alloc_stats(d, n_shards, dev)
        if call in ("fused", "adamw", "accumulate_adamw"):
            s["p"], s["m"], s["v"] = synth.adam_state(d, 200 + i, dev, zero_moments=False)
        if call in ("normtest", "adamw", "accumulate", "accumulate_adamw") or gbar:
            s["gbar"] = torch.zeros(d, dtype=torch.float32, device=dev)
            if call == "adamw":
                s["gbar"].normal_().mul_(0.02)
        if call == "persample":
            s["G"] = torch.empty(b, d, dtype=torch.float32, device=dev).normal_().mul_(0.3).to(tdt)
            s["stats"] = B.alloc_persample_stats(b, d, dev)
            s["gbar"] = torch.zeros(d, dtype=torch.float32, device=dev)
        s["b_next"] = torch.zeros(1, dtype=torch.int64, device=dev)
        if mixed:
            s["p16"] = torch.zeros(d, dtype=torch.bfloat16, device=dev)
        if call == "fused":  # marshal once; each timed call is then a single C call
            s["prepared"] = B.FusedStep(s["grads"], s["stats"], s.get("gbar"), s["b_next"], s["p"],
                                        s["m"], s["v"], HP, shard_offsets=offs,
                                        params_bf16_out=s.get("p16"), coordwise=coordwise)
        sets.append(s)

    def one(i):
        s = sets[i % n_sets]
        if call == "fused":
            s["prepared"].run(0.1, 512, 100 + i)
        elif call == "normtest":
            fn = (B.abs_norm_test_coordwise if coordwise
                  else (B.abs_norm_test_q if with_q else B.abs_norm_test))
            fn(s["grads"], 0.1, 512, s["stats"], s["gbar"], s["b_next"], shard_offsets=offs)
        elif call == "adamw" and mixed:
            B.abs_adamw_step_mixed(s["p"], s["gbar"], s["m"], s["v"], s["p16"], HP, 100 + i)
        elif call == "adamw":
            B.abs_adamw_step(s["p"], s["gbar"], s["m"], s["v"], HP, 100 + i)
        elif call == "accumulate":  # a later call of a step: the running mean is read and written
            B.abs_norm_test_accumulate(s["grads"], 8 * K, 0.1, 512, s["stats"], s["gbar"],
                                       s["b_next"], shard_offsets=offs)
        elif call == "accumulate_adamw":  # the closing call of a step, the mean not written
            B.abs_norm_test_accumulate_adamw(s["grads"], 8 * K, 0.1, 512, s["stats"], s["gbar"],
                                             None, s["b_next"], s["p"], s["m"], s["v"], HP,
                                             100 + i, shard_offsets=offs)
        else:
            fn = B.abs_persample_norm_test_coordwise if coordwise else B.abs_persample_norm_test
            fn(s["G"], 0.1, s["stats"], s["gbar"], s["b_next"])

    for i in range(warmup):
        one(i)
    torch.cuda.synchronize()
    est_ms = None
    if steps is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        one(0)
        e1.record()
        torch.cuda.synchronize()
        est_ms = max(e0.elapsed_time(e1), 1e-3)
        steps = int(max(10, min(400, 300.0 / est_ms)))
    if graph is None:  # short calls are bound by the host's per-call cost, which the estimate includes
        graph = est_ms is not None and est_ms < 0.2
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    t_begin = None
    if graph:
        # capture the calls once, replay them: device-side time of back-to-back calls
        per_graph = max(n_sets, min(steps, 64))
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for i in range(per_graph):
                    one(i)
        torch.cuda.current_stream().wait_stream(side)
        replays = max(1, steps // per_graph)
        g.replay()
        torch.cuda.synchronize()
        # short calls: replay for at least ~150 ms so that the clock record has samples
        per_replay_ms = max(est_ms if est_ms is not None else 0.05, 1e-3) * per_graph
        replays = int(max(replays, min(2000, 150.0 / per_replay_ms)))
        t_begin = time.perf_counter()
        e0.record()
        for _ in range(replays):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        steps = replays * per_graph
    else:
        stream = torch.cuda.current_stream()
        t_begin = time.perf_counter()
        e0.record(stream)
        for i in range(steps):
            one(warmup + i)
        e1.record(stream)
        torch.cuda.synchronize()
    t_end = time.perf_counter()
    sampler.stop()
    ms = e0.elapsed_time(e1) / steps
    out = {"call": call, "d": d, "K": K, "dtype": dtype, "n_shards": n_shards, "gbar": bool(gbar),
           "mixed": bool(mixed), "coordwise": bool(coordwise), "with_q": bool(with_q),
           "steps": steps, "buffer_sets": n_sets, "cuda_graph": bool(graph),
           "ms": ms,
           "bytes": nbytes, "GBps": nbytes / (ms * 1e-3) / 1e9}
    if call == "persample":
        out["b"] = b
    ck = sampler.summary(t_begin, t_end)
    out["clocks"] = {"sm_mhz": ck["sm_mhz"], "sm_max_mhz": ck["sm_max_mhz"],
                     "reasons": ck["reasons"], "power_w_max": ck.get("power_w_max"),
                     "samples": ck["samples"], "window": ck["window"]}
    return out


# Every per-call number quoted beside the d x K grid, as (call, d, K, dtype, shards, extras).
GPT2, LLAMA = 124_439_808, 1_235_814_400
REPORT_POINTS = (
    [("normtest", LLAMA, 8, "bf16", 8, {})]
    + [("normtest", GPT2, K, dt, 1, {}) for K in (1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12, 13, 14,
                                                  15, 16, 24, 32) for dt in ("bf16", "f32")]
    + [("adamw", GPT2, 0, "f32", 1, {}), ("adamw", LLAMA, 0, "f32", 1, {}),
       ("adamw", GPT2, 0, "f32", 1, {"mixed": True})]
    + [("persample", 16_384, 0, "f32", 1, {"b": b}) for b in (4096, 1024, 256, 32)]
    + [("persample", 65_536, 0, "f32", 1, {"b": 4096}), ("persample", 16_384, 0, "bf16", 1, {"b": 4096}),
       ("persample", 65_536, 0, "bf16", 1, {"b": 8192}),
       ("persample", 16_384, 0, "f32", 1, {"b": 4096, "coordwise": True})]
    + [("fused", GPT2, 8, "bf16", 1, {"gbar": True}), ("fused", GPT2, 8, "bf16", 1, {"mixed": True}),
       ("fused", 1_048_576, 4, "f32", 1, {})]
    + [("fused", GPT2, K, "bf16", 1, {}) for K in (6, 12, 20, 24, 27, 31, 36, 40, 44, 48, 52, 56,
                                                   60, 64)]
    + [("fused", GPT2, K, "f32", 1, {}) for K in (12, 20, 31, 48, 64)]
    # the diagnostic variant and the coordinate-wise test
    + [("normtest", GPT2, 8, "bf16", 1, {"q": True}), ("normtest", GPT2, 32, "bf16", 1, {"q": True}),
       ("normtest", GPT2, 8, "bf16", 1, {"coordwise": True}),
       ("fused", GPT2, 8, "bf16", 1, {"coordwise": True}),
       ("fused", GPT2, 4, "f32", 1, {"coordwise": True}),
       ("fused", GPT2, 32, "bf16", 1, {"coordwise": True})]
    # the carry-in form: K new gradients merged into the running mean per call
    + [("accumulate", GPT2, K, dt, 1, {}) for K in (1, 2, 4, 8, 9, 12, 16, 32) for dt in ("bf16", "f32")]
    + [("accumulate_adamw", GPT2, K, "bf16", 1, {}) for K in (1, 4, 8, 16)]
    # the paper's own model sizes (Table 4), J = 4 workers, bf16
    + [("fused", d, 4, "bf16", 1, {}) for d in (304_600_000, 1_100_000_000, 3_400_000_000)])


def sweep(args, graph):
    for dtype in ("bf16", "f32"):
        esz = 2 if dtype == "bf16" else 4
        for d in SWEEP_D:
            for K in SWEEP_K:
                if K * d * esz + 16 * d > MEM_CAP:
                    print(json.dumps({"call": "fused", "d": d, "K": K, "dtype": dtype, "sweep": True,
                                      "skipped": "K*d*s + 16*d exceeds 160 GB"}), flush=True)
                    continue
                r = run_point("fused", d, K, dtype, steps=args.steps, warmup=args.warmup, graph=graph)
                r["sweep"] = True
                print(json.dumps(r), flush=True)
                torch.cuda.empty_cache()


def report(args, graph):
    sweep(args, graph)
    for call, d, K, dtype, shards, extra in REPORT_POINTS:
        r = run_point(call, d, K, dtype, shards, args.steps, args.warmup, extra.get("gbar", False),
                      extra.get("b", 4096), graph=graph, mixed=extra.get("mixed", False),
                      coordwise=extra.get("coordwise", False), with_q=extra.get("q", False))
        print(json.dumps(r), flush=True)
        torch.cuda.empty_cache()


def _measured_peak():
    here = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    try:
        with open(os.path.join(here, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"])
    except Exception:
        return None


def format_markdown(path):
    """The JSON lines of --sweep / --report as two markdown tables (stdout)."""
    rows = [json.loads(line) for line in open(path) if line.startswith("{")]
    peak = _measured_peak()

    def clk(r):
        c = r.get("clocks") or {}
        if c.get("sm_mhz") is None:
            return "-", "-"
        watts = "%.0f W" % c["power_w_max"] if c.get("power_w_max") else ""
        return "%d" % c["sm_mhz"], (",".join(c.get("reasons") or []) or "none") + " " + watts

    print("| dtype | d | K | ms | GB/s | of 8000 | of measured | steps | graph | SM MHz | reasons, peak power |")
    print("|---|---|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        if not r.get("sweep"):
            continue
        if "skipped" in r:
            print("| %s | %d | %d | skipped: %s | | | | | | | |" % (r["dtype"], r["d"], r["K"],
                                                                  r["skipped"]))
            continue
        mhz, why = clk(r)
        print("| %s | %d | %d | %.4f | %.0f | %.3f | %s | %d | %s | %s | %s |" % (
            r["dtype"], r["d"], r["K"], r["ms"], r["GBps"], r["GBps"] / 8000.0,
            "%.3f" % (r["GBps"] / peak) if peak else "-", r["steps"],
            "yes" if r["cuda_graph"] else "", mhz, why))
    print()
    print("| call | d | K / b | dtype | shards | ms | GB/s | of 8000 | graph | SM MHz | reasons, peak power |")
    print("|---|---|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        if r.get("sweep"):
            continue
        name = r["call"] + (" +gbar" if r.get("gbar") and r["call"] == "fused" else "") + (
            " +bf16 copy" if r.get("mixed") else "") + (" +Q" if r.get("with_q") else "") + (
            " coordinate-wise" if r.get("coordwise") else "")
        kb = r["b"] if r["call"] == "persample" else (r["K"] if r["call"] != "adamw" else "-")
        mhz, why = clk(r)
        print("| %s | %d | %s | %s | %d | %.4f | %.0f | %.3f | %s | %s | %s |" % (
            name, r["d"], kb, r["dtype"], r["n_shards"], r["ms"], r["GBps"], r["GBps"] / 8000.0,
            "yes" if r["cuda_graph"] else "", mhz, why))


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--call", choices=["fused", "normtest", "adamw", "persample", "accumulate",
                                       "accumulate_adamw"], default="fused")
    ap.add_argument("--d", type=int, default=33_554_432)
    ap.add_argument("--K", type=int, default=8)
    ap.add_argument("--dtype", choices=["bf16", "f32"], default="bf16")
    ap.add_argument("--shards", type=int, default=1)
    ap.add_argument("--b", type=int, default=4096, help="rows of the per-sample matrix")
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--gbar", action="store_true", help="fused: also write gbar")
    ap.add_argument("--mixed", action="store_true",
                    help="fused / adamw: also write the bf16 copy of the parameters")
    ap.add_argument("--q", action="store_true",
                    help="normtest: abs_norm_test_q (also the diagnostic Q)")
    ap.add_argument("--coordwise", action="store_true",
                    help="fused / normtest: the coordinate-wise test as the decision")
    ap.add_argument("--sweep", action="store_true", help="fused call over the d x K x dtype grid")
    ap.add_argument("--report", action="store_true",
                    help="the grid and the per-call points quoted beside it, in one run")
    ap.add_argument("--format", metavar="JSONL", default=None,
                    help="print the JSON lines of a --sweep/--report run as markdown tables")
    ap.add_argument("--graph", choices=["auto", "on", "off"], default="auto",
                    help="time replays of a captured CUDA graph (auto: for calls under 200 us)")
    args = ap.parse_args(argv)
    if args.format:
        format_markdown(args.format)
        return
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device (there is no CPU fallback)")
    B.lib()
    graph = {"auto": None, "on": True, "off": False}[args.graph]
    if args.report:
        report(args, graph)
    elif args.sweep:
        sweep(args, graph)
    else:
        print(json.dumps(run_point(args.call, args.d, args.K, args.dtype, args.shards, args.steps,
                                   args.warmup, args.gbar, args.b, graph=graph,
                                   mixed=args.mixed, coordwise=args.coordwise,
                                   with_q=args.q)), flush=True)


if __name__ == "__main__":
    main(sys.argv[1:])
