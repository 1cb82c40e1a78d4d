"""world_size-2 gloo test (CPU) of the multi-process host logic: index ranges cover the
vector, per-rank sums combined in rank order reproduce the oracle's sharded totals and
decision on every rank, every rank's batch-size schedule advances identically, and the timing
reduction is a max."""
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import sys, json
sys.path.insert(0, %(root)r)
import numpy as np, torch
from paper_2412_21124_b200 import dist as adist, synth
from oracle import abs_oracle as orc
rank, world, _ = adist.init_from_env(backend="gloo")
K, d, eta, b_cur = 4, 50_003, 0.1, 16
grads = synth.worker_grads([d], K, torch.float32, 42, "cpu")       # same seed on every rank
host = [g.numpy() for g in grads]
lo, hi = adist.rank_range(d, rank, world)
mine = orc.norm_test([h[lo:hi] for h in host], eta, b_cur, want_gbar=False)  # this rank's range
out = adist.combine_rank_sums(mine["n2"], mine["S"], mine["Q"], K, eta, b_cur)
offs = [adist.rank_range(d, r, world)[0] for r in range(world)] + [d]
full = orc.norm_test(host, eta, b_cur, shard_offsets=offs, want_gbar=False)
t = adist.max_over_ranks(1.0 + rank)
# every rank advances its own copy of the schedule with the decision it computed
from paper_2412_21124_b200 import binding
sched = binding.abs_schedule_init(world, 2, 4, 4096, 8, 1)   # J = world, M = 2, microbatch 4: b = 16
assert sched.b == b_cur and binding.abs_schedule_test_due(sched)
binding.abs_schedule_advance(sched, out["b_next"])
adist.barrier()
print(json.dumps({"rank": rank, "out": out, "full": {k: full[k] for k in ("n2", "S", "Q", "T", "b_next", "flags")},
                  "offs": offs, "tmax": t,
                  "sched": {k: getattr(sched, k) for k in ("J", "M", "micro", "b", "step", "samples")}}))
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def test_rank_ranges_cover():
    from paper_2412_21124_b200 import dist as adist
    for d, w in ((10, 3), (7, 8), (1_235_814_400, 8), (5, 1)):
        prev = 0
        for r in range(w):
            lo, hi = adist.rank_range(d, r, w)
            assert lo == prev and hi >= lo
            prev = hi
        assert prev == d
    # whole units of `align` coordinates: every range starts on a unit boundary, the ranges still
    # tile [0, d), and ranks beyond the last unit get empty ranges
    for d, w, al in ((1000, 3, 64), (64, 4, 64), (65, 4, 64), (124_439_808, 8, 64), (7, 2, 64)):
        prev = 0
        for r in range(w):
            lo, hi = adist.rank_range(d, r, w, al)
            assert lo == prev and hi >= lo and (lo % al == 0 or lo == d)
            prev = hi
        assert prev == d
        sizes = [adist.rank_range(d, r, w, al) for r in range(w)]
        assert max(h - l for l, h in sizes) - min(h - l for l, h in sizes) < 2 * al


def test_two_rank_combine_matches_oracle():
    import json
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER % {"root": ROOT}], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE))
    outs = []
    for p in procs:
        so, se = p.communicate(timeout=300)
        assert p.returncode == 0, se.decode()[-2000:]
        outs.append(json.loads(so.decode().strip().splitlines()[-1]))
    a, b = outs
    assert a["out"] == b["out"]  # every rank takes the same bit-identical decision
    for r in outs:
        for k in ("n2", "S", "Q", "T", "b_next", "flags"):
            assert r["out"][k] == r["full"][k], k  # rank-ordered sum == shard-ordered sum
        assert r["tmax"] == 2.0
    assert a["out"]["b_next"] > 16
    # identical schedules on both ranks, the new batch a multiple of J*M that covers b_next
    assert a["sched"] == b["sched"]
    sc = a["sched"]
    assert sc["b"] == sc["J"] * sc["M"] * sc["micro"] and sc["micro"] <= 8
    assert sc["b"] >= min(a["out"]["b_next"], 4096) or sc["b"] == 4096 // (sc["J"] * sc["M"]) * sc["J"] * sc["M"]
    assert sc["step"] == 2 and sc["samples"] == 16
