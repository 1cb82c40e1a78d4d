"""FSDP-Norm with one process per rank (Sec. 3.3): every rank runs the fused norm-test + AdamW
kernels on its own index range and only the three sums per rank are exchanged.

Two rank processes share the one GPU that is there (their kernels are independent launches:
none waits on the other rank) and exchange the sums over gloo on the host.  Each rank checks
the combined sums, the decision and its slice of the updated state against the fp64 oracle run
on the whole vector with the rank ranges as shards; the parent checks that both ranks took
the same decision bit for bit.
"""
import json
import os
import socket
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import sys, json, datetime
sys.path.insert(0, %(root)r)
sys.path.insert(0, %(root)r + "/tests")
import numpy as np, torch, torch.distributed as tdist
from paper_2412_21124_b200 import dist as adist, synth, binding
from oracle import abs_oracle as orc
import util
import os
tdist.init_process_group("gloo", timeout=datetime.timedelta(seconds=120))
rank, world = tdist.get_rank(), tdist.get_world_size()
dev = "cuda:0"
K, d, eta, b_cur, step = 4, %(d)d, 0.1, 64, 3
tdt = torch.bfloat16 if %(bf16)d else torch.float32
hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)
seed = 7
while True:   # same seeds on every rank: identical full vectors; reseed near a decision boundary
    grads = synth.worker_grads([d], K, tdt, seed, dev)
    host = [util.to_host(g) for g in grads]
    offs = [adist.rank_range(d, r, world)[0] for r in range(world)] + [d]
    ref = orc.norm_test(host, eta, b_cur, shard_offsets=offs)
    if util.margin_ok(ref["T"], b_cur):
        break
    seed += 1
p, m, v = synth.adam_state(d, 11, dev, zero_moments=False)
p0, m0, v0 = (t.cpu().numpy().copy() for t in (p, m, v))
lo, hi = adist.rank_range(d, rank, world)
stats = binding.alloc_stats(hi - lo, 1, dev)
b_next = torch.zeros(1, dtype=torch.int64, device=dev)
gbar = torch.zeros(hi - lo, dtype=torch.float32, device=dev)
out = adist.sharded_normtest_adamw([g[lo:hi] for g in grads], eta, b_cur, stats, gbar, b_next,
                                   p[lo:hi], m[lo:hi], v[lo:hi], hp, step)
torch.cuda.synchronize()
util.assert_sum_close(out["n2"], ref["n2"], "n2")
util.assert_sum_close(out["S"], ref["S"], "S")
assert out["b_next"] == ref["b_next"], (out, ref["T"], ref["b_next"])
assert abs(out["T"] - ref["T"]) <= 2e-6 * abs(ref["T"])
# this rank's own sums are the oracle's shard record of its range
mine = binding.read_stats(stats)
util.assert_sum_close(mine["n2"], ref["shards"][rank][0], "n2 of the range")
util.assert_sum_close(mine["S"], ref["shards"][rank][1], "S of the range")
util.assert_vec_close(gbar, ref["gbar"][lo:hi], "gbar")
w_ref, m_ref, v_ref = util.oracle_adamw(orc, p0, m0, v0, ref["gbar"], hp, step)
util.assert_vec_close(p[lo:hi], w_ref[lo:hi], "params")
util.assert_vec_close(m[lo:hi], m_ref[lo:hi], "m")
util.assert_vec_close(v[lo:hi], v_ref[lo:hi], "v")
# outside its range a rank touches nothing
other = slice(0, lo) if lo > 0 else slice(hi, d)
assert np.array_equal(p[other].cpu().numpy(), p0[other])
tdist.barrier()
print(json.dumps({"rank": rank, "lo": lo, "hi": hi,
                  "out": {k: (repr(x) if isinstance(x, float) else x) for k, x in out.items()}}))
"""


# DDP-Norm (Sec. 3.2): every rank owns the gradient of its own minibatch for the whole vector and
# opens the other rank's buffer through an inter-process handle; its fused kernel then reads
# index range r of both buffers.  Neither kernel waits on the other rank: the ordering is two
# host rendezvous around the call.
DDP_WORKER = r"""
import sys, json, datetime
sys.path.insert(0, %(root)r)
sys.path.insert(0, %(root)r + "/tests")
import numpy as np, torch, torch.distributed as tdist
from paper_2412_21124_b200 import dist as adist, synth, binding
from oracle import abs_oracle as orc
import util
tdist.init_process_group("gloo", timeout=datetime.timedelta(seconds=120))
rank, world = tdist.get_rank(), tdist.get_world_size()
dev = "cuda:0"
torch.cuda.set_device(0)
d, eta, b_cur = %(d)d, 0.1, 64
tdt = torch.bfloat16 if %(bf16)d else torch.float32
hp = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)
p, m, v = synth.adam_state(d, 11, dev, zero_moments=False)     # the same replica on every rank
lo, hi = adist.rank_range(d, rank, world, adist.kDdpRangeAlign)
m_loc, v_loc = m[lo:hi].clone(), v[lo:hi].clone()
p_ref, m_ref, v_ref = (t.cpu().numpy().copy() for t in (p, m, v))
mine = torch.empty(d, dtype=tdt, device=dev)                   # this rank's gradient buffer
peers = adist.share_across_ranks(mine)
assert len(peers) == world and peers[rank] is mine
stats = binding.alloc_stats(hi - lo, 1, dev)
b_next = torch.zeros(1, dtype=torch.int64, device=dev)
outs, seed = [], 100
for step in (1, 2, 3):
    while True:   # all workers' gradients are known to every rank (same seeds), for the oracle
        grads = synth.worker_grads([d], world, tdt, seed, dev)
        host = [util.to_host(g) for g in grads]
        ref = orc.norm_test(host, eta, b_cur)
        seed += 1
        if util.margin_ok(ref["T"], b_cur):
            break
    mine.copy_(grads[rank])        # only this rank's own gradient goes into the shared buffer
    out = adist.ddp_normtest_adamw(peers, eta, b_cur, stats, b_next, p, m_loc, v_loc, hp, step)
    torch.cuda.synchronize()
    util.assert_sum_close(out["n2"], ref["n2"], "n2")
    util.assert_sum_close(out["S"], ref["S"], "S")
    assert out["b_next"] == ref["b_next"], (out, ref["T"], ref["b_next"])
    p_ref, m_ref, v_ref = util.oracle_adamw(orc, p_ref.astype(np.float32), m_ref.astype(np.float32),
                                            v_ref.astype(np.float32), ref["gbar"], hp, step)
    # the whole replica is up to date on every rank; the moments of this rank's range too
    util.assert_vec_close(p, p_ref, "params (whole replica)")
    util.assert_vec_close(m_loc, m_ref[lo:hi], "m")
    util.assert_vec_close(v_loc, v_ref[lo:hi], "v")
    # the oracle's next step starts from the values this GPU holds (parameters: everywhere;
    # moments: on its own range, the other range keeps the oracle's), so that one step's
    # rounding is not carried into the next comparison
    p_ref = p.cpu().numpy().copy()
    m_ref[lo:hi] = m_loc.cpu().numpy(); v_ref[lo:hi] = v_loc.cpu().numpy()
    outs.append({k: (repr(x) if isinstance(x, float) else x) for k, x in out.items()})
    tdist.barrier()
print(json.dumps({"rank": rank, "lo": lo, "hi": hi, "outs": outs,
                  "p_sum": repr(float(p.double().sum()))}))
"""


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


@pytest.mark.parametrize("d,bf16", [(300_007, 1), (65_539, 0)], ids=["bf16-odd-split", "f32"])
def test_two_rank_processes_index_ranges(d, bf16):
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK="0",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen(
            [sys.executable, "-c", WORKER % {"root": ROOT, "d": d, "bf16": bf16}], env=env,
            stdout=subprocess.PIPE, stderr=subprocess.PIPE))
    outs = []
    for proc in procs:
        so, se = proc.communicate(timeout=600)
        assert proc.returncode == 0, se.decode()[-3000:]
        outs.append(json.loads(so.decode().strip().splitlines()[-1]))
    outs.sort(key=lambda r: r["rank"])
    assert outs[0]["hi"] == outs[1]["lo"] and outs[0]["lo"] == 0 and outs[1]["hi"] == d
    assert outs[0]["out"] == outs[1]["out"]  # the same decision from the same bits on both ranks


def _run_two(script):
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK="0",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable, "-c", script], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE))
    outs = []
    for proc in procs:
        so, se = proc.communicate(timeout=600)
        assert proc.returncode == 0, se.decode()[-3000:]
        outs.append(json.loads(so.decode().strip().splitlines()[-1]))
    return sorted(outs, key=lambda r: r["rank"])


@pytest.mark.parametrize("d,bf16", [(300_007, 1), (65_539, 0)], ids=["bf16", "f32"])
def test_two_rank_processes_ddp_layout_over_shared_gradients(d, bf16):
    """Each rank contributes only its own worker gradient; the other rank's is read through the
    inter-process mapping by the fused kernel.  Three steps: the sums, the decision, the whole
    parameter replica and the rank's moments against the oracle on both workers' gradients; both
    ranks take the same decisions and end with the same replica, bit for bit."""
    a, b = _run_two(DDP_WORKER % {"root": ROOT, "d": d, "bf16": bf16})
    assert a["lo"] == 0 and a["hi"] == b["lo"] and b["hi"] == d and a["hi"] % 64 == 0
    assert a["outs"] == b["outs"] and len(a["outs"]) == 3
    assert a["p_sum"] == b["p_sum"]
