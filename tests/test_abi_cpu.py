"""CPU-side checks of the C ABI: the library loads, exports every declared symbol, its
host helpers agree with the hand-worked fixtures, and every invalid-argument path returns
its status before anything could be launched.

The reject cases hand fabricated addresses to launching entry points.  They are safe because
every check comes before the first launch -- and, so that this does not rest on every check
being right, the whole module runs with CUDA_VISIBLE_DEVICES set to the empty string: the
library initialises CUDA lazily, on its first runtime call, so with no device visible a launch
that slipped through a regressed check returns ABS_ERR_CUDA (and fails the test) instead of
running on an unmapped address."""
import ctypes
import json
import math
import os
import re
import subprocess
import sys

import pytest

import __graft_entry__ as entry
from paper_2412_21124_b200 import binding


@pytest.fixture(scope="module", autouse=True)
def _no_visible_device():
    """Hide every GPU from the CUDA runtime for the life of this module.  The variable is read
    when the runtime initialises, which nothing here triggers when all checks hold; it is put
    back afterwards for the modules that follow."""
    old = os.environ.get("CUDA_VISIBLE_DEVICES")
    os.environ["CUDA_VISIBLE_DEVICES"] = ""
    yield
    if old is None:
        os.environ.pop("CUDA_VISIBLE_DEVICES", None)
    else:
        os.environ["CUDA_VISIBLE_DEVICES"] = old

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "abs_normtest.h")
GOLDEN = os.path.join(ROOT, "tests", "golden", "hand_cases.json")


@pytest.fixture(scope="module")
def L():
    entry.build()
    return binding.lib()


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(abs_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = declared_functions()
    assert {"abs_norm_test", "abs_adamw_step", "abs_normtest_adamw",
            "abs_persample_norm_test"} <= set(names)
    for n in names:
        assert hasattr(L, n), "header declares %s but the library does not export it" % n


def test_header_is_plain_c_and_links_from_c(L, tmp_path):
    """The boundary is a C ABI: the header compiles as C99 and a C program can call the
    host-side helpers of the shared library."""
    import subprocess
    src = tmp_path / "use_abi.c"
    src.write_text(
        '#include "abs_normtest.h"\n#include <stdio.h>\n'
        "int main(void) {\n"
        "  double T; int flags;\n"
        "  long long b = (long long)abs_decide(4.0, 8.0, 2.0, 0.25, 3, &T, &flags);\n"
        "  abs_adamw_hparams hp = {1e-3f, 0.9f, 0.999f, 1e-8f, 0.1f};\n"
        "  int rc = abs_adamw_step(0, 0, 0, 0, 10, &hp, 1, 0);\n"
        '  printf("%lld %.1f %d %lld %d %zu\\n", b, T, flags, (long long)abs_round_batch(259, 4, 16), rc,\n'
        "         abs_stats_bytes(1, 1));\n"
        "  abs_schedule s;\n"
        "  if (abs_schedule_init(&s, 4, 16, 4, 8192, 8, 1) != ABS_OK || !abs_schedule_test_due(&s)) return 1;\n"
        "  if (abs_schedule_advance(&s, 1000) != ABS_OK) return 2;\n"
        '  printf("%lld %lld %lld\\n", (long long)s.M, (long long)s.micro, (long long)s.b);\n'
        "  return 0;\n}\n")
    exe = tmp_path / "use_abi"
    lib_dir = os.path.dirname(binding._build.LIB_PATH)
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-pedantic", "-I",
                           os.path.join(ROOT, "include"), str(src), "-o", str(exe), "-L", lib_dir,
                           "-labs_normtest", "-Wl,-rpath," + lib_dir])
    out = subprocess.check_output([str(exe)]).decode().split()
    assert out == ["4", "4.0", "4", "320", str(binding.ABS_ERR_NULL), str(8 * 8 + 4 * 8 + 2 * 32),
                   "32", "8", "1024"]


def _sched_state(s):
    return {k: getattr(s, k) for k in ("J", "M", "micro", "b", "step", "samples")}


def test_schedule_hand_cases(L):
    for c in json.load(open(GOLDEN))["schedule"]:
        i = c["init"]
        s = binding.abs_schedule_init(i["J"], i["M"], i["micro0"], i["b_max"], i["max_micro"],
                                      i["interval"])
        assert s.b == i["J"] * i["M"] * i["micro0"] and s.step == 1 and s.samples == 0
        for st in c["steps"]:
            assert binding.abs_schedule_test_due(s) == st["due"], c["name"]
            binding.abs_schedule_advance(s, st["b_test"])
            got = _sched_state(s)
            assert {k: got[k] for k in st["after"]} == st["after"], c["name"]


def test_schedule_matches_oracle_on_random_runs(L):
    import numpy as np
    from oracle import abs_oracle as orc
    rng = np.random.default_rng(23)
    for trial in range(100):
        J, M, micro0 = int(rng.integers(1, 9)), int(rng.integers(1, 33)), int(rng.integers(1, 9))
        max_micro = int(rng.integers(micro0, 4 * micro0 + 1)) if trial % 4 else 0
        b_max = J * M * micro0 * int(rng.integers(1, 200)) + int(rng.integers(0, 50))
        interval = int(rng.integers(1, 5))
        s = binding.abs_schedule_init(J, M, micro0, b_max, max_micro, interval)
        o = orc.Schedule(J, M, micro0, b_max, max_micro, interval)
        for _ in range(40):
            assert binding.abs_schedule_test_due(s) == o.test_due()
            b_test = int(rng.integers(1, 3 * b_max)) if o.test_due() else o.b
            binding.abs_schedule_advance(s, b_test)
            o.advance(b_test)
            assert _sched_state(s) == o.state()
    # near the largest accepted cap: Python integers on one side, int64 on the other
    big = 1 << 60
    s = binding.abs_schedule_init(3, 5, 7, big, 11, 1)
    o = orc.Schedule(3, 5, 7, big, 11, 1)
    for b_test in (10**6, 10**12, big - 12345, big, 2**63 - 1):
        binding.abs_schedule_advance(s, b_test)
        o.advance(b_test)
        assert _sched_state(s) == o.state()
    assert s.b <= big and not binding.abs_schedule_test_due(s) == (s.b == big)


def test_schedule_rejects(L):
    s = binding.AbsSchedule()
    ref = ctypes.byref(s)
    assert L.abs_schedule_init(None, 4, 16, 4, 8192, 8, 1) == binding.ABS_ERR_NULL
    for args in ((0, 16, 4, 8192, 8, 1), (4, 0, 4, 8192, 8, 1), (4, 16, 0, 8192, 8, 1),
                 (4, 16, 4, 0, 8, 1), (4, 16, 4, 8192, -1, 1), (4, 16, 4, 8192, 8, 0),
                 (4, 16, 4, 255, 8, 1),        # base batch 256 above the cap
                 (4, 16, 9, 8192, 8, 1),       # base microbatch above its maximum
                 (4, 16, 4, (1 << 60) + 1, 8, 1),
                 (1 << 31, 1 << 31, 4, 1 << 60, 0, 1)):  # J*M*micro passes 2^60
        assert L.abs_schedule_init(ref, *args) == binding.ABS_ERR_RANGE, args
    assert L.abs_schedule_test_due(None) == -1
    assert L.abs_schedule_advance(None, 5) == binding.ABS_ERR_NULL
    assert L.abs_schedule_init(ref, 4, 16, 4, 8192, 8, 1) == 0
    before = _sched_state(s)
    assert L.abs_schedule_advance(ref, 0) == binding.ABS_ERR_RANGE
    assert _sched_state(s) == before
    with pytest.raises(binding.AbsError):
        binding.abs_schedule_init(4, 16, 4, 255)


def test_status_strings(L):
    seen = set()
    for s in range(0, -9, -1):
        msg = L.abs_status_string(s).decode()
        assert msg and msg != "unknown status"
        seen.add(msg)
    assert len(seen) == 9
    assert L.abs_status_string(-99).decode() == "unknown status"
    assert L.abs_last_cuda_error() == 0


def test_decide_matches_hand_cases(L):
    cases = json.load(open(GOLDEN))["norm_test"]
    for c in cases:
        K = len(c["grads"])
        for dec in c["decisions_worker"]:
            b_next, T, flags = binding.abs_decide(c["S"], c["n2"], K, c["eta"], dec["b_cur"])
            assert b_next == dec["b_next"]
            assert bool(flags & binding.ABS_FLAG_VIOLATED) == dec["violated"]
        b_next, T, flags = binding.abs_decide(c["S"], c["n2"], K - 1, c["eta"], K)
        assert b_next == c["b_next_persample"]


def test_decide_edge_cases(L):
    b_next, T, flags = binding.abs_decide(0.0, 0.0, 4, 0.1, 9)
    assert b_next == 9 and math.isnan(T) and flags == binding.ABS_FLAG_DEGENERATE
    b_next, T, flags = binding.abs_decide(1.0, 0.0, 4, 0.1, 9)
    assert b_next == 2 ** 63 - 1 and T == math.inf
    assert flags == binding.ABS_FLAG_DEGENERATE | binding.ABS_FLAG_VIOLATED
    for bad in (math.nan, math.inf):
        b_next, T, flags = binding.abs_decide(bad, 1.0, 4, 0.1, 9)
        assert b_next == 9 and flags == binding.ABS_FLAG_NONFINITE
    b_next, T, flags = binding.abs_decide(1.0, 1.0, 2.0, 1e-12, 5)
    assert b_next == 2 ** 63 - 1 and flags == binding.ABS_FLAG_VIOLATED
    # ties keep the batch size (the test is satisfied with equality)
    assert binding.abs_decide(4.0, 8.0, 2.0, 0.25, 4)[0] == 4


def test_round_batch_hand_cases(L):
    for c in json.load(open(GOLDEN))["round_batch"]:
        for case in c["cases"]:
            assert binding.abs_round_batch(case["b_next"], case["J"], case["M"]) == case["b"]
    assert binding.abs_round_batch(0, 4, 4) == -1
    assert binding.abs_round_batch(5, 0, 4) == -1
    assert binding.abs_round_batch(5, 4, 0) == -1


def test_stats_bytes(L):
    assert binding.abs_stats_bytes(0, 1) == 0
    assert binding.abs_stats_bytes(10, 0) == 0
    assert binding.abs_stats_bytes(10, binding.ABS_MAX_SHARDS + 1) == 0
    hdr = binding.ABS_STATS_HEADER * 8
    # one chunk + one spare per shard
    assert binding.abs_stats_bytes(1, 1) == hdr + 4 * 8 + 2 * 32
    big = binding.abs_stats_bytes(124_439_808, 8)
    assert big % 16 == 0 and big < (1 << 20)
    assert binding.abs_persample_stats_bytes(1, 10) == 0
    # two doubles per (row block, column), row blocks of at most 512 rows
    assert binding.abs_persample_stats_bytes(4096, 16384) > 2 * (4096 // 512) * 16384 * 8


# ---- invalid arguments: every path returns its status before any CUDA call ---------------
FAKE = 0x10000  # a non-null, 16-byte aligned value that is never dereferenced


def _nt_args(**over):
    K = over.pop("K", 2)
    table = over.pop("table", (ctypes.c_void_p * 64)(*([FAKE] * 64)))
    a = dict(grads=table, K=K, d=100, dtype=0, offs=None, n_shards=1, eta=0.1, b_cur=8,
             stats=FAKE, gbar=FAKE, b_next=FAKE, stream=None)
    a.update(over)
    return [a[k] for k in ("grads", "K", "d", "dtype", "offs", "n_shards", "eta", "b_cur",
                           "stats", "gbar", "b_next", "stream")]


def _offs(*vals):
    return (ctypes.c_int64 * len(vals))(*vals)


@pytest.mark.parametrize("over,status", [
    (dict(grads=None), binding.ABS_ERR_NULL),
    (dict(stats=None), binding.ABS_ERR_NULL),
    (dict(gbar=None), binding.ABS_ERR_NULL),
    (dict(b_next=None), binding.ABS_ERR_NULL),
    (dict(dtype=2), binding.ABS_ERR_DTYPE),
    (dict(K=0), binding.ABS_ERR_RANGE),
    (dict(K=binding.ABS_MAX_WORKERS + 1), binding.ABS_ERR_RANGE),
    (dict(d=0), binding.ABS_ERR_RANGE),
    (dict(b_cur=0), binding.ABS_ERR_RANGE),
    (dict(eta=0.0), binding.ABS_ERR_RANGE),
    (dict(eta=-0.1), binding.ABS_ERR_RANGE),
    (dict(eta=math.nan), binding.ABS_ERR_RANGE),
    (dict(eta=math.inf), binding.ABS_ERR_RANGE),
    (dict(stats=FAKE + 8), binding.ABS_ERR_ALIGN),
    (dict(gbar=FAKE + 2), binding.ABS_ERR_ALIGN),
    (dict(b_next=FAKE + 4), binding.ABS_ERR_ALIGN),
    (dict(table=(ctypes.c_void_p * 32)(FAKE, 0)), binding.ABS_ERR_NULL),
    (dict(table=(ctypes.c_void_p * 32)(FAKE, FAKE + 2)), binding.ABS_ERR_ALIGN),
    (dict(offs=_offs(0, 100), n_shards=0), binding.ABS_ERR_RANGE),
    (dict(offs=_offs(0, 100), n_shards=129), binding.ABS_ERR_RANGE),
    (dict(offs=_offs(1, 100), n_shards=1), binding.ABS_ERR_SHARDS),
    (dict(offs=_offs(0, 99), n_shards=1), binding.ABS_ERR_SHARDS),
    (dict(offs=_offs(0, 60, 50, 100), n_shards=3), binding.ABS_ERR_SHARDS),
])
def test_norm_test_rejects(L, over, status):
    assert L.abs_norm_test(*_nt_args(**over)) == status


def _acc_args(**over):
    K = over.pop("K", 2)
    table = over.pop("table", (ctypes.c_void_p * 64)(*([FAKE] * 64)))
    a = dict(grads=table, K=K, d=100, dtype=0, offs=None, n_shards=1, count_in=0, eta=0.1,
             b_cur=8, stats=FAKE, mean=FAKE, b_next=FAKE, stream=None)
    a.update(over)
    return [a[k] for k in ("grads", "K", "d", "dtype", "offs", "n_shards", "count_in", "eta",
                           "b_cur", "stats", "mean", "b_next", "stream")]


@pytest.mark.parametrize("over,status", [
    (dict(grads=None), binding.ABS_ERR_NULL),
    (dict(stats=None), binding.ABS_ERR_NULL),
    (dict(mean=None), binding.ABS_ERR_NULL),
    (dict(b_next=None), binding.ABS_ERR_NULL),
    (dict(dtype=2), binding.ABS_ERR_DTYPE),
    (dict(K=0), binding.ABS_ERR_RANGE),
    (dict(K=65), binding.ABS_ERR_RANGE),          # more per call than the carry-in form takes
    (dict(count_in=-1), binding.ABS_ERR_RANGE),
    (dict(d=0), binding.ABS_ERR_RANGE),
    (dict(b_cur=0), binding.ABS_ERR_RANGE),
    (dict(eta=0.0), binding.ABS_ERR_RANGE),
    (dict(eta=math.nan), binding.ABS_ERR_RANGE),
    (dict(stats=FAKE + 8), binding.ABS_ERR_ALIGN),
    (dict(mean=FAKE + 2), binding.ABS_ERR_ALIGN),
    (dict(table=(ctypes.c_void_p * 32)(FAKE, 0)), binding.ABS_ERR_NULL),
    (dict(offs=_offs(0, 99), n_shards=1), binding.ABS_ERR_SHARDS),
    # the running mean is read and written while the gradients are read: no overlap allowed
    (dict(), binding.ABS_ERR_ALIAS),
    (dict(table=(ctypes.c_void_p * 32)(FAKE + 0x100000, FAKE + 0x200000), mean=FAKE + 0x100000 + 40,
          stats=FAKE + 0x300000, b_next=FAKE + 0x400000), binding.ABS_ERR_ALIAS),
])
def test_accumulate_rejects(L, over, status):
    assert L.abs_norm_test_accumulate(*_acc_args(**over)) == status


def test_accumulate_adamw_rejects(L):
    hp = binding.abs_adamw_hparams(1e-3, 0.9, 0.999, 1e-8, 0.1)
    far = [FAKE + i * 0x100000 for i in range(1, 12)]
    table = (ctypes.c_void_p * 4)(far[0], far[1])

    def call(**over):
        a = dict(grads=table, K=2, d=100, dtype=0, offs=None, n_shards=1, count_in=3, eta=0.1,
                 b_cur=8, stats=far[2], mean=far[3], gbar=far[3], b_next=far[4], p=far[5], m=far[6],
                 v=far[7], hp=ctypes.byref(hp), step=1, stream=None)
        a.update(over)
        return L.abs_norm_test_accumulate_adamw(*[a[k] for k in (
            "grads", "K", "d", "dtype", "offs", "n_shards", "count_in", "eta", "b_cur", "stats",
            "mean", "gbar", "b_next", "p", "m", "v", "hp", "step", "stream")])

    assert call(mean=None) == binding.ABS_ERR_NULL            # a running step needs its mean
    assert call(p=None) == binding.ABS_ERR_NULL
    assert call(hp=None) == binding.ABS_ERR_NULL
    assert call(step=0) == binding.ABS_ERR_RANGE
    assert call(K=65) == binding.ABS_ERR_RANGE
    assert call(m=far[6] + 2) == binding.ABS_ERR_ALIGN
    assert call(gbar=far[3] + 16) == binding.ABS_ERR_ALIAS     # overlaps the mean without being it
    assert call(gbar=far[5]) == binding.ABS_ERR_ALIAS          # the mean output on the parameters
    assert call(mean=far[6]) == binding.ABS_ERR_ALIAS          # the running mean on a moment
    assert call(v=far[0] + 8) == binding.ABS_ERR_ALIAS         # an output on a gradient buffer


def _hp(**over):
    v = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)
    v.update(over)
    return binding.abs_adamw_hparams(v["lr"], v["beta1"], v["beta2"], v["eps"], v["weight_decay"])


@pytest.mark.parametrize("hp,step,status", [
    (None, 1, binding.ABS_ERR_NULL),
    (_hp(), 0, binding.ABS_ERR_RANGE),
    (_hp(beta1=1.0), 1, binding.ABS_ERR_RANGE),
    (_hp(beta2=-0.1), 1, binding.ABS_ERR_RANGE),
    (_hp(lr=-1.0), 1, binding.ABS_ERR_RANGE),
    (_hp(eps=math.nan), 1, binding.ABS_ERR_RANGE),
    (_hp(weight_decay=math.inf), 1, binding.ABS_ERR_RANGE),
])
def test_adamw_and_fused_reject_hparams(L, hp, step, status):
    ref = ctypes.byref(hp) if hp is not None else None
    assert L.abs_adamw_step(FAKE, FAKE, FAKE, FAKE, 10, ref, step, None) == status
    args = _nt_args() [:-1] + [FAKE, FAKE, FAKE, ref, step, None]
    assert L.abs_normtest_adamw(*args) == status


def test_clipped_adamw_rejects(L):
    hp = _hp()
    r = ctypes.byref(hp)
    f = L.abs_adamw_step_clipped
    assert f(FAKE, FAKE, FAKE, FAKE, 10, r, 1, 1.0, None, None) == binding.ABS_ERR_NULL
    assert f(FAKE, FAKE, FAKE, FAKE, 10, r, 1, 0.0, FAKE, None) == binding.ABS_ERR_RANGE
    assert f(FAKE, FAKE, FAKE, FAKE, 10, r, 1, math.nan, FAKE, None) == binding.ABS_ERR_RANGE
    assert f(FAKE, FAKE, FAKE, FAKE, 10, r, 1, 1.0, FAKE + 4, None) == binding.ABS_ERR_ALIGN
    assert f(None, FAKE, FAKE, FAKE, 10, r, 1, 1.0, FAKE, None) == binding.ABS_ERR_NULL
    assert f(FAKE, FAKE, FAKE, FAKE, 10, r, 0, 1.0, FAKE, None) == binding.ABS_ERR_RANGE


def test_clip_prev_rejects(L):
    hp = _hp()
    r = ctypes.byref(hp)
    base = _nt_args(gbar=None)[:-1]
    f = L.abs_normtest_adamw_clip_prev
    far = [FAKE + 0x100000 * i for i in range(1, 4)]   # params, m, v apart from each other
    assert f(*(base + far + [r, 1, 0.0, FAKE, None])) == binding.ABS_ERR_RANGE
    assert f(*(base + far + [r, 1, math.nan, FAKE, None])) == binding.ABS_ERR_RANGE
    assert f(*(base + far + [r, 1, 1.0, FAKE + 4, None])) == binding.ABS_ERR_ALIGN
    assert f(*(base + [None] + far[1:] + [r, 1, 1.0, FAKE, None])) == binding.ABS_ERR_NULL
    assert f(*(base + far + [r, 0, 1.0, None, None])) == binding.ABS_ERR_RANGE   # step, no clipping


def test_mixed_precision_rejects(L):
    hp = binding.abs_adamw_hparams(1e-3, 0.9, 0.999, 1e-8, 0.1)
    r = ctypes.byref(hp)
    f = L.abs_adamw_step_mixed
    assert f(FAKE, FAKE, FAKE, FAKE, None, 10, r, 1, 0.0, None, None) == binding.ABS_ERR_NULL
    assert f(FAKE, FAKE, FAKE, FAKE, FAKE + 1, 10, r, 1, 0.0, None, None) == binding.ABS_ERR_ALIGN
    assert f(None, FAKE, FAKE, FAKE, FAKE, 10, r, 1, 0.0, None, None) == binding.ABS_ERR_NULL
    assert f(FAKE, FAKE, FAKE, FAKE, FAKE, 0, r, 1, 0.0, None, None) == binding.ABS_ERR_RANGE
    # clipping is on exactly when stats_in is given: then max_norm must be finite and positive
    assert f(FAKE, FAKE, FAKE, FAKE, FAKE, 10, r, 1, 0.0, FAKE, None) == binding.ABS_ERR_RANGE
    assert f(FAKE, FAKE, FAKE, FAKE, FAKE, 10, r, 1, math.inf, FAKE, None) == binding.ABS_ERR_RANGE
    assert f(FAKE, FAKE, FAKE, FAKE, FAKE, 10, r, 1, 1.0, FAKE + 4, None) == binding.ABS_ERR_ALIGN
    base = _nt_args()[:-1]
    g = L.abs_normtest_adamw_mixed
    assert g(*(base + [FAKE, FAKE, FAKE, None, r, 1, None])) == binding.ABS_ERR_NULL
    assert g(*(base + [FAKE, FAKE, FAKE, FAKE + 1, r, 1, None])) == binding.ABS_ERR_ALIGN
    assert g(*(base + [None, FAKE, FAKE, FAKE, r, 1, None])) == binding.ABS_ERR_NULL
    assert g(*(base + [FAKE, FAKE, FAKE, FAKE, r, 0, None])) == binding.ABS_ERR_RANGE


def test_adamw_rejects_pointers(L):
    hp = _hp()
    r = ctypes.byref(hp)
    assert L.abs_adamw_step(None, FAKE, FAKE, FAKE, 10, r, 1, None) == binding.ABS_ERR_NULL
    assert L.abs_adamw_step(FAKE, FAKE, FAKE, None, 10, r, 1, None) == binding.ABS_ERR_NULL
    assert L.abs_adamw_step(FAKE, FAKE, FAKE, FAKE, 0, r, 1, None) == binding.ABS_ERR_RANGE
    assert L.abs_adamw_step(FAKE + 2, FAKE, FAKE, FAKE, 10, r, 1, None) == binding.ABS_ERR_ALIGN
    # fused: params/m/v required, gbar optional
    base = _nt_args(gbar=None)[:-1]
    assert L.abs_normtest_adamw(*(base + [None, FAKE, FAKE, r, 1, None])) == binding.ABS_ERR_NULL
    assert L.abs_normtest_adamw(*(base + [FAKE, FAKE + 2, FAKE, r, 1, None])) == binding.ABS_ERR_ALIGN


@pytest.mark.parametrize("args,status", [
    ((None, 4, 10, 10, 0, 0.1, FAKE, FAKE, FAKE, None), binding.ABS_ERR_NULL),
    ((FAKE, 4, 10, 10, 0, 0.1, None, FAKE, FAKE, None), binding.ABS_ERR_NULL),
    ((FAKE, 4, 10, 10, 2, 0.1, FAKE, FAKE, FAKE, None), binding.ABS_ERR_DTYPE),
    ((FAKE + 1, 4, 10, 10, 1, 0.1, FAKE, FAKE, FAKE, None), binding.ABS_ERR_ALIGN),
    ((FAKE, 1, 10, 10, 0, 0.1, FAKE, FAKE, FAKE, None), binding.ABS_ERR_RANGE),
    ((FAKE, 4, 0, 10, 0, 0.1, FAKE, FAKE, FAKE, None), binding.ABS_ERR_RANGE),
    ((FAKE, 4, 10, 9, 0, 0.1, FAKE, FAKE, FAKE, None), binding.ABS_ERR_RANGE),
    ((FAKE, 4, 10, 10, 0, 0.0, FAKE, FAKE, FAKE, None), binding.ABS_ERR_RANGE),
    ((FAKE + 2, 4, 10, 10, 0, 0.1, FAKE, FAKE, FAKE, None), binding.ABS_ERR_ALIGN),
    ((FAKE, 4, 10, 10, 0, 0.1, FAKE + 8, FAKE, FAKE, None), binding.ABS_ERR_ALIGN),
])
def test_persample_rejects(L, args, status):
    assert L.abs_persample_norm_test(*args) == status
    assert L.abs_persample_norm_test_coordwise(*args) == status


# ---- aliasing: outputs may not overlap the gradients or each other ------------------------
def _fused_args(table, K, d, dtype, stats, gbar, b_next, p, m, v):
    hp = _hp()
    return [table, K, d, dtype, None, 1, 0.1, 8, stats, gbar, b_next, p, m, v, ctypes.byref(hp), 1,
            None], hp


def test_overlapping_buffers_are_rejected(L):
    d = 1000                       # fp32: 4000 bytes per buffer
    A = 0x100000                   # fabricated, 16-byte aligned, never dereferenced
    g0, g1 = A, A + 0x10000
    stats, b_next = A + 0x80000, A + 0x90000
    table = (ctypes.c_void_p * 2)(g0, g1)
    ok_gbar = A + 0x20000
    nt = lambda gbar, st=stats, bn=b_next: L.abs_norm_test(table, 2, d, 0, None, 1, 0.1, 8, st,
                                                           gbar, bn, None)
    # gbar_out inside, at the start of, or straddling the end of a gradient buffer
    for gbar in (g0, g1, g0 + 4 * (d - 1), g1 - 4 * (d - 1), g0 + 2000):
        assert nt(gbar) == binding.ABS_ERR_ALIAS, hex(gbar)
    # stats_out or b_next_out inside a gradient buffer or inside gbar_out
    assert nt(ok_gbar, st=g1 + 16) == binding.ABS_ERR_ALIAS
    assert nt(ok_gbar, bn=ok_gbar + 8) == binding.ABS_ERR_ALIAS
    assert nt(ok_gbar, st=ok_gbar + 4 * d - 16) == binding.ABS_ERR_ALIAS
    # fused: params/m/v against the gradients, gbar_out and each other
    p, m, v = A + 0x30000, A + 0x40000, A + 0x50000
    for bad in (dict(p=g0), dict(m=g1 + 4), dict(v=p), dict(m=p + 4 * (d - 1)), dict(gbar=v),
                dict(gbar=g0 + 400)):
        a = dict(p=p, m=m, v=v, gbar=ok_gbar)
        a.update(bad)
        args, hp = _fused_args(table, 2, d, 0, stats, a["gbar"], b_next, a["p"], a["m"], a["v"])
        assert L.abs_normtest_adamw(*args) == binding.ABS_ERR_ALIAS, bad
        assert L.abs_normtest_adamw_noalloc(*args) == binding.ABS_ERR_ALIAS, bad
    # the bf16 copy of the parameters (2-byte elements) against a gradient and against params
    for p16 in (g1 + 2 * (2 * d - 1), p + 4 * d - 2):
        args, hp = _fused_args(table, 2, d, 0, stats, ok_gbar, b_next, p, m, v)
        assert L.abs_normtest_adamw_mixed(*(args[:14] + [p16] + args[14:])) == binding.ABS_ERR_ALIAS
    # (ranges that merely touch are accepted: see test_cuda_failure_is_a_status_not_a_crash)
    # per-sample: gbar_out inside the matrix
    assert L.abs_persample_norm_test(A, 4, 10, 12, 0, 0.1, stats, A + 4 * 40, b_next,
                                     None) == binding.ABS_ERR_ALIAS


def test_combine_sums_adds_in_rank_order_and_decides(L):
    # three ranks whose sums only add up exactly in one order: 1e16 + 1 + 1 differs from
    # 1 + 1 + 1e16 in fp64
    rows = [(1e16, 2.0, 0.0), (1.0, 1.0, 0.0), (1.0, 1.0, 0.0)]
    out = binding.abs_combine_sums(rows, 2, 0.25, 3)
    assert out["n2"] == (1e16 + 1.0) + 1.0 == 1e16 and out["S"] == 4.0
    out = binding.abs_combine_sums(rows[::-1], 2, 0.25, 3)
    assert out["n2"] == (1.0 + 1.0) + 1e16 == 1e16 + 2.0
    # hand case H1 split over two ranks (coordinate 0 on rank 0, coordinate 1 on rank 1)
    c = json.load(open(GOLDEN))["norm_test"][0]
    assert c["n2"] == 8 and c["S"] == 4
    out = binding.abs_combine_sums([(4.0, 2.0, 10.0), (4.0, 2.0, 10.0)], 2, c["eta"], 3)
    assert (out["n2"], out["S"], out["Q"], out["T"], out["b_next"]) == (8.0, 4.0, 20.0, 4.0, 4)
    assert out["flags"] == binding.ABS_FLAG_VIOLATED
    b, T, flags = binding.abs_decide(4.0, 8.0, 2, c["eta"], 3)
    assert (b, T, flags) == (out["b_next"], out["T"], out["flags"])
    # a non-finite rank poisons the decision, the batch size is kept
    out = binding.abs_combine_sums([(4.0, 2.0, 0.0), (math.nan, 2.0, 0.0)], 2, 0.25, 3)
    assert out["flags"] == binding.ABS_FLAG_NONFINITE and out["b_next"] == 3
    assert L.abs_combine_sums(None, 2, 2.0, 0.25, 3, None, None, None) == -1
    one = (ctypes.c_double * 3)(1.0, 1.0, 1.0)
    assert L.abs_combine_sums(one, 0, 2.0, 0.25, 3, None, None, None) == -1


def test_noalloc_size_limit_is_a_host_check(L):
    """Problems that would not fit the array built into the library are refused before anything
    touches the GPU; abs_noalloc_fits answers the same question."""
    cap = binding.ABS_NOALLOC_MAX_CHUNKS
    assert binding.abs_noalloc_fits(1)
    assert binding.abs_noalloc_fits(cap * 8192)            # exactly the capacity
    assert not binding.abs_noalloc_fits(cap * 8192 + 1)
    assert not binding.abs_noalloc_fits(0)
    # shard cuts add ragged chunks: the same d no longer fits when every shard ends mid-chunk
    d = cap * 8192 - 5
    assert binding.abs_noalloc_fits(d)
    assert not binding.abs_noalloc_fits(d, [0, 1, 2, d])
    assert not binding.abs_noalloc_fits(100, [0, 50, 40, 100])   # invalid table
    table = (ctypes.c_void_p * 2)(FAKE, FAKE + 0x1000)
    hp = _hp()
    big = 1 << 50  # fabricated, far apart: the alias check is passed on the way
    rc = L.abs_normtest_adamw_noalloc(table, 2, cap * 8192 + 1, binding.ABS_BF16, None, 1, 0.1, 8,
                                      big, None, big + 64, 2 * big, 3 * big, 4 * big,
                                      ctypes.byref(hp), 1, None)
    assert rc == binding.ABS_ERR_TOO_LARGE
    assert "ABS_NOALLOC_MAX_CHUNKS" in L.abs_status_string(rc).decode()


class _FakeCudaTensor:
    """Just enough of a tensor for the binding's buffer checks (no GPU here)."""
    is_cuda = True

    def __init__(self, nbytes, ptr=0x10000, itemsize=8):
        self._n, self._ptr, self._sz = nbytes // itemsize, ptr, itemsize

    def numel(self):
        return self._n

    def element_size(self):
        return self._sz

    def is_contiguous(self):
        return True

    def data_ptr(self):
        return self._ptr


def test_binding_refuses_short_or_misplaced_stats_buffers(L):
    need = binding.abs_stats_bytes(1 << 20, 4)
    binding._check_stats(_FakeCudaTensor(need), need)
    with pytest.raises(ValueError, match="abs_stats_bytes"):
        binding._check_stats(_FakeCudaTensor(need - 8), need)
    # a header-only buffer (what the no-alloc call takes) handed to the plain call
    with pytest.raises(ValueError):
        binding._check_stats(_FakeCudaTensor(8 * (binding.ABS_STATS_HEADER + 4 * 4)), need)
    with pytest.raises(ValueError, match="aligned"):
        binding._check_stats(_FakeCudaTensor(need, ptr=0x10008), need)
    import torch
    with pytest.raises(TypeError):
        binding._check_stats(torch.zeros(need // 8, dtype=torch.float64), need)  # host memory
    with pytest.raises(TypeError):
        binding._check_b_next(torch.zeros(1, dtype=torch.int64))
    with pytest.raises(ValueError):
        binding._check_stats(_FakeCudaTensor(64), 0)


def test_cuda_failure_is_a_status_not_a_crash():
    """Valid arguments but no usable device: the first runtime call fails, the entry point
    returns ABS_ERR_CUDA, abs_last_cuda_error holds the code, nothing ran.  In a child process,
    so that the failed initialisation stays out of this one."""
    code = (
        "import ctypes, sys\n"
        "sys.path.insert(0, %r)\n"
        "from paper_2412_21124_b200 import binding as B\n"
        "L = B.lib()\n"
        "hp = B.abs_adamw_hparams(1e-3, 0.9, 0.999, 1e-8, 0.1)\n"
        "A = 0x100000\n"
        "rc = L.abs_adamw_step(A, A + 0x10000, A + 0x20000, A + 0x30000, 100, ctypes.byref(hp), 1, None)\n"
        "print(rc, L.abs_last_cuda_error())\n"
        "# buffers that touch end to start do not overlap: the alias check lets them through\n"
        "d = 1000\n"
        "table = (ctypes.c_void_p * 2)(A, A + 2 * d)\n"
        "rc = L.abs_norm_test(table, 2, d, 1, None, 1, 0.1, 8, A + 0x80000, A + 4 * d, A + 0x90000, None)\n"
        "print(rc, L.abs_last_cuda_error())\n" % ROOT)
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="")
    out = subprocess.check_output([sys.executable, "-c", code], env=env).decode().split()
    assert int(out[0]) == binding.ABS_ERR_CUDA and int(out[1]) != 0
    assert int(out[2]) == binding.ABS_ERR_CUDA and int(out[3]) != 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding._build, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.lib()
