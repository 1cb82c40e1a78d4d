"""GPU parity: the CUDA library, called through its C ABI, against the fp64 CPU oracle on
the same seeded inputs.  Sums within relative 1e-6, vectors within 1e-6*max|ref|, batch
size decisions bit-exact (inputs are reseeded until the oracle's T keeps a 1e-4 relative
margin from the threshold and from every integer)."""
import math

import numpy as np
import pytest
import torch

import paper_2412_21124_b200 as absnt
from oracle import abs_oracle as orc
from paper_2412_21124_b200 import synth
from tests.util import (assert_sum_close, assert_vec_close, f32, margin_ok, oracle_adamw,
                        to_host)

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
HP = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)
SENTINEL = -12345.5
GUARD = 64


@pytest.fixture(scope="module", autouse=True)
def _device():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    torch.cuda.set_device(0)
    absnt.binding.lib()  # raises if the CUDA library is missing
    yield
    torch.cuda.synchronize()


def guarded(n, dtype=torch.float32, shift=0):
    """An n-element view inside a sentinel-filled buffer; `shift` elements off alignment."""
    buf = torch.full((n + 2 * GUARD + shift,), SENTINEL, dtype=dtype, device=DEV)
    return buf, buf[GUARD + shift:GUARD + shift + n]


def check_guards(buf, n, shift=0):
    lo = buf[:GUARD + shift]
    hi = buf[GUARD + shift + n:]
    assert bool((lo == SENTINEL).all()) and bool((hi == SENTINEL).all()), "write outside the output"


def shifted_copy(t, shift):
    """A copy of t that starts `shift` elements past a 256-byte aligned address."""
    if shift == 0:
        return t
    buf = torch.empty(t.numel() + shift, dtype=t.dtype, device=t.device)
    v = buf[shift:]
    v.copy_(t)
    return v


def make_case(K, d, dtype, eta, b_cur, seed, sigma=0.05, noise="normal", shard_offsets=None):
    """Worker gradients whose oracle statistic respects the decision margin."""
    for attempt in range(8):
        grads = synth.worker_grads([d], K, dtype, seed + 1000 * attempt, DEV, sigma=sigma,
                                   noise=noise)
        ref = orc.norm_test([to_host(g) for g in grads], eta, b_cur, shard_offsets=shard_offsets)
        if margin_ok(ref["T"], b_cur):
            return grads, ref
    raise AssertionError("no seed met the decision margin")


def run_and_check(K, d, dtype, *, fused, eta=0.1, b_cur=64, seed=1, shard_offsets=None,
                  grad_shift=0, state_shift=0, zero_moments=True, step=1, want_gbar=True,
                  sigma=0.05, with_q=None):
    """One call through the C ABI, every output against the oracle.  The unfused test exists
    with and without the diagnostic Q (abs_norm_test_q / abs_norm_test): with_q=None runs
    both and returns the results of the one with Q."""
    if not fused and with_q is None:
        run_and_check(K, d, dtype, fused=False, eta=eta, b_cur=b_cur, seed=seed,
                      shard_offsets=shard_offsets, grad_shift=grad_shift, state_shift=state_shift,
                      sigma=sigma, with_q=False)
        with_q = True
    grads, ref = make_case(K, d, dtype, eta, b_cur, seed, sigma=sigma, shard_offsets=shard_offsets)
    grads = [shifted_copy(g, grad_shift) for g in grads]
    n_shards = 1 if shard_offsets is None else len(shard_offsets) - 1
    stats = absnt.alloc_stats(d, n_shards, DEV)
    gbuf, gbar = guarded(d, shift=state_shift)
    b_next = torch.full((1,), -7, dtype=torch.int64, device=DEV)
    if fused:
        p, m, v = synth.adam_state(d, seed + 17, DEV, zero_moments=zero_moments)
        p0, m0, v0 = to_host(p), to_host(m), to_host(v)
        bufs = []
        views = []
        for t in (p, m, v):
            b, w = guarded(d, shift=state_shift)
            w.copy_(t)
            bufs.append(b)
            views.append(w)
        absnt.abs_normtest_adamw(grads, eta, b_cur, stats, gbar if want_gbar else None, b_next,
                                 views[0], views[1], views[2], HP, step,
                                 shard_offsets=shard_offsets)
    else:
        entry = absnt.abs_norm_test_q if with_q else absnt.abs_norm_test
        entry(grads, eta, b_cur, stats, gbar, b_next, shard_offsets=shard_offsets)
    torch.cuda.synchronize()
    got = absnt.read_stats(stats, n_shards)

    assert_sum_close(got["n2"], ref["n2"], "n2")
    assert_sum_close(got["S"], ref["S"], "S")
    # only abs_norm_test_q computes Q; everywhere else its slots read NaN
    keys = ("n2", "S", "Q") if with_q else ("n2", "S")
    if with_q:
        assert_sum_close(got["Q"], ref["Q"], "Q")
    else:
        offs_ = shard_offsets if shard_offsets is not None else [0, d]
        assert math.isnan(got["Q"])
        for s_, rec in enumerate(got["shards"]):  # an empty shard has nothing to add: 0
            assert math.isnan(rec[2]) or (offs_[s_ + 1] == offs_[s_] and rec[2] == 0.0)
    assert got["norm"] == K
    assert got["T"] == pytest.approx(ref["T"], rel=3e-6)
    assert int(b_next.item()) == ref["b_next"]
    assert got["flags"] == ref["flags"]
    # header totals are the shard records added in shard order, exactly
    for j, key in enumerate(keys):
        acc = 0.0
        for rec in got["shards"]:
            acc += rec[j]
        assert acc == got[key]
    for s in range(n_shards):
        for j in range(len(keys)):
            r = ref["shards"][s, j]
            assert abs(got["shards"][s][j] - r) <= 1e-6 * abs(r) + 1e-300
    if want_gbar or not fused:
        assert_vec_close(gbar, ref["gbar"], "gbar")
        check_guards(gbuf, d, state_shift)
    else:
        assert bool((gbuf == SENTINEL).all())
    if fused:
        w_ref, m_ref, v_ref = oracle_adamw(orc, p0, m0, v0, ref["gbar"], HP, step)
        assert_vec_close(views[0], w_ref, "params")
        assert_vec_close(views[1], m_ref, "m")
        assert_vec_close(views[2], v_ref, "v")
        for b in bufs:
            check_guards(b, d, state_shift)
    return got, ref


# ----------------------------------------------------------------------------- config 1
def test_config1_unfused_then_adamw_and_fused():
    K, d, eta, b_cur = 4, 1 << 20, 0.1, 64
    grads, ref = make_case(K, d, torch.float32, eta, b_cur, seed=11)
    assert 150 < ref["T"] < 400  # sanity band of the generator: E[T] ~ 259
    p, m, v = synth.adam_state(d, 12, DEV, zero_moments=True)
    p0, m0, v0 = to_host(p), to_host(m), to_host(v)
    w_ref, m_ref, v_ref = oracle_adamw(orc, p0, m0, v0, ref["gbar"], HP, 1)

    stats = absnt.alloc_stats(d, 1, DEV)
    gbar = torch.empty(d, dtype=torch.float32, device=DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    absnt.abs_norm_test(grads, eta, b_cur, stats, gbar, b_next)
    absnt.abs_adamw_step(p, gbar, m, v, HP, 1)
    torch.cuda.synchronize()
    got = absnt.read_stats(stats)
    assert_sum_close(got["n2"], ref["n2"], "n2")
    assert_sum_close(got["S"], ref["S"], "S")
    assert int(b_next.item()) == ref["b_next"] and ref["b_next"] > b_cur
    assert got["flags"] == absnt.ABS_FLAG_VIOLATED
    assert_vec_close(gbar, ref["gbar"], "gbar")
    assert_vec_close(p, w_ref, "params")
    assert_vec_close(m, m_ref, "m")
    assert_vec_close(v, v_ref, "v")

    # the fused call gives bit-identical results to the two-call sequence
    p2 = torch.from_numpy(p0).to(DEV)
    m2 = torch.zeros_like(p2)
    v2 = torch.zeros_like(p2)
    stats2 = absnt.alloc_stats(d, 1, DEV)
    gbar2 = torch.empty_like(gbar)
    b_next2 = torch.zeros_like(b_next)
    absnt.abs_normtest_adamw(grads, eta, b_cur, stats2, gbar2, b_next2, p2, m2, v2, HP, 1)
    torch.cuda.synchronize()
    assert torch.equal(stats[:2], stats2[:2]) and torch.equal(stats[3:6], stats2[3:6])
    assert torch.equal(stats[8:10], stats2[8:10]) and torch.equal(b_next, b_next2)
    assert torch.equal(gbar, gbar2)
    assert torch.equal(p, p2) and torch.equal(m, m2) and torch.equal(v, v2)


# ------------------------------------------------------------------ K / dtype / raggedness
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("K", list(range(1, 33)))
def test_fused_all_K(K, dtype):
    run_and_check(K, 50_001, dtype, fused=True, seed=100 + K, zero_moments=(K % 2 == 0),
                  step=1 if K % 2 == 0 else 5)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("K", [2, 5, 6, 8, 9, 11, 12, 14, 15, 17, 21, 24, 29, 31, 32])
def test_unfused_some_K(K, dtype):
    run_and_check(K, 33_333, dtype, fused=False, seed=200 + K)


@pytest.mark.parametrize("d", [1, 2, 3, 7, 8, 9, 2047, 2048, 2049, 4095, 4096, 4097])
def test_tiny_and_boundary_lengths(d):
    run_and_check(2, d, torch.bfloat16, fused=True, seed=300 + d, b_cur=1)
    run_and_check(3, d, torch.float32, fused=True, seed=400 + d, b_cur=1)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("grad_shift,state_shift", [(1, 0), (0, 1), (3, 2)])
def test_misaligned_buffers(dtype, grad_shift, state_shift):
    run_and_check(4, 20_011, dtype, fused=True, seed=500, grad_shift=grad_shift,
                  state_shift=state_shift)
    run_and_check(4, 20_011, dtype, fused=False, seed=501, grad_shift=grad_shift,
                  state_shift=state_shift)


@pytest.mark.parametrize("K,dtype", [(32, torch.bfloat16), (32, torch.float32), (20, torch.float32)],
                         ids=["K32-bf16", "K32-f32", "K20-f32"])
def test_many_workers_ragged_and_misaligned(K, dtype):
    # the split kernels: vector rows, a ragged tail, and the element-wise path of shifted buffers
    run_and_check(K, 9_999, dtype, fused=True, seed=540 + K)
    run_and_check(K, 9_999, dtype, fused=True, seed=541 + K, grad_shift=1, state_shift=3)
    run_and_check(K, 9_999, dtype, fused=False, seed=542 + K, shard_offsets=[0, 5, 4101, 9_999])


@pytest.mark.parametrize("K,dtype", [(33, torch.bfloat16), (48, torch.float32), (64, torch.bfloat16),
                                     (64, torch.float32)]
                         + [(K, torch.bfloat16) for K in (36, 40, 44, 48, 52, 56, 60)]
                         + [(40, torch.float32), (47, torch.bfloat16)],
                         ids=lambda x: str(x).replace("torch.", ""))
def test_more_than_32_workers(K, dtype):
    """33..64 buffers (e.g. the J*M micro-batch gradients of a step): compile-time groups for
    bf16 multiples of four, run-time groups of 8 otherwise."""
    run_and_check(K, 2 * 4096 + 1_234, dtype, fused=True, seed=560 + K, zero_moments=False, step=3)
    run_and_check(K, 9_999, dtype, fused=False, seed=561 + K, shard_offsets=[0, 5, 4101, 9_999],
                  grad_shift=1 if K == 48 else 0)


@pytest.mark.parametrize("K,dtype", [(65, torch.bfloat16), (65, torch.float32), (100, torch.bfloat16),
                                     (128, torch.float32), (333, torch.bfloat16),
                                     (1024, torch.bfloat16), (1024, torch.float32)],
                         ids=lambda x: str(x).replace("torch.", ""))
def test_more_than_64_workers(K, dtype):
    """65..1024 buffers (4 workers x 256 accumulation steps is the largest layout of the paper's
    Table 5): the pointer table travels as a kernel parameter of its own."""
    d = 2 * 4096 + 1_234 if K <= 333 else 4096 + 321
    run_and_check(K, d, dtype, fused=True, seed=580 + K, zero_moments=False, step=3)
    run_and_check(K, d, dtype, fused=True, seed=581 + K, zero_moments=True, step=1,
                  grad_shift=1, state_shift=3)
    run_and_check(K, d, dtype, fused=False, seed=582 + K, shard_offsets=[0, 5, 4101, d])


def _random_case(i):
    rng = np.random.default_rng(9000 + i)
    K = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 9, 11, 13, 16, 17, 23, 24, 31, 32, 33, 47, 48, 63, 64]))
    d = int(rng.choice([1, 17, 255, 4096, 4097, 9_999, 40_000, 100_003, 262_144, 1_000_003]))
    if K > 16:
        d = min(d, 100_003)
    dtype = torch.bfloat16 if rng.integers(2) else torch.float32
    fused = bool(rng.integers(2))
    n_sh = int(rng.choice([1, 1, 2, 5, 17]))
    offs = None
    if n_sh > 1 and d >= n_sh:
        cuts = sorted(int(c) for c in rng.integers(0, d + 1, size=n_sh - 1))
        offs = [0] + cuts + [d]
    grad_shift = int(rng.choice([0, 0, 0, 1, 3]))
    state_shift = int(rng.choice([0, 0, 1]))
    return K, d, dtype, fused, offs, grad_shift, state_shift


@pytest.mark.parametrize("i", range(40))
def test_randomized_configurations(i):
    """Seeded random draws over worker count, length, dtype, entry point, ragged shard cuts
    (empty shards included) and buffer alignment: every combination goes through the same
    element-by-element comparison with the oracle."""
    K, d, dtype, fused, offs, grad_shift, state_shift = _random_case(i)
    run_and_check(K, d, dtype, fused=fused, seed=9100 + i, shard_offsets=offs, grad_shift=grad_shift,
                  state_shift=state_shift, zero_moments=bool(i % 2), step=1 + (i % 7))


def test_fused_without_gbar_output():
    run_and_check(8, 40_000, torch.bfloat16, fused=True, seed=600, want_gbar=False)


def test_large_d_uses_bigger_chunks():
    # d >= 2^23 switches the reduction chunk; several chunks plus a ragged tail
    got, _ = run_and_check(2, (1 << 23) + 12_345, torch.bfloat16, fused=True, seed=650,
                           zero_moments=False, step=9)
    assert got["n_chunks"] == 1026  # 8192 per chunk in the fused call
    got, _ = run_and_check(2, (1 << 23) + 12_345, torch.bfloat16, fused=False, seed=651)
    assert got["n_chunks"] == 513   # 16384 per chunk in the unfused test


# ----------------------------------------------------------------------------- shards
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_ragged_shards(dtype):
    d = 60_013
    offs = [0, 1, 4097, 4097, 12_289, 30_000, 30_003, d]  # odd starts, one empty shard
    got, ref = run_and_check(4, d, dtype, fused=True, seed=700, shard_offsets=offs)
    assert got["shards"][2][:2] == (0.0, 0.0)
    got, ref = run_and_check(4, d, dtype, fused=False, seed=701, shard_offsets=offs)
    assert got["shards"][2] == (0.0, 0.0, 0.0)   # the results of abs_norm_test_q


def test_shards_spanning_several_record_slices():
    # chunk counts 1, 128, 129, 0, 257 and a ragged rest: the final reduction cuts each shard's
    # chunk records into slices of 128, so these sit on both sides of every slice boundary
    c = 4096
    offs = [0, c, 129 * c, 258 * c, 258 * c, 515 * c, 515 * c + 700 * c + 77]
    d = offs[-1]
    got, _ = run_and_check(2, d, torch.bfloat16, fused=True, seed=705, shard_offsets=offs)
    assert got["n_chunks"] == 1 + 128 + 129 + 257 + 701
    run_and_check(3, d, torch.float32, fused=False, seed=706, shard_offsets=offs)


def test_equal_shards_and_max_shards():
    d = 100_000
    run_and_check(8, d, torch.bfloat16, fused=False, seed=710,
                  shard_offsets=synth.equal_shard_offsets(d, 8))
    run_and_check(2, d, torch.float32, fused=True, seed=711,
                  shard_offsets=synth.equal_shard_offsets(d, absnt.binding.ABS_MAX_SHARDS))


def test_sharding_does_not_change_gbar_or_update():
    K, d = 4, 70_001
    grads, _ = make_case(K, d, torch.bfloat16, 0.1, 64, seed=720)
    outs = []
    for offs in (None, synth.equal_shard_offsets(d, 5)):
        n_sh = 1 if offs is None else 5
        p, m, v = synth.adam_state(d, 721, DEV, zero_moments=False)
        stats = absnt.alloc_stats(d, n_sh, DEV)
        gbar = torch.empty(d, dtype=torch.float32, device=DEV)
        b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
        absnt.abs_normtest_adamw(grads, 0.1, 64, stats, gbar, b_next, p, m, v, HP, 4,
                                 shard_offsets=offs)
        outs.append((gbar, p, m, v, absnt.read_stats(stats, n_sh), int(b_next.item())))
    for a, b in zip(outs[0][:4], outs[1][:4]):
        assert torch.equal(a, b)
    assert outs[0][4]["S"] == pytest.approx(outs[1][4]["S"], rel=1e-7)  # row grouping differs
    assert outs[0][5] == outs[1][5]


def test_prepared_fused_step_matches_plain_call():
    K, d = 4, 30_001
    grads, _ = make_case(K, d, torch.bfloat16, 0.1, 64, seed=760)
    outs = []
    for prepared in (False, True):
        p, m, v = synth.adam_state(d, 761, DEV, zero_moments=False)
        stats = absnt.alloc_stats(d, 1, DEV)
        gbar = torch.empty(d, dtype=torch.float32, device=DEV)
        b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
        if prepared:
            step = absnt.FusedStep(grads, stats, gbar, b_next, p, m, v, HP)
            step.run(0.1, 64, 4)
        else:
            absnt.abs_normtest_adamw(grads, 0.1, 64, stats, gbar, b_next, p, m, v, HP, 4)
        torch.cuda.synchronize()
        outs.append((stats[:2].clone(), gbar, p, m, v, b_next))
    for a, b in zip(*outs):
        assert torch.equal(a, b)
    # the prepared object with a bf16 copy of the parameters
    p, m, v = synth.adam_state(d, 761, DEV, zero_moments=False)
    p16 = torch.zeros(d, dtype=torch.bfloat16, device=DEV)
    step = absnt.FusedStep(grads, stats, gbar, b_next, p, m, v, HP, params_bf16_out=p16)
    step.run(0.1, 64, 4)
    torch.cuda.synchronize()
    assert torch.equal(p, outs[0][2]) and torch.equal(p16, p.to(torch.bfloat16))


def test_calls_can_be_captured_in_a_cuda_graph():
    """The library only enqueues kernels on the caller's stream, so a sequence of calls can be
    captured once and replayed (how a launch-bound small-d loop avoids per-call host cost)."""
    K, d = 4, 200_003
    grads, ref = make_case(K, d, torch.bfloat16, 0.1, 64, seed=770)
    p, m, v = synth.adam_state(d, 771, DEV, zero_moments=False)
    p0, m0, v0 = p.clone(), m.clone(), v.clone()
    stats = absnt.alloc_stats(d, 1, DEV)
    gbar = torch.empty(d, dtype=torch.float32, device=DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    # eager reference (also the first, un-captured call of every kernel involved)
    absnt.abs_normtest_adamw(grads, 0.1, 64, stats, gbar, b_next, p, m, v, HP, 4)
    absnt.abs_adamw_step(p, gbar, m, v, HP, 5)
    torch.cuda.synchronize()
    want = (stats[:2].clone(), gbar.clone(), p.clone(), m.clone(), v.clone(), b_next.clone())
    for t, t0 in ((p, p0), (m, m0), (v, v0)):
        t.copy_(t0)
    gbar.zero_()
    b_next.zero_()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            absnt.abs_normtest_adamw(grads, 0.1, 64, stats, gbar, b_next, p, m, v, HP, 4)
            absnt.abs_adamw_step(p, gbar, m, v, HP, 5)
    torch.cuda.current_stream().wait_stream(side)
    for t, t0 in ((p, p0), (m, m0), (v, v0)):  # capture does not execute; start from the same state
        t.copy_(t0)
    graph.replay()
    torch.cuda.synchronize()
    got = (stats[:2], gbar, p, m, v, b_next)
    for a, b in zip(got, want):
        assert torch.equal(a, b)
    assert int(b_next.item()) == ref["b_next"]


# ------------------------------------------------------------------------- determinism
def test_bit_identical_across_runs():
    K, d = 8, 3_000_017
    grads, _ = make_case(K, d, torch.bfloat16, 0.1, 512, seed=800)
    res = []
    for _ in range(3):
        p, m, v = synth.adam_state(d, 801, DEV, zero_moments=False)
        stats = absnt.alloc_stats(d, 1, DEV)
        gbar = torch.empty(d, dtype=torch.float32, device=DEV)
        b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
        absnt.abs_normtest_adamw(grads, 0.1, 512, stats, gbar, b_next, p, m, v, HP, 2)
        torch.cuda.synchronize()
        res.append((stats[:2].clone(), stats[3:6].clone(), gbar, p, m, v, b_next))
    for r in res[1:]:
        for a, b in zip(res[0], r):
            assert torch.equal(a, b)


# --------------------------------------------------------------------- degenerate inputs
@pytest.mark.parametrize("K", [2, 3, 4, 5, 8])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_identical_buffers_keep_batch_size(K, dtype):
    d = 10_001
    g = synth.worker_grads([d], 1, dtype, 900 + K, DEV)[0]
    grads = [g.clone() for _ in range(K)]
    stats = absnt.alloc_stats(d, 1, DEV)
    gbar = torch.empty(d, dtype=torch.float32, device=DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    absnt.abs_norm_test_q(grads, 0.1, 77, stats, gbar, b_next)
    got = absnt.read_stats(stats)
    assert got["S"] == 0.0 and got["T"] == 0.0 and got["flags"] == 0
    assert int(b_next.item()) == 77
    assert torch.equal(gbar, g.float())
    assert got["Q"] == pytest.approx(K * got["n2"], rel=1e-6)  # fp32 row partials


def test_degenerate_and_nonfinite_flags():
    d = 5000
    z = torch.zeros(d, dtype=torch.float32, device=DEV)
    stats = absnt.alloc_stats(d, 1, DEV)
    gbar = torch.empty(d, dtype=torch.float32, device=DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)

    absnt.abs_norm_test([z, z, z], 0.1, 9, stats, gbar, b_next)
    got = absnt.read_stats(stats)
    assert got["flags"] == absnt.ABS_FLAG_DEGENERATE and math.isnan(got["T"])
    assert int(b_next.item()) == 9

    a = synth.worker_grads([d], 1, torch.float32, 950, DEV)[0]
    absnt.abs_norm_test([a, -a], 0.1, 9, stats, gbar, b_next)
    got = absnt.read_stats(stats)
    assert got["flags"] == absnt.ABS_FLAG_DEGENERATE | absnt.ABS_FLAG_VIOLATED
    assert got["T"] == math.inf and int(b_next.item()) == 2 ** 63 - 1
    assert not gbar.any()

    for bad in (math.inf, math.nan):
        c = a.clone()
        c[1234] = bad
        absnt.abs_norm_test([a, c], 0.1, 9, stats, gbar, b_next)
        got = absnt.read_stats(stats)
        assert got["flags"] & absnt.ABS_FLAG_NONFINITE and int(b_next.item()) == 9


def test_identity_Q_minus_K_n2_on_device_sums():
    for K, dtype in ((4, torch.float32), (8, torch.bfloat16), (32, torch.bfloat16)):
        got, _ = run_and_check(K, 123_457, dtype, fused=False, seed=980 + K)
        assert got["S"] == pytest.approx(got["Q"] - K * got["n2"], rel=2e-6)


def test_eta_sweep_decisions_and_host_decide():
    K, d, b_cur = 8, 200_003, 1024
    grads = synth.worker_grads([d], K, torch.bfloat16, 990, DEV, noise="student_t3")
    host = [to_host(g) for g in grads]
    stats = absnt.alloc_stats(d, 1, DEV)
    gbar = torch.empty(d, dtype=torch.float32, device=DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    seen = []
    for eta in (0.05, 0.1, 0.2, 0.4, 1.5):
        ref = orc.norm_test(host, eta, b_cur, want_gbar=False)
        if not margin_ok(ref["T"], b_cur):
            continue
        absnt.abs_norm_test(grads, eta, b_cur, stats, gbar, b_next)
        got = absnt.read_stats(stats)
        assert int(b_next.item()) == ref["b_next"]
        # the host-side decision from the device sums agrees with the device decision
        hb, hT, hflags = absnt.abs_decide(got["S"], got["n2"], K, eta, b_cur)
        assert hb == int(b_next.item()) and hT == got["T"] and hflags == got["flags"]
        seen.append(ref["b_next"])
    assert len(seen) >= 3 and seen == sorted(seen, reverse=True)


# -------------------------------------------------------------------- stand-alone AdamW
@pytest.mark.parametrize("d,shift", [(1, 0), (5, 0), (4096, 0), (100_003, 0), (100_003, 1),
                                     (77_777, 3)])
def test_adamw_step_sequence(d, shift):
    p, m, v = synth.adam_state(d, 1100 + d % 97, DEV, zero_moments=True)
    bufs, views = [], []
    for t in (p, m, v):
        b, w = guarded(d, shift=shift)
        w.copy_(t)
        bufs.append(b)
        views.append(w)
    for step in (1, 2, 3):
        g = shifted_copy(synth.worker_grads([d], 1, torch.float32, 1200 + step, DEV)[0], shift)
        p0, m0, v0 = (to_host(x) for x in views)
        absnt.abs_adamw_step(views[0], g, views[1], views[2], HP, step)
        torch.cuda.synchronize()
        w_ref, m_ref, v_ref = oracle_adamw(orc, p0, m0, v0, to_host(g).astype(np.float64), HP, step)
        assert_vec_close(views[0], w_ref, "params")
        assert_vec_close(views[1], m_ref, "m")
        assert_vec_close(views[2], v_ref, "v")
    for b in bufs:
        check_guards(b, d, shift)


@pytest.mark.parametrize("shift", [0, 1])
def test_adamw_step_large_vector(shift):
    """From 2^25 coordinates on the update runs as the one-worker fused kernel (bulk-staged, with
    its element-wise path for a misaligned vector): plain, clipped and with the bf16 copy, against
    the oracle; and the clipped update agrees bit for bit with the small-vector kernel's on the
    same values."""
    d = (1 << 25) + 4097
    g = shifted_copy(synth.worker_grads([d], 1, torch.float32, 1290, DEV)[0], shift)
    p, m, v = (shifted_copy(t, shift) for t in synth.adam_state(d, 1291, DEV, zero_moments=False))
    p0, m0, v0 = to_host(p), to_host(m), to_host(v)
    g64 = to_host(g).astype(np.float64)
    absnt.abs_adamw_step(p, g, m, v, HP, 7)
    torch.cuda.synchronize()
    w_ref, m_ref, v_ref = oracle_adamw(orc, p0, m0, v0, g64, HP, 7)
    assert_vec_close(p, w_ref, "params")
    assert_vec_close(m, m_ref, "m")
    assert_vec_close(v, v_ref, "v")
    # clipped, with the bf16 copy; n2 comes from a stats header as a norm test would write it
    n2 = float((g.double() ** 2).sum())
    stats = torch.zeros(absnt.binding.ABS_STATS_HEADER, dtype=torch.float64, device=DEV)
    stats[absnt.binding.ABS_STAT_N2] = n2
    p16 = torch.zeros(d, dtype=torch.bfloat16, device=DEV)
    p1, m1, v1 = to_host(p), to_host(m), to_host(v)
    absnt.abs_adamw_step_mixed(p, g, m, v, p16, HP, 8, max_norm=1.0, stats_in=stats)
    torch.cuda.synchronize()
    assert orc.clip_scale(n2, 1.0) < 1.0
    w_ref, m_ref, v_ref = orc.adamw_clipped(p1, m1, v1, g64, f32(HP["lr"]), f32(HP["beta1"]),
                                            f32(HP["beta2"]), f32(HP["eps"]),
                                            f32(HP["weight_decay"]), 8, 1.0, n2)
    assert_vec_close(p, w_ref, "params")
    assert_vec_close(m, m_ref, "m")
    assert_vec_close(v, v_ref, "v")
    assert np.array_equal(bf16_bits(p16), orc.bf16_round(to_host(p)))
    # the first 100,000 coordinates through the small-vector kernel: identical bits
    n = 100_000
    q, mq, vq = (torch.from_numpy(x[:n].copy()).to(DEV) for x in (p1, m1, v1))
    absnt.abs_adamw_step_clipped(q, g[:n].clone(), mq, vq, HP, 8, 1.0, stats)
    torch.cuda.synchronize()
    assert torch.equal(q, p[:n]) and torch.equal(mq, m[:n]) and torch.equal(vq, v[:n])


@pytest.mark.parametrize("max_norm", [1.0, 0.05, 1e3])
@pytest.mark.parametrize("d,shift", [(100_003, 0), (50_001, 1)])
def test_norm_test_then_clipped_adamw(max_norm, d, shift):
    """Clipping by global norm (what the paper's experiments add to Algorithm 1): the norm
    test writes gbar and ||gbar||^2, the clipped update reads both on the device."""
    K, eta, b_cur, step = 4, 0.1, 64, 6
    grads, ref = make_case(K, d, torch.bfloat16, eta, b_cur, seed=1250 + d % 7)
    p, m, v = synth.adam_state(d, 1251, DEV, zero_moments=False)
    bufs, views = [], []
    for t in (p, m, v):
        b, w = guarded(d, shift=shift)
        w.copy_(t)
        bufs.append(b)
        views.append(w)
    p0, m0, v0 = (to_host(x) for x in views)
    stats = absnt.alloc_stats(d, 1, DEV)
    gbar = torch.empty(d, dtype=torch.float32, device=DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    absnt.abs_norm_test(grads, eta, b_cur, stats, gbar, b_next)
    absnt.abs_adamw_step_clipped(views[0], gbar, views[1], views[2], HP, step, max_norm, stats)
    torch.cuda.synchronize()
    scale = orc.clip_scale(ref["n2"], max_norm)
    assert (scale < 1.0) == (max_norm < 1e3)
    w_ref, m_ref, v_ref = orc.adamw_clipped(p0, m0, v0, ref["gbar"], f32(HP["lr"]), f32(HP["beta1"]),
                                            f32(HP["beta2"]), f32(HP["eps"]),
                                            f32(HP["weight_decay"]), step, max_norm, ref["n2"])
    assert_vec_close(views[0], w_ref, "params")
    assert_vec_close(views[1], m_ref, "m")
    assert_vec_close(views[2], v_ref, "v")
    for b in bufs:
        check_guards(b, d, shift)
    if max_norm == 1e3:  # inactive clipping is the plain update, bit for bit
        q, mq, vq = (torch.from_numpy(x).to(DEV) for x in (p0, m0, v0))
        absnt.abs_adamw_step(q, gbar, mq, vq, HP, step)
        assert torch.equal(q, views[0]) and torch.equal(mq, views[1]) and torch.equal(vq, views[2])


@pytest.mark.parametrize("K,dtype,d", [(8, torch.bfloat16, 5 * 8192 + 777), (4, torch.float32, 50_001),
                                       (12, torch.float32, 33_000), (32, torch.bfloat16, 20_481),
                                       (100, torch.bfloat16, 9_999)],
                         ids=["k8-bf16", "k4-f32", "k12-f32", "k32-bf16", "k100-bf16"])
def test_fused_step_clipped_by_the_previous_norm(K, dtype, d):
    """abs_normtest_adamw_clip_prev over three steps: step 1 unclipped (no previous norm), steps
    2 and 3 clipped by the norm the step before wrote into the same stats buffer.  The oracle
    clips by its own previous n2; the test's statistics stay those of the unclipped gradient."""
    eta, b_cur, max_norm = 0.1, 64, 0.5
    p, m, v = synth.adam_state(d, 1701, DEV, zero_moments=True)
    ph, mh, vh = to_host(p), to_host(m), to_host(v)
    stats = absnt.alloc_stats(d, 1, DEV)
    gbar = torch.empty(d, dtype=torch.float32, device=DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    n2_prev, clipped_steps = None, 0
    for step in (1, 2, 3):
        grads, ref = make_case(K, d, dtype, eta, b_cur, seed=1700 + 10 * step + K)
        absnt.abs_normtest_adamw_clip_prev(grads, eta, b_cur, stats, gbar, b_next, p, m, v, HP, step,
                                           max_norm, stats if step > 1 else None)
        torch.cuda.synchronize()
        got = absnt.read_stats(stats)
        assert_sum_close(got["n2"], ref["n2"], "n2")
        assert_sum_close(got["S"], ref["S"], "S")
        assert int(b_next.item()) == ref["b_next"]
        assert_vec_close(gbar, ref["gbar"], "gbar")
        hp = [f32(HP[k]) for k in ("lr", "beta1", "beta2", "eps", "weight_decay")]
        if n2_prev is None:
            w_ref, m_ref, v_ref = orc.adamw(ph, mh, vh, ref["gbar"], *hp, step)
        else:
            clipped_steps += orc.clip_scale(n2_prev, max_norm) < 1.0
            w_ref, m_ref, v_ref = orc.adamw_clipped(ph, mh, vh, ref["gbar"], *hp, step, max_norm,
                                                    n2_prev)
        assert_vec_close(p, w_ref, "params")
        assert_vec_close(m, m_ref, "m")
        assert_vec_close(v, v_ref, "v")
        # the next step starts from the library's stored state and the oracle's previous norm
        ph, mh, vh = to_host(p), to_host(m), to_host(v)
        n2_prev = ref["n2"]
    assert clipped_steps == 2  # ||gbar|| is about 0.05 sqrt(d/K) + ..., well above 0.5
    # a threshold the norm does not reach: the plain fused step, bit for bit
    q, mq, vq = p.clone(), m.clone(), v.clone()
    stats2 = absnt.alloc_stats(d, 1, DEV)
    absnt.abs_normtest_adamw_clip_prev(grads, eta, b_cur, stats2, gbar, b_next, q, mq, vq, HP, 4,
                                       1e9, stats)
    absnt.abs_normtest_adamw(grads, eta, b_cur, stats, gbar, b_next, p, m, v, HP, 4)
    torch.cuda.synchronize()
    assert torch.equal(p, q) and torch.equal(m, mq) and torch.equal(v, vq)
    assert torch.equal(stats[:2], stats2[:2])


# ------------------------------------------------------------------- mixed precision
def bf16_bits(t):
    return t.detach().cpu().view(torch.int16).numpy().view(np.uint16)


def guarded_bf16(n, shift=0):
    buf = torch.full((n + 2 * GUARD + shift,), 7.0, dtype=torch.bfloat16, device=DEV)
    return buf, buf[GUARD + shift:GUARD + shift + n]


def check_bf16_copy(p16_buf, p16, p_f32, n, shift):
    """The bf16 copy is the stored fp32 value rounded to nearest even, bit for bit (the oracle
    decides the code from the same fp32 value the kernel rounded), and nothing else was written."""
    want = orc.bf16_round(to_host(p_f32))
    assert np.array_equal(bf16_bits(p16), want)
    assert bool((p16_buf[:GUARD + shift] == 7.0).all())
    assert bool((p16_buf[GUARD + shift + n:] == 7.0).all())


@pytest.mark.parametrize("K,dtype,d,offs,shift", [
    (8, torch.bfloat16, 5 * 8192 + 777, None, 0),        # staged kernel + ragged last chunk
    (8, torch.bfloat16, 3 * 8192, None, 1),              # copy off 16-byte alignment: scalar rows
    (4, torch.float32, 50_001, [0, 5, 20_000, 50_001], 0),
    (2, torch.bfloat16, 70_003, None, 0),                # 256-bit stores
    (5, torch.bfloat16, 33_000, None, 0),
    (32, torch.bfloat16, 20_481, None, 0),               # split kernel
    (20, torch.float32, 9_999, None, 0),
], ids=["k8", "k8-shifted", "k4-f32-shards", "k2", "k5", "k32", "k20-f32"])
def test_mixed_precision_fused_step(K, dtype, d, offs, shift):
    """abs_normtest_adamw_mixed = abs_normtest_adamw bit for bit, plus the bf16 copy."""
    eta, b_cur, step = 0.1, 64, 5
    grads, ref = make_case(K, d, dtype, eta, b_cur, seed=1600 + K, shard_offsets=offs)
    n_sh = 1 if offs is None else len(offs) - 1
    outs = []
    for mixed in (False, True):
        p, m, v = synth.adam_state(d, 1601, DEV, zero_moments=False)
        stats = absnt.alloc_stats(d, n_sh, DEV)
        gbar = torch.empty(d, dtype=torch.float32, device=DEV)
        b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
        if mixed:
            p16_buf, p16 = guarded_bf16(d, shift)
            absnt.abs_normtest_adamw_mixed(grads, eta, b_cur, stats, gbar, b_next, p, m, v, p16, HP,
                                           step, shard_offsets=offs)
        else:
            absnt.abs_normtest_adamw(grads, eta, b_cur, stats, gbar, b_next, p, m, v, HP, step,
                                     shard_offsets=offs)
        torch.cuda.synchronize()
        outs.append((p, m, v, gbar, absnt.read_stats(stats, n_sh), int(b_next.item())))
    for a, b in zip(outs[0][:4], outs[1][:4]):
        assert torch.equal(a, b)
    # an output off 16-byte alignment moves the rows to the element-wise path, whose partial sums
    # group differently (same values, different fp32 row grouping)
    rel = 0.0 if shift == 0 else 1e-7
    for key in ("n2", "S"):
        assert abs(outs[0][4][key] - outs[1][4][key]) <= rel * outs[0][4][key]
    assert outs[0][5] == outs[1][5] == ref["b_next"]
    check_bf16_copy(p16_buf, p16, outs[1][0], d, shift)
    assert np.array_equal(bf16_bits(p16), bf16_bits(outs[1][0].to(torch.bfloat16)))


@pytest.mark.parametrize("d,shift,clip", [(100_003, 0, False), (100_003, 1, False), (4096, 0, True),
                                          (50_001, 3, True), (7, 0, False)])
def test_mixed_precision_adamw_step(d, shift, clip):
    grads, ref = make_case(4, d, torch.float32, 0.1, 64, seed=1650 + d % 5)
    stats = absnt.alloc_stats(d, 1, DEV)
    gbar = torch.empty(d, dtype=torch.float32, device=DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    absnt.abs_norm_test(grads, 0.1, 64, stats, gbar, b_next)
    p, m, v = synth.adam_state(d, 1651, DEV, zero_moments=False)
    q, mq, vq = p.clone(), m.clone(), v.clone()
    p16_buf, p16 = guarded_bf16(d, shift)
    if clip:
        absnt.abs_adamw_step_clipped(q, gbar, mq, vq, HP, 3, 0.05, stats)
        absnt.abs_adamw_step_mixed(p, gbar, m, v, p16, HP, 3, max_norm=0.05, stats_in=stats)
    else:
        absnt.abs_adamw_step(q, gbar, mq, vq, HP, 3)
        absnt.abs_adamw_step_mixed(p, gbar, m, v, p16, HP, 3)
    torch.cuda.synchronize()
    assert torch.equal(p, q) and torch.equal(m, mq) and torch.equal(v, vq)
    check_bf16_copy(p16_buf, p16, p, d, shift)


# --------------------------------------------------------------------- per-sample form
def persample_check(G, eta):
    b, d = G.shape
    stats = absnt.alloc_persample_stats(b, d, DEV)
    gbuf, gbar = guarded(d)
    b_next = torch.full((1,), -7, dtype=torch.int64, device=DEV)
    absnt.abs_persample_norm_test(G, eta, stats, gbar, b_next)
    torch.cuda.synchronize()
    got = absnt.read_stats(stats)
    Gh = G.detach().cpu()
    if Gh.dtype == torch.bfloat16:   # the oracle takes bf16 as uint16 bit patterns
        Gh = Gh.view(torch.int16).numpy().view(np.uint16)
    else:
        Gh = Gh.numpy()
    ref = orc.persample(Gh, eta)
    assert_sum_close(got["n2"], ref["n2"], "n2")
    assert_sum_close(got["S"], ref["S"], "S")
    assert math.isnan(got["Q"])   # the per-sample call does not compute the diagnostic
    assert got["norm"] == b - 1
    assert got["T"] == pytest.approx(ref["T"], rel=3e-6)
    assert_vec_close(gbar, ref["gbar"], "gbar")
    check_guards(gbuf, d)
    if margin_ok(ref["T"], b):
        assert int(b_next.item()) == ref["b_next"]
        assert got["flags"] == ref["flags"]
    return got, ref, int(b_next.item())


@pytest.mark.parametrize("b,d,ld,shift", [(2, 5, 5, 0), (7, 4100, 4100, 0), (32, 1000, 1000, 0),
                                          (33, 300, 320, 0), (100, 2051, 2052, 1),
                                          (257, 4096, 4096, 0), (1000, 777, 800, 0),
                                          (2049, 515, 516, 0),
                                          (130, 700, 700, 0),      # few rows per row block
                                          (4096, 1000, 1000, 0),   # narrow and tall: many row blocks
                                          (1500, 300, 304, 2),     # the same, rows misaligned, ragged last block
                                          (65, 40_000, 40_000, 0)])
def test_persample_shapes(b, d, ld, shift):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(b * 131 + d)
    buf = torch.empty(b * ld + shift, dtype=torch.float32, device=DEV)
    buf.normal_(generator=gen)
    buf.mul_(0.3).add_(0.02)
    G = buf[shift:].view(b, ld)[:, :d]
    persample_check(G, 0.1)


@pytest.mark.parametrize("b,d,ld,shift", [(2, 5, 5, 0), (7, 4100, 4100, 0), (33, 300, 320, 0),
                                          (100, 2051, 2052, 1),    # rows off the 8-byte boundary
                                          (257, 4096, 4096, 0), (1000, 777, 780, 0),
                                          (2049, 515, 516, 0), (4096, 1000, 1000, 0),
                                          (1500, 300, 302, 0),     # odd row pitch: element loads
                                          (65, 40_000, 40_000, 0)])
def test_persample_bf16_shapes(b, d, ld, shift):
    """bfloat16 per-sample gradients (the paper trains in bfloat16): same sums, exact widening."""
    gen = torch.Generator(device=DEV)
    gen.manual_seed(b * 137 + d)
    buf = torch.empty(b * ld + shift, dtype=torch.float32, device=DEV)
    buf.normal_(generator=gen)
    buf.mul_(0.3).add_(0.02)
    G = buf.to(torch.bfloat16)[shift:].view(b, ld)[:, :d]
    persample_check(G, 0.1)


def test_persample_identical_and_cancelling_rows_are_exact():
    """Column sums are carried in fp64 and divided once: identical rows give their common value
    as the mean, bit for bit, with S = 0; rows that cancel in pairs give a mean of exactly zero
    (n2 = 0, T = +inf: DEGENERATE | VIOLATED), as the oracle's plain sums do."""
    gen = torch.Generator(device=DEV)
    gen.manual_seed(77)
    for dtype in (torch.float32, torch.bfloat16):
        for b, d in ((48, 1000), (1100, 515)):
            row = (torch.empty(d, device=DEV).normal_(generator=gen) * 0.3).to(dtype)
            G = row.repeat(b, 1).contiguous()
            got, ref, b_next = persample_check(G, 0.1)
            assert got["S"] == 0.0 and got["T"] == 0.0 and b_next == b
            half = (torch.empty(b // 2, d, device=DEV).normal_(generator=gen) * 0.3).to(dtype)
            G = torch.cat([half, -half]).contiguous()
            got, ref, b_next = persample_check(G, 0.1)
            assert got["n2"] == 0.0 and got["T"] == math.inf and b_next == 2 ** 63 - 1
            assert got["flags"] == absnt.ABS_FLAG_DEGENERATE | absnt.ABS_FLAG_VIOLATED


def test_persample_stats_buffer_is_reusable_and_calls_are_bit_identical():
    """The call counts its thread blocks off in ticket counters kept in stats_out and leaves them
    at zero: the same buffer serves call after call (here also inside a captured graph), and
    which block happens to do a merge does not change a bit of the result."""
    b, d = 777, 5000
    gen = torch.Generator(device=DEV)
    gen.manual_seed(5)
    G = torch.empty(b, d, dtype=torch.float32, device=DEV).normal_(generator=gen).mul_(0.3).add_(0.02)
    stats = absnt.alloc_persample_stats(b, d, DEV)
    gbar = torch.empty(d, dtype=torch.float32, device=DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    outs = []
    for _ in range(4):
        gbar.fill_(-1.0)
        absnt.abs_persample_norm_test(G, 0.1, stats, gbar, b_next)
        torch.cuda.synchronize()
        outs.append((stats[:12].clone(), gbar.clone(), b_next.clone()))
    for o in outs[1:]:
        assert torch.equal(o[0].view(torch.int64), outs[0][0].view(torch.int64))
        assert torch.equal(o[1], outs[0][1]) and torch.equal(o[2], outs[0][2])
    ref = orc.persample(G.cpu().numpy(), 0.1)
    assert_sum_close(float(outs[0][0][1]), ref["S"], "S")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            absnt.abs_persample_norm_test(G, 0.1, stats, gbar, b_next)
            absnt.abs_persample_norm_test(G, 0.1, stats, gbar, b_next)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        gbar.fill_(-1.0)
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(stats[:12].view(torch.int64), outs[0][0].view(torch.int64))
        assert torch.equal(gbar, outs[0][1])
    # the same buffer, now full of another shape's records, serves a smaller problem as it is
    G2 = G[:300, :1234].contiguous()
    gbar2 = torch.empty(1234, dtype=torch.float32, device=DEV)
    absnt.abs_persample_norm_test(G2, 0.1, stats, gbar2, b_next)
    torch.cuda.synchronize()
    ref2 = orc.persample(G2.cpu().numpy(), 0.1)
    assert_sum_close(float(stats[1]), ref2["S"], "S")
    assert_sum_close(float(stats[0]), ref2["n2"], "n2")
    assert_vec_close(gbar2, ref2["gbar"], "gbar")


def test_persample_more_rows_than_one_grid_dimension_of_512_row_blocks():
    """b above 65535 x 512 rows: the row blocks must grow past 512 rows to fit the grid."""
    b, d, ld = 65535 * 512 + 70_001, 3, 4
    gen = torch.Generator(device=DEV)
    gen.manual_seed(99)
    buf = torch.empty(b * ld, dtype=torch.float32, device=DEV)
    buf.normal_(generator=gen)
    buf.mul_(0.3).add_(0.05)
    persample_check(buf.view(b, ld)[:, :d], 0.1)


def test_persample_matches_worker_form_factor():
    K, d = 8, 30_001
    grads, ref = make_case(K, d, torch.float32, 0.1, 1, seed=1300)
    G = torch.stack(grads)
    got, _, _ = persample_check(G, 0.1)
    assert got["T"] == pytest.approx(ref["T"] * K / (K - 1), rel=3e-6)


@pytest.mark.parametrize("b", [32, 256, 1024, 4096])
def test_persample_least_squares_batches(b):
    d = 16_384
    w_star, w0 = synth.lsq_problem(d, 1400, DEV)
    x, y = synth.lsq_batch(b, w_star, 1400, 0)
    G = synth.lsq_persample_grads(x, y, w0)
    got, ref, b_next = persample_check(G, 0.1)
    assert ref["T"] > b  # noise-dominated: the test fails and asks for a larger batch


@pytest.mark.parametrize("eta", [0.1, 0.5])
def test_least_squares_schedule_step_locked(eta):
    """200 steps from b=32, capped at 4096; at every tested step the oracle sees the same
    batch and the library's current weights, so state drift cannot hide a decision bug."""
    d, b_max, steps = 16_384, 4096, 200
    w_star, w = synth.lsq_problem(d, 1500, DEV)
    w = w.clone()
    m = torch.zeros_like(w)
    v = torch.zeros_like(w)
    gbar = torch.empty(d, dtype=torch.float32, device=DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    sched = absnt.abs_schedule_init(1, 1, 32, b_max)  # J = M = 1: the microbatch is the batch
    traj, checked = [], 0
    for t in range(steps):
        b = int(sched.b)
        assert int(sched.step) == t + 1
        x, y = synth.lsq_batch(b, w_star, 1500, t)
        G = synth.lsq_persample_grads(x, y, w)
        stats = absnt.alloc_persample_stats(b, d, DEV)
        absnt.abs_persample_norm_test(G, eta, stats, gbar, b_next)
        testing = absnt.abs_schedule_test_due(sched)
        assert testing == (b < b_max)
        if testing or t % 40 == 0:
            ref = orc.persample(G.cpu().numpy(), eta)
            got = absnt.read_stats(stats)
            assert_sum_close(got["S"], ref["S"], "S")
            assert_sum_close(got["n2"], ref["n2"], "n2")
            assert_vec_close(gbar, ref["gbar"], "gbar")
            if margin_ok(ref["T"], b):
                assert int(b_next.item()) == ref["b_next"], (t, b, ref["T"])
            p0, m0, v0 = to_host(w), to_host(m), to_host(v)
            w_ref, m_ref, v_ref = oracle_adamw(orc, p0, m0, v0, ref["gbar"], HP, t + 1)
            checked += 1
        else:
            w_ref = None
        absnt.abs_adamw_step(w, gbar, m, v, HP, t + 1)
        if w_ref is not None:
            assert_vec_close(w, w_ref, "w")
            assert_vec_close(m, m_ref, "m")
            assert_vec_close(v, v_ref, "v")
        traj.append(b)
        # the paper's device->host crossing, once per tested step
        absnt.abs_schedule_advance(sched, int(b_next.item()) if testing else b)
    assert int(sched.samples) == sum(traj)
    assert traj[0] == 32 and traj[-1] == b_max
    assert all(a <= c for a, c in zip(traj, traj[1:]))  # never decreases
    assert checked >= 5
    if eta == 0.5:
        assert len(set(traj)) >= 4  # a ramp with several distinct sizes


# ------------------------------------------------------------- full-size configurations
def test_config2_full_size_fused():
    """GPT-2-small-shaped vector, K=8 bf16, fused call in the benchmark's launch shape."""
    sizes = synth.gpt2_small_tensor_sizes()
    d, K, eta, b_cur, step = sum(sizes), 8, 0.1, 512, 100
    sig = synth.per_tensor_sigma(sizes, 2001)
    for attempt in range(4):
        grads = synth.worker_grads(sizes, K, torch.bfloat16, 2000 + attempt, DEV, sigma=sig)
        ref = orc.norm_test([to_host(g) for g in grads], eta, b_cur)
        if margin_ok(ref["T"], b_cur):
            break
    p, m, v = synth.adam_state(d, 2002, DEV, zero_moments=False)
    p0, m0, v0 = to_host(p), to_host(m), to_host(v)
    stats = absnt.alloc_stats(d, 1, DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    absnt.abs_normtest_adamw(grads, eta, b_cur, stats, None, b_next, p, m, v, HP, step)
    torch.cuda.synchronize()
    got = absnt.read_stats(stats)
    assert_sum_close(got["n2"], ref["n2"], "n2")
    assert_sum_close(got["S"], ref["S"], "S")
    assert int(b_next.item()) == ref["b_next"]
    w_ref, m_ref, v_ref = oracle_adamw(orc, p0, m0, v0, ref["gbar"], HP, step)
    assert_vec_close(p, w_ref, "params")
    assert_vec_close(m, m_ref, "m")
    assert_vec_close(v, v_ref, "v")


def test_config3_full_size_fsdp_shards():
    """Llama-style 1.24B vector in 8 equal shards, heavy-tailed noise; the oracle is fed
    shard by shard so the host never holds more than one shard of the K buffers."""
    sizes = synth.llama_1b_tensor_sizes()
    d, K, b_cur, n_sh = sum(sizes), 8, 1024, 8
    offs = synth.equal_shard_offsets(d, n_sh)
    grads = synth.worker_grads([d], K, torch.bfloat16, 3000, DEV, sigma=0.05, noise="student_t3")
    stats = absnt.alloc_stats(d, n_sh, DEV)
    gbar = torch.empty(d, dtype=torch.float32, device=DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    absnt.abs_norm_test(grads, 0.1, b_cur, stats, gbar, b_next, shard_offsets=offs)
    torch.cuda.synchronize()
    got = absnt.read_stats(stats, n_sh)
    dev_b_next = int(b_next.item())

    tot = [0.0, 0.0]
    for s in range(n_sh):
        lo, hi = offs[s], offs[s + 1]
        ref = orc.norm_test([to_host(g[lo:hi]) for g in grads], 0.1, b_cur)
        for j, key in enumerate(("n2", "S")):
            assert abs(got["shards"][s][j] - ref[key]) <= 1e-6 * ref[key], (s, key)
            tot[j] += ref[key]  # shard order, as the oracle itself combines shards
        assert_vec_close(gbar[lo:hi], ref["gbar"], "gbar shard %d" % s)
    assert_sum_close(got["n2"], tot[0], "n2")
    assert_sum_close(got["S"], tot[1], "S")
    decided = 0
    for eta in (0.05, 0.1, 0.2):
        ob, oT, oflags = orc.decide(tot[1], tot[0], K, eta, b_cur)
        hb, hT, hflags = absnt.abs_decide(got["S"], got["n2"], K, eta, b_cur)
        assert hT == pytest.approx(oT, rel=3e-6)
        if margin_ok(oT, b_cur):
            assert hb == ob and hflags == oflags
            decided += 1
            if eta == 0.1:
                assert dev_b_next == ob
    assert decided >= 2


def test_more_than_2_to_31_coordinates():
    """64-bit indexing: d just above 2^31 with shard boundaries on both sides of 2^31.  The
    unfused test is checked shard by shard against the oracle; the fused call must reproduce the
    sums and is checked element-wise on three 1M-coordinate windows (start, across 2^31, end)."""
    d = (1 << 31) + 3 * 4096 + 5
    K, eta, b_cur, step = 2, 0.1, 64, 3
    offs = [0, (1 << 30) + 17, (1 << 31) - 1000, d]
    grads = synth.worker_grads([d], K, torch.bfloat16, 4000, DEV)
    stats = absnt.alloc_stats(d, 3, DEV)
    gbar = torch.empty(d, dtype=torch.float32, device=DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    absnt.abs_norm_test(grads, eta, b_cur, stats, gbar, b_next, shard_offsets=offs)
    torch.cuda.synchronize()
    got = absnt.read_stats(stats, 3)
    tot = [0.0, 0.0]
    for s in range(3):
        lo, hi = offs[s], offs[s + 1]
        ref = orc.norm_test([to_host(g[lo:hi]) for g in grads], eta, b_cur, want_gbar=False)
        for j, key in enumerate(("n2", "S")):
            assert abs(got["shards"][s][j] - ref[key]) <= 1e-6 * ref[key], (s, key)
            tot[j] += ref[key]
    assert_sum_close(got["n2"], tot[0], "n2")
    assert_sum_close(got["S"], tot[1], "S")
    ob, oT, _ = orc.decide(tot[1], tot[0], K, eta, b_cur)
    if margin_ok(oT, b_cur):
        assert int(b_next.item()) == ob

    p, m, v = synth.adam_state(d, 4001, DEV, zero_moments=False)
    windows = [(0, 1 << 20), ((1 << 31) - (1 << 19), (1 << 31) + (1 << 19)), (d - (1 << 20), d)]
    before = [[to_host(x[lo:hi]) for x in (p, m, v)] for lo, hi in windows]
    stats2 = absnt.alloc_stats(d, 1, DEV)
    gbar.fill_(-1.0)
    absnt.abs_normtest_adamw(grads, eta, b_cur, stats2, gbar, b_next, p, m, v, HP, step)
    torch.cuda.synchronize()
    got2 = absnt.read_stats(stats2)
    assert_sum_close(got2["n2"], tot[0], "n2 fused")
    assert_sum_close(got2["S"], tot[1], "S fused")
    for (lo, hi), (p0, m0, v0) in zip(windows, before):
        ref = orc.norm_test([to_host(g[lo:hi]) for g in grads], eta, b_cur)
        assert_vec_close(gbar[lo:hi], ref["gbar"], "gbar window")
        w_ref, m_ref, v_ref = oracle_adamw(orc, p0, m0, v0, ref["gbar"], HP, step)
        assert_vec_close(p[lo:hi], w_ref, "params window")
        assert_vec_close(m[lo:hi], m_ref, "m window")
        assert_vec_close(v[lo:hi], v_ref, "v window")
