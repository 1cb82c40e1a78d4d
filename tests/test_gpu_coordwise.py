"""GPU parity of the coordinate-wise norm test (Sec. 4, Proposition 1) against the fp64 oracle.

The kernels form each per-coordinate ratio in fp32, so the statistic T = max_i T_i is compared
within a relative tolerance (2e-6 up to 16 workers; 2e-5 beyond, where the deviations come
from the shifted one-pass form), and the reported coordinate must be one whose oracle ratio
reaches the oracle's maximum within the same tolerance (several coordinates can be correct;
what is unique -- the value -- is compared, the index is checked for validity).  b_next is
exact under the margin rule; gbar, n2, S and the fused AdamW update are the ordinary parity.
"""
import json
import math
import os

import numpy as np
import pytest
import torch

import paper_2412_21124_b200 as absnt
from oracle import abs_oracle as orc
from paper_2412_21124_b200 import synth
from tests.util import (assert_sum_close, assert_vec_close, margin_ok, oracle_adamw, to_host)

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
HP = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_cases.json")
INT64_MAX = 2 ** 63 - 1


@pytest.fixture(scope="module", autouse=True)
def _device():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    torch.cuda.set_device(0)
    absnt.binding.lib()
    yield
    torch.cuda.synchronize()


def tol_for(K):
    return 2e-6 if K <= 16 else (2e-5 if K <= 64 else 1e-4)


def close_or_both_inf(got, ref, rel):
    if math.isinf(ref) or math.isinf(got):
        return got == ref
    return abs(got - ref) <= rel * abs(ref)


def run_coordwise(grads, eta, b_cur, fused, shard_offsets=None, step=3, seed=9):
    K, d = len(grads), grads[0].numel()
    n_shards = 1 if shard_offsets is None else len(shard_offsets) - 1
    stats = absnt.alloc_stats(d, n_shards, DEV)
    gbar = torch.full((d,), -3.0, dtype=torch.float32, device=DEV)
    b_next = torch.full((1,), -7, dtype=torch.int64, device=DEV)
    state = None
    if fused:
        p, m, v = synth.adam_state(d, seed, DEV, zero_moments=False)
        state = (p, m, v, to_host(p), to_host(m), to_host(v))
        absnt.abs_normtest_adamw_coordwise(grads, eta, b_cur, stats, gbar, b_next, p, m, v, HP,
                                           step, shard_offsets=shard_offsets)
    else:
        absnt.abs_norm_test_coordwise(grads, eta, b_cur, stats, gbar, b_next,
                                      shard_offsets=shard_offsets)
    torch.cuda.synchronize()
    return absnt.read_stats(stats, n_shards), int(b_next.item()), gbar, state


def check_against_oracle(grads, eta, b_cur, fused, shard_offsets=None, step=3):
    K, d = len(grads), grads[0].numel()
    rel = tol_for(K)
    ref = orc.norm_test_coordwise([to_host(g) for g in grads], eta, b_cur,
                                  shard_offsets=shard_offsets, want_ratios=True)
    got, b_next, gbar, state = run_coordwise(grads, eta, b_cur, fused, shard_offsets, step)
    assert_sum_close(got["n2"], ref["n2"], "n2")
    assert_sum_close(got["S"], ref["S"], "S")
    assert math.isnan(got["Q"]) and got["norm"] == K
    assert close_or_both_inf(got["T"], ref["T"], rel), (got["T"], ref["T"])
    # the reported coordinate attains the maximum (within the accuracy of the fp32 ratios)
    i = got["argmax"]
    assert 0 <= i < d
    if math.isinf(ref["T"]):
        assert math.isinf(ref["ratios"][i])
    else:
        assert ref["ratios"][i] >= (1.0 - rel) * ref["T"], (i, ref["ratios"][i], ref["T"])
    assert got["flags"] == ref["flags"]
    if margin_ok(ref["T"], b_cur):
        assert b_next == ref["b_next"]
    # shard records: the same sums, the shard's largest T_i and a coordinate inside the shard
    # that attains it
    if shard_offsets is not None:
        for s in range(len(shard_offsets) - 1):
            lo, hi = shard_offsets[s], shard_offsets[s + 1]
            assert close_or_both_inf(got["shard_max"][s], ref["shard_max"][s], rel), s
            j = int(got["shards"][s][2])
            if hi > lo:
                assert lo <= j < hi
                want = ref["shard_max"][s]
                assert (math.isinf(ref["ratios"][j]) if math.isinf(want)
                        else ref["ratios"][j] >= (1.0 - rel) * want)
            else:
                assert j == lo and got["shard_max"][s] == 0.0
        assert got["T"] == max(got["shard_max"])
    assert_vec_close(gbar, ref["gbar"], "gbar")
    if fused:
        p, m, v, p0, m0, v0 = state
        w_ref, m_ref, v_ref = oracle_adamw(orc, p0, m0, v0, ref["gbar"], HP, step)
        assert_vec_close(p, w_ref, "params")
        assert_vec_close(m, m_ref, "m")
        assert_vec_close(v, v_ref, "v")
    return got, ref


# worker counts that reach every kernel family (see tests/test_gpu_edge_cases.py)
FAMILY_K = [1, 2, 3, 4, 8, 12, 16, 24, 32, 33, 47, 64, 130]
D = 4 * 4096 + 1234


@pytest.mark.parametrize("fused", [True, False], ids=["fused", "unfused"])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("K", FAMILY_K)
def test_coordwise_every_kernel_family(K, dtype, fused):
    eta = 0.1
    for attempt in range(6):
        # a mean well away from zero keeps T finite and moderate; the plain generator below
        # (mean ~ 0.01) exercises the large ratios
        grads = synth.worker_grads([D], K, dtype, 8000 + 10 * K + attempt, DEV, sigma=0.05,
                                   mu_std=0.01)
        for g in grads:
            g += 0.5
        ref = orc.norm_test_coordwise([to_host(g) for g in grads], eta, 1)
        if margin_ok(ref["T"], 1):
            break
    b_cur = max(1, int(ref["T"] / 2)) if K > 1 else 5
    check_against_oracle(grads, eta, b_cur, fused)
    # the same with shards whose cuts fall inside chunks and thread-rows, one of them empty
    offs = [0, 5, 4101, 4101, 9_999, D]
    check_against_oracle(grads, eta, b_cur, fused, shard_offsets=offs)
    # small means: huge ratios, possibly +inf (a bf16 mean can cancel to exactly zero)
    grads = synth.worker_grads([D], K, dtype, 8500 + K, DEV)
    check_against_oracle(grads, eta, 64, fused)
    # a batch size the statistic does not reach: the test holds, b is kept
    got, ref = check_against_oracle(grads, 1e6, 64, fused)
    assert ref["b_next"] == 64 or math.isinf(ref["T"])


def test_coordwise_hand_cases_on_the_device():
    cases = json.load(open(GOLDEN))["coordwise"]
    c = cases[0]
    grads = [torch.tensor(g, dtype=torch.float32, device=DEV) for g in c["grads"]]
    for dec in c["decisions"]:
        got, b_next, gbar, _ = run_coordwise(grads, c["eta"], dec["b_cur"], fused=False)
        assert got["T"] == c["T"] and got["argmax"] == c["argmax"] and b_next == dec["b_next"]
        assert bool(got["flags"] & absnt.ABS_FLAG_VIOLATED) == dec["violated"]
        # the summed test on the same data, through the plain entry point
        stats = absnt.alloc_stats(2, 1, DEV)
        bn = torch.zeros(1, dtype=torch.int64, device=DEV)
        absnt.abs_norm_test(grads, c["eta"], dec["b_cur"], stats, gbar, bn)
        assert int(bn.item()) == dec["b_next_summed"]
    c = cases[1]
    grads = [torch.tensor(g, dtype=torch.float32, device=DEV) for g in c["grads"]]
    got, b_next, _, _ = run_coordwise(grads, c["eta"], 7, fused=False)
    assert got["T"] == math.inf and got["argmax"] == c["argmax"] and got["flags"] == c["flags"]
    assert b_next == INT64_MAX
    got, b_next, _, _ = run_coordwise([g[1:].contiguous() for g in grads], c["eta"], 7, fused=False)
    assert got["T"] == 0.0 and got["flags"] == 0 and b_next == 7 and got["argmax"] == 0
    z = [torch.zeros(3, dtype=torch.bfloat16, device=DEV)] * 2
    got, b_next, _, _ = run_coordwise(z, c["eta"], 7, fused=True)
    assert got["T"] == 0.0 and got["flags"] == absnt.ABS_FLAG_DEGENERATE and b_next == 7


@pytest.mark.parametrize("K,dtype", [(4, torch.float32), (8, torch.bfloat16), (32, torch.bfloat16),
                                     (47, torch.float32)], ids=["k4-f32", "k8-bf16", "k32-bf16",
                                                                "k47-f32"])
def test_coordwise_ties_zero_rules_and_nonfinite(K, dtype):
    d = 3 * 4096 + 77
    base = synth.worker_grads([d], K, dtype, 8600 + K, DEV)
    for g in base:
        g += 0.5
    # plant the same extreme coordinate twice: the lower index is reported
    hot = [(-1.0) ** k * 0.25 + 0.03125 for k in range(K)]
    if K % 2:
        hot[-1] = 0.03125
    grads = [g.clone() for g in base]
    for k in range(K):
        for i in (4096 + 900, 700, 2 * 4096 + 5):
            grads[k][i] = hot[k]
    got, ref = check_against_oracle(grads, 0.1, 64, fused=True)
    assert ref["argmax"] == 700 and got["argmax"] == 700
    # zero mean with positive variance in one coordinate: +inf, DEGENERATE | VIOLATED
    grads = [g.clone() for g in base]
    for k in range(K):
        grads[k][d - 2] = 0.0
    grads[0][d - 2], grads[1 % K][d - 2] = 0.125, -0.125
    if K > 1:
        got, ref = check_against_oracle(grads, 0.1, 64, fused=False)
        assert got["T"] == math.inf and got["argmax"] == d - 2
        assert got["flags"] == absnt.ABS_FLAG_DEGENERATE | absnt.ABS_FLAG_VIOLATED
    # identical buffers: every coordinate passes for any batch size
    same = [base[0].clone() for _ in range(K)]
    got, b_next, _, _ = run_coordwise(same, 0.1, 3, fused=True)
    assert got["T"] == 0.0 and b_next == 3 and got["flags"] == 0 and got["argmax"] == 0
    # a non-finite input: flag, T = NaN, b kept (as the oracle says)
    bad = [g.clone() for g in base]
    bad[K - 1][5000] = math.nan
    ref = orc.norm_test_coordwise([to_host(g) for g in bad], 0.1, 64)
    got, b_next, _, _ = run_coordwise(bad, 0.1, 64, fused=False)
    assert ref["flags"] == orc.FLAG_NONFINITE
    assert got["flags"] == absnt.ABS_FLAG_NONFINITE and math.isnan(got["T"]) and b_next == 64
    # a statistic beyond 2^62 saturates
    got, ref = check_against_oracle(base, 1e-12, 64, fused=False)
    assert ref["b_next"] == INT64_MAX


def test_coordwise_config1_and_large_chunks():
    # config 1's shape: K=4 fp32, d = 2^20, unfused then fused
    grads = synth.worker_grads([1 << 20], 4, torch.float32, 8700, DEV)
    check_against_oracle(grads, 0.1, 64, fused=False)
    check_against_oracle(grads, 0.1, 64, fused=True)
    # d >= 2^23: 8192 / 16384-coordinate chunks, a ragged tail, shards
    d = (1 << 23) + 3 * 8192 + 321
    grads = synth.worker_grads([d], 8, torch.bfloat16, 8701, DEV)
    for g in grads:
        g += 0.25
    offs = synth.equal_shard_offsets(d, 5)
    check_against_oracle(grads, 0.1, 512, fused=True, shard_offsets=offs)
    check_against_oracle(grads, 0.1, 512, fused=False, shard_offsets=offs)


def test_coordwise_config2_full_size():
    """The benchmark's workload (GPT-2-small-shaped vector, K=8 bf16, fused) with the
    coordinate-wise decision; the sums and the update are those of the plain fused call."""
    sizes = synth.gpt2_small_tensor_sizes()
    d, K, eta, b_cur, step = sum(sizes), 8, 0.1, 512, 100
    sig = synth.per_tensor_sigma(sizes, 2001)
    grads = synth.worker_grads(sizes, K, torch.bfloat16, 2000, DEV, sigma=sig)
    ref = orc.norm_test_coordwise([to_host(g) for g in grads], eta, b_cur, want_ratios=True)
    p, m, v = synth.adam_state(d, 2002, DEV, zero_moments=False)
    q, mq, vq = p.clone(), m.clone(), v.clone()
    stats = absnt.alloc_stats(d, 1, DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    absnt.abs_normtest_adamw_coordwise(grads, eta, b_cur, stats, None, b_next, p, m, v, HP, step)
    torch.cuda.synchronize()
    got = absnt.read_stats(stats)
    assert_sum_close(got["n2"], ref["n2"], "n2")
    assert_sum_close(got["S"], ref["S"], "S")
    assert close_or_both_inf(got["T"], ref["T"], 2e-6)
    i = got["argmax"]
    assert (math.isinf(ref["ratios"][i]) if math.isinf(ref["T"])
            else ref["ratios"][i] >= (1 - 2e-6) * ref["T"])
    assert got["flags"] == ref["flags"] and int(b_next.item()) == ref["b_next"]
    # same update, bit for bit, as the plain fused call
    stats2 = absnt.alloc_stats(d, 1, DEV)
    absnt.abs_normtest_adamw(grads, eta, b_cur, stats2, None, b_next, q, mq, vq, HP, step)
    torch.cuda.synchronize()
    assert torch.equal(p, q) and torch.equal(m, mq) and torch.equal(v, vq)
    assert torch.equal(stats[:2], stats2[:2])


# ------------------------------------------------------------- per-sample form
def persample_cw_check(G, eta, rel=1e-5):
    """abs_persample_norm_test_coordwise against the oracle's per-sample coordinate-wise test."""
    b, d = G.shape
    stats = absnt.alloc_persample_stats(b, d, DEV)
    gbar = torch.full((d,), -3.0, dtype=torch.float32, device=DEV)
    b_next = torch.full((1,), -7, dtype=torch.int64, device=DEV)
    absnt.abs_persample_norm_test_coordwise(G, eta, stats, gbar, b_next)
    torch.cuda.synchronize()
    got = absnt.read_stats(stats)
    host = to_host(G) if G.dtype == torch.bfloat16 else G.cpu().numpy()
    ref = orc.persample_coordwise(host, eta, want_ratios=True)
    assert got["norm"] == b - 1 and math.isnan(got["Q"])
    if math.isfinite(ref["n2"]) and math.isfinite(ref["S"]):
        assert_sum_close(got["n2"], ref["n2"], "n2")
        if ref["S"] == 0.0:
            assert got["S"] == 0.0
        else:
            assert_sum_close(got["S"], ref["S"], "S")
        assert_vec_close(gbar, ref["gbar"], "gbar")
    assert got["flags"] == ref["flags"], (got, ref["flags"])
    if math.isnan(ref["T"]):
        assert math.isnan(got["T"])
    else:
        assert close_or_both_inf(got["T"], ref["T"], rel), (got["T"], ref["T"])
        i = got["argmax"]
        assert 0 <= i < d
        if math.isinf(ref["T"]):
            assert math.isinf(ref["ratios"][i])
        else:
            assert ref["ratios"][i] >= (1.0 - rel) * ref["T"]
        assert got["shards"][0][2] == i and got["shard_max"][0] == got["T"]
    if margin_ok(ref["T"], b):
        assert int(b_next.item()) == ref["b_next"]
    return got, ref, int(b_next.item())


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("b,d,ld,shift", [(2, 5, 5, 0), (33, 300, 320, 0), (100, 2051, 2052, 1),
                                          (257, 4096, 4096, 0), (1000, 777, 780, 0),
                                          (2049, 515, 516, 0), (65, 40_000, 40_000, 0)])
def test_persample_coordwise_shapes(b, d, ld, shift, dtype):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(b * 139 + d)
    buf = torch.empty(b * ld + shift, dtype=torch.float32, device=DEV)
    buf.normal_(generator=gen)
    buf.mul_(0.3).add_(0.2)
    G = buf.to(dtype)[shift:].view(b, ld)[:, :d]
    persample_cw_check(G, 0.3)


def test_persample_coordwise_disagrees_with_the_summed_test():
    """One column with a mean close to zero dominates the coordinate-wise statistic while the
    summed test (Eq. 3) still passes: the two calls decide differently on the same matrix."""
    b, d = 64, 3000
    gen = torch.Generator(device=DEV)
    gen.manual_seed(3)
    G = torch.empty(b, d, device=DEV).normal_(generator=gen).mul_(0.05).add_(1.0)
    G[:, 1234] -= G[:, 1234].mean() - 1e-4    # this column's mean is 1e-4, its spread stays
    eta = 0.5
    got, ref, b_cw = persample_cw_check(G, eta)
    assert got["argmax"] == 1234 and b_cw > b
    stats = absnt.alloc_persample_stats(b, d, DEV)
    gbar = torch.empty(d, dtype=torch.float32, device=DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    absnt.abs_persample_norm_test(G, eta, stats, gbar, b_next)
    torch.cuda.synchronize()
    assert int(b_next.item()) == b    # the summed test keeps the batch size


def test_persample_coordwise_zero_rules_ties_and_nonfinite():
    b, d = 40, 700
    gen = torch.Generator(device=DEV)
    gen.manual_seed(4)
    base = torch.empty(b, d, device=DEV).normal_(generator=gen).mul_(0.1).add_(0.5)
    # a column of identical values has T_i = 0, also when that value is zero
    G = base.clone()
    G[:, 10] = 0.25
    G[:, 11] = 0.0
    got, ref, _ = persample_cw_check(G, 0.3)
    assert ref["ratios"][10] == 0.0 and ref["ratios"][11] == 0.0
    # two identical columns tie: the lower index is reported
    G = base.clone()
    G[:, 5] = G[:, 600] = torch.linspace(-1.0, 1.001, b, device=DEV)
    got, ref, _ = persample_cw_check(G, 0.3)
    assert got["argmax"] == 5 == ref["argmax"]
    # a column whose values cancel exactly: positive variance, zero mean -> +inf, DEGENERATE
    G = base.clone()
    half = torch.linspace(0.1, 1.0, b // 2, device=DEV)
    G[:, 77] = torch.cat([half, -half])
    got, ref, b_next = persample_cw_check(G, 0.3)
    assert got["T"] == math.inf and got["argmax"] == 77 and b_next == INT64_MAX
    assert got["flags"] == absnt.ABS_FLAG_DEGENERATE | absnt.ABS_FLAG_VIOLATED
    # a NaN anywhere: NONFINITE, the batch size stays
    G = base.clone()
    G[17, 300] = float("nan")
    got, ref, b_next = persample_cw_check(G, 0.3)
    assert got["flags"] & absnt.ABS_FLAG_NONFINITE and b_next == b


def test_persample_coordwise_hand_cases():
    """Hand cases H8 and H9 with their rows as the samples (b = 2, normalisation b - 1 = 1)."""
    cases = json.load(open(GOLDEN))["coordwise"]
    c = cases[0]
    G = torch.tensor(c["grads"], dtype=torch.float32, device=DEV)
    got, ref, b_next = persample_cw_check(G, c["eta"])
    assert got["T"] == c["T_persample"] and got["argmax"] == c["argmax"]
    assert b_next == c["b_next_persample"]
    c = cases[1]
    G = torch.tensor(c["grads"], dtype=torch.float32, device=DEV)
    got, ref, b_next = persample_cw_check(G, c["eta"])
    assert got["T"] == math.inf and got["argmax"] == c["argmax"] and got["flags"] == c["flags"]
    assert b_next == INT64_MAX
