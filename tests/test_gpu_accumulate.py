"""GPU parity of the carry-in form of the norm test (`abs_norm_test_accumulate`) against the
fp64 oracle.

The gradients of a step reach the library a few per call; after every call the running mean, the
sums, the statistic and the decision must be those of the oracle's plain norm test over all the
gradients merged so far -- the oracle knows nothing of the carry, it is simply given the buffers
side by side.  Sums within relative 1e-6; b_next exact under the margin rule; the mean within
1e-6 * max|gbar|, widened by sqrt(calls)/4 beyond 16 calls because the running mean is rounded to
fp32 once per call.
"""
import math

import pytest
import torch

import paper_2412_21124_b200 as absnt
from oracle import abs_oracle as orc
from paper_2412_21124_b200 import synth
from tests.util import (REL_VEC, assert_sum_close, assert_vec_close, margin_ok, oracle_adamw,
                        to_host)

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
D = 4 * 4096 + 1234   # several chunks of 4096 and a ragged tail
HP = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)


@pytest.fixture(scope="module", autouse=True)
def _device():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    torch.cuda.set_device(0)
    absnt.binding.lib()
    yield
    torch.cuda.synchronize()


def shifted_copy(t, shift):
    """A copy of t that starts `shift` elements into a fresh allocation (misaligned for shift > 0)."""
    buf = torch.empty(t.numel() + shift + 8, dtype=t.dtype, device=t.device)
    view = buf[shift:shift + t.numel()]
    view.copy_(t)
    return view


def mean_tolerance(calls):
    return REL_VEC * max(1.0, math.sqrt(calls) / 4.0)


def accumulate_and_check(grads, parts, eta, b_cur, shard_offsets=None, check_every_call=True,
                         mean=None):
    """Feeds `grads` in consecutive pieces of the sizes in `parts`; returns the final stats."""
    d = grads[0].numel()
    n_shards = 1 if shard_offsets is None else len(shard_offsets) - 1
    stats = absnt.alloc_stats(d, n_shards, DEV)
    if mean is None:
        mean = torch.full((d,), float("nan"), dtype=torch.float32, device=DEV)  # only written at first
    b_next = torch.full((1,), -7, dtype=torch.int64, device=DEV)
    host = [to_host(g) for g in grads]
    count = 0
    assert sum(parts) == len(grads)
    for call, m in enumerate(parts, start=1):
        absnt.abs_norm_test_accumulate(grads[count:count + m], count, eta, b_cur, stats, mean,
                                       b_next, shard_offsets=shard_offsets)
        count += m
        if not (check_every_call or count == len(grads)):
            continue
        torch.cuda.synchronize()
        ref = orc.norm_test(host[:count], eta, b_cur, shard_offsets=shard_offsets)
        got = absnt.read_stats(stats, n_shards)
        assert got["norm"] == count and math.isnan(got["Q"])
        assert_sum_close(got["n2"], ref["n2"], "n2 after %d gradients" % count)
        if ref["S"] == 0.0:
            assert got["S"] == 0.0
        else:
            assert_sum_close(got["S"], ref["S"], "S after %d gradients" % count)
        assert got["flags"] == ref["flags"]
        if margin_ok(ref["T"], b_cur):
            assert int(b_next.item()) == ref["b_next"], (count, got["T"], ref["T"])
        assert_vec_close(mean, ref["gbar"], "mean after %d gradients" % count,
                         rel=mean_tolerance(call))
        if shard_offsets is not None:
            for s in range(n_shards):
                assert_sum_close(got["shards"][s][0], ref["shards"][s][0], "n2 of shard %d" % s)
                if ref["shards"][s][1] == 0.0:
                    assert got["shards"][s][1] == 0.0
                else:
                    assert_sum_close(got["shards"][s][1], ref["shards"][s][1], "S of shard %d" % s)
    return absnt.read_stats(stats, n_shards), mean, int(b_next.item())


SPLITS = [
    [8],                       # one call: the plain test through this kernel
    [1] * 8,                   # one gradient per call (a micro-batch at a time)
    [3, 5],
    [2, 2, 4, 1, 7],           # multi-row kernels (K <= 2, K <= 4) and the general one
    [16, 17],                  # a whole group of 16 (bf16) / two of 8 (fp32) and a remainder
    [64, 36],                  # the largest call
    [1, 2, 4, 8, 16, 2],
    [12, 9, 6, 15],            # part of a group: the predicated batch of the two-row kernels
]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("parts", SPLITS, ids=["-".join(map(str, p)) for p in SPLITS])
def test_accumulate_matches_the_oracle_after_every_call(parts, dtype):
    K = sum(parts)
    grads = synth.worker_grads([D], K, dtype, 300 + K, DEV)
    accumulate_and_check(grads, parts, 0.1, 64)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_accumulate_with_shards_empty_shards_and_large_chunks(dtype):
    """Shard records are carried shard by shard; an empty shard carries nothing; at 2^23
    coordinates and more the chunks are 16384 coordinates."""
    grads = synth.worker_grads([D], 12, dtype, 77, DEV)
    offs = [0, 0, 5000, 5000, 5003, D - 1, D, D]
    accumulate_and_check(grads, [5, 4, 3], 0.07, 32, shard_offsets=offs)
    d_big = (1 << 23) + 16384 + 77
    grads = synth.worker_grads([d_big], 4, dtype, 78, DEV)
    accumulate_and_check(grads, [1, 3], 0.1, 64, shard_offsets=[0, 3_000_001, d_big],
                         check_every_call=False)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("shift", [1, 3])
def test_accumulate_misaligned_buffers_give_the_same_bits(dtype, shift):
    """Buffers that are not 16-byte aligned take the element-wise path: same operations in the
    same order, so the results are bit-identical to the aligned run's."""
    grads = synth.worker_grads([D], 7, dtype, 31, DEV)
    ref_stats, ref_mean, ref_b = accumulate_and_check(grads, [2, 5], 0.1, 64)
    moved = [shifted_copy(g, shift) for g in grads]
    mean = shifted_copy(torch.zeros(D, dtype=torch.float32, device=DEV), shift)
    stats, mean, b = accumulate_and_check(moved, [2, 5], 0.1, 64, mean=mean)
    for key in ("n2", "S", "T", "flags", "norm"):   # Q is NaN in both
        assert stats[key] == ref_stats[key], key
    assert b == ref_b
    assert torch.equal(mean, ref_mean)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_accumulate_identical_gradients_have_zero_variance(dtype):
    """Eq. 5 with identical worker gradients: the variance sum is exactly zero after every call,
    the mean is that gradient bit for bit and the batch size stays."""
    g = synth.worker_grads([D], 1, dtype, 5, DEV)[0]
    grads = [g.clone() for _ in range(9)]
    stats, mean, b_next = accumulate_and_check(grads, [1, 3, 5], 0.1, 64)
    assert stats["S"] == 0.0 and stats["T"] == 0.0 and b_next == 64
    assert torch.equal(mean, g.float())


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_accumulate_nonfinite_stays_until_a_new_step(dtype):
    """A NaN merged by one call stays in the sums of the later calls of the step (flag raised,
    batch size kept); a call with count_in = 0 starts clean in the same buffers."""
    grads = synth.worker_grads([D], 6, dtype, 8, DEV)
    bad = [g.clone() for g in grads]
    bad[2][4097] = float("nan")
    stats = absnt.alloc_stats(D, 1, DEV)
    mean = torch.zeros(D, dtype=torch.float32, device=DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    count = 0
    for m in (2, 2, 2):
        absnt.abs_norm_test_accumulate(bad[count:count + m], count, 0.1, 64, stats, mean, b_next)
        count += m
        torch.cuda.synchronize()
        got = absnt.read_stats(stats)
        if count >= 3:
            assert got["flags"] & absnt.ABS_FLAG_NONFINITE and int(b_next.item()) == 64
        else:
            assert got["flags"] & absnt.ABS_FLAG_NONFINITE == 0
    # the same buffers, a new step
    absnt.abs_norm_test_accumulate(grads, 0, 0.1, 64, stats, mean, b_next)
    torch.cuda.synchronize()
    ref = orc.norm_test([to_host(g) for g in grads], 0.1, 64)
    got = absnt.read_stats(stats)
    assert got["flags"] == ref["flags"]
    assert_sum_close(got["S"], ref["S"], "S")
    assert_vec_close(mean, ref["gbar"], "mean")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_accumulate_agrees_with_the_one_call_test(dtype):
    """The same 32 gradients through abs_norm_test at once and through 32 calls of one gradient:
    sums within 1e-6 of each other, the same decision."""
    K, eta, b_cur = 32, 0.1, 64
    seed = 900
    while True:
        grads = synth.worker_grads([D], K, dtype, seed, DEV)
        ref = orc.norm_test([to_host(g) for g in grads], eta, b_cur)
        if margin_ok(ref["T"], b_cur):
            break
        seed += 1
    stats1 = absnt.alloc_stats(D, 1, DEV)
    gbar = torch.zeros(D, dtype=torch.float32, device=DEV)
    b1 = torch.zeros(1, dtype=torch.int64, device=DEV)
    absnt.abs_norm_test(grads, eta, b_cur, stats1, gbar, b1)
    got, mean, b2 = accumulate_and_check(grads, [1] * K, eta, b_cur, check_every_call=False)
    torch.cuda.synchronize()
    one = absnt.read_stats(stats1)
    assert_sum_close(got["S"], one["S"], "S")
    assert_sum_close(got["n2"], one["n2"], "n2")
    assert b2 == int(b1.item()) == ref["b_next"]
    assert_vec_close(mean, gbar.double().cpu().numpy(), "mean", rel=mean_tolerance(K))


def test_accumulate_many_calls_keeps_the_stated_accuracy():
    """256 calls of one bf16 gradient (Table 5's largest accumulation count for one worker):
    the running mean is rounded 256 times; the sums still meet 1e-6."""
    K = 256
    d = 3 * 4096 + 5
    grads = synth.worker_grads([d], K, torch.bfloat16, 4242, DEV)
    accumulate_and_check(grads, [1] * K, 0.1, 256, check_every_call=False)


def test_accumulate_spread_far_below_the_mean():
    """sigma/|mu| = 1e-3: the centre of every call is the running mean, so the deviations are
    formed without cancellation and the sums keep 1e-6."""
    K, d = 16, D
    gen = torch.Generator(device="cpu").manual_seed(99)
    base = torch.ones(d) + 0.25 * torch.rand(d, generator=gen)
    grads = [(base * (1.0 + 1e-3 * torch.randn(d, generator=gen))).to(DEV) for _ in range(K)]
    accumulate_and_check(grads, [4, 4, 8], 1e-4, 64)


def test_accumulate_config2_size_sampled():
    """The benchmark's vector (124,439,808 coordinates, bf16) merged in 8 calls of one gradient:
    sums and decision against the oracle on the whole vector, the mean on the whole vector."""
    d, K, eta, b_cur = 124_439_808, 8, 0.1, 512
    sizes = synth.gpt2_small_tensor_sizes()
    assert sum(sizes) == d
    sig = synth.per_tensor_sigma(sizes, 2001)
    for attempt in range(4):
        grads = synth.worker_grads(sizes, K, torch.bfloat16, 2000 + attempt, DEV, sigma=sig)
        if margin_ok(orc.norm_test([to_host(g) for g in grads], eta, b_cur, want_gbar=False)["T"],
                     b_cur):
            break
    accumulate_and_check(grads, [1] * K, eta, b_cur, check_every_call=False)


# ------------------------------------------------------------- closing call fused with AdamW
CLOSING = [([8], "whole step"), ([7, 1], "one"), ([4, 4], "two rows"), ([3, 9], "general"),
           ([1] * 5, "micro-batches"), ([20, 33], "groups"), ([2, 6], "batch of six"),
           ([3, 13], "batch of thirteen")]


@pytest.mark.parametrize("inplace", [True, False], ids=["mean in place", "mean not written"])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("parts", [c[0] for c in CLOSING], ids=[c[1] for c in CLOSING])
def test_accumulate_closing_call_with_adamw(parts, dtype, inplace):
    """All calls but the last merge; the last one merges and applies AdamW with the final mean
    (Algorithm 1: the test, then the update on the batch gradient).  Sums, decision, parameters
    and moments against the oracle's plain test + AdamW on all buffers."""
    K, eta, b_cur, step = sum(parts), 0.1, 64, 4
    seed = 500 + K
    while True:
        grads = synth.worker_grads([D], K, dtype, seed, DEV)
        ref = orc.norm_test([to_host(g) for g in grads], eta, b_cur)
        if margin_ok(ref["T"], b_cur):
            break
        seed += 1
    p, m, v = synth.adam_state(D, 12, DEV, zero_moments=False)
    p0, m0, v0 = to_host(p), to_host(m), to_host(v)
    stats = absnt.alloc_stats(D, 1, DEV)
    mean = torch.zeros(D, dtype=torch.float32, device=DEV)
    b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
    count = 0
    for mpart in parts[:-1]:
        absnt.abs_norm_test_accumulate(grads[count:count + mpart], count, eta, b_cur, stats, mean,
                                       b_next)
        count += mpart
    before = mean.clone()
    absnt.abs_norm_test_accumulate_adamw(grads[count:], count, eta, b_cur, stats,
                                         mean if count else None, mean if inplace else None,
                                         b_next, p, m, v, HP, step)
    torch.cuda.synchronize()
    got = absnt.read_stats(stats)
    assert got["norm"] == K
    assert_sum_close(got["n2"], ref["n2"], "n2")
    assert_sum_close(got["S"], ref["S"], "S")
    assert int(b_next.item()) == ref["b_next"] and got["flags"] == ref["flags"]
    if inplace:
        assert_vec_close(mean, ref["gbar"], "final mean", rel=mean_tolerance(len(parts)))
    else:
        assert torch.equal(mean, before)   # the running mean was only read
    w_ref, m_ref, v_ref = oracle_adamw(orc, p0, m0, v0, ref["gbar"], HP, step)
    assert_vec_close(p, w_ref, "params")
    assert_vec_close(m, m_ref, "m")
    assert_vec_close(v, v_ref, "v")


def test_accumulate_closing_call_equals_merge_then_adamw():
    """The fused closing call against the two-call form (abs_norm_test_accumulate, then
    abs_adamw_step on the final mean): the same mean, sums and decision bit for bit, and the
    same update (both run adamw on the same fp32 mean)."""
    K = 6
    grads = synth.worker_grads([D], K, torch.bfloat16, 77, DEV)
    outs = []
    for fused in (False, True):
        p, m, v = synth.adam_state(D, 13, DEV, zero_moments=False)
        stats = absnt.alloc_stats(D, 1, DEV)
        mean = torch.zeros(D, dtype=torch.float32, device=DEV)
        b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
        absnt.abs_norm_test_accumulate(grads[:4], 0, 0.1, 64, stats, mean, b_next)
        if fused:
            absnt.abs_norm_test_accumulate_adamw(grads[4:], 4, 0.1, 64, stats, mean, mean, b_next,
                                                 p, m, v, HP, 9)
        else:
            absnt.abs_norm_test_accumulate(grads[4:], 4, 0.1, 64, stats, mean, b_next)
            absnt.abs_adamw_step(p, mean, m, v, HP, 9)
        torch.cuda.synchronize()
        outs.append((absnt.read_stats(stats), mean, int(b_next.item()), p, m, v))
    a, b = outs
    for key in ("n2", "S", "T", "flags"):
        assert a[0][key] == b[0][key], key
    assert a[2] == b[2]
    for x, y in zip(a[1:2] + a[3:], b[1:2] + b[3:]):
        assert torch.equal(x, y)


def test_accumulate_adamw_misaligned_and_ragged():
    """State vectors that are not 16-byte aligned take the element-wise path of the fused
    closing call: the same bits as the aligned run."""
    grads = synth.worker_grads([D], 5, torch.float32, 61, DEV)
    res = []
    for shift in (0, 1):
        p, m, v = (shifted_copy(t, shift) for t in synth.adam_state(D, 14, DEV, zero_moments=False))
        stats = absnt.alloc_stats(D, 1, DEV)
        mean = shifted_copy(torch.zeros(D, dtype=torch.float32, device=DEV), shift)
        b_next = torch.zeros(1, dtype=torch.int64, device=DEV)
        absnt.abs_norm_test_accumulate(grads[:2], 0, 0.1, 64, stats, mean, b_next)
        absnt.abs_norm_test_accumulate_adamw(grads[2:], 2, 0.1, 64, stats, mean, mean, b_next,
                                             p, m, v, HP, 2)
        torch.cuda.synchronize()
        res.append((absnt.read_stats(stats)["S"], mean.clone(), p.clone(), m.clone(), v.clone()))
    assert res[0][0] == res[1][0]
    for x, y in zip(res[0][1:], res[1][1:]):
        assert torch.equal(x, y)
