"""abs_normtest_adamw_noalloc: the fused step for callers that cannot allocate device memory
(plugin execute hooks, latency-critical callbacks, processes whose device memory belongs to
another allocator).  It keeps its per-chunk partial sums in an array built into the library
instead of a caller-sized tail of stats_out, so the caller only supplies the fixed header and
the shard records.

Checked here, through the C ABI, on two calls in a row (different sizes, so the second call
sees stale records of the first in the shared array):
  * against the fp64 CPU oracle, element by element, within the parity tolerances of the other
    GPU tests (sums relative 1e-6, vectors 1e-6 * max|reference|, b_next exact);
  * against abs_normtest_adamw on the same inputs, bit for bit -- both entry points run the
    same kernels on the same chunk layout, which is what the header promises.
That the size limit is refused on the host, before anything is launched, is checked without a
GPU in tests/test_abi_cpu.py.

This file is collected last on purpose: a run that stops at the first failure has then already
run every other test.  It passes alone in a fresh process as well as after the other tests.
"""
import pytest
import torch

import paper_2412_21124_b200 as absnt
from oracle import abs_oracle as orc
from paper_2412_21124_b200 import binding, synth
from tests.util import (assert_sum_close, assert_vec_close, margin_ok, oracle_adamw, to_host)

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
HP = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)


def _run_pair(K, d, dtype, n_shards, step, seed):
    """The same inputs through the existing entry point and through the no-alloc variant, and
    through the oracle."""
    eta, b_cur = 0.1, 64
    offs = synth.equal_shard_offsets(d, n_shards) if n_shards > 1 else None
    for attempt in range(8):
        grads = synth.worker_grads([d], K, dtype, seed + 100 * attempt, DEV)
        ref = orc.norm_test([to_host(g) for g in grads], eta, b_cur, shard_offsets=offs)
        if margin_ok(ref["T"], b_cur):
            break
    else:
        raise AssertionError("no seed met the decision margin")
    p0, m0, v0 = (to_host(t) for t in synth.adam_state(d, seed + 1, DEV, zero_moments=False))
    w_ref, m_ref, v_ref = oracle_adamw(orc, p0, m0, v0, ref["gbar"], HP, step)
    n_hdr = binding.ABS_STATS_HEADER + n_shards * binding.ABS_SHARD_STRIDE
    outs = []
    for variant in ("existing", "noalloc"):
        p, m, v = synth.adam_state(d, seed + 1, DEV, zero_moments=False)
        gbar = torch.empty(d, dtype=torch.float32, device=DEV)
        b_next = torch.full((1,), -1, dtype=torch.int64, device=DEV)
        if variant == "existing":
            stats = absnt.alloc_stats(d, n_shards, DEV)
            absnt.abs_normtest_adamw(grads, eta, b_cur, stats, gbar, b_next, p, m, v, HP, step,
                                     shard_offsets=offs)
        else:
            # header + shard records only: nothing here grows with d
            stats = torch.full((n_hdr,), -1.0, dtype=torch.float64, device=DEV)
            assert absnt.abs_noalloc_fits(d, offs)
            absnt.abs_normtest_adamw_noalloc(grads, eta, b_cur, stats, gbar, b_next, p, m, v, HP,
                                             step, shard_offsets=offs)
        torch.cuda.synchronize()
        outs.append((stats[:n_hdr].clone(), b_next, gbar, p, m, v))
    (sa, ba, ga, pa, ma, va), (sb, bb, gb, pb, mb, vb) = outs

    # the no-alloc call against the oracle
    got = absnt.read_stats(sb, n_shards)
    assert_sum_close(got["n2"], ref["n2"], "n2")
    assert_sum_close(got["S"], ref["S"], "S")
    assert got["T"] == pytest.approx(ref["T"], rel=3e-6)
    assert got["flags"] == ref["flags"] and got["norm"] == K
    assert int(bb.item()) == ref["b_next"]
    for s in range(n_shards):
        for j in range(2):
            assert_sum_close(got["shards"][s][j], ref["shards"][s, j], "shard %d sum %d" % (s, j))
    assert_vec_close(gb, ref["gbar"], "gbar")
    assert_vec_close(pb, w_ref, "params")
    assert_vec_close(mb, m_ref, "m")
    assert_vec_close(vb, v_ref, "v")

    # ... and against the existing entry point: identical bits (Q is NaN in both: compare the
    # header and shard records as bit patterns)
    assert torch.equal(sa.view(torch.int64), sb.view(torch.int64))
    assert torch.equal(ba, bb)
    for a, b in ((ga, gb), (pa, pb), (ma, mb), (va, vb)):
        assert torch.equal(a, b)


def test_noalloc_matches_oracle_and_existing_entry_point_twice_in_a_row():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    torch.cuda.set_device(0)
    # first call: large problem (8192-element chunks), several shards
    _run_pair(K=8, d=(1 << 23) + 40_001, dtype=torch.bfloat16, n_shards=4, step=7, seed=41)
    # second call straight after it: smaller problem, other dtype and chunk size; the shared
    # array still holds the first call's records beyond this call's chunks
    _run_pair(K=3, d=100_003, dtype=torch.float32, n_shards=1, step=1, seed=43)


def test_binding_refuses_a_stats_buffer_without_the_shard_records():
    torch.cuda.set_device(0)
    p = torch.zeros(8, device=DEV)
    with pytest.raises(ValueError):
        absnt.abs_normtest_adamw_noalloc([p.bfloat16()], 0.1, 8,
                                         torch.zeros(4, dtype=torch.float64, device=DEV), None,
                                         torch.zeros(1, dtype=torch.int64, device=DEV), p,
                                         p.clone(), p.clone(), HP, 1)
    # and the reverse mistake: a header-only buffer handed to the plain call
    with pytest.raises(ValueError):
        absnt.abs_normtest_adamw([p.bfloat16()], 0.1, 8,
                                 torch.zeros(binding.ABS_STATS_HEADER + binding.ABS_SHARD_STRIDE,
                                             dtype=torch.float64, device=DEV), None,
                                 torch.zeros(1, dtype=torch.int64, device=DEV), p, p.clone(),
                                 p.clone(), HP, 1)
