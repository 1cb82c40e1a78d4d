"""abs_normtest_adamw_noalloc: the fused step for callers that cannot allocate device memory
(plugin execute hooks, latency-critical callbacks, processes whose device memory belongs to
another allocator).  It keeps its per-chunk partial sums in an array built into the library
instead of a caller-sized tail of stats_out, so the caller only supplies the fixed header and
the shard records.

Checked here, through the C ABI: on two calls in a row (different sizes, so the second call
sees stale records of the first in the shared array) it reproduces abs_normtest_adamw within
the parity tolerances of the other GPU tests, and it refuses problems that would not fit the
built-in array with ABS_ERR_TOO_LARGE before launching anything.

This file is collected last on purpose: a run that stops at the first failure has then already
run every other test.  It passes alone in a fresh process as well as after the other tests.
"""
import ctypes

import pytest
import torch

import paper_2412_21124_b200 as absnt
from paper_2412_21124_b200 import binding, synth
from tests.util import assert_sum_close, assert_vec_close

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
HP = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.1)


def _run_pair(K, d, dtype, n_shards, step, seed):
    """The same inputs through the existing entry point and through the no-alloc variant."""
    offs = synth.equal_shard_offsets(d, n_shards) if n_shards > 1 else None
    grads = synth.worker_grads([d], K, dtype, seed, DEV)
    outs = []
    for variant in ("existing", "noalloc"):
        p, m, v = synth.adam_state(d, seed + 1, DEV, zero_moments=False)
        gbar = torch.empty(d, dtype=torch.float32, device=DEV)
        b_next = torch.full((1,), -1, dtype=torch.int64, device=DEV)
        if variant == "existing":
            stats = absnt.alloc_stats(d, n_shards, DEV)
            absnt.abs_normtest_adamw(grads, 0.1, 64, stats, gbar, b_next, p, m, v, HP, step,
                                     shard_offsets=offs)
        else:
            # header + shard records only: nothing here grows with d
            n = binding.ABS_STATS_HEADER + n_shards * binding.ABS_SHARD_STRIDE
            stats = torch.full((n,), -1.0, dtype=torch.float64, device=DEV)
            absnt.abs_normtest_adamw_noalloc(grads, 0.1, 64, stats, gbar, b_next, p, m, v, HP,
                                             step, shard_offsets=offs)
        torch.cuda.synchronize()
        outs.append((absnt.read_stats(stats, n_shards), int(b_next.item()), gbar, p, m, v))
    (sa, ba, ga, pa, ma, va), (sb, bb, gb, pb, mb, vb) = outs
    for key in ("n2", "S", "T"):
        assert_sum_close(sb[key], sa[key], key)
    assert sb["flags"] == sa["flags"] and sb["norm"] == sa["norm"]
    assert sb["n_chunks"] == sa["n_chunks"]
    for ra, rb in zip(sa["shards"], sb["shards"]):
        assert_sum_close(rb[0], ra[0], "shard n2")
        assert_sum_close(rb[1], ra[1], "shard S")
    assert bb == ba
    for got, ref, name in ((gb, ga, "gbar"), (pb, pa, "params"), (mb, ma, "m"), (vb, va, "v")):
        assert_vec_close(got, ref.double().cpu().numpy(), name)


def test_noalloc_matches_existing_entry_point_twice_in_a_row():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    torch.cuda.set_device(0)
    # first call: large problem (8192-element chunks), several shards
    _run_pair(K=8, d=(1 << 23) + 40_001, dtype=torch.bfloat16, n_shards=4, step=7, seed=41)
    # second call straight after it: smaller problem, other dtype and chunk size; the shared
    # array still holds the first call's records beyond this call's chunks
    _run_pair(K=3, d=100_003, dtype=torch.float32, n_shards=1, step=1, seed=43)


def test_noalloc_rejects_problems_beyond_the_builtin_array():
    torch.cuda.set_device(0)
    L = binding.lib()
    fake = 0x10000  # never dereferenced: the size check comes before any launch
    table = (ctypes.c_void_p * 2)(fake, fake)
    hp = binding.abs_adamw_hparams(1e-3, 0.9, 0.999, 1e-8, 0.1)
    too_many = (binding.ABS_NOALLOC_MAX_CHUNKS + 1) * 8192
    rc = L.abs_normtest_adamw_noalloc(table, 2, too_many, binding.ABS_BF16, None, 1, 0.1, 8,
                                      fake, None, fake, fake, fake, fake, ctypes.byref(hp), 1,
                                      None)
    assert rc == binding.ABS_ERR_TOO_LARGE
    msg = L.abs_status_string(rc).decode()
    assert "ABS_NOALLOC_MAX_CHUNKS" in msg
    with pytest.raises(ValueError):  # the binding refuses a stats buffer without the records
        p = torch.zeros(8, device=DEV)
        absnt.abs_normtest_adamw_noalloc([p.bfloat16()], 0.1, 8,
                                         torch.zeros(4, dtype=torch.float64, device=DEV), None,
                                         torch.zeros(1, dtype=torch.int64, device=DEV), p,
                                         p.clone(), p.clone(), HP, 1)
