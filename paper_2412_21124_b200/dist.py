"""Multi-process plumbing (one process per GPU, torch.distributed).

The norm-test + AdamW step is separable per coordinate, so it needs no data-path
collective: ranks either run independent replicas, or each rank owns an index range of
the flat vector (the FSDP layout of Sec. 3.3) and only the three fp64 sums per rank
cross the wire.  This module holds that small host-side logic:

  rank_range          the contiguous index range a rank owns
  combine_rank_sums   all-gather of {n2, S, Q} per rank; the rank-ordered sum and the
                      decision are the library's abs_combine_sums, called with the same
                      rows on every rank (so all ranks take the same bit-identical decision)
  sharded_normtest_adamw
                      the fused step on this rank's index range followed by that exchange:
                      the multi-GPU form of FSDP-Norm (Sec. 3.3; Algorithm 1 with the shard
                      sums "concatenated")
  max_over_ranks      max-reduction used for timing
"""
import os

import torch
import torch.distributed as dist

from . import binding


def init_from_env(backend=None):
    """Initialises the default process group from RANK / WORLD_SIZE / MASTER_* when
    WORLD_SIZE > 1.  Returns (rank, world_size, local_rank)."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", str(rank)))
    if world > 1 and not dist.is_initialized():
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if backend == "nccl":
            torch.cuda.set_device(local_rank)
            dist.init_process_group(backend, device_id=torch.device("cuda", local_rank))
        else:
            dist.init_process_group(backend)
    return rank, world, local_rank


def rank_range(d, rank, world):
    """[lo, hi) of the flat vector owned by `rank`: equal contiguous ranges, the first
    d % world ranks holding one extra coordinate."""
    q, r = divmod(int(d), int(world))
    lo = rank * q + min(rank, r)
    return lo, lo + q + (1 if rank < r else 0)


def combine_rank_sums(n2, S, Q, K, eta, b_cur, device="cpu", group=None):
    """Each rank passes the sums of its own index range; every rank returns the same
    dict of totals (added in rank order), statistic, flags and b_next."""
    local = torch.tensor([n2, S, Q], dtype=torch.float64, device=device)
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        parts = [torch.empty_like(local) for _ in range(dist.get_world_size(group))]
        dist.all_gather(parts, local, group=group)
    else:
        parts = [local]
    # the rank-ordered sum and the decision are the library's (abs_combine_sums)
    return binding.abs_combine_sums([part.tolist() for part in parts], K, eta, b_cur)


def _gather_rank_rows(local, group=None):
    """all-gather of one small fp64 row per rank -> list of rows in rank order.  The row
    travels on the device the backend works with (NCCL: this rank's GPU, gloo: the host)."""
    if not (dist.is_initialized() and dist.get_world_size(group) > 1):
        return [local.tolist()]
    on_gpu = dist.get_backend(group) == "nccl"
    if on_gpu and not local.is_cuda:
        local = local.cuda()
    if not on_gpu and local.is_cuda:
        local = local.cpu()  # synchronises with the stream that wrote the sums
    parts = [torch.empty_like(local) for _ in range(dist.get_world_size(group))]
    dist.all_gather(parts, local.contiguous(), group=group)
    return [part.tolist() for part in parts]


def sharded_normtest_adamw(grads_local, eta, b_cur, stats_out, gbar_out, b_next_out, params_local,
                           m_local, v_local, hparams, step, group=None):
    """FSDP-Norm step (Sec. 3.3) with one process per GPU.  Every rank holds the same index
    range [lo, hi) of all K gradient buffers and of params / m / v (`rank_range`) and passes
    those slices.  The rank's GPU runs the fused norm-test + AdamW call on its range; the only
    exchange is an all-gather of the three sums of the rank (24 bytes), added in rank order on
    every rank, so that all ranks compute the same T and b_next bit for bit.  AdamW is
    element-wise and needs no exchange.

    `b_next_out` receives the local range's own decision (what the kernel wrote); the global
    one is in the returned dict: n2, S, Q (NaN: the fused call does not compute it), T, flags,
    b_next.  Synchronises the host with the stream (the sums are read back)."""
    binding.abs_normtest_adamw(grads_local, eta, b_cur, stats_out, gbar_out, b_next_out,
                               params_local, m_local, v_local, hparams, step)
    local = stats_out.view(torch.float64)[binding.ABS_STAT_N2:binding.ABS_STAT_Q + 1]
    return binding.abs_combine_sums(_gather_rank_rows(local, group), len(grads_local), eta, b_cur)


def barrier(device=None):
    if dist.is_initialized() and dist.get_world_size() > 1:
        if device is not None and torch.device(device).type == "cuda":
            dist.barrier(device_ids=[torch.device(device).index])
        else:
            dist.barrier()


def max_over_ranks(x, device="cpu"):
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    if dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def max_over_ranks_vec(xs, device="cpu"):
    """Element-wise max over ranks of a list of floats (one all-reduce)."""
    t = torch.tensor([float(x) for x in xs], dtype=torch.float64, device=device)
    if dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def sum_over_ranks(x, device="cpu"):
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    if dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
