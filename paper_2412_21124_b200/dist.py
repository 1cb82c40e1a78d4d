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
  share_across_ranks, ddp_normtest_adamw
                      the DDP layout of Sec. 3.2 (DDP-Norm): every rank holds the gradient of
                      its own minibatch for the whole vector and makes it addressable by its
                      peers; rank r then runs the fused call on index range r of all ranks'
                      buffers, so the gradient exchange is the kernel's own loads over NVLink
                      (no all-reduce of d elements, no second all-reduce for the variance)
  max_over_ranks      max-reduction used for timing
"""
import os
import pickle

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


def rank_range(d, rank, world, align=1):
    """[lo, hi) of the flat vector owned by `rank`: equal contiguous ranges of whole units of
    `align` coordinates (the last unit may be short), the first ranks holding one extra unit
    where the units do not divide evenly.  align = 1: the first d % world ranks hold one
    extra coordinate."""
    units = -(-int(d) // int(align))
    q, r = divmod(units, int(world))
    lo = rank * q + min(rank, r)
    hi = lo + q + (1 if rank < r else 0)
    return min(lo * align, int(d)), min(hi * align, int(d))


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


def share_across_ranks(t, group=None):
    """Makes this rank's CUDA tensor `t` addressable by every rank of the group and returns the
    list, in rank order, of all ranks' tensors as this process sees them (its own entry is `t`
    itself; the others are views of the owners' device memory, opened from inter-process
    handles, living on the owner's device index).  Collective; call it once per buffer and
    keep `t` alive while any rank uses the views.  Every process must see all GPUs of the node
    under the same indices."""
    from multiprocessing.reduction import ForkingPickler
    import torch.multiprocessing.reductions  # noqa: F401  (registers the CUDA tensor reducer)
    if not (dist.is_initialized() and dist.get_world_size(group) > 1):
        return [t]
    if not t.is_cuda:
        raise ValueError("only CUDA tensors can be shared across ranks")
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    blobs = [None] * world
    dist.all_gather_object(blobs, bytes(ForkingPickler.dumps(t)), group=group)
    return [t if r == rank else pickle.loads(blobs[r]) for r in range(world)]


def _all_ranks_reached(group=None):
    """Everything this rank has enqueued on its current stream so far is complete, on every
    rank, before anything enqueued after this call runs.  NCCL: a one-element all-reduce on
    the stream (the host does not wait); other backends: stream synchronise + host barrier."""
    if not (dist.is_initialized() and dist.get_world_size(group) > 1):
        return
    if dist.get_backend(group) == "nccl":
        dist.all_reduce(torch.zeros(1, device="cuda"), group=group)
    else:
        torch.cuda.current_stream().synchronize()
        dist.barrier(group=group)


kDdpRangeAlign = 64   # coordinates: rank ranges start on 128-byte (bf16) / 256-byte (fp32) lines


def ddp_normtest_adamw(peer_grads, eta, b_cur, stats_out, b_next_out, params, m_local, v_local,
                       hparams, step, group=None):
    """DDP-Norm step (Sec. 3.2; Algorithm 1 with J workers) with one process per GPU.

    `peer_grads` is `share_across_ranks` of the ranks' own gradient buffers (rank j's entry
    holds the gradient of worker j's minibatch for the whole flat vector, d elements).  Rank r
    runs the fused norm-test + AdamW call on index range r (`rank_range` with
    align = kDdpRangeAlign, so that every range starts on a vector boundary) of ALL J buffers:
    its loads of the other ranks' ranges cross NVLink once, which is the reduce-scatter of
    the gradient average done by the kernel's own loads, and the variance sum of Eq. 5 comes
    out of the same pass.  `params` is this rank's full replica (d fp32 values) and is
    updated in place on range r; `m_local`, `v_local` are the moments of range r only (no
    other rank needs them).  Then the three sums per rank are gathered and added in rank
    order (every rank takes the same decision from the same bits) and the updated ranges are
    broadcast so that every replica of `params` is whole again.

    Ordering: the call starts with a rendezvous -- no rank reads a peer's gradient before that
    peer's stream has finished writing it -- and the closing broadcasts are the second one:
    when they return on a rank, every rank's kernel has read what it needed, so the gradient
    buffers may be overwritten.  Returns the dict of `abs_combine_sums`."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    if len(peer_grads) != world:
        raise ValueError("peer_grads must hold one buffer per rank")
    d = params.numel()
    lo, hi = rank_range(d, rank, world, kDdpRangeAlign)
    _all_ranks_reached(group)
    binding.abs_normtest_adamw([g[lo:hi] for g in peer_grads], eta, b_cur, stats_out, None,
                               b_next_out, params[lo:hi], m_local, v_local, hparams, step,
                               peer_grads=True)
    local = stats_out.view(torch.float64)[binding.ABS_STAT_N2:binding.ABS_STAT_Q + 1]
    out = binding.abs_combine_sums(_gather_rank_rows(local, group), world, eta, b_cur)
    if world > 1:
        for r in range(world):
            r_lo, r_hi = rank_range(d, r, world, kDdpRangeAlign)
            if r_hi > r_lo:
                dist.broadcast(params[r_lo:r_hi], src=dist.get_global_rank(group, r)
                               if group is not None else r, group=group)
    return out


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
