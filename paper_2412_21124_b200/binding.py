"""Thin ctypes binding of ``include/abs_normtest.h``.

Argument marshalling only: every function here validates tensor types, collects raw
device pointers and the current CUDA stream, and calls the C entry point of the same
name.  All arithmetic of the path runs in the CUDA kernels of ``libabs_normtest.so``.
There is no CPU fallback: if the library has not been built, the first call raises.
"""
import ctypes
import os

import torch

from . import build as _build

ABS_F32, ABS_BF16 = 0, 1
ABS_OK = 0
ABS_ERR_NULL, ABS_ERR_RANGE, ABS_ERR_SHARDS, ABS_ERR_ALIGN, ABS_ERR_DTYPE, ABS_ERR_CUDA = (
    -1, -2, -3, -4, -5, -6)
ABS_ERR_TOO_LARGE = -7
ABS_ERR_ALIAS = -8
ABS_NOALLOC_MAX_CHUNKS = 131072
ABS_MAX_WORKERS, ABS_MAX_SHARDS = 1024, 128
(ABS_STAT_N2, ABS_STAT_S, ABS_STAT_Q, ABS_STAT_T, ABS_STAT_FLAGS, ABS_STAT_NORM,
 ABS_STAT_NCHUNKS, ABS_STAT_ARGMAX) = range(8)
ABS_STATS_HEADER, ABS_SHARD_STRIDE = 8, 4
ABS_FLAG_DEGENERATE, ABS_FLAG_NONFINITE, ABS_FLAG_VIOLATED = 1, 2, 4


class abs_adamw_hparams(ctypes.Structure):
    _fields_ = [("lr", ctypes.c_float), ("beta1", ctypes.c_float), ("beta2", ctypes.c_float),
                ("eps", ctypes.c_float), ("weight_decay", ctypes.c_float)]


class AbsError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        msg = lib().abs_status_string(status).decode()
        if status == ABS_ERR_CUDA:
            msg += " [cudaError %d]" % lib().abs_last_cuda_error()
        super().__init__("%s: %s (status %d)" % (where, msg, status))


_lib = None


def lib():
    """The loaded shared library.  Raises when it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    # ABS_NORMTEST_LIB: a library built elsewhere (another build of the same sources)
    path = os.environ.get("ABS_NORMTEST_LIB") or _build.LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError(
            "libabs_normtest.so is missing: build it with `python -m paper_2412_21124_b200.build` "
            "(there is no CPU fallback)")
    L = ctypes.CDLL(path)
    i64, dbl, ptr, cint, sz = (ctypes.c_int64, ctypes.c_double, ctypes.c_void_p, ctypes.c_int,
                               ctypes.c_size_t)
    L.abs_stats_bytes.restype = sz
    L.abs_stats_bytes.argtypes = [i64, cint]
    L.abs_persample_stats_bytes.restype = sz
    L.abs_persample_stats_bytes.argtypes = [i64, i64]
    L.abs_norm_test.restype = cint
    L.abs_norm_test.argtypes = [ptr, cint, i64, cint, ptr, cint, dbl, i64, ptr, ptr, ptr, ptr]
    L.abs_adamw_step.restype = cint
    L.abs_adamw_step.argtypes = [ptr, ptr, ptr, ptr, i64, ptr, i64, ptr]
    L.abs_adamw_step_clipped.restype = cint
    L.abs_adamw_step_clipped.argtypes = [ptr, ptr, ptr, ptr, i64, ptr, i64, dbl, ptr, ptr]
    L.abs_normtest_adamw.restype = cint
    L.abs_normtest_adamw.argtypes = [ptr, cint, i64, cint, ptr, cint, dbl, i64, ptr, ptr, ptr,
                                     ptr, ptr, ptr, ptr, i64, ptr]
    L.abs_normtest_adamw_noalloc.restype = cint
    L.abs_normtest_adamw_noalloc.argtypes = list(L.abs_normtest_adamw.argtypes)
    L.abs_normtest_adamw_clip_prev.restype = cint
    L.abs_normtest_adamw_clip_prev.argtypes = [ptr, cint, i64, cint, ptr, cint, dbl, i64, ptr, ptr,
                                               ptr, ptr, ptr, ptr, ptr, i64, dbl, ptr, ptr]
    L.abs_norm_test_coordwise.restype = cint
    L.abs_norm_test_coordwise.argtypes = list(L.abs_norm_test.argtypes)
    L.abs_norm_test_q.restype = cint
    L.abs_norm_test_q.argtypes = list(L.abs_norm_test.argtypes)
    L.abs_norm_test_accumulate.restype = cint
    L.abs_norm_test_accumulate.argtypes = [ptr, cint, i64, cint, ptr, cint, i64, dbl, i64, ptr,
                                           ptr, ptr, ptr]
    L.abs_norm_test_accumulate_adamw.restype = cint
    L.abs_norm_test_accumulate_adamw.argtypes = [ptr, cint, i64, cint, ptr, cint, i64, dbl, i64,
                                                 ptr, ptr, ptr, ptr, ptr, ptr, ptr, ptr, i64, ptr]
    L.abs_normtest_adamw_coordwise.restype = cint
    L.abs_normtest_adamw_coordwise.argtypes = list(L.abs_normtest_adamw.argtypes)
    L.abs_normtest_adamw_mixed.restype = cint
    L.abs_normtest_adamw_mixed.argtypes = [ptr, cint, i64, cint, ptr, cint, dbl, i64, ptr, ptr,
                                           ptr, ptr, ptr, ptr, ptr, ptr, i64, ptr]
    L.abs_adamw_step_mixed.restype = cint
    L.abs_adamw_step_mixed.argtypes = [ptr, ptr, ptr, ptr, ptr, i64, ptr, i64, dbl, ptr, ptr]
    L.abs_persample_norm_test.restype = cint
    L.abs_persample_norm_test.argtypes = [ptr, i64, i64, i64, cint, dbl, ptr, ptr, ptr, ptr]
    L.abs_persample_norm_test_coordwise.restype = cint
    L.abs_persample_norm_test_coordwise.argtypes = list(L.abs_persample_norm_test.argtypes)
    L.abs_noalloc_fits.restype = cint
    L.abs_noalloc_fits.argtypes = [i64, ptr, cint]
    L.abs_combine_sums.restype = i64
    L.abs_combine_sums.argtypes = [ptr, cint, dbl, dbl, i64, ptr, ptr, ptr]
    L.abs_decide.restype = i64
    L.abs_decide.argtypes = [dbl, dbl, dbl, dbl, i64, ptr, ptr]
    L.abs_round_batch.restype = i64
    L.abs_round_batch.argtypes = [i64, i64, i64]
    L.abs_schedule_init.restype = cint
    L.abs_schedule_init.argtypes = [ptr, i64, i64, i64, i64, i64, i64]
    L.abs_schedule_test_due.restype = cint
    L.abs_schedule_test_due.argtypes = [ptr]
    L.abs_schedule_advance.restype = cint
    L.abs_schedule_advance.argtypes = [ptr, i64]
    L.abs_selftest_bounded_wait.restype = cint
    L.abs_selftest_bounded_wait.argtypes = [cint, ptr, ptr]
    L.abs_status_string.restype = ctypes.c_char_p
    L.abs_status_string.argtypes = [cint]
    L.abs_last_cuda_error.restype = cint
    L.abs_last_cuda_error.argtypes = []
    _lib = L
    return L


# ------------------------------------------------------------------------- marshalling
def _dtype_code(t):
    if t.dtype == torch.float32:
        return ABS_F32
    if t.dtype == torch.bfloat16:
        return ABS_BF16
    raise TypeError("gradient buffers must be float32 or bfloat16, got %s" % t.dtype)


def _check_f32_vec(t, d, name):
    if t.dtype != torch.float32 or t.dim() != 1 or t.numel() != d or t.stride(0) != 1:
        raise TypeError("%s must be a contiguous float32 vector of %d elements" % (name, d))
    if not t.is_cuda:
        raise TypeError("%s must live on a CUDA device" % name)


def _check_stats(t, nbytes, name="stats_out"):
    """stats_out must be a CUDA buffer of at least `nbytes` bytes, 16-byte aligned: the kernels
    write every chunk record (and the per-sample work space) without a bounds check."""
    if nbytes <= 0:
        raise ValueError("invalid problem size for %s" % name)
    if not getattr(t, "is_cuda", False) or not t.is_contiguous():
        raise TypeError("%s must be a contiguous CUDA tensor" % name)
    if t.numel() * t.element_size() < nbytes:
        raise ValueError("%s holds %d bytes, the call needs %d (see abs_stats_bytes)"
                         % (name, t.numel() * t.element_size(), nbytes))
    if t.data_ptr() % 16:
        raise ValueError("%s must be 16-byte aligned" % name)


def _check_b_next(t):
    if (not getattr(t, "is_cuda", False) or t.dtype != torch.int64 or t.numel() < 1
            or not t.is_contiguous()):
        raise TypeError("b_next_out must be a CUDA int64 tensor with at least one element")


def _check_one_device(*tensors):
    """All buffers of a call live on the CUDA device that is current: the library launches on
    the current device and caches per-device kernel attributes under its index."""
    cur = torch.cuda.current_device()
    for t in tensors:
        if t is None:
            continue
        if not t.is_cuda or t.device.index != cur:
            raise ValueError("every buffer must live on the current CUDA device (cuda:%d), got %s"
                             % (cur, t.device))


def _check_peer_grads(grads):
    """Gradient buffers that may live on other GPUs: each on the current device or on one whose
    memory the current device can address (peer access; a buffer opened from another process's
    handle counts as living on its owner's device)."""
    cur = torch.cuda.current_device()
    for g in grads:
        if not g.is_cuda:
            raise ValueError("gradient buffers must be CUDA tensors, got %s" % g.device)
        if g.device.index != cur and not torch.cuda.can_device_access_peer(cur, g.device.index):
            raise ValueError("cuda:%d cannot address the memory of %s" % (cur, g.device))


def _stream(stream):
    if stream is None:
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, torch.cuda.Stream):
        return ctypes.c_void_p(stream.cuda_stream)
    return ctypes.c_void_p(int(stream))


def _grad_table(grads):
    K = len(grads)
    if K < 1:
        raise ValueError("need at least one gradient buffer")
    g0 = grads[0]
    d, code = g0.numel(), _dtype_code(g0)
    for g in grads:
        if (not g.is_cuda or g.dtype != g0.dtype or g.dim() != 1 or g.numel() != d
                or g.stride(0) != 1):
            raise TypeError("gradient buffers must be contiguous CUDA vectors of one dtype/length")
    table = (ctypes.c_void_p * K)(*[g.data_ptr() for g in grads])
    return table, K, d, code


def _offsets(shard_offsets):
    if shard_offsets is None:
        return None, 1
    offs = (ctypes.c_int64 * len(shard_offsets))(*[int(o) for o in shard_offsets])
    return offs, len(shard_offsets) - 1


def _hparams(hp):
    if isinstance(hp, abs_adamw_hparams):
        return hp
    return abs_adamw_hparams(float(hp["lr"]), float(hp["beta1"]), float(hp["beta2"]),
                             float(hp["eps"]), float(hp["weight_decay"]))


def abs_stats_bytes(d, n_shards=1):
    return int(lib().abs_stats_bytes(int(d), int(n_shards)))


def abs_persample_stats_bytes(b, d):
    return int(lib().abs_persample_stats_bytes(int(b), int(d)))


def alloc_stats(d, n_shards=1, device="cuda"):
    """A stats_out buffer (float64 tensor) of the size abs_stats_bytes asks for."""
    nbytes = abs_stats_bytes(d, n_shards)
    if nbytes == 0:
        raise ValueError("invalid (d, n_shards)")
    return torch.empty(nbytes // 8, dtype=torch.float64, device=device)


def alloc_persample_stats(b, d, device="cuda"):
    """A zero-filled stats_out for abs_persample_norm_test (its ticket counters start at 0)."""
    nbytes = abs_persample_stats_bytes(b, d)
    if nbytes == 0:
        raise ValueError("invalid (b, d)")
    return torch.zeros(nbytes // 8, dtype=torch.float64, device=device)


# ------------------------------------------------------------------------- entry points
def abs_norm_test(grads, eta, b_cur, stats_out, gbar_out, b_next_out, shard_offsets=None,
                  stream=None, _entry="abs_norm_test"):
    table, K, d, code = _grad_table(grads)
    offs, n_shards = _offsets(shard_offsets)
    _check_f32_vec(gbar_out, d, "gbar_out")
    _check_stats(stats_out, abs_stats_bytes(d, n_shards))
    _check_b_next(b_next_out)
    _check_one_device(*grads, stats_out, gbar_out, b_next_out)
    rc = getattr(lib(), _entry)(table, K, d, code, offs, n_shards, float(eta), int(b_cur),
                                stats_out.data_ptr(), gbar_out.data_ptr(), b_next_out.data_ptr(),
                                _stream(stream))
    if rc != ABS_OK:
        raise AbsError(rc, _entry)


def abs_norm_test_accumulate(grads, count_in, eta, b_cur, stats_inout, mean_inout, b_next_out,
                             shard_offsets=None, stream=None):
    """Merges the K new gradient buffers into the running mean (`mean_inout`, d floats) and the
    running sums (`stats_inout`) of the `count_in` gradients merged by the earlier calls of this
    step; count_in = 0 starts a step.  After the call the outputs are those of the test over all
    count_in + K gradients."""
    table, K, d, code = _grad_table(grads)
    offs, n_shards = _offsets(shard_offsets)
    _check_f32_vec(mean_inout, d, "mean_inout")
    _check_stats(stats_inout, abs_stats_bytes(d, n_shards))
    _check_b_next(b_next_out)
    _check_one_device(*grads, stats_inout, mean_inout, b_next_out)
    rc = lib().abs_norm_test_accumulate(table, K, d, code, offs, n_shards, int(count_in),
                                        float(eta), int(b_cur), stats_inout.data_ptr(),
                                        mean_inout.data_ptr(), b_next_out.data_ptr(),
                                        _stream(stream))
    if rc != ABS_OK:
        raise AbsError(rc, "abs_norm_test_accumulate")


def abs_norm_test_accumulate_adamw(grads, count_in, eta, b_cur, stats_inout, mean_in, gbar_out,
                                   b_next_out, params, m, v, hparams, step, shard_offsets=None,
                                   stream=None):
    """The closing call of a step in the carry-in form, fused with AdamW: merges the last K
    buffers into the running mean `mean_in` (None when count_in = 0) and updates params / m / v
    with the final mean in the same pass; `gbar_out` (None, or `mean_in` itself) receives it."""
    table, K, d, code = _grad_table(grads)
    offs, n_shards = _offsets(shard_offsets)
    for t, name in ((params, "params"), (m, "m"), (v, "v")):
        _check_f32_vec(t, d, name)
    for t, name in ((mean_in, "mean_in"), (gbar_out, "gbar_out")):
        if t is not None:
            _check_f32_vec(t, d, name)
    if count_in > 0 and mean_in is None:
        raise ValueError("count_in > 0 needs the running mean")
    _check_stats(stats_inout, abs_stats_bytes(d, n_shards))
    _check_b_next(b_next_out)
    _check_one_device(*grads, stats_inout, mean_in, gbar_out, b_next_out, params, m, v)
    hp = _hparams(hparams)
    rc = lib().abs_norm_test_accumulate_adamw(
        table, K, d, code, offs, n_shards, int(count_in), float(eta), int(b_cur),
        stats_inout.data_ptr(), mean_in.data_ptr() if mean_in is not None else None,
        gbar_out.data_ptr() if gbar_out is not None else None, b_next_out.data_ptr(),
        params.data_ptr(), m.data_ptr(), v.data_ptr(), ctypes.byref(hp), int(step),
        _stream(stream))
    if rc != ABS_OK:
        raise AbsError(rc, "abs_norm_test_accumulate_adamw")


def abs_norm_test_q(grads, eta, b_cur, stats_out, gbar_out, b_next_out, shard_offsets=None,
                    stream=None):
    """abs_norm_test that also computes the diagnostic Q = sum_k ||g_k||^2."""
    abs_norm_test(grads, eta, b_cur, stats_out, gbar_out, b_next_out, shard_offsets, stream,
                  _entry="abs_norm_test_q")


def abs_norm_test_coordwise(grads, eta, b_cur, stats_out, gbar_out, b_next_out,
                            shard_offsets=None, stream=None):
    """The coordinate-wise test: T = max_i T_i, its coordinate in the ABS_STAT_ARGMAX slot."""
    abs_norm_test(grads, eta, b_cur, stats_out, gbar_out, b_next_out, shard_offsets, stream,
                  _entry="abs_norm_test_coordwise")


def abs_adamw_step(params, gbar, m, v, hparams, step, stream=None):
    d = params.numel()
    for t, name in ((params, "params"), (gbar, "gbar"), (m, "m"), (v, "v")):
        _check_f32_vec(t, d, name)
    _check_one_device(params, gbar, m, v)
    hp = _hparams(hparams)
    rc = lib().abs_adamw_step(params.data_ptr(), gbar.data_ptr(), m.data_ptr(), v.data_ptr(), d,
                              ctypes.byref(hp), int(step), _stream(stream))
    if rc != ABS_OK:
        raise AbsError(rc, "abs_adamw_step")


def abs_adamw_step_clipped(params, gbar, m, v, hparams, step, max_norm, stats_in, stream=None):
    """AdamW on gbar clipped to global norm max_norm; ||gbar||^2 is read on the device from
    `stats_in` (the stats_out of the abs_norm_test that produced gbar)."""
    d = params.numel()
    for t, name in ((params, "params"), (gbar, "gbar"), (m, "m"), (v, "v")):
        _check_f32_vec(t, d, name)
    _check_stats(stats_in, 8 * ABS_STATS_HEADER, "stats_in")
    _check_one_device(params, gbar, m, v, stats_in)
    hp = _hparams(hparams)
    rc = lib().abs_adamw_step_clipped(params.data_ptr(), gbar.data_ptr(), m.data_ptr(),
                                      v.data_ptr(), d, ctypes.byref(hp), int(step),
                                      float(max_norm), stats_in.data_ptr(), _stream(stream))
    if rc != ABS_OK:
        raise AbsError(rc, "abs_adamw_step_clipped")


def abs_normtest_adamw(grads, eta, b_cur, stats_out, gbar_out, b_next_out, params, m, v, hparams,
                       step, shard_offsets=None, stream=None, _entry="abs_normtest_adamw",
                       peer_grads=False):
    """The fused step.  `peer_grads=True` lets the gradient buffers (read-only inputs) live on
    other GPUs whose memory the current device can address: the kernel then loads them over
    NVLink (plain loads and non-multicast bulk copies); everything written stays local."""
    table, K, d, code = _grad_table(grads)
    offs, n_shards = _offsets(shard_offsets)
    for t, name in ((params, "params"), (m, "m"), (v, "v")):
        _check_f32_vec(t, d, name)
    if gbar_out is not None:
        _check_f32_vec(gbar_out, d, "gbar_out")
    _check_stats(stats_out, abs_stats_bytes(d, n_shards))
    _check_b_next(b_next_out)
    if peer_grads:
        _check_peer_grads(grads)
        _check_one_device(stats_out, gbar_out, b_next_out, params, m, v)
    else:
        _check_one_device(*grads, stats_out, gbar_out, b_next_out, params, m, v)
    hp = _hparams(hparams)
    rc = getattr(lib(), _entry)(table, K, d, code, offs, n_shards, float(eta), int(b_cur),
                                stats_out.data_ptr(),
                                gbar_out.data_ptr() if gbar_out is not None else None,
                                b_next_out.data_ptr(), params.data_ptr(), m.data_ptr(),
                                v.data_ptr(), ctypes.byref(hp), int(step), _stream(stream))
    if rc != ABS_OK:
        raise AbsError(rc, _entry)


def abs_normtest_adamw_coordwise(grads, eta, b_cur, stats_out, gbar_out, b_next_out, params, m, v,
                                 hparams, step, shard_offsets=None, stream=None):
    """The fused step with the coordinate-wise test as its decision."""
    abs_normtest_adamw(grads, eta, b_cur, stats_out, gbar_out, b_next_out, params, m, v, hparams,
                       step, shard_offsets, stream, _entry="abs_normtest_adamw_coordwise")


def abs_normtest_adamw_clip_prev(grads, eta, b_cur, stats_out, gbar_out, b_next_out, params, m, v,
                                 hparams, step, max_norm, stats_prev, shard_offsets=None,
                                 stream=None):
    """The fused step with the gradient clipped by the previous step's global norm, read on the
    device from `stats_prev` (the previous call's stats_out; may be `stats_out` itself; None =
    no clipping).  A single-pass approximation, not what the paper's experiments compute."""
    table, K, d, code = _grad_table(grads)
    offs, n_shards = _offsets(shard_offsets)
    for t, name in ((params, "params"), (m, "m"), (v, "v")):
        _check_f32_vec(t, d, name)
    if gbar_out is not None:
        _check_f32_vec(gbar_out, d, "gbar_out")
    _check_stats(stats_out, abs_stats_bytes(d, n_shards))
    if stats_prev is not None:
        _check_stats(stats_prev, 8 * ABS_STATS_HEADER, "stats_prev")
    _check_b_next(b_next_out)
    _check_one_device(*grads, stats_out, gbar_out, b_next_out, params, m, v, stats_prev)
    hp = _hparams(hparams)
    rc = lib().abs_normtest_adamw_clip_prev(
        table, K, d, code, offs, n_shards, float(eta), int(b_cur), stats_out.data_ptr(),
        gbar_out.data_ptr() if gbar_out is not None else None, b_next_out.data_ptr(),
        params.data_ptr(), m.data_ptr(), v.data_ptr(), ctypes.byref(hp), int(step),
        float(max_norm), stats_prev.data_ptr() if stats_prev is not None else None,
        _stream(stream))
    if rc != ABS_OK:
        raise AbsError(rc, "abs_normtest_adamw_clip_prev")


def _check_bf16_vec(t, d, name):
    if t.dtype != torch.bfloat16 or t.dim() != 1 or t.numel() != d or t.stride(0) != 1:
        raise TypeError("%s must be a contiguous bfloat16 vector of %d elements" % (name, d))
    if not t.is_cuda:
        raise TypeError("%s must live on a CUDA device" % name)


def abs_normtest_adamw_mixed(grads, eta, b_cur, stats_out, gbar_out, b_next_out, params, m, v,
                             params_bf16_out, hparams, step, shard_offsets=None, stream=None):
    """abs_normtest_adamw that also writes a bfloat16 copy of the updated parameters."""
    table, K, d, code = _grad_table(grads)
    offs, n_shards = _offsets(shard_offsets)
    for t, name in ((params, "params"), (m, "m"), (v, "v")):
        _check_f32_vec(t, d, name)
    _check_bf16_vec(params_bf16_out, d, "params_bf16_out")
    if gbar_out is not None:
        _check_f32_vec(gbar_out, d, "gbar_out")
    _check_stats(stats_out, abs_stats_bytes(d, n_shards))
    _check_b_next(b_next_out)
    _check_one_device(*grads, stats_out, gbar_out, b_next_out, params, m, v, params_bf16_out)
    hp = _hparams(hparams)
    rc = lib().abs_normtest_adamw_mixed(table, K, d, code, offs, n_shards, float(eta),
                                        int(b_cur), stats_out.data_ptr(),
                                        gbar_out.data_ptr() if gbar_out is not None else None,
                                        b_next_out.data_ptr(), params.data_ptr(), m.data_ptr(),
                                        v.data_ptr(), params_bf16_out.data_ptr(),
                                        ctypes.byref(hp), int(step), _stream(stream))
    if rc != ABS_OK:
        raise AbsError(rc, "abs_normtest_adamw_mixed")


def abs_adamw_step_mixed(params, gbar, m, v, params_bf16_out, hparams, step, max_norm=0.0,
                         stats_in=None, stream=None):
    """abs_adamw_step (clipped to max_norm when stats_in is given) that also writes a bfloat16
    copy of the updated parameters."""
    d = params.numel()
    for t, name in ((params, "params"), (gbar, "gbar"), (m, "m"), (v, "v")):
        _check_f32_vec(t, d, name)
    _check_bf16_vec(params_bf16_out, d, "params_bf16_out")
    if stats_in is not None:
        _check_stats(stats_in, 8 * ABS_STATS_HEADER, "stats_in")
    _check_one_device(params, gbar, m, v, params_bf16_out, stats_in)
    hp = _hparams(hparams)
    rc = lib().abs_adamw_step_mixed(params.data_ptr(), gbar.data_ptr(), m.data_ptr(),
                                    v.data_ptr(), params_bf16_out.data_ptr(), d,
                                    ctypes.byref(hp), int(step), float(max_norm),
                                    stats_in.data_ptr() if stats_in is not None else None,
                                    _stream(stream))
    if rc != ABS_OK:
        raise AbsError(rc, "abs_adamw_step_mixed")


def abs_normtest_adamw_noalloc(grads, eta, b_cur, stats_out, gbar_out, b_next_out, params, m, v,
                               hparams, step, shard_offsets=None, stream=None):
    """abs_normtest_adamw for callers that cannot allocate device memory: `stats_out` only
    needs ABS_STATS_HEADER + n_shards*ABS_SHARD_STRIDE doubles, the per-chunk records live
    in an array built into the library (shared by all calls on a device, so calls whose GPU
    work overlaps race).  Raises AbsError(ABS_ERR_TOO_LARGE) beyond ABS_NOALLOC_MAX_CHUNKS
    chunks.  Make the first call on a device outside of stream capture."""
    table, K, d, code = _grad_table(grads)
    offs, n_shards = _offsets(shard_offsets)
    for t, name in ((params, "params"), (m, "m"), (v, "v")):
        _check_f32_vec(t, d, name)
    if gbar_out is not None:
        _check_f32_vec(gbar_out, d, "gbar_out")
    _check_stats(stats_out, 8 * (ABS_STATS_HEADER + n_shards * ABS_SHARD_STRIDE))
    _check_b_next(b_next_out)
    _check_one_device(*grads, stats_out, gbar_out, b_next_out, params, m, v)
    hp = _hparams(hparams)
    rc = lib().abs_normtest_adamw_noalloc(table, K, d, code, offs, n_shards, float(eta),
                                          int(b_cur), stats_out.data_ptr(),
                                          gbar_out.data_ptr() if gbar_out is not None else None,
                                          b_next_out.data_ptr(), params.data_ptr(), m.data_ptr(),
                                          v.data_ptr(), ctypes.byref(hp), int(step),
                                          _stream(stream))
    if rc != ABS_OK:
        raise AbsError(rc, "abs_normtest_adamw_noalloc")


class FusedStep:
    """abs_normtest_adamw with the argument marshalling done once.

    A training loop calls the fused step with the same buffers every iteration; only eta,
    b_cur and the step counter change.  This object validates the tensors and builds the
    pointer table once, so each ``run`` is a single C call (a few microseconds of host time
    instead of ~20) -- which matters when d is small enough for the call to be launch-bound.
    The tensors must stay alive and must not be reallocated while the object is in use.
    """

    def __init__(self, grads, stats_out, gbar_out, b_next_out, params, m, v, hparams,
                 shard_offsets=None, params_bf16_out=None, coordwise=False):
        self._keep = (list(grads), stats_out, gbar_out, b_next_out, params, m, v, params_bf16_out)
        self._table, self._K, self._d, self._code = _grad_table(grads)
        self._offs, self._n_shards = _offsets(shard_offsets)
        for t, name in ((params, "params"), (m, "m"), (v, "v")):
            _check_f32_vec(t, self._d, name)
        if gbar_out is not None:
            _check_f32_vec(gbar_out, self._d, "gbar_out")
        _check_stats(stats_out, abs_stats_bytes(self._d, self._n_shards))
        _check_b_next(b_next_out)
        _check_one_device(*grads, stats_out, gbar_out, b_next_out, params, m, v, params_bf16_out)
        self._hp = _hparams(hparams)
        self._hp_ref = ctypes.byref(self._hp)
        self._ptrs = (stats_out.data_ptr(), gbar_out.data_ptr() if gbar_out is not None else None,
                      b_next_out.data_ptr(), params.data_ptr(), m.data_ptr(), v.data_ptr())
        self._fn = lib().abs_normtest_adamw_coordwise if coordwise else lib().abs_normtest_adamw
        self._p16 = None
        if coordwise and params_bf16_out is not None:
            raise ValueError("the coordinate-wise step has no mixed-precision variant")
        if params_bf16_out is not None:  # mixed precision: also the bf16 copy of the parameters
            _check_bf16_vec(params_bf16_out, self._d, "params_bf16_out")
            self._p16 = params_bf16_out.data_ptr()
            self._fn = lib().abs_normtest_adamw_mixed

    def run(self, eta, b_cur, step, stream=None):
        st, gb, bn, p, m, v = self._ptrs
        cu_stream = torch.cuda.current_stream().cuda_stream if stream is None else _stream(stream)
        if self._p16 is None:
            rc = self._fn(self._table, self._K, self._d, self._code, self._offs, self._n_shards,
                          eta, b_cur, st, gb, bn, p, m, v, self._hp_ref, step, cu_stream)
        else:
            rc = self._fn(self._table, self._K, self._d, self._code, self._offs, self._n_shards,
                          eta, b_cur, st, gb, bn, p, m, v, self._p16, self._hp_ref, step, cu_stream)
        if rc != ABS_OK:
            raise AbsError(rc, "abs_normtest_adamw")


def abs_persample_norm_test(G, eta, stats_out, gbar_out, b_next_out, stream=None,
                            _entry="abs_persample_norm_test"):
    if G.dim() != 2 or G.stride(1) != 1 or not G.is_cuda:
        raise TypeError("G must be a CUDA matrix [b, d] with unit column stride")
    b, d, ld = G.shape[0], G.shape[1], G.stride(0)
    _check_f32_vec(gbar_out, d, "gbar_out")
    _check_stats(stats_out, abs_persample_stats_bytes(b, d))
    _check_b_next(b_next_out)
    _check_one_device(G, stats_out, gbar_out, b_next_out)
    rc = getattr(lib(), _entry)(G.data_ptr(), b, d, ld, _dtype_code(G), float(eta),
                                stats_out.data_ptr(), gbar_out.data_ptr(),
                                b_next_out.data_ptr(), _stream(stream))
    if rc != ABS_OK:
        raise AbsError(rc, _entry)


def abs_persample_norm_test_coordwise(G, eta, stats_out, gbar_out, b_next_out, stream=None):
    """The per-sample call with the coordinate-wise test as its decision (T = max over columns,
    the column in the ABS_STAT_ARGMAX slot)."""
    abs_persample_norm_test(G, eta, stats_out, gbar_out, b_next_out, stream,
                            _entry="abs_persample_norm_test_coordwise")


def abs_decide(S, n2, norm, eta, b_cur):
    """Host-side decision; returns (b_next, T, flags)."""
    T, flags = ctypes.c_double(0.0), ctypes.c_int(0)
    b_next = lib().abs_decide(float(S), float(n2), float(norm), float(eta), int(b_cur),
                              ctypes.byref(T), ctypes.byref(flags))
    return int(b_next), T.value, flags.value


def abs_combine_sums(rows, norm, eta, b_cur):
    """rows: one (n2, S, Q) triple per rank, in rank order.  Returns a dict with the totals
    (added in rank order by the library), T, flags and b_next."""
    n = len(rows)
    flat = (ctypes.c_double * (3 * n))(*[float(x) for row in rows for x in row])
    tot = (ctypes.c_double * 3)()
    T, flags = ctypes.c_double(0.0), ctypes.c_int(0)
    b_next = lib().abs_combine_sums(flat, n, float(norm), float(eta), int(b_cur), tot,
                                    ctypes.byref(T), ctypes.byref(flags))
    if b_next < 0:
        raise ValueError("abs_combine_sums rejected its arguments")
    return {"n2": tot[0], "S": tot[1], "Q": tot[2], "T": T.value, "flags": flags.value,
            "b_next": int(b_next)}


def abs_noalloc_fits(d, shard_offsets=None):
    offs, n_shards = _offsets(shard_offsets)
    return bool(lib().abs_noalloc_fits(int(d), offs, n_shards))


def abs_selftest_bounded_wait(polls, stream=None):
    """Runs the staged kernels' bounded wait on a barrier nothing completes.  Returns
    (gave_up, nanoseconds)."""
    out = torch.zeros(2, dtype=torch.int64, device="cuda")
    rc = lib().abs_selftest_bounded_wait(int(polls), out.data_ptr(), _stream(stream))
    if rc != ABS_OK:
        raise AbsError(rc, "abs_selftest_bounded_wait")
    gave_up, ns = out.tolist()  # synchronises
    return bool(gave_up), int(ns)


def abs_round_batch(b_next, J, M):
    return int(lib().abs_round_batch(int(b_next), int(J), int(M)))


class AbsSchedule(ctypes.Structure):
    """struct abs_schedule of the C header (host-side state of Algorithm 1's loop)."""
    _fields_ = [(name, ctypes.c_int64) for name in
                ("J", "M", "micro", "b", "b_max", "max_micro", "interval", "step", "samples")]


def abs_schedule_init(J, M, micro0, b_max, max_micro=0, interval=1):
    s = AbsSchedule()
    rc = lib().abs_schedule_init(ctypes.byref(s), int(J), int(M), int(micro0), int(b_max),
                                 int(max_micro), int(interval))
    if rc != 0:
        raise AbsError(rc, "abs_schedule_init")
    return s


def abs_schedule_test_due(s):
    return bool(lib().abs_schedule_test_due(ctypes.byref(s)))


def abs_schedule_advance(s, b_test):
    rc = lib().abs_schedule_advance(ctypes.byref(s), int(b_test))
    if rc != 0:
        raise AbsError(rc, "abs_schedule_advance")


def read_stats(stats_out, n_shards=1):
    """Copies the header and shard records to the host (synchronises) and names them."""
    n = ABS_STATS_HEADER + n_shards * ABS_SHARD_STRIDE
    h = stats_out[:n].cpu().tolist()
    shards = [tuple(h[ABS_STATS_HEADER + s * ABS_SHARD_STRIDE + j] for j in range(3))
              for s in range(n_shards)]
    # fourth slot of a shard record: 0, or the shard's largest T_i (coordinate-wise calls)
    shard_max = [h[ABS_STATS_HEADER + s * ABS_SHARD_STRIDE + 3] for s in range(n_shards)]
    return {"n2": h[ABS_STAT_N2], "S": h[ABS_STAT_S], "Q": h[ABS_STAT_Q], "T": h[ABS_STAT_T],
            "flags": int(h[ABS_STAT_FLAGS]), "norm": h[ABS_STAT_NORM],
            "n_chunks": int(h[ABS_STAT_NCHUNKS]), "argmax": int(h[ABS_STAT_ARGMAX]),
            "shards": shards, "shard_max": shard_max}
