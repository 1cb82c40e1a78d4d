"""ctypes front end of the fp64 CPU oracle (``abs_oracle.c``).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only the test-suite, the smoke check and the
benchmark's CPU-baseline / reference legs may import this module.  It holds no
arithmetic of its own -- it marshals numpy arrays into the C functions and builds the
shared object with gcc when it is missing.  bf16 data is passed as ``uint16`` bit
patterns; fp32 as ``float32``.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "abs_oracle.c")
_LIB = os.path.join(_HERE, "libabs_oracle.so")

F32, BF16 = 0, 1
FLAG_DEGENERATE, FLAG_NONFINITE, FLAG_VIOLATED = 1, 2, 4
TOT_N2, TOT_S, TOT_Q, TOT_T, TOT_FLAGS, TOT_NORM, TOT_COUNT = 0, 1, 2, 3, 4, 5, 8


def build(force=False):
    """Compile abs_oracle.c -> libabs_oracle.so (gcc, OpenMP, no FMA contraction)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-shared",
                           "-fPIC", "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i64, dbl, ptr, cint = ctypes.c_int64, ctypes.c_double, ctypes.c_void_p, ctypes.c_int
        L.abs_oracle_threads.restype = cint
        L.abs_oracle_decide.restype = i64
        L.abs_oracle_decide.argtypes = [dbl, dbl, dbl, dbl, i64, ptr, ptr]
        L.abs_oracle_round_batch.restype = i64
        L.abs_oracle_round_batch.argtypes = [i64, i64, i64]
        L.abs_oracle_norm_test.restype = cint
        L.abs_oracle_norm_test.argtypes = [ptr, cint, i64, cint, ptr, cint, dbl, i64, ptr, ptr,
                                           ptr, ptr]
        L.abs_oracle_persample.restype = cint
        L.abs_oracle_persample.argtypes = [ptr, i64, i64, i64, cint, dbl, ptr, ptr, ptr]
        L.abs_oracle_norm_test_coordwise.restype = cint
        L.abs_oracle_norm_test_coordwise.argtypes = [ptr, cint, i64, cint, ptr, cint, dbl, i64,
                                                     ptr, ptr, ptr, ptr, ptr, ptr]
        L.abs_oracle_persample_coordwise.restype = cint
        L.abs_oracle_persample_coordwise.argtypes = [ptr, i64, i64, i64, cint, dbl, ptr, ptr, ptr,
                                                     ptr, ptr]
        L.abs_oracle_adamw.restype = cint
        L.abs_oracle_adamw.argtypes = [ptr, ptr, ptr, ptr, i64, dbl, dbl, dbl, dbl, dbl, i64,
                                       ptr, ptr, ptr]
        L.abs_oracle_bf16_round.restype = cint
        L.abs_oracle_bf16_round.argtypes = [ptr, i64, ptr]
        L.abs_oracle_clip_scale.restype = dbl
        L.abs_oracle_clip_scale.argtypes = [dbl, dbl]
        L.abs_oracle_adamw_clipped.restype = cint
        L.abs_oracle_adamw_clipped.argtypes = [ptr, ptr, ptr, ptr, i64, dbl, dbl, dbl, dbl, dbl,
                                               i64, dbl, dbl, ptr, ptr, ptr]
        _lib = L
    return _lib


def threads():
    return int(lib().abs_oracle_threads())


def _dtype_code(a):
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError("oracle inputs are float32 or uint16 (bf16 bits), got %s" % a.dtype)


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _totals_dict(tot, b_next):
    return {"n2": float(tot[TOT_N2]), "S": float(tot[TOT_S]), "Q": float(tot[TOT_Q]),
            "T": float(tot[TOT_T]), "flags": int(tot[TOT_FLAGS]), "norm": float(tot[TOT_NORM]),
            "b_next": int(b_next)}


def norm_test(grads, eta, b_cur, shard_offsets=None, want_gbar=True):
    """grads: sequence of K 1-D contiguous arrays (float32 or uint16 bf16 bits), equal length."""
    grads = [np.ascontiguousarray(g) for g in grads]
    K, d = len(grads), int(grads[0].shape[0])
    code = _dtype_code(grads[0])
    for g in grads:
        assert g.ndim == 1 and g.shape[0] == d and _dtype_code(g) == code
    ptrs = (ctypes.c_void_p * K)(*[g.ctypes.data for g in grads])
    if shard_offsets is None:
        offs, n_shards, offs_p = None, 1, None
    else:
        offs = np.ascontiguousarray(np.asarray(shard_offsets, dtype=np.int64))
        n_shards, offs_p = int(offs.shape[0]) - 1, _p(offs)
    gbar = np.empty(d, dtype=np.float64) if want_gbar else None
    tot = np.zeros(TOT_COUNT, dtype=np.float64)
    shard = np.zeros((n_shards, 3), dtype=np.float64)
    b_next = ctypes.c_int64(0)
    rc = lib().abs_oracle_norm_test(ptrs, K, d, code, offs_p, n_shards, float(eta), int(b_cur),
                                    _p(gbar) if want_gbar else None, _p(tot), _p(shard),
                                    ctypes.byref(b_next))
    if rc != 0:
        raise ValueError("abs_oracle_norm_test rejected its arguments")
    out = _totals_dict(tot, b_next.value)
    out["gbar"] = gbar
    out["shards"] = shard
    return out


def persample(G, eta, want_gbar=True):
    """G: 2-D array [b, d] (float32 or uint16 bf16 bits); rows may be strided by ld >= d."""
    assert G.ndim == 2 and G.strides[1] == G.itemsize and G.strides[0] % G.itemsize == 0
    b, d = int(G.shape[0]), int(G.shape[1])
    ld = G.strides[0] // G.itemsize
    gbar = np.empty(d, dtype=np.float64) if want_gbar else None
    tot = np.zeros(TOT_COUNT, dtype=np.float64)
    b_next = ctypes.c_int64(0)
    rc = lib().abs_oracle_persample(_p(G), b, d, ld, _dtype_code(G), float(eta),
                                    _p(gbar) if want_gbar else None, _p(tot),
                                    ctypes.byref(b_next))
    if rc != 0:
        raise ValueError("abs_oracle_persample rejected its arguments")
    out = _totals_dict(tot, b_next.value)
    out["gbar"] = gbar
    return out


def norm_test_coordwise(grads, eta, b_cur, shard_offsets=None, want_ratios=False):
    """Coordinate-wise test, worker form.  Returns the dict of norm_test (T, flags and b_next
    are those of the coordinate-wise test) plus "argmax", "shard_max" and, on request,
    "ratios" (the d per-coordinate statistics T_i)."""
    grads = [np.ascontiguousarray(g) for g in grads]
    K, d = len(grads), int(grads[0].shape[0])
    code = _dtype_code(grads[0])
    for g in grads:
        assert g.ndim == 1 and g.shape[0] == d and _dtype_code(g) == code
    ptrs = (ctypes.c_void_p * K)(*[g.ctypes.data for g in grads])
    if shard_offsets is None:
        n_shards, offs_p = 1, None
    else:
        offs = np.ascontiguousarray(np.asarray(shard_offsets, dtype=np.int64))
        n_shards, offs_p = int(offs.shape[0]) - 1, _p(offs)
    gbar = np.empty(d, dtype=np.float64)
    ratios = np.empty(d, dtype=np.float64) if want_ratios else None
    tot = np.zeros(TOT_COUNT, dtype=np.float64)
    shard_max = np.zeros(n_shards, dtype=np.float64)
    b_next, arg = ctypes.c_int64(0), ctypes.c_int64(0)
    rc = lib().abs_oracle_norm_test_coordwise(ptrs, K, d, code, offs_p, n_shards, float(eta),
                                              int(b_cur), _p(gbar),
                                              _p(ratios) if want_ratios else None, _p(tot),
                                              _p(shard_max), ctypes.byref(arg),
                                              ctypes.byref(b_next))
    if rc != 0:
        raise ValueError("abs_oracle_norm_test_coordwise rejected its arguments")
    out = _totals_dict(tot, b_next.value)
    out.update(gbar=gbar, ratios=ratios, argmax=int(arg.value), shard_max=shard_max)
    return out


def persample_coordwise(G, eta, want_ratios=False):
    """Coordinate-wise test, per-sample form (rows of G are the samples)."""
    assert G.ndim == 2 and G.strides[1] == G.itemsize and G.strides[0] % G.itemsize == 0
    b, d = int(G.shape[0]), int(G.shape[1])
    ld = G.strides[0] // G.itemsize
    gbar = np.empty(d, dtype=np.float64)
    ratios = np.empty(d, dtype=np.float64) if want_ratios else None
    tot = np.zeros(TOT_COUNT, dtype=np.float64)
    b_next, arg = ctypes.c_int64(0), ctypes.c_int64(0)
    rc = lib().abs_oracle_persample_coordwise(_p(G), b, d, ld, _dtype_code(G), float(eta),
                                              _p(gbar), _p(ratios) if want_ratios else None,
                                              _p(tot), ctypes.byref(arg), ctypes.byref(b_next))
    if rc != 0:
        raise ValueError("abs_oracle_persample_coordwise rejected its arguments")
    out = _totals_dict(tot, b_next.value)
    out.update(gbar=gbar, ratios=ratios, argmax=int(arg.value))
    return out


def decide(S, n2, norm, eta, b_cur):
    T, flags = ctypes.c_double(0), ctypes.c_int(0)
    b_next = lib().abs_oracle_decide(float(S), float(n2), float(norm), float(eta), int(b_cur),
                                     ctypes.byref(T), ctypes.byref(flags))
    return int(b_next), T.value, flags.value


def round_batch(b_next, J, M):
    return int(lib().abs_oracle_round_batch(int(b_next), int(J), int(M)))


def _least(holds, lo, hi):
    """Smallest integer in [lo, hi] at which the monotone predicate `holds` (false, ..., false,
    true, ..., true) is true; it must be true at hi.  Bisection, so that any size is exact."""
    assert holds(hi)
    while lo < hi:
        mid = (lo + hi) // 2
        if holds(mid):
            hi = mid
        else:
            lo = mid + 1
    return lo


def _greatest(holds, lo, hi):
    """Largest integer in [lo, hi] at which the monotone predicate `holds` (true, ..., true,
    false, ..., false) is true; it must be true at lo."""
    assert holds(lo)
    while lo < hi:
        mid = (lo + hi + 1) // 2
        if holds(mid):
            lo = mid
        else:
            hi = mid - 1
    return lo


class Schedule:
    """Algorithm 1's loop state around the test, in Python integers (exact at any size): the
    If branch (microbatch rounded up, minibatch = M * microbatch, global = J * minibatch), the
    Else branch, and the counters k and i; with the maximum global batch size and test interval
    of Sec. 5 ("Training Specifications") and the maximum micro batch size of Tables 5-7.  The
    paper prints no rule for the last two beyond their values; the reading here is: when the
    rounded microbatch would pass the maximum, M becomes the smallest count that keeps it
    within the maximum; a batch that rounding pushes over the cap falls back to the largest
    microbatch under the cap and is ignored if that is no increase."""

    def __init__(self, J, M, micro0, b_max, max_micro=0, interval=1):
        self.J, self.M, self.micro = J, M, micro0
        self.b = J * M * micro0
        self.b_max, self.max_micro, self.interval = b_max, max_micro, interval
        self.step, self.samples = 1, 0
        assert self.b <= b_max and (max_micro == 0 or micro0 <= max_micro)

    def test_due(self):
        return self.b < self.b_max and self.step % self.interval == 0

    def advance(self, b_test):
        """One pass of the loop body after the test.  The new layout is stated as what it has
        to satisfy and found by search over the integers (`_least`, `_greatest`), not by a
        rounding formula."""
        J, used = self.J, self.b
        target = min(b_test, self.b_max)
        if target > self.b:   # the If branch (the Else branch changes nothing)
            def covers(M, micro):
                return J * M * micro >= target
            # the paper's M, unless even the largest allowed microbatch does not cover the
            # target with it: then the smallest count of accumulation steps that does
            M = self.M
            if self.max_micro and not covers(M, self.max_micro):
                M = _least(lambda c: covers(c, self.max_micro), self.M, target)
            # the smallest microbatch that covers the target ...
            micro = _least(lambda u: covers(M, u), 1, target)
            if J * M * micro > self.b_max:
                # ... or, should that pass the cap, the largest one that stays under it
                micro = _greatest(lambda u: J * M * u <= self.b_max, 0, micro)
            if micro >= 1 and J * M * micro > self.b:   # only ever an increase
                self.M, self.micro, self.b = M, micro, J * M * micro
        self.samples += used
        self.step += 1

    def state(self):
        return dict(J=self.J, M=self.M, micro=self.micro, b=self.b, step=self.step,
                    samples=self.samples)


def adamw(w, m, v, g, lr, beta1, beta2, eps, wd, step):
    """w, m, v float32 arrays (the stored state), g float64; returns fp64 (w', m', v')."""
    w, m, v = (np.ascontiguousarray(x, dtype=np.float32) for x in (w, m, v))
    g = np.ascontiguousarray(g, dtype=np.float64)
    d = int(w.shape[0])
    assert m.shape[0] == d and v.shape[0] == d and g.shape[0] == d
    wo, mo, vo = (np.empty(d, dtype=np.float64) for _ in range(3))
    rc = lib().abs_oracle_adamw(_p(w), _p(m), _p(v), _p(g), d, float(lr), float(beta1),
                                float(beta2), float(eps), float(wd), int(step), _p(wo), _p(mo),
                                _p(vo))
    if rc != 0:
        raise ValueError("abs_oracle_adamw rejected its arguments")
    return wo, mo, vo


def bf16_round(x):
    """float32 array -> uint16 array of bfloat16 bit patterns, round to nearest even."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    if lib().abs_oracle_bf16_round(_p(x), int(x.size), _p(out)) != 0:
        raise ValueError("abs_oracle_bf16_round rejected its arguments")
    return out


def clip_scale(n2, max_norm):
    return float(lib().abs_oracle_clip_scale(float(n2), float(max_norm)))


def adamw_clipped(w, m, v, g, lr, beta1, beta2, eps, wd, step, max_norm, n2):
    """AdamW on the gradient clipped to global norm max_norm (n2 = ||g||^2); fp64 (w', m', v')."""
    w, m, v = (np.ascontiguousarray(x, dtype=np.float32) for x in (w, m, v))
    g = np.ascontiguousarray(g, dtype=np.float64)
    d = int(w.shape[0])
    assert m.shape[0] == d and v.shape[0] == d and g.shape[0] == d
    wo, mo, vo = (np.empty(d, dtype=np.float64) for _ in range(3))
    rc = lib().abs_oracle_adamw_clipped(_p(w), _p(m), _p(v), _p(g), d, float(lr), float(beta1),
                                        float(beta2), float(eps), float(wd), int(step),
                                        float(max_norm), float(n2), _p(wo), _p(mo), _p(vo))
    if rc != 0:
        raise ValueError("abs_oracle_adamw_clipped rejected its arguments")
    return wo, mo, vo
