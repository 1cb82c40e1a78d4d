"""Helpers shared by the tests: host copies for the oracle, tolerances, decision margins."""
import math

import numpy as np
import torch

# Parity tolerances: sums within relative 1e-6; vectors within 1e-6 * max|reference|.
REL_SUM = 1e-6
REL_VEC = 1e-6
# Decision parity is asserted bit-exact only when the oracle's T keeps this relative
# distance from the threshold b_cur and from every integer (ceil is then insensitive to
# the 1e-6 agreement of the sums).
MARGIN = 1e-4


def to_host(t):
    """torch tensor (fp32 or bf16, any device) -> numpy array the oracle accepts."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def f32(x):
    """The double value of x after rounding to fp32 (what the C ABI's float fields hold)."""
    return float(np.float32(x))


def margin_ok(T, b_cur, margin=MARGIN):
    if not math.isfinite(T):
        return True
    tol = margin * max(abs(T), 1.0)
    if abs(T - b_cur) < tol:
        return False
    if T > b_cur and abs(T - round(T)) < tol:
        return False
    return True


def assert_sum_close(got, ref, name, rel=REL_SUM):
    assert abs(got - ref) <= rel * abs(ref) + 1e-300, "%s: got %r ref %r" % (name, got, ref)


def assert_vec_close(got, ref, name, rel=REL_VEC):
    got = got.detach().cpu().numpy().astype(np.float64) if torch.is_tensor(got) else got
    scale = float(np.abs(ref).max())
    err = float(np.abs(got - ref).max())
    assert err <= rel * scale + 1e-300, "%s: max abs err %g > %g * %g" % (name, err, rel, scale)


def oracle_adamw(orc, p0, m0, v0, gbar64, hp, step):
    return orc.adamw(p0, m0, v0, gbar64, f32(hp["lr"]), f32(hp["beta1"]), f32(hp["beta2"]),
                     f32(hp["eps"]), f32(hp["weight_decay"]), step)
