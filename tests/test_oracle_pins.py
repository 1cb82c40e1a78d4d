"""Pins for the fp64 CPU oracle: none of the expected values below come from the oracle.

They come from (a) hand-worked fixtures, (b) exact rational arithmetic on tiny inputs,
(c) numpy / torch library routines for the special cases that reduce to them,
(d) closed forms and invariants of the definitions.  Each is chosen so that a plausible
slip in the oracle (dropped term, wrong normalisation, wrong sign, transposed operand,
wrong decay order) fails at least one of them.
"""
import json
import math
import os
import subprocess
import sys
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import abs_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_cases.json")


def bf16_bits(x):
    """float array -> uint16 bf16 bit patterns (round-to-nearest-even, by torch)."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bf16_to_f64(bits):
    t = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)
    return t.to(torch.float64).numpy()


def frac_stats(rows):
    """Exact rational mean / n2 / S / Q of a list of rows (each a list of floats)."""
    K, d = len(rows), len(rows[0])
    F = [[Fraction(float(x)) for x in r] for r in rows]
    gbar = [sum(F[k][i] for k in range(K)) / K for i in range(d)]
    n2 = sum(g * g for g in gbar)
    S = sum((F[k][i] - gbar[i]) ** 2 for k in range(K) for i in range(d))
    Q = sum(F[k][i] ** 2 for k in range(K) for i in range(d))
    return gbar, n2, S, Q


def frac_decide(S, n2, norm, eta, b_cur):
    T = (S / norm) / (Fraction(float(eta)) ** 2 * n2)
    if T > b_cur:
        return math.ceil(T), T
    return b_cur, T


# ----------------------------------------------------------------------------- hand cases
def test_hand_cases_norm_test():
    cases = json.load(open(GOLDEN))["norm_test"]
    for c in cases:
        grads = [np.asarray(g, dtype=np.float32) for g in c["grads"]]
        K = len(grads)
        T_w = c.get("T_worker", None)
        if T_w is None:
            n, dnm = c["T_worker_fraction"]
            T_w = n / dnm
        T_p = c.get("T_persample", None)
        if T_p is None:
            n, dnm = c["T_persample_fraction"]
            T_p = n / dnm
        for dec in c["decisions_worker"]:
            r = orc.norm_test(grads, c["eta"], dec["b_cur"])
            assert r["n2"] == c["n2"] and r["S"] == c["S"] and r["Q"] == c["Q"], c["name"]
            assert list(r["gbar"]) == c["gbar"]
            assert r["T"] == pytest.approx(T_w, rel=1e-15)
            assert r["b_next"] == dec["b_next"], (c["name"], dec)
            assert bool(r["flags"] & orc.FLAG_VIOLATED) == dec["violated"]
            assert r["norm"] == K
        G = np.stack(grads)
        r = orc.persample(G, c["eta"])
        assert r["n2"] == c["n2"] and r["S"] == c["S"] and r["Q"] == c["Q"]
        assert r["T"] == pytest.approx(T_p, rel=1e-15)
        assert r["b_next"] == c["b_next_persample"]
        assert r["norm"] == K - 1


def test_hand_case_adamw():
    for c in json.load(open(GOLDEN))["adamw"]:
        w, m, v = orc.adamw([c["w"]], [c["m"]], [c["v"]], [c["g"]], c["lr"], c["beta1"],
                            c["beta2"], c["eps"], c["wd"], c["step"])
        assert abs(w[0] - c["w_out"]) < c["tol"]
        assert abs(m[0] - c["m_out"]) < c["tol"]
        assert abs(v[0] - c["v_out"]) < c["tol"]


def test_hand_case_round_batch():
    for c in json.load(open(GOLDEN))["round_batch"]:
        for case in c["cases"]:
            assert orc.round_batch(case["b_next"], case["J"], case["M"]) == case["b"]


def test_round_batch_properties():
    rng = np.random.default_rng(5)
    for _ in range(200):
        b, J, M = int(rng.integers(1, 10**6)), int(rng.integers(1, 65)), int(rng.integers(1, 33))
        r = orc.round_batch(b, J, M)
        assert r % (J * M) == 0 and b <= r < b + J * M


def test_hand_case_schedule():
    for c in json.load(open(GOLDEN))["schedule"]:
        i = c["init"]
        s = orc.Schedule(i["J"], i["M"], i["micro0"], i["b_max"], i["max_micro"], i["interval"])
        for st in c["steps"]:
            assert s.test_due() == st["due"], c["name"]
            s.advance(st["b_test"])
            got = s.state()
            assert {k: got[k] for k in st["after"]} == st["after"], c["name"]


def test_schedule_properties_and_brute_force_layout():
    """Invariants of Algorithm 1's If/Else with the cap and the micro-batch limit, and the
    layout checked against an exhaustive search on small numbers."""
    rng = np.random.default_rng(11)
    for trial in range(150):
        J, M0, micro0 = int(rng.integers(1, 6)), int(rng.integers(1, 5)), int(rng.integers(1, 4))
        max_micro = int(rng.integers(micro0, micro0 + 4)) if trial % 3 else 0
        b0 = J * M0 * micro0
        b_max = b0 + int(rng.integers(0, 400))
        s = orc.Schedule(J, M0, micro0, b_max, max_micro, int(rng.integers(1, 4)))
        total = 0
        for k in range(1, 30):
            before = s.state()
            b_test = int(rng.integers(1, 2 * b_max))
            s.advance(b_test)
            after = s.state()
            total += before["b"]
            assert after["step"] == k + 1 and after["samples"] == total
            assert after["b"] == J * after["M"] * after["micro"]
            assert before["b"] <= after["b"] <= b_max            # never shrinks, never passes the cap
            assert max_micro == 0 or after["micro"] <= max_micro
            assert after["M"] >= before["M"] and (max_micro or after["M"] == M0)
            target = min(b_test, b_max)
            if target <= before["b"]:
                assert after == dict(before, step=k + 1, samples=total)  # Else branch
                continue
            # If branch: among layouts (M', micro') allowed by the limit, with M' the paper's M
            # when its rounded microbatch fits and otherwise the smallest M' that fits, the
            # batch is the smallest J*M'*micro' >= target; found here by exhaustive search
            M_fit = None
            for Mc in range(before["M"], b_max + 1):
                mic = -(-target // (J * Mc))
                if max_micro == 0 or mic <= max_micro:
                    M_fit = (Mc, mic)
                    break
            Mc, mic = M_fit
            want = J * Mc * mic
            if want <= b_max:
                assert (after["M"], after["micro"], after["b"]) == (Mc, mic, want)
                assert target <= after["b"] < target + J * Mc
                if Mc == before["M"]:
                    assert after["b"] == orc.round_batch(target, J, before["M"])
            else:  # rounding passed the cap: largest multiple of J*Mc under it, if an increase
                fb = (b_max // (J * Mc)) * J * Mc
                if fb > before["b"]:
                    assert after["b"] == fb and after["M"] == Mc
                else:
                    assert after["b"] == before["b"] and after["M"] == before["M"]


# ------------------------------------------------------------- exact rational brute force
@pytest.mark.parametrize("K,d", [(1, 1), (2, 3), (3, 5), (4, 8), (5, 7), (7, 2)])
@pytest.mark.parametrize("kind", ["f32", "bf16"])
def test_brute_force_rational(K, d, kind):
    rng = np.random.default_rng(1000 * K + d)
    for trial in range(6):
        raw = (rng.standard_normal((K, d)) * 0.3 + 0.1).astype(np.float32)
        if kind == "bf16":
            grads = [bf16_bits(raw[k]) for k in range(K)]
            rows = [list(bf16_to_f64(g)) for g in grads]
        else:
            grads = [raw[k].copy() for k in range(K)]
            rows = [list(raw[k].astype(np.float64)) for k in range(K)]
        gbar, n2, S, Q = frac_stats(rows)
        eta, b_cur = 0.25, 1 + trial
        r = orc.norm_test(grads, eta, b_cur)
        assert r["n2"] == pytest.approx(float(n2), rel=1e-14)
        assert r["Q"] == pytest.approx(float(Q), rel=1e-14)
        assert r["S"] == pytest.approx(float(S), rel=1e-13, abs=1e-300)
        np.testing.assert_allclose(r["gbar"], [float(g) for g in gbar], rtol=1e-15, atol=0)
        if n2 > 0:
            b_next, T = frac_decide(S, n2, K, eta, b_cur)
            assert r["T"] == pytest.approx(float(T), rel=1e-13, abs=1e-300)
            if abs(float(T) - round(float(T))) > 1e-9 and abs(float(T) - b_cur) > 1e-9:
                assert r["b_next"] == b_next
        if K >= 2:
            G = (np.stack(grads))
            rp = orc.persample(G, eta)
            assert rp["S"] == pytest.approx(float(S), rel=1e-13, abs=1e-300)
            assert rp["n2"] == pytest.approx(float(n2), rel=1e-14)
            b_next, T = frac_decide(S, n2, K - 1, eta, K)
            assert rp["T"] == pytest.approx(float(T), rel=1e-13, abs=1e-300)
            if abs(float(T) - round(float(T))) > 1e-9:
                assert rp["b_next"] == b_next


# ------------------------------------------------------------- library-routine special cases
@pytest.mark.parametrize("K,d", [(2, 4096), (4, 4097), (8, 20000), (3, 12289), (32, 5000)])
def test_against_numpy_mean_var(K, d):
    rng = np.random.default_rng(K * 7 + d)
    mu = rng.standard_normal(d) * 0.01
    A = (mu + 0.05 * rng.standard_normal((K, d))).astype(np.float32)
    r = orc.norm_test([A[k] for k in range(K)], 0.1, 64)
    A64 = A.astype(np.float64)
    mean = A64.mean(axis=0)
    np.testing.assert_allclose(r["gbar"], mean, rtol=1e-14, atol=1e-18)
    assert r["n2"] == pytest.approx(float(np.dot(mean, mean)), rel=1e-12)
    # \hat Var = population variance across workers (1/K), so S = K * sum_i var_i
    assert r["S"] == pytest.approx(K * float(A64.var(axis=0, ddof=0).sum()), rel=1e-12)
    assert r["Q"] == pytest.approx(float((A64 * A64).sum()), rel=1e-12)
    T = (r["S"] / K) / (0.1 ** 2 * r["n2"])
    assert r["T"] == pytest.approx(T, rel=1e-14)
    assert r["b_next"] == (math.ceil(T) if T > 64 else 64)


@pytest.mark.parametrize("b,d,ld", [(2, 5, 5), (7, 4100, 4100), (33, 300, 320), (64, 8193, 8200)])
def test_persample_against_numpy(b, d, ld):
    rng = np.random.default_rng(b * 31 + d)
    buf = (0.02 + 0.3 * rng.standard_normal((b, ld))).astype(np.float32)
    G = buf[:, :d]
    r = orc.persample(G, 0.1)
    G64 = G.astype(np.float64)
    mean = G64.mean(axis=0)
    np.testing.assert_allclose(r["gbar"], mean, rtol=1e-14, atol=1e-18)
    var1 = float(G64.var(axis=0, ddof=1).sum())  # ||Var||_1 with 1/(b-1)
    assert r["S"] / (b - 1) == pytest.approx(var1, rel=1e-12)
    T = var1 / (0.01 * float(np.dot(mean, mean)))
    assert r["T"] == pytest.approx(T, rel=1e-12)
    assert r["norm"] == b - 1
    assert r["b_next"] == (math.ceil(r["T"]) if r["T"] > b else b)


def test_persample_is_not_transposed():
    # rows are samples: with b != d a transposed read changes gbar's length-d content
    G = np.arange(12, dtype=np.float32).reshape(3, 4)
    r = orc.persample(G, 0.5)
    assert list(r["gbar"]) == [4.0, 5.0, 6.0, 7.0]
    assert r["S"] == 4 * 32.0  # each column deviates by (-4, 0, 4)


def test_bf16_widening_matches_torch():
    rng = np.random.default_rng(3)
    x = (rng.standard_normal(5000) * np.exp(rng.uniform(-20, 20, 5000))).astype(np.float32)
    bits = bf16_bits(x)
    r = orc.norm_test([bits], 0.1, 1)
    np.testing.assert_array_equal(r["gbar"], bf16_to_f64(bits))


# --------------------------------------------------------------------------- invariants
@pytest.mark.parametrize("K", [1, 2, 3, 4, 5, 8, 32])
def test_identity_S_equals_Q_minus_K_n2(K):
    rng = np.random.default_rng(K)
    d = 9001
    A = (0.01 * rng.standard_normal(d) + 0.05 * rng.standard_normal((K, d))).astype(np.float32)
    r = orc.norm_test([A[k] for k in range(K)], 0.1, 8)
    assert r["S"] == pytest.approx(r["Q"] - K * r["n2"], rel=1e-11, abs=1e-12 * r["Q"])
    if K == 1:
        assert r["S"] == 0.0 and r["b_next"] == 8


@pytest.mark.parametrize("K", [2, 3, 4, 5, 8])
def test_identical_buffers_keep_batch_size(K):
    rng = np.random.default_rng(11)
    g = rng.standard_normal(5000).astype(np.float32)
    r = orc.norm_test([g.copy() for _ in range(K)], 0.1, 77)
    if K & (K - 1) == 0:
        assert r["S"] == 0.0
    assert r["S"] <= 1e-30 * r["Q"]
    assert r["b_next"] == 77 and not (r["flags"] & orc.FLAG_VIOLATED)
    assert r["T"] < 1e-20


def test_degenerate_and_nonfinite():
    z = np.zeros(16, dtype=np.float32)
    r = orc.norm_test([z, z, z, z], 0.1, 9)
    assert r["flags"] == orc.FLAG_DEGENERATE and r["b_next"] == 9 and math.isnan(r["T"])
    a = np.array([1.0, -1.0], dtype=np.float32)
    r = orc.norm_test([a, -a], 0.1, 9)  # gbar = 0 but S > 0
    assert r["flags"] == orc.FLAG_DEGENERATE | orc.FLAG_VIOLATED
    assert r["T"] == math.inf and r["b_next"] == 2 ** 63 - 1
    bad = np.array([1.0, np.inf], dtype=np.float32)
    r = orc.norm_test([bad, a], 0.1, 9)
    assert r["flags"] & orc.FLAG_NONFINITE and r["b_next"] == 9
    bad = np.array([1.0, np.nan], dtype=np.float32)
    r = orc.norm_test([bad, a], 0.1, 9)
    assert r["flags"] & orc.FLAG_NONFINITE and r["b_next"] == 9
    # saturation: tiny eta drives T past 2^62
    b_next, T, flags = orc.decide(1.0, 1.0, 2.0, 1e-12, 5)
    assert T > 2.0 ** 62 and b_next == 2 ** 63 - 1 and flags == orc.FLAG_VIOLATED


def test_decide_strictness_and_monotonicity():
    # T == b exactly: satisfied (Eq. 5 holds with equality), batch unchanged
    assert orc.decide(4.0, 8.0, 2.0, 0.25, 4)[0] == 4
    assert orc.decide(4.0, 8.0, 2.0, 0.25, 3)[0] == 4
    rng = np.random.default_rng(2)
    for _ in range(100):
        S, n2 = float(rng.uniform(0.1, 1e4)), float(rng.uniform(0.1, 1e2))
        b = int(rng.integers(1, 5000))
        prev = None
        for eta in [0.05, 0.1, 0.2, 0.4, 0.8]:
            bn, T, fl = orc.decide(S, n2, 8.0, eta, b)
            assert bn >= b  # never decreases
            assert bn == (math.ceil(T) if T > b else b)
            if prev is not None:
                assert bn <= prev  # larger eta tolerates more variance
            prev = bn


def test_shard_sums_add_up_and_match_slices():
    rng = np.random.default_rng(8)
    K, d = 4, 30011
    A = (0.05 * rng.standard_normal((K, d))).astype(np.float32)
    offs = [0, 1, 4097, 4097, 12289, 30000, d]  # ragged, one empty shard
    r = orc.norm_test([A[k] for k in range(K)], 0.1, 16, shard_offsets=offs)
    sh = r["shards"]
    assert sh.shape == (6, 3)
    assert r["n2"] == pytest.approx(sh[:, 0].sum(), rel=1e-15)
    assert r["S"] == pytest.approx(sh[:, 1].sum(), rel=1e-15)
    assert r["Q"] == pytest.approx(sh[:, 2].sum(), rel=1e-15)
    for s in range(6):
        lo, hi = offs[s], offs[s + 1]
        if hi == lo:
            assert tuple(sh[s]) == (0.0, 0.0, 0.0)
            continue
        A64 = A[:, lo:hi].astype(np.float64)
        mean = A64.mean(axis=0)
        assert sh[s, 0] == pytest.approx(float(np.dot(mean, mean)), rel=1e-12)
        assert sh[s, 1] == pytest.approx(float(((A64 - mean) ** 2).sum()), rel=1e-12)
    # the unsharded call agrees to summation-order rounding
    r1 = orc.norm_test([A[k] for k in range(K)], 0.1, 16)
    assert r1["S"] == pytest.approx(r["S"], rel=1e-13)
    np.testing.assert_array_equal(r1["gbar"], r["gbar"])


def test_persample_vs_worker_form_factor():
    rng = np.random.default_rng(21)
    K, d = 6, 5000
    A = (0.02 + 0.05 * rng.standard_normal((K, d))).astype(np.float32)
    rw = orc.norm_test([A[k] for k in range(K)], 0.1, 1)
    rp = orc.persample(A, 0.1)
    assert rp["T"] == pytest.approx(rw["T"] * K / (K - 1), rel=1e-13)


# ------------------------------------------------------------------------------- AdamW
def test_adamw_against_torch_optimizer_fp64():
    """torch.optim.AdamW run in fp64 is a library statement of the same update."""
    rng = np.random.default_rng(4)
    d = 1000
    lr, b1, b2, eps, wd = [float(np.float32(x)) for x in (1e-3, 0.9, 0.95, 1e-8, 0.1)]
    for step in (1, 2, 7, 1000):
        w32 = (0.02 * rng.standard_normal(d)).astype(np.float32)
        m32 = (0.01 * rng.standard_normal(d)).astype(np.float32) if step > 1 else np.zeros(d, np.float32)
        v32 = (1e-4 * rng.random(d)).astype(np.float32) if step > 1 else np.zeros(d, np.float32)
        g = 0.1 * rng.standard_normal(d)
        p = torch.nn.Parameter(torch.from_numpy(w32.astype(np.float64)))
        opt = torch.optim.AdamW([p], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd)
        p.grad = torch.zeros(d, dtype=torch.float64)
        opt.step()  # creates the state entries
        st = opt.state[p]
        with torch.no_grad():
            p.copy_(torch.from_numpy(w32.astype(np.float64)))
            st["exp_avg"].copy_(torch.from_numpy(m32.astype(np.float64)))
            st["exp_avg_sq"].copy_(torch.from_numpy(v32.astype(np.float64)))
            st["step"].fill_(step - 1)  # the next call is step number `step`
        p.grad = torch.from_numpy(g.copy())
        opt.step()
        wo, mo, vo = orc.adamw(w32, m32, v32, g, lr, b1, b2, eps, wd, step)
        np.testing.assert_allclose(wo, p.detach().numpy(), rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(mo, st["exp_avg"].numpy(), rtol=1e-12, atol=1e-18)
        np.testing.assert_allclose(vo, st["exp_avg_sq"].numpy(), rtol=1e-12, atol=1e-20)


def test_adamw_closed_form_first_step():
    rng = np.random.default_rng(6)
    d = 2000
    lr, b1, b2, eps, wd = 1e-3, 0.9, 0.999, 1e-8, 0.1
    w = (0.02 * rng.standard_normal(d)).astype(np.float32)
    g = 0.05 * rng.standard_normal(d)
    z = np.zeros(d, dtype=np.float32)
    wo, mo, vo = orc.adamw(w, z, z, g, lr, b1, b2, eps, wd, 1)
    np.testing.assert_allclose(mo, (1 - b1) * g, rtol=1e-15)
    np.testing.assert_allclose(vo, (1 - b2) * g * g, rtol=1e-15)
    expect = (1 - lr * wd) * w.astype(np.float64) - lr * g / (np.abs(g) + eps)
    np.testing.assert_allclose(wo, expect, rtol=0, atol=1e-12)
    # zero gradient: only the decoupled decay acts
    wo, mo, vo = orc.adamw(w, z, z, np.zeros(d), lr, b1, b2, eps, wd, 1)
    np.testing.assert_allclose(wo, (1 - lr * wd) * w.astype(np.float64), rtol=1e-15)
    assert not mo.any() and not vo.any()


def test_adamw_decay_multiplies_old_weight_and_eps_outside_sqrt():
    # large eps and large decay make the two classic slips visible
    w, m, v, g = [2.0], [0.5], [0.25], [1.0]
    lr, b1, b2, eps, wd, step = 0.5, 0.5, 0.5, 1.0, 0.5, 2
    m1 = 0.5 * 0.5 + 0.5 * 1.0  # 0.75
    v1 = 0.5 * 0.25 + 0.5 * 1.0  # 0.625
    mh, vh = m1 / (1 - 0.25), v1 / (1 - 0.25)
    expect = (1 - 0.25) * 2.0 - 0.5 * mh / (math.sqrt(vh) + 1.0)
    wo, mo, vo = orc.adamw(w, m, v, g, lr, b1, b2, eps, wd, step)
    assert wo[0] == pytest.approx(expect, rel=1e-15)
    assert mo[0] == m1 and vo[0] == v1


def test_clipped_adamw_against_torch_clip_grad_norm():
    """torch.nn.utils.clip_grad_norm_ + torch.optim.AdamW in fp64 is the library statement of
    clipping by global norm followed by the update."""
    rng = np.random.default_rng(12)
    d = 800
    lr, b1, b2, eps, wd = [float(np.float32(x)) for x in (1e-3, 0.9, 0.95, 1e-8, 0.1)]
    for gscale, max_norm in ((0.5, 1.0), (0.001, 1.0), (0.2, 0.25)):
        w32 = (0.02 * rng.standard_normal(d)).astype(np.float32)
        m32 = (0.01 * rng.standard_normal(d)).astype(np.float32)
        v32 = (1e-4 * rng.random(d)).astype(np.float32)
        g = gscale * rng.standard_normal(d)
        n2 = float(np.dot(g, g))
        p = torch.nn.Parameter(torch.from_numpy(w32.astype(np.float64)))
        opt = torch.optim.AdamW([p], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd)
        p.grad = torch.zeros(d, dtype=torch.float64)
        opt.step()
        st = opt.state[p]
        with torch.no_grad():
            p.copy_(torch.from_numpy(w32.astype(np.float64)))
            st["exp_avg"].copy_(torch.from_numpy(m32.astype(np.float64)))
            st["exp_avg_sq"].copy_(torch.from_numpy(v32.astype(np.float64)))
            st["step"].fill_(4)
        p.grad = torch.from_numpy(g.copy())
        total = torch.nn.utils.clip_grad_norm_([p], max_norm)
        assert float(total) == pytest.approx(math.sqrt(n2), rel=1e-13)
        scale = orc.clip_scale(n2, max_norm)
        np.testing.assert_allclose(p.grad.numpy(), scale * g, rtol=1e-13, atol=0)
        assert (scale < 1.0) == (math.sqrt(n2) + 1e-6 > max_norm)
        opt.step()
        wo, mo, vo = orc.adamw_clipped(w32, m32, v32, g, lr, b1, b2, eps, wd, 5, max_norm, n2)
        np.testing.assert_allclose(wo, p.detach().numpy(), rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(mo, st["exp_avg"].numpy(), rtol=1e-12, atol=1e-18)
        np.testing.assert_allclose(vo, st["exp_avg_sq"].numpy(), rtol=1e-12, atol=1e-20)
    # no clipping needed: identical to the plain update
    g = 1e-3 * rng.standard_normal(d)
    a = orc.adamw_clipped(w32, m32, v32, g, lr, b1, b2, eps, wd, 3, 1.0, float(np.dot(g, g)))
    b = orc.adamw(w32, m32, v32, g, lr, b1, b2, eps, wd, 3)
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)
    assert orc.clip_scale(4.0, 1.0) == pytest.approx(1.0 / (2.0 + 1e-6), rel=1e-15)
    assert orc.clip_scale(0.0, 1.0) == 1.0


# ------------------------------------------------------------------- thread independence
def test_bf16_round_against_torch_and_hand_cases():
    """The bfloat16 working copy: against torch's conversion on random values and around every
    kind of boundary, and against hand-worked ties (1 + 2^-8 is halfway between the bfloat16
    neighbours 1 and 1 + 2^-7: ties go to the even significand)."""
    rng = np.random.default_rng(77)
    x = np.concatenate([
        rng.standard_normal(20000).astype(np.float32),
        (rng.standard_normal(2000) * 1e-30).astype(np.float32),
        (rng.standard_normal(2000) * 1e30).astype(np.float32),
        np.array([0.0, -0.0, 1.0, -1.0, np.inf, -np.inf, 3.3895314e38, -3.3895314e38,
                  3.4028235e38, 1e-45, -1e-45, 1.17549435e-38, 9.18e-41], dtype=np.float32)])
    # exact ties and their neighbours: k * 2^-8 + tiny offsets around odd k
    base = (1.0 + np.arange(0, 64) * 2.0 ** -8).astype(np.float32)
    ties = np.concatenate([base, np.nextafter(base, np.float32(2)), np.nextafter(base, np.float32(0)),
                           -base])
    x = np.concatenate([x, ties]).astype(np.float32)
    got = orc.bf16_round(x)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, want)
    # hand-worked: 1 = 0x3F80; 1 + 2^-7 = 0x3F81; 1 + 2^-6 = 0x3F82
    hand = {1.0 + 2.0 ** -8: 0x3F80,               # tie between 0x3F80 and 0x3F81 -> even
            1.0 + 2.0 ** -7 + 2.0 ** -8: 0x3F82,   # tie between 0x3F81 and 0x3F82 -> even
            1.0 + 2.0 ** -8 + 2.0 ** -20: 0x3F81,  # just above the tie
            -(1.0 + 2.0 ** -8): 0xBF80,
            0.5: 0x3F00, 3.0: 0x4040}
    for val, code in hand.items():
        assert int(orc.bf16_round(np.array([val], dtype=np.float32))[0]) == code, val
    # the largest finite bfloat16 is 0x7F7F; halfway to 2^128 and beyond rounds to infinity
    big = np.array([3.3895314e38, 3.3961775e38, 3.4028235e38], dtype=np.float32)
    assert list(orc.bf16_round(big)) == [0x7F7F, 0x7F80, 0x7F80]
    nan = orc.bf16_round(np.array([np.nan], dtype=np.float32))[0]
    assert (nan & 0x7F80) == 0x7F80 and (nan & 0x007F) != 0


# --------------------------------------------------------------- coordinate-wise test
def frac_coordwise(rows, norm, eta):
    """Exact per-coordinate statistics T_i (Fractions; None stands for +inf)."""
    K, d = len(rows), len(rows[0])
    F = [[Fraction(float(x)) for x in r] for r in rows]
    e2 = Fraction(float(eta)) ** 2
    out = []
    for i in range(d):
        gbar = sum(F[k][i] for k in range(K)) / K
        var = sum((F[k][i] - gbar) ** 2 for k in range(K)) / norm
        if var == 0:
            out.append(Fraction(0))
        elif gbar == 0:
            out.append(None)
        else:
            out.append(var / (e2 * gbar * gbar))
    return out


def test_hand_cases_coordwise():
    cases = json.load(open(GOLDEN))["coordwise"]
    c = cases[0]
    grads = [np.asarray(g, dtype=np.float32) for g in c["grads"]]
    for dec in c["decisions"]:
        r = orc.norm_test_coordwise(grads, c["eta"], dec["b_cur"], want_ratios=True)
        assert list(r["ratios"]) == c["ratios"] and r["T"] == c["T"] and r["argmax"] == c["argmax"]
        assert r["b_next"] == dec["b_next"]
        assert bool(r["flags"] & orc.FLAG_VIOLATED) == dec["violated"]
        # the summed test on the same data decides differently at b = 2
        s = orc.norm_test(grads, c["eta"], dec["b_cur"])
        assert Fraction(s["T"]).limit_denominator(1000) == Fraction(*c["T_sum_fraction"])
        assert s["b_next"] == dec["b_next_summed"]
    r = orc.persample_coordwise(np.stack(grads), c["eta"])
    assert r["T"] == c["T_persample"] and r["b_next"] == c["b_next_persample"]
    c = cases[1]
    grads = [np.asarray(g, dtype=np.float32) for g in c["grads"]]
    r = orc.norm_test_coordwise(grads, c["eta"], 7, want_ratios=True)
    assert [("inf" if math.isinf(x) else x) for x in r["ratios"]] == c["ratios"]
    assert r["T"] == math.inf and r["argmax"] == c["argmax"] and r["flags"] == c["flags"]
    assert r["b_next"] == 2 ** 63 - 1
    r = orc.norm_test_coordwise([g[1:] for g in grads], c["eta"], 7)
    assert r["T"] == 0.0 and r["flags"] == 0 and r["b_next"] == 7
    z = [np.zeros(3, dtype=np.float32)] * 2
    r = orc.norm_test_coordwise(z, c["eta"], 7)
    assert r["T"] == 0.0 and r["flags"] == orc.FLAG_DEGENERATE and r["b_next"] == 7


@pytest.mark.parametrize("K,d", [(1, 1), (2, 3), (3, 5), (4, 8), (5, 7), (7, 2)])
@pytest.mark.parametrize("kind", ["f32", "bf16"])
def test_coordwise_brute_force_rational(K, d, kind):
    rng = np.random.default_rng(300 + 10 * K + d)
    raw = rng.normal(0.1, 1.0, size=(K, d)).astype(np.float32)
    raw[:, 0] = raw[0, 0]                      # a zero-variance coordinate
    if kind == "bf16":
        bits = [bf16_bits(r) for r in raw]
        vals = [bf16_to_f64(b) for b in bits]
        grads = bits
    else:
        vals = [r.astype(np.float64) for r in raw]
        grads = [r for r in raw]
    eta = 0.375
    want = frac_coordwise([list(v) for v in vals], K, eta)
    finite = [w for w in want if w is not None]
    T = max(finite)
    arg = want.index(T)
    for b_cur in (1, 3, 10 ** 6):
        r = orc.norm_test_coordwise(grads, eta, b_cur, want_ratios=True)
        for got, w in zip(r["ratios"], want):
            assert got == pytest.approx(float(w), rel=1e-13)
        assert r["ratios"][0] == 0.0
        assert r["T"] == pytest.approx(float(T), rel=1e-13) and r["argmax"] == arg
        assert r["b_next"] == (math.ceil(T) if T > b_cur else b_cur)
    # per-sample form: the rows are the samples, normalisation b-1
    if K >= 2 and kind == "f32":
        want = frac_coordwise([list(v) for v in vals], K - 1, eta)
        r = orc.persample_coordwise(raw, eta, want_ratios=True)
        for got, w in zip(r["ratios"], want):
            assert got == pytest.approx(float(w), rel=1e-13)
        T = max(want)
        assert r["b_next"] == (math.ceil(T) if T > K else K) and r["argmax"] == want.index(T)


def test_coordwise_against_numpy_and_invariants():
    rng = np.random.default_rng(31)
    K, d, eta = 8, 12_345, 0.2
    grads = [rng.normal(0.05, 0.3, size=d).astype(np.float32) for _ in range(K)]
    G = np.stack(grads).astype(np.float64)
    t = G.var(axis=0, ddof=0) / (eta ** 2 * G.mean(axis=0) ** 2)
    offs = [0, 100, 100, 5000, d]
    r = orc.norm_test_coordwise(grads, eta, 64, shard_offsets=offs, want_ratios=True)
    np.testing.assert_allclose(r["ratios"], t, rtol=1e-11)
    assert r["argmax"] == int(np.argmax(t)) and r["T"] == pytest.approx(t.max(), rel=1e-11)
    # shard maxima: the maximum over the shard's slice; an empty shard reports 0
    for s in range(4):
        want = t[offs[s]:offs[s + 1]].max() if offs[s + 1] > offs[s] else 0.0
        assert r["shard_max"][s] == pytest.approx(want, rel=1e-11)
    assert r["T"] == r["shard_max"].max()
    # the sums are those of the summed test, and the coordinate-wise statistic dominates the
    # summed one (which is a weighted mean of the T_i with weights gbar_i^2)
    s = orc.norm_test(grads, eta, 64, shard_offsets=offs)
    for key in ("n2", "S", "Q"):   # same sums, another order of additions
        assert r[key] == pytest.approx(s[key], rel=1e-12)
    assert r["T"] >= s["T"]
    # one coordinate: the two statistics are the same expression
    one = [g[7:8] for g in grads]
    assert orc.norm_test_coordwise(one, eta, 64)["T"] == orc.norm_test(one, eta, 64)["T"]
    # scaling every gradient by a power of two changes no ratio; a permutation of the
    # coordinates moves the argmax with it
    r2 = orc.norm_test_coordwise([4.0 * g for g in grads], eta, 64, want_ratios=True)
    assert np.array_equal(r2["ratios"], r["ratios"])
    perm = rng.permutation(d)
    r3 = orc.norm_test_coordwise([g[perm] for g in grads], eta, 64)
    assert r3["T"] == r["T"] and perm[r3["argmax"]] == r["argmax"]
    # T scales with 1/eta^2, so b_next never grows with eta
    seen = [orc.norm_test_coordwise(grads, e, 64)["b_next"] for e in (0.05, 0.1, 0.2, 0.4, 3.0, 1e4)]
    assert seen == sorted(seen, reverse=True) and seen[-1] == 64
    # per-sample form against numpy's ddof=1
    Gs = rng.normal(0.02, 0.3, size=(33, 700)).astype(np.float32)
    tp = Gs.astype(np.float64).var(axis=0, ddof=1) / (eta ** 2 * Gs.astype(np.float64).mean(axis=0) ** 2)
    rp = orc.persample_coordwise(Gs, eta, want_ratios=True)
    np.testing.assert_allclose(rp["ratios"], tp, rtol=1e-11)
    assert rp["argmax"] == int(np.argmax(tp)) and rp["norm"] == 32
    # a strided matrix is read row by row, not transposed
    wide = np.zeros((33, 704), dtype=np.float32)
    wide[:, :700] = Gs
    assert orc.persample_coordwise(wide[:, :700], eta)["T"] == rp["T"]
    # non-finite input: flag, T = NaN, batch size kept
    bad = [g.copy() for g in grads]
    bad[3][17] = np.nan
    rb = orc.norm_test_coordwise(bad, eta, 64)
    assert rb["flags"] == orc.FLAG_NONFINITE and math.isnan(rb["T"]) and rb["b_next"] == 64


def test_thread_count_does_not_change_results():
    code = (
        "import sys, numpy as np; sys.path.insert(0, %r)\n"
        "from oracle import abs_oracle as orc\n"
        "rng = np.random.default_rng(9)\n"
        "A = (0.05*rng.standard_normal((4, 100003))).astype(np.float32)\n"
        "r = orc.norm_test([A[k] for k in range(4)], 0.1, 64, shard_offsets=[0, 5, 50001, 100003])\n"
        "print(repr((r['n2'], r['S'], r['Q'], r['T'], r['b_next'], r['shards'].tolist())))\n"
    ) % os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    outs = []
    for nt in ("1", "3"):
        env = dict(os.environ, OMP_NUM_THREADS=nt)
        outs.append(subprocess.check_output([sys.executable, "-c", code], env=env).decode())
    assert outs[0] == outs[1]
