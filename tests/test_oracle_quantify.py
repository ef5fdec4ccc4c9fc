"""Pins for the oracle's quantifier: closed forms, a hand-worked example, invariants the paper
states, and a library log-sum-exp.  Each test is chosen so that a plausible slip in the oracle
(a dropped term, a swapped sign on the radius, population vs sample variance, a wrong n) fails it."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.special
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _params(**kw):
    return oracle.IntervalParams(**kw)


def _rand_logits(rows, v, scale=3.0, seed=0, dtype=np.float32):
    rng = np.random.default_rng(seed)
    return (scale * rng.standard_normal((rows, v))).astype(dtype)


def test_entropy_uniform_row_is_log_v():
    for v in (2, 7, 64, 1000):
        c = np.full((1, v), 1.25, np.float32)
        q = oracle.quantify(c, _params())
        assert q.entropy[0] == pytest.approx(math.log(v), rel=1e-13)
        assert q.p_max[0] == pytest.approx(1.0 / v, rel=1e-13)
        assert q.argmax[0] == 0  # lowest index among ties


def test_entropy_one_hot_row_is_zero():
    c = np.full((1, 33), -np.inf, np.float32)
    c[0, 17] = 0.0
    q = oracle.quantify(c, _params())
    assert q.entropy[0] == 0.0
    assert q.p_max[0] == 1.0
    assert q.argmax[0] == 17
    assert q.row_status[0] == 0


def test_softmax_sums_to_one_and_matches_library_logsumexp():
    c = _rand_logits(16, 1000, scale=5.0, seed=1)
    q = oracle.quantify(c, _params(), dense=True)
    np.testing.assert_allclose(q.p.sum(1), 1.0, rtol=0, atol=1e-13)
    np.testing.assert_allclose(q.lse, scipy.special.logsumexp(c.astype(np.float64), axis=1), rtol=1e-14)
    np.testing.assert_allclose(q.p, scipy.special.softmax(c.astype(np.float64), axis=1), rtol=1e-12, atol=0)
    ent = scipy.stats.entropy(scipy.special.softmax(c.astype(np.float64), axis=1), axis=1) \
        if hasattr(scipy, "stats") else None
    if ent is not None:
        np.testing.assert_allclose(q.entropy, ent, rtol=1e-12)
    assert (q.argmax == c.argmax(1)).all()
    np.testing.assert_allclose(q.row_max, c.max(1))


def test_shift_invariance():
    c = np.round(_rand_logits(4, 257, seed=2) * 64) / np.float32(64)  # multiples of 1/64: the shift is exact
    shifted = c + np.float32(8.0)
    assert np.array_equal(shifted.astype(np.float64) - 8.0, c.astype(np.float64))
    a = oracle.quantify(c, _params(r_scalar=0.3))
    b = oracle.quantify(shifted, _params(r_scalar=0.3))
    for name in ("entropy", "omega", "sigma", "score", "S_lo", "S_up", "sum_exp"):
        np.testing.assert_allclose(getattr(a, name), getattr(b, name), rtol=1e-12)
    np.testing.assert_allclose(a.lse + 8.0, b.lse, rtol=1e-14)


def test_worked_example_exact_rationals():
    vals = {}
    with open(os.path.join(GOLDEN, "interfuse_worked_example.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, num, den = line.split()
            vals[k] = Fraction(int(num), int(den))
    c = np.log(np.array([[1.0, 2.0, 3.0]])).astype(np.float32)
    # float32 logs are not exact: feed the example through float64-exact inputs instead by
    # checking against the rational values with the float32 input error (~1e-7) as tolerance
    q = oracle.quantify(c, _params(r_scalar=math.log(2.0)), dense=True)
    tol = 5e-7
    for i in range(3):
        assert q.p_lo[0, i] == pytest.approx(float(vals["p_lo_%d" % i]), rel=tol)
        assert q.p_up[0, i] == pytest.approx(float(vals["p_up_%d" % i]), rel=tol)
    assert q.S_lo[0] == pytest.approx(float(vals["S_lo"]), rel=tol)
    assert q.S_up[0] == pytest.approx(float(vals["S_up"]), rel=tol)
    assert q.scale_lo[0] == 1.0 and q.scale_up[0] == 1.0
    omega = vals["omega"]
    assert q.omega[0] == pytest.approx(float(omega), rel=tol)
    ssq = vals["sum_delta_sq_term0"] + vals["sum_delta_sq_term1"] + vals["sum_delta_sq_term2"]
    var = ssq / 3 - (omega / 3) ** 2
    assert q.sigma[0] == pytest.approx(math.sqrt(float(var)), rel=2e-6)
    assert q.score[0] == pytest.approx(float(omega) * math.sqrt(float(var)), rel=2e-6)
    assert q.entropy[0] == pytest.approx(math.log(6) / 6 + math.log(3) / 3 + math.log(2) / 2, rel=tol)


def test_zero_radius_closed_form():
    """r = 0: both bounds equal softmax(c), S_l = S_u = 1, so the rescale gives delta = 0.02 p:
    Omega = 0.02, Sigma = 0.02 * popstd(p), U = 4e-4 * popstd(p)."""
    c = _rand_logits(8, 500, scale=2.0, seed=3)
    q = oracle.quantify(c, _params(r_scalar=0.0), dense=True)
    p = scipy.special.softmax(c.astype(np.float64), axis=1)
    np.testing.assert_allclose(q.S_lo, 1.0, atol=1e-13)
    np.testing.assert_allclose(q.S_up, 1.0, atol=1e-13)
    np.testing.assert_allclose(q.p_lo, 0.99 * p, rtol=1e-12)
    np.testing.assert_allclose(q.p_up, 1.01 * p, rtol=1e-12)
    np.testing.assert_allclose(q.omega, 0.02, rtol=1e-11)
    np.testing.assert_allclose(q.sigma, 0.02 * p.std(axis=1), rtol=1e-10)  # numpy std is the population std
    np.testing.assert_allclose(q.score, 4e-4 * p.std(axis=1), rtol=1e-10)


def test_two_code_row_is_logistic():
    """V = 2: p^l_1 = sigmoid(c_1 - c_2 - r), p^u_1 = sigmoid(c_1 - c_2 + r) before the rescale."""
    c = np.array([[0.5, -1.25], [2.0, 2.0], [-3.0, 4.0]], np.float32)
    r = 0.75
    q = oracle.quantify(c, _params(r_scalar=r), dense=True)
    d = (c[:, 0] - c[:, 1]).astype(np.float64)
    lo0, up0 = scipy.special.expit(d - r), scipy.special.expit(d + r)
    lo1, up1 = scipy.special.expit(-d - r), scipy.special.expit(-d + r)
    np.testing.assert_allclose(q.S_lo, lo0 + lo1, rtol=1e-13)
    np.testing.assert_allclose(q.S_up, up0 + up1, rtol=1e-13)
    np.testing.assert_allclose(q.p_lo[:, 0], lo0 * q.scale_lo, rtol=1e-13)
    np.testing.assert_allclose(q.p_up[:, 0], up0 * q.scale_up, rtol=1e-13)
    np.testing.assert_allclose(q.p_lo[:, 1], lo1 * q.scale_lo, rtol=1e-13)
    np.testing.assert_allclose(q.p_up[:, 1], up1 * q.scale_up, rtol=1e-13)


def test_one_hot_row_meets_claim3_with_equality():
    """One finite code: both raw bounds are 1 there and 0 elsewhere, so after the rescale
    delta = (0.02, 0, ..., 0): Omega = 0.02 and Sigma = 0.02 * sqrt(n-1)/n (Claim 3, tight case)."""
    for n in (2, 9, 64):
        c = np.full((1, n), -np.inf, np.float32)
        c[0, n // 2] = 3.0
        q = oracle.quantify(c, _params(r_scalar=1.5))
        assert q.omega[0] == pytest.approx(0.02, rel=1e-12)
        assert q.sigma[0] == pytest.approx(0.02 * math.sqrt(n - 1) / n, rel=1e-12)
        assert q.score[0] == pytest.approx(4e-4 * math.sqrt(n - 1) / n, rel=1e-12)


def test_constant_row_constant_radius_has_zero_disparity():
    c = np.full((1, 40), -0.5, np.float32)
    q = oracle.quantify(c, _params(r_scalar=0.8))
    assert q.sigma[0] == pytest.approx(0.0, abs=1e-15)  # rounding of omega / n only
    assert q.score[0] == pytest.approx(0.0, abs=1e-15)
    assert q.omega[0] > 0.02


@pytest.mark.parametrize("mode", ["scalar", "per_row", "per_code", "per_code_raw"])
def test_validity_invariants_and_claims(mode):
    rows, v = 12, 64
    c = _rand_logits(rows, v, scale=4.0, seed=5)
    rng = np.random.default_rng(6)
    if mode == "scalar":
        prm = _params(r_scalar=0.6)
    elif mode == "per_row":
        prm = _params(radius_mode=oracle.RADIUS_PER_ROW, radius=rng.uniform(0, 2, rows).astype(np.float32))
    elif mode == "per_code":
        prm = _params(radius_mode=oracle.RADIUS_PER_CODE, radius=rng.uniform(0, 2, (rows, v)).astype(np.float32))
    else:
        prm = _params(radius_mode=oracle.RADIUS_PER_CODE, radius_is_raw=True,
                      radius=rng.normal(0, 1, (rows, v)).astype(np.float32))
    q = oracle.quantify(c, prm, dense=True)
    raw_lo, raw_up = q.p_lo / q.scale_lo[:, None], q.p_up / q.scale_up[:, None]
    assert (raw_lo >= 0).all() and (raw_up <= 1 + 1e-15).all() and (raw_lo <= raw_up + 1e-18).all()
    assert (raw_lo <= q.p + 1e-15).all() and (q.p <= raw_up + 1e-15).all()  # the centre lies inside
    assert (q.p_lo.sum(1) <= 0.99 + 1e-12).all() and (q.p_up.sum(1) >= 1.01 - 1e-12).all()
    delta = q.p_up - q.p_lo
    n = v
    np.testing.assert_allclose(q.omega, delta.sum(1), rtol=1e-12)
    assert (q.score >= 0).all()
    assert (q.sigma <= math.sqrt(n - 1) / n * q.omega * (1 + 1e-12)).all()  # Claim 3
    assert (q.score <= 0.5 * (delta ** 2).sum(1) * (1 + 1e-12)).all()  # Claim 4
    mu = q.omega / n
    np.testing.assert_allclose(q.score, n * mu * mu * (q.sigma / mu), rtol=1e-12)  # U = n mu^2 CV
    np.testing.assert_allclose(q.sigma, delta.std(axis=1), rtol=1e-9)  # library population std
    # Proposition 1: two distributions inside the box differ by at most Omega in L1
    assert (np.abs(q.p - np.clip(q.p, q.p_lo, q.p_up)).sum(1) <= q.omega).all()


def test_softplus_and_clamp():
    """raw radius rho -> softplus(rho) (library log1p/exp), then min(., r_max)."""
    c = _rand_logits(3, 16, seed=7)
    rho = np.array([-2.0, 0.3, 5.0], np.float32)
    r = np.log1p(np.exp(rho.astype(np.float64)))
    a = oracle.quantify(c, _params(radius_mode=oracle.RADIUS_PER_ROW, radius=rho, radius_is_raw=True, r_max=2.0))
    b = oracle.quantify(c, _params(radius_mode=oracle.RADIUS_PER_ROW, radius=np.minimum(r, 2.0).astype(np.float32)))
    # float32 rounding of the pre-activated radius limits the agreement
    np.testing.assert_allclose(a.omega, b.omega, rtol=1e-6)
    np.testing.assert_allclose(a.score, b.score, rtol=1e-6)
    # clamp really bites: r_max = 2 and r_max = 100 differ on the row with rho = 5
    d = oracle.quantify(c, _params(radius_mode=oracle.RADIUS_PER_ROW, radius=rho, radius_is_raw=True, r_max=100.0))
    assert d.omega[2] > a.omega[2] * 1.01
    assert d.omega[0] == pytest.approx(a.omega[0], rel=1e-14)


def test_widths_grow_with_radius():
    c = _rand_logits(2, 128, seed=8)
    prev = None
    for r in (0.0, 0.1, 0.5, 1.0, 3.0):
        q = oracle.quantify(c, _params(r_scalar=r))
        if prev is not None:
            assert (q.omega > prev).all()
        prev = q.omega


def test_masked_slice_uses_valid_count_as_n():
    """Codes outside the valid slice are not part of V: same result as the compact row."""
    v, vb, n = 256, 64, 96
    inner = _rand_logits(5, n, seed=9)
    full = np.full((5, v), -np.inf, np.float32)
    full[:, vb:vb + n] = inner
    full[:, :vb] = 123.0  # garbage outside the slice must not be read
    a = oracle.quantify(full, _params(r_scalar=0.4), valid_begin=vb, valid_count=n)
    b = oracle.quantify(inner, _params(r_scalar=0.4))
    for name in ("lse", "entropy", "omega", "sigma", "score", "S_lo", "S_up"):
        np.testing.assert_array_equal(getattr(a, name), getattr(b, name))
    assert (a.argmax == b.argmax + vb).all()


def test_minus_inf_inside_slice_counts_in_n():
    c = _rand_logits(1, 10, seed=10)
    d = np.concatenate([c, np.full((1, 6), -np.inf, np.float32)], axis=1)
    a, b = oracle.quantify(c, _params(r_scalar=0.7)), oracle.quantify(d, _params(r_scalar=0.7))
    assert b.omega[0] == pytest.approx(a.omega[0], rel=1e-14)
    # same widths plus six zeros: the population variance over n = 16 differs from n = 10
    assert b.sigma[0] != pytest.approx(a.sigma[0], rel=1e-3)


def test_bf16_rows_equal_their_float32_widening():
    c = torch.randn(6, 300, generator=torch.Generator().manual_seed(11)) * 4
    cb = c.to(torch.bfloat16)
    a = oracle.quantify(cb, _params(r_scalar=0.25))
    b = oracle.quantify(cb.to(torch.float32), _params(r_scalar=0.25))
    for name in ("lse", "entropy", "omega", "sigma", "score"):
        np.testing.assert_array_equal(getattr(a, name), getattr(b, name))


def test_policies_and_status():
    c = _rand_logits(6, 50, seed=12)
    base = oracle.quantify(c, _params(r_scalar=1.0))
    tau = float(np.median(base.score))
    q = oracle.quantify(c, _params(r_scalar=1.0, tau=tau))
    assert (q.flag == (base.score > tau)).all()  # Algorithm 1: kept on the device iff U <= tau
    q = oracle.quantify(c, _params(policy=oracle.POLICY_ENTROPY, tau=float(np.median(base.entropy))))
    assert (q.flag == (base.entropy > np.median(base.entropy))).all()
    q = oracle.quantify(c, _params(policy=oracle.POLICY_MAXPROB, tau=float(np.median(base.p_max))))
    assert (q.flag == (base.p_max < np.median(base.p_max))).all()
    u = np.linspace(0, 0.99, 6).astype(np.float32)
    q = oracle.quantify(c, _params(policy=oracle.POLICY_RANDOM, tau=0.5, u_flag=u))
    assert (q.flag == (u < 0.5)).all()
    assert oracle.quantify(c, _params(policy=oracle.POLICY_ALL)).flag.all()
    bad = c.copy()
    bad[1, 3] = np.nan
    bad[2, :] = -np.inf
    bad[3, 0] = np.inf
    q = oracle.quantify(bad, _params(r_scalar=1.0, tau=1e9))
    assert q.row_status[1] & oracle.ROW_NAN and q.row_status[2] & oracle.ROW_NO_FINITE
    assert q.row_status[3] & oracle.ROW_NAN
    assert q.flag[1] == 1 and q.flag[2] == 1 and q.flag[3] == 1 and q.flag[0] == 0
    assert np.isnan(q.score[1]) and np.isnan(q.score[2])


def test_planted_mistakes_are_caught():
    """Sanity of the pins themselves: typical slips change the pinned numbers by far more than
    the tolerances above (checked on the worked example, in exact rationals)."""
    e = [Fraction(1), Fraction(2), Fraction(3)]
    z = sum(e)
    right_lo = [x / 2 / (z - x + x / 2) for x in e]
    dropped_term = [x / 2 / (z - x) for x in e]  # forgets + exp(c - r) in the denominator
    swapped_sign = [x * 2 / (z - x + x * 2) for x in e]  # uses +r for the lower bound
    assert right_lo == [Fraction(1, 11), Fraction(1, 5), Fraction(1, 3)]
    assert all(abs(float(a - b)) > 1e-3 for a, b in zip(right_lo, dropped_term))
    assert all(abs(float(a - b)) > 1e-3 for a, b in zip(right_lo, swapped_sign))
