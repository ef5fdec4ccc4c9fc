"""Pins of the oracle's score variants, multi-head aggregation and Inter-DRO forward value against
closed forms, the paper's own scaling claim, special cases that reduce to functions pinned
elsewhere, and library routines (paper: uncertainty appendix, "Practical Remarks for Thresholding
and Normalization"; appendix "Impact of Inter-Head Capacity"; method section, "Inter-DRO Loss")."""
import math

import numpy as np
import pytest
from scipy.special import log_softmax, rel_entr, softmax

import oracle


# ---------------------------------------------------------------- score variants
def _widths_stats(delta):
    om = delta.sum(axis=1)
    sg = delta.std(axis=1)  # population std
    return om, sg


def test_variants_follow_the_scaling_claim():
    # U(alpha delta) = alpha^2 U(delta) (scaling claim of the uncertainty appendix): PER_OMEGA2 is
    # scale free, PER_N scales like U, ADDITIVE with lambda2 = 0 is linear in the widths
    rng = np.random.default_rng(1)
    delta = rng.uniform(0.0, 1e-2, size=(6, 50))
    om, sg = _widths_stats(delta)
    om3, sg3 = _widths_stats(3.0 * delta)
    u, _, _ = oracle.score_variant(om, sg, 50, oracle.SCORE_PRODUCT)
    u3, _, _ = oracle.score_variant(om3, sg3, 50, oracle.SCORE_PRODUCT)
    np.testing.assert_allclose(u3, 9.0 * u, rtol=1e-13)
    np.testing.assert_allclose(u, delta.sum(axis=1) * delta.std(axis=1), rtol=1e-14)
    a, _, _ = oracle.score_variant(om, sg, 50, oracle.SCORE_PER_OMEGA2)
    a3, _, _ = oracle.score_variant(om3, sg3, 50, oracle.SCORE_PER_OMEGA2)
    np.testing.assert_allclose(a3, a, rtol=1e-13)
    # Sigma / Omega = CV / n (the appendix's rewrite U = n mu^2 CV... in its dimensionless form)
    np.testing.assert_allclose(a, (delta.std(axis=1) / delta.mean(axis=1)) / 50, rtol=1e-13)
    b, _, _ = oracle.score_variant(om, sg, 50, oracle.SCORE_PER_N)
    np.testing.assert_allclose(b, u / 50, rtol=1e-14)
    lin, _, _ = oracle.score_variant(om, sg, 50, oracle.SCORE_ADDITIVE, lambda1=0.25, lambda2=0.0)
    np.testing.assert_allclose(lin, 0.25 * om, rtol=1e-14)


def test_variants_reduce_to_the_product():
    rng = np.random.default_rng(2)
    om, sg = rng.uniform(0.02, 2, 9), rng.uniform(0, 0.1, 9)
    u, fu, _ = oracle.score_variant(om, sg, 10, oracle.SCORE_PRODUCT, tau=0.05)
    s, fs, _ = oracle.score_variant(om, sg, 10, oracle.SCORE_SMOOTHED, eps=0.0, tau=0.05)
    a, fa, _ = oracle.score_variant(om, sg, 10, oracle.SCORE_ADDITIVE, lambda1=0.0, lambda2=1.0, tau=0.05)
    np.testing.assert_allclose(s, u, rtol=1e-14)
    np.testing.assert_array_equal(a, u)
    assert np.array_equal(fu, fs) and np.array_equal(fu, fa)
    assert np.array_equal(fu, (u > 0.05).astype(np.uint8))


def test_uniform_widths_answer_only_in_the_smoothed_and_additive_forms():
    # remark 2: the product vanishes for equal widths; sqrt(Sigma^2 + eps) and the additive form do not
    om, sg = np.array([0.8]), np.array([0.0])
    assert oracle.score_variant(om, sg, 100, oracle.SCORE_PRODUCT)[0][0] == 0.0
    assert oracle.score_variant(om, sg, 100, oracle.SCORE_SMOOTHED, eps=1e-4)[0][0] == pytest.approx(0.8e-2, rel=1e-14)
    assert oracle.score_variant(om, sg, 100, oracle.SCORE_ADDITIVE, lambda1=0.1, lambda2=1.0)[0][0] == pytest.approx(0.08, rel=1e-14)
    v, f, _ = oracle.score_variant(np.array([np.nan]), np.array([0.1]), 4, oracle.SCORE_PER_N, tau=1.0)
    assert np.isnan(v[0]) and f[0] == 1


# ---------------------------------------------------------------- several heads
def test_one_head_and_identical_heads_are_the_single_head_quantifier():
    rng = np.random.default_rng(3)
    c = (2.0 * rng.standard_normal((5, 40))).astype(np.float32)
    rad = rng.uniform(0.1, 1.2, 5).astype(np.float32)
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=rad, tau=3e-3)
    q = oracle.quantify(c, prm)
    for heads in (1, 3):
        prm_h = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=np.tile(rad, (heads, 1)), tau=3e-3)
        e = oracle.ensemble(np.stack([c] * heads), prm_h, dense=True)
        for name in ("p_max", "entropy", "S_lo", "S_up", "omega", "sigma", "score"):
            np.testing.assert_allclose(getattr(e, name), getattr(q, name), rtol=1e-11, atol=1e-15)
        np.testing.assert_allclose(e.pbar, softmax(c.astype(np.float64), axis=1), rtol=1e-12)
        assert np.array_equal(e.flag, q.flag)


def test_ensemble_averages_distributions_not_logits():
    # two heads whose distributions are mirror images: the average is uniform although neither head is;
    # a uniform distribution with a constant radius has equal widths, so Sigma = 0 and U = 0
    v = 8
    a = np.linspace(-0.4, 0.4, v).astype(np.float32)
    pa = softmax(a.astype(np.float64))
    pb = 2.0 / v - pa
    assert (pb > 0).all()
    b = np.log(pb).astype(np.float32)
    heads = np.stack([a[None, :], b[None, :]])
    e = oracle.ensemble(heads, oracle.IntervalParams(r_scalar=0.7, tau=1e-9), dense=True)
    np.testing.assert_allclose(e.pbar[0], 1.0 / v, rtol=1e-6)
    assert e.entropy[0] == pytest.approx(math.log(v), rel=1e-6)
    assert e.sigma[0] == pytest.approx(0.0, abs=1e-8)
    # the order of the heads does not matter, and the radius is the mean of the heads' radii
    rng = np.random.default_rng(4)
    hh = rng.standard_normal((3, 4, 24)).astype(np.float32)
    rr = rng.uniform(0.1, 1, (3, 4)).astype(np.float32)
    e1 = oracle.ensemble(hh, oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=rr))
    e2 = oracle.ensemble(hh[[2, 0, 1]], oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=rr[[2, 0, 1]]))
    np.testing.assert_allclose(e1.score, e2.score, rtol=1e-12)
    pbar = softmax(hh.astype(np.float64), axis=2).mean(axis=0)
    single = oracle.quantify(np.log(pbar).astype(np.float32),
                             oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=rr.astype(np.float64).mean(axis=0).astype(np.float32)))
    np.testing.assert_allclose(e1.score, single.score, rtol=1e-5)  # ln pbar rounded to fp32 on the way in


def test_vote_is_a_strict_majority():
    flags = np.array([[1, 1, 0, 0, 1], [1, 0, 0, 1, 1], [1, 0, 0, 0, 0]], np.uint8)
    out, votes = oracle.vote(flags)
    assert list(votes) == [3, 1, 0, 1, 2] and list(out) == [1, 0, 0, 0, 1]
    out2, _ = oracle.vote(flags[:2])  # two heads: both must flag
    assert list(out2) == [1, 0, 0, 0, 1]
    out1, _ = oracle.vote(flags[:1])
    assert np.array_equal(out1, flags[0])


# ---------------------------------------------------------------- Inter-DRO forward
def _softplus_inv(r):
    return np.log(np.expm1(r))


def test_interdro_matches_library_pieces():
    rng = np.random.default_rng(5)
    rows, v = 6, 32
    c = (2 * rng.standard_normal((rows, v))).astype(np.float32)
    rho = rng.standard_normal((rows, v)).astype(np.float32)
    t = (c + 0.5 * rng.standard_normal((rows, v))).astype(np.float32)
    lv, lp, lb, al = 0.7, 1.3, 0.4, 2.5
    res = oracle.interdro(c, rho, t, radius_is_raw=True, lambda_v=lv, lambda_p=lp, lambda_beta=lb, alpha=al)
    r = np.log1p(np.exp(rho.astype(np.float64)))
    q = softmax(t.astype(np.float64), axis=1)
    for x, o in enumerate((c.astype(np.float64), c + r, c - r)):
        lpx = log_softmax(o, axis=1)
        np.testing.assert_allclose(res.l1[x], np.abs(np.exp(lpx) - q).sum(axis=1), rtol=1e-12)
        np.testing.assert_allclose(res.ce[x], -(q * lpx).sum(axis=1), rtol=1e-12)
    np.testing.assert_allclose(res.kl, rel_entr(q, softmax(c.astype(np.float64), axis=1)).sum(axis=1), rtol=1e-9, atol=1e-15)
    # cross-entropy = entropy of the cloud distribution + KL
    hq = -(q * np.log(q)).sum(axis=1)
    np.testing.assert_allclose(res.ce[0] - hq, res.kl, rtol=1e-9, atol=1e-14)
    w = softmax(al * res.ce[2])
    np.testing.assert_allclose(res.weights, w, rtol=1e-12)
    assert res.weights.sum() == pytest.approx(1.0, rel=1e-14)
    dro = (w * res.ce[2]).sum()
    anchor = [lv * res.l1[x].mean() + lp * res.ce[x].mean() for x in range(3)]
    align = lb * res.kl.mean()
    np.testing.assert_allclose(res.loss, [anchor[0] + align + anchor[1] + anchor[2] + dro, anchor[0] + align,
                                          anchor[1], anchor[2] + dro, dro, align], rtol=1e-12)
    assert (res.l1 <= 2.0).all() and (res.kl >= -1e-15).all()


def test_interdro_special_cases():
    rng = np.random.default_rng(6)
    c = rng.standard_normal((4, 20)).astype(np.float32)
    # a constant radius shifts every logit alike: the three distributions coincide; with cloud = centre
    # the L1 and KL terms vanish and every cross-entropy is the entropy of the distribution
    res = oracle.interdro(c, np.full_like(c, 0.8), c, radius_is_raw=False)
    q = softmax(c.astype(np.float64), axis=1)
    hq = -(q * np.log(q)).sum(axis=1)
    np.testing.assert_allclose(res.l1, 0.0, atol=1e-14)
    np.testing.assert_allclose(res.kl, 0.0, atol=1e-14)
    for x in range(3):
        np.testing.assert_allclose(res.ce[x], hq, rtol=1e-12)
    # alpha = 0: uniform weights, the DRO term is the batch mean; large alpha: it tends to the worst sample
    t = (c + rng.standard_normal(c.shape)).astype(np.float32)
    rho = rng.standard_normal(c.shape).astype(np.float32)
    r0 = oracle.interdro(c, rho, t, alpha=0.0)
    np.testing.assert_allclose(r0.weights, 0.25, rtol=1e-14)
    assert r0.loss[4] == pytest.approx(r0.ce[2].mean(), rel=1e-13)
    rbig = oracle.interdro(c, rho, t, alpha=1e4)
    assert rbig.loss[4] == pytest.approx(rbig.ce[2].max(), rel=1e-9)
    # the clamp: a huge raw radius acts as r_max
    big = oracle.interdro(c, np.full_like(c, 50.0), t, radius_is_raw=True, r_max=2.0)
    ref = oracle.interdro(c, np.full_like(c, 2.0), t, radius_is_raw=False, r_max=10.0)
    np.testing.assert_allclose(big.loss, ref.loss, rtol=1e-13)


def test_interdro_two_codes_closed_form():
    # V = 2: p_mid = sigma(c0 - c1), p_up = sigma(c0 - c1 + r0 - r1), p_lo = sigma(c0 - c1 - r0 + r1)
    c = np.array([[0.5, -0.25]], np.float32)
    r = np.array([[1.0, 0.25]], np.float32)
    t = np.array([[0.0, 1.0]], np.float32)
    res = oracle.interdro(c, r, t, radius_is_raw=False)
    sig = lambda x: 1.0 / (1.0 + math.exp(-x))
    q0 = sig(-1.0)
    for x, d in enumerate((0.75, 0.75 + 0.75, 0.75 - 0.75)):
        p0 = sig(d)
        assert res.l1[x, 0] == pytest.approx(2 * abs(p0 - q0), rel=1e-12)
        assert res.ce[x, 0] == pytest.approx(-(q0 * math.log(p0) + (1 - q0) * math.log(1 - p0)), rel=1e-12)
