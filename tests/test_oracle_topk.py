"""Pins of the oracle's discrete top-k quantifier (orc_topk) against what does not depend on it:
brute-force rank counting on small rows, the reductions k = V (the continuous quantifier) and
k = 1, and closed forms for constant and geometric rows (paper: the discrete-vs-continuous
comparison; the paper prints no formula, so the pins fix the reading stated in the oracle)."""
import math

import numpy as np
import pytest

import oracle


def _params(r=0.5, tau=1e-3):
    return oracle.IntervalParams(radius_mode=oracle.RADIUS_SCALAR, r_scalar=r, tau=tau)


def _brute_set(c, k):
    """Codes whose rank (number of codes that beat them: larger logit, or equal logit and lower
    index) is below k -- O(V^2), no sort."""
    n = len(c)
    keep = []
    for i in range(n):
        rank = sum(1 for j in range(n) if c[j] > c[i] or (c[j] == c[i] and j < i))
        if rank < k:
            keep.append(i)
    return keep


@pytest.mark.parametrize("v,k", [(5, 1), (8, 3), (17, 17), (64, 10), (64, 63)])
def test_set_matches_rank_counting(v, k):
    rng = np.random.default_rng(100 + v + k)
    # a coarse grid of values so that ties are frequent
    c = (rng.integers(-6, 6, size=(7, v)) * 0.5).astype(np.float32)
    res = oracle.topk(c, k, _params(), indices=True)
    for row in range(c.shape[0]):
        keep = _brute_set(c[row], k)
        assert list(res.indices[row]) == keep
        kth = min(c[row][i] for i in keep)
        assert res.kth_logit[row] == kth
        assert res.n_above[row] == int((c[row] > kth).sum())
        p = np.exp(c[row].astype(np.float64) - c[row].max())
        p /= p.sum()
        assert res.mass[row] == pytest.approx(p[keep].sum(), rel=1e-13)
        pk = p[keep] / p[keep].sum()
        assert res.entropy[row] == pytest.approx(-(pk * np.log(pk)).sum(), rel=1e-12, abs=1e-14)


def test_k_equal_v_is_the_continuous_quantifier():
    rng = np.random.default_rng(7)
    c = (3.0 * rng.standard_normal((9, 48))).astype(np.float32)
    rad = rng.uniform(0.05, 1.5, size=9).astype(np.float32)
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=rad, tau=2e-3)
    q = oracle.quantify(c, prm)
    t = oracle.topk(c, 48, prm, indices=True)
    for name in ("entropy", "S_lo", "S_up", "omega", "sigma", "score"):
        np.testing.assert_allclose(getattr(t, name), getattr(q, name), rtol=1e-13, atol=0)
    np.testing.assert_allclose(t.mass, 1.0, rtol=1e-14)
    assert np.array_equal(t.flag, q.flag)
    assert np.array_equal(t.indices, np.tile(np.arange(48, dtype=np.int32), (9, 1)))
    assert np.array_equal(t.kth_logit, c.min(axis=1).astype(np.float64))


def test_k_one():
    rng = np.random.default_rng(8)
    c = rng.standard_normal((6, 33)).astype(np.float32)
    q = oracle.quantify(c, _params())
    t = oracle.topk(c, 1, _params(), indices=True)
    np.testing.assert_allclose(t.mass, q.p_max, rtol=1e-14)
    assert np.array_equal(t.indices[:, 0], q.argmax)
    # one code: p = 1, bounds 1 and 1 before the rescale -> 0.99 and 1.01 after it
    np.testing.assert_allclose(t.omega, 0.02, rtol=1e-12)
    np.testing.assert_allclose(t.sigma, 0.0, atol=1e-15)
    np.testing.assert_allclose(t.entropy, 0.0, atol=1e-15)
    assert not t.flag.any()


def test_constant_and_geometric_rows():
    v = 40
    const = np.full((1, v), 1.25, np.float32)
    for k in (1, 7, 40):
        t = oracle.topk(const, k, _params(), indices=True)
        assert t.mass[0] == pytest.approx(k / v, rel=1e-14)
        assert t.entropy[0] == pytest.approx(math.log(k), rel=1e-13, abs=1e-15)
        assert list(t.indices[0]) == list(range(k))  # equal logits: lowest indices
        assert t.n_above[0] == 0
        assert t.sigma[0] == pytest.approx(0.0, abs=1e-15)  # equal widths
    # c_i = -i ln 2 (exact in fp32 up to rounding of ln 2): mass of the first k = (1 - 2^-k) / (1 - 2^-v)
    geo = (-np.arange(v) * np.float32(math.log(2.0))).astype(np.float32)[None, :]
    g = np.exp(geo[0].astype(np.float64))
    for k in (1, 3, 12):
        t = oracle.topk(geo, k, _params(), indices=True)
        assert t.mass[0] == pytest.approx(g[:k].sum() / g.sum(), rel=1e-13)
        assert t.mass[0] == pytest.approx((1 - 2.0 ** -k) / (1 - 2.0 ** -v), rel=1e-5)
        assert list(t.indices[0]) == list(range(k))
        assert t.n_above[0] == k - 1


def test_mass_grows_with_k_and_slice_is_respected():
    rng = np.random.default_rng(9)
    c = rng.standard_normal((5, 64)).astype(np.float32)
    last = np.zeros(5)
    for k in (1, 2, 8, 30, 40):
        t = oracle.topk(c, k, _params(), valid_begin=16, valid_count=40, indices=True)
        assert (t.mass > last).all()
        last = t.mass
        assert t.indices.min() >= 16 and t.indices.max() < 56
    sub = np.ascontiguousarray(c[:, 16:56])
    a = oracle.topk(c, 8, _params(), valid_begin=16, valid_count=40, indices=True)
    b = oracle.topk(sub, 8, _params(), indices=True)
    assert np.array_equal(a.indices, b.indices + 16)
    np.testing.assert_array_equal(a.score, b.score)


def test_unusable_rows():
    c = np.zeros((3, 16), np.float32)
    c[0, 3] = np.nan
    c[1, :] = -np.inf
    t = oracle.topk(c, 4, _params(), indices=True)
    assert t.row_status[0] & oracle.ROW_NAN and t.row_status[1] & oracle.ROW_NO_FINITE and t.row_status[2] == 0
    assert np.isnan(t.score[:2]).all() and t.flag[0] == 1 and t.flag[1] == 1
    assert (t.indices[:2] == -1).all()
    with pytest.raises(ValueError):
        oracle.topk(c, 17, _params())
