"""Pins for the oracle's cloud-side test: the acceptance probability and the emitted-token
distribution that the speculative accept / resample rule must have, residual mass = total
variation, inverse-CDF end points, window bookkeeping by brute force, and the decode loop's
replay and conservation laws."""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats
import torch

import oracle
from paper_2603_25463_b200 import synth


def _softmax(x):
    return scipy.special.softmax(np.asarray(x, np.float64), axis=-1)


def _sample_tokens(p, n, rng):
    return rng.choice(len(p), size=n, p=p).astype(np.int32)


@pytest.mark.parametrize("v", [4, 8])
def test_acceptance_probability_and_emitted_distribution(v):
    """Over x ~ p and u ~ U[0,1): P(accept) = sum_i min(p_i, q_i) = 1 - TV(p, q), and the emitted
    token (x if accepted, else the residual sample) is distributed exactly as q."""
    rng = np.random.default_rng(100 + v)
    c = rng.normal(0, 1.2, v).astype(np.float32)
    t = (c + rng.normal(0, 0.9, v)).astype(np.float32)
    p, q = _softmax(c), _softmax(t)
    n = 1_000_000
    draft = np.broadcast_to(c, (n, v)).copy()
    target = np.broadcast_to(t, (n, v)).copy()
    x = _sample_tokens(p, n, rng)
    ua = rng.random(n, dtype=np.float32)
    ur = rng.random(n, dtype=np.float32)
    r = oracle.verify(draft, target, x, None, ua, ur, window=1, mode=oracle.VERIFY_ALL)
    alpha = np.minimum(p, q).sum()
    acc = r.accept.mean()
    assert abs(acc - alpha) < 5 * math.sqrt(alpha * (1 - alpha) / n)
    assert (r.accepted_len == r.accept).all()  # window of one row
    assert ((r.resampled_token >= 0) == (r.accept == 0)).all()
    emitted = np.where(r.accept == 1, x, r.resampled_token)
    counts = np.bincount(emitted, minlength=v)
    chi2, pval = scipy.stats.chisquare(counts, q * n)
    assert pval > 1e-4, (chi2, pval)
    # a wrong residual (e.g. p - q instead of q - p) or a non-strict test shifts mass visibly:
    wrong = np.maximum(p - q, 0)
    assert np.abs(wrong / wrong.sum() - np.maximum(q - p, 0) / np.maximum(q - p, 0).sum()).max() > 0.05
    np.testing.assert_allclose(r.p_draft_tok, p[x], rtol=1e-12)
    np.testing.assert_allclose(r.p_target_tok, q[x], rtol=1e-12)


def test_accept_rule_is_strict_and_handles_zero_mass():
    c = np.array([[0.0, 0.0, -np.inf, 0.0]], np.float32).repeat(4, 0)
    t = np.array([[0.0, 0.0, 0.0, -np.inf]], np.float32).repeat(4, 0)
    tok = np.array([0, 2, 3, 1], np.int32)
    ua = np.array([0.999, 0.5, 0.0, 0.0], np.float32)
    r = oracle.verify(c, t, tok, None, ua, np.zeros(4, np.float32), window=1, mode=oracle.VERIFY_ALL)
    # row 0: p = q = 1/3 -> u*p < q holds for every u < 1
    # row 1: p_x = 0 < q_x -> accept;  row 2: q_x = 0 -> 0 < 0 is false -> reject even with u = 0
    assert r.accept.tolist() == [1, 1, 0, 1]
    # residual of row 2: q - p > 0 only at code 2 (q = 1/3, p = 0)
    assert r.resampled_token[2] == 2
    assert r.residual_mass[2] == pytest.approx(1.0 / 3.0, rel=1e-12)


def test_residual_mass_is_total_variation_and_cdf_endpoints():
    rng = np.random.default_rng(7)
    v, rows = 64, 32
    c = rng.normal(0, 2, (rows, v)).astype(np.float32)
    t = (c + rng.normal(0, 1, (rows, v))).astype(np.float32)
    p, q = _softmax(c), _softmax(t)
    # force a rejection on every row: pick the token with the smallest q/p and u close to 1
    tok = np.argmin(q / p, axis=1).astype(np.int32)
    ua = np.full(rows, 1 - 2.0 ** -24, np.float32)
    res = np.maximum(q - p, 0)
    tv = 0.5 * np.abs(p - q).sum(1)
    for u_val, pick in ((0.0, "first"), (1 - 2.0 ** -24, "last")):
        ur = np.full(rows, u_val, np.float32)
        r = oracle.verify(c, t, tok, None, ua, ur, window=1, mode=oracle.VERIFY_ALL)
        assert (r.accept == 0).all()
        np.testing.assert_allclose(r.residual_mass, tv, rtol=1e-11)
        pos = res > 0
        expect = pos.argmax(1) if pick == "first" else v - 1 - pos[:, ::-1].argmax(1)
        assert (r.resampled_token == expect).all()
    # generic u: brute-force inverse CDF with a library cumulative sum
    ur = rng.random(rows, dtype=np.float32)
    r = oracle.verify(c, t, tok, None, ua, ur, window=1, mode=oracle.VERIFY_ALL)
    cum = np.cumsum(res, axis=1)
    expect = (cum > (ur.astype(np.float64) * cum[:, -1])[:, None]).argmax(1)
    assert (r.resampled_token == expect).all()


def _brute_window(flags, accept_bits, mode):
    w = len(flags)
    f = next((j for j in range(w) if flags[j]), w) if mode != oracle.VERIFY_ALL else 0
    a = w
    for j in range(w):
        tested = mode == oracle.VERIFY_ALL or (mode == oracle.VERIFY_ANCHORED and j >= f) or \
            (mode == oracle.VERIFY_PER_TOKEN and flags[j])
        if tested and not accept_bits[j]:
            a = j
            break
    return f, a


@pytest.mark.parametrize("mode", [oracle.VERIFY_ANCHORED, oracle.VERIFY_PER_TOKEN, oracle.VERIFY_ALL])
def test_window_bookkeeping_brute_force(mode):
    rng = np.random.default_rng(11 + mode)
    v, w, nw = 16, 4, 200
    rows = w * nw
    c = rng.normal(0, 1.5, (rows, v)).astype(np.float32)
    t = (c + rng.normal(0, 1.0, (rows, v))).astype(np.float32)
    p, q = _softmax(c), _softmax(t)
    tok = np.array([rng.choice(v, p=p[i]) for i in range(rows)], np.int32)
    flags = (rng.random(rows) < 0.3).astype(np.uint8)
    ua, ur = rng.random(rows, dtype=np.float32), rng.random(rows, dtype=np.float32)
    r = oracle.verify(c, t, tok, flags, ua, ur, window=w, mode=mode)
    idx = np.arange(rows)
    would_accept = ua.astype(np.float64) * p[idx, tok] < q[idx, tok]
    seen = set()
    for k in range(nw):
        sl = slice(k * w, (k + 1) * w)
        f, a = _brute_window(flags[sl], would_accept[sl], mode)
        seen.add((f, a))
        assert r.first_flag[k] == f and r.accepted_len[k] == a
        assert r.cloud_call[k] == (f < w)
        assert (r.resampled_token[k] >= 0) == (a < w)
        for j in range(w):
            tested = mode == oracle.VERIFY_ALL or (mode == oracle.VERIFY_ANCHORED and j >= f) or \
                (mode == oracle.VERIFY_PER_TOKEN and flags[k * w + j])
            assert r.accept[k * w + j] == (would_accept[k * w + j] if tested else 1)
        if a < w:  # the resample uses row a and ITS uniform
            res = np.maximum(q[k * w + a] - p[k * w + a], 0)
            cum = np.cumsum(res)
            assert r.resampled_token[k] == int((cum > float(ur[k * w + a]) * cum[-1]).argmax())
    assert len(seen) >= (5 if mode == oracle.VERIFY_ALL else 8)  # the cases really vary


def test_expected_accepted_length_iid_rows():
    """Rows tested independently with acceptance probability alpha: E[a] = alpha (1 - alpha^W) / (1 - alpha)."""
    rng = np.random.default_rng(21)
    v, w, nw = 6, 8, 40_000
    c = rng.normal(0, 1, v).astype(np.float32)
    t = (c + rng.normal(0, 0.8, v)).astype(np.float32)
    p, q = _softmax(c), _softmax(t)
    alpha = np.minimum(p, q).sum()
    rows = w * nw
    draft, target = np.broadcast_to(c, (rows, v)).copy(), np.broadcast_to(t, (rows, v)).copy()
    tok = _sample_tokens(p, rows, rng)
    r = oracle.verify(draft, target, tok, None, rng.random(rows, dtype=np.float32),
                      rng.random(rows, dtype=np.float32), window=w, mode=oracle.VERIFY_ALL)
    expect = alpha * (1 - alpha ** w) / (1 - alpha)
    a = r.accepted_len.astype(np.float64)
    assert abs(a.mean() - expect) < 5 * a.std() / math.sqrt(nw)


@pytest.mark.parametrize("sigma,expect", [(0.5, 0.8026), (0.3, 0.8808)])
def test_flat_rows_acceptance_tends_to_two_phi(sigma, expect):
    """Flat rows with target = draft + N(0, sigma^2) over a large vocabulary accept with probability
    2 * Phi(-sigma / 2); this pins the input generator and the oracle together."""
    assert 2 * scipy.stats.norm.cdf(-sigma / 2) == pytest.approx(expect, abs=5e-5)
    wl = synth.Workload("flat", 4, 16, 16, 4096, "f32", 8, sigma, seed=9, boundary_frac=1.0)
    inp = synth.make_inputs(wl)
    assert bool(inp.boundary.all())
    r = oracle.verify(inp.draft, inp.target, inp.tokens, None, inp.u_accept, inp.u_resample,
                      window=wl.window, mode=oracle.VERIFY_ALL)
    n = wl.rows
    assert abs(r.accept.mean() - expect) < 4 * math.sqrt(expect * (1 - expect) / n) + 0.004
    p, q = _softmax(inp.draft.numpy()), _softmax(inp.target.numpy())
    assert np.minimum(p, q).sum(1).mean() == pytest.approx(expect, abs=0.004)


def test_bad_token_and_invalid_arguments():
    c = np.zeros((2, 8), np.float32)
    r = oracle.verify(c, c, np.array([9, -1], np.int32), None, np.zeros(2, np.float32), np.zeros(2, np.float32),
                      window=1, mode=oracle.VERIFY_ALL)
    assert (r.row_status & oracle.ROW_BAD_TOKEN).all() and (r.accept == 0).all()
    with pytest.raises(ValueError):
        oracle.verify(c, c, np.zeros(2, np.int32), None, np.zeros(2, np.float32), np.zeros(2, np.float32), window=3)
    with pytest.raises(ValueError):  # flags are required unless every row is tested
        oracle.verify(c, c, np.zeros(2, np.int32), None, np.zeros(2, np.float32), np.zeros(2, np.float32),
                      window=1, mode=oracle.VERIFY_ANCHORED)


def _decode_workload():
    return synth.Workload("dec", 6, 5, 8, 512, "bf16", 8, 0.5, seed=13, decode=True)


def test_decode_loop_replays_verify_and_conserves_tokens():
    wl = _decode_workload()
    inp = synth.make_inputs(wl)
    seq = wl.tokens_per_image
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=inp.radius_row, tau=2e-3)
    q = oracle.quantify(inp.draft, prm)
    assert 0.05 < q.flag.mean() < 0.95
    st = oracle.DecodeState(wl.images, seq)
    steps = 0
    draft, target = inp.draft.view(torch.int16).numpy().view(np.uint16), inp.target.view(torch.int16).numpy().view(np.uint16)
    tok, ua, ur = inp.tokens.numpy(), inp.u_accept.numpy(), inp.u_resample.numpy()
    while (st.pos < seq).any():
        before = st.pos.copy()
        emitted_before = (st.tokens_out >= 0).sum(1)
        oracle.decode_step(st, inp.draft, inp.target, inp.tokens, inp.u_accept, inp.u_resample, prm, wl.window)
        steps += 1
        for rq in range(wl.images):
            p0 = int(before[rq])
            if p0 >= seq:
                assert st.pos[rq] == p0
                continue
            wlen = min(wl.window, seq - p0)
            r0 = rq * seq + p0
            sl = slice(r0, r0 + wlen)
            # replay: the same window through orc_verify (window length = the cut window)
            r = oracle.verify(draft[sl], target[sl], tok[sl], q.flag[sl], ua[sl], ur[sl], window=wlen)
            a = int(r.accepted_len[0])
            adv = a + (1 if a < wlen else 0)
            assert st.pos[rq] == p0 + adv
            assert (st.tokens_out[rq, p0:p0 + a] == tok[r0:r0 + a]).all()
            if a < wlen:
                assert st.tokens_out[rq, p0 + a] == r.resampled_token[0]
            assert (st.tokens_out[rq] >= 0).sum() == emitted_before[rq] + adv
        assert steps <= seq
    assert (st.pos == seq).all()
    assert (st.tokens_out >= 0).all()  # every request emitted exactly seq_len tokens
    assert steps >= math.ceil(seq / wl.window)
    cnt = st.counters
    assert cnt[4] + cnt[5] == wl.images * seq  # kept drafts + resampled tokens
    assert cnt[7] == wl.images
    assert cnt[1] <= cnt[0] and cnt[2] <= cnt[6]
