"""Element-by-element comparison of the CUDA path (through the C ABI binding) with the CPU oracle
on the same input bytes.  Used by the GPU tests and by the smoke check.

Bar: integer / byte results (flags, accept bits, accepted lengths, token ids, arg-max, status)
bit-exact, except rows whose oracle decision margin is below 1e-6 (relative), which are counted
and reported separately; floating-point results within 1e-5 relative or 1e-7 absolute.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np
import torch

import oracle
from paper_2603_25463_b200 import ciar

RTOL, ATOL = 1e-5, 1e-7
NEAR_TIE = 1e-6

Q_FLOAT_FIELDS = ("row_max", "sum_exp", "lse", "p_max", "entropy", "S_lo", "S_up", "omega", "sigma", "score")


@dataclass
class Report:
    rows: int = 0
    windows: int = 0
    near_tie_flags: int = 0
    near_tie_accepts: int = 0
    near_tie_resamples: int = 0
    excluded_windows: int = 0
    max_rel_err: dict = field(default_factory=dict)

    def merge(self, other: "Report") -> "Report":
        for k in ("rows", "windows", "near_tie_flags", "near_tie_accepts", "near_tie_resamples", "excluded_windows"):
            setattr(self, k, getattr(self, k) + getattr(other, k))
        for k, v in other.max_rel_err.items():
            self.max_rel_err[k] = max(v, self.max_rel_err.get(k, 0.0))
        return self


def assert_close(name, got, want, rep: Optional[Report] = None, rtol=RTOL, atol=ATOL):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    assert got.shape == want.shape, (name, got.shape, want.shape)
    both_nan = np.isnan(got) & np.isnan(want)
    err = np.abs(got - want)
    tol = atol + rtol * np.abs(want)
    bad = ~both_nan & ~(err <= tol)
    if rep is not None and want.size:
        with np.errstate(divide="ignore", invalid="ignore"):
            rel = np.where(both_nan | (err <= atol), 0.0, err / np.maximum(np.abs(want), 1e-300))
        rep.max_rel_err[name] = max(float(np.nanmax(rel)) if rel.size else 0.0, rep.max_rel_err.get(name, 0.0))
    if bad.any():
        i = np.flatnonzero(bad.ravel())[0]
        raise AssertionError("%s: %d of %d outside tolerance; first at %d: got %.9g want %.9g" %
                             (name, bad.sum(), bad.size, i, got.ravel()[i], want.ravel()[i]))


GUARD = 64  # canary elements on either side of every output array


class Guarded:
    """Puts every tensor of an output object (QuantifyOut, VerifyOut) between two runs of a byte pattern inside a larger
    buffer; check() says whether a kernel wrote outside any of them."""

    def __init__(self, out):
        self.out, self.bufs = out, []
        for name, t in list(vars(out).items()):
            if not isinstance(t, torch.Tensor):
                continue
            n = t.numel()
            buf = torch.empty(n + 2 * GUARD, dtype=t.dtype, device=t.device)
            buf.view(torch.uint8).fill_(0xA5)
            setattr(out, name, buf[GUARD:GUARD + n].view(t.shape))
            self.bufs.append((name, buf, n))

    def check(self):
        for name, buf, n in self.bufs:
            edge = torch.cat([buf[:GUARD], buf[GUARD + n:]]).view(torch.uint8)
            assert bool((edge == 0xA5).all()), "a kernel wrote outside the output array %s" % name


def to_ciar_params(p: oracle.IntervalParams, device) -> ciar.IntervalParams:
    def dev(x, dtype=None):
        if x is None:
            return None
        t = x if isinstance(x, torch.Tensor) else torch.as_tensor(np.asarray(x))
        if dtype is not None:
            t = t.to(dtype)
        return t.to(device).contiguous()
    radius = None
    if p.radius_mode == oracle.RADIUS_PER_ROW:
        radius = dev(p.radius, torch.float32)
    elif p.radius_mode == oracle.RADIUS_PER_CODE:
        radius = dev(p.radius)
    return ciar.IntervalParams(p.radius_mode, radius, p.radius_is_raw, p.r_scalar, p.r_max, p.lo_cap, p.hi_cap,
                               p.policy, p.tau, dev(p.u_flag, torch.float32))


def check_quantify(logits_cpu: torch.Tensor, params: oracle.IntervalParams, valid_begin=0, valid_count=None,
                   dense=False, device="cuda", logits_dev: Optional[torch.Tensor] = None, threads=0,
                   radius_dev: Optional[torch.Tensor] = None):
    """Runs both sides on the same rows; returns (oracle result, gpu QuantifyOut, Report).
    logits_dev / radius_dev: device tensors to use instead of copies of the CPU ones (strided views)."""
    rows, vocab = logits_cpu.shape
    n = vocab - valid_begin if valid_count is None else valid_count
    ref = oracle.quantify(logits_cpu, params, valid_begin, n, dense=dense, threads=threads)
    ld = logits_cpu.to(device) if logits_dev is None else logits_dev
    out = ciar.QuantifyOut.allocate(rows, device, dense_width=n if dense else 0)
    guard = Guarded(out)
    gp = to_ciar_params(params, device)
    if radius_dev is not None:
        gp.radius = radius_dev
    ciar.quantify(ld, gp, out, valid_begin, n)
    torch.cuda.synchronize()
    guard.check()
    rep = Report(rows=rows)
    for name in Q_FLOAT_FIELDS:
        assert_close(name, getattr(out, name).cpu().numpy(), getattr(ref, name), rep)
    assert np.array_equal(out.row_status.cpu().numpy(), ref.row_status), "row_status"
    assert np.array_equal(out.argmax.cpu().numpy(), ref.argmax), "argmax"
    gflag = out.flag.cpu().numpy()
    near = ref.margin < NEAR_TIE
    rep.near_tie_flags = int(near.sum())
    mism = gflag != ref.flag
    assert not (mism & ~near).any(), "flag differs on %d rows away from the threshold" % int((mism & ~near).sum())
    if dense:
        assert_close("dense_p", out.dense_p.cpu().numpy(), ref.p, rep)
        assert_close("dense_lo", out.dense_lo.cpu().numpy(), ref.p_lo, rep)
        assert_close("dense_up", out.dense_up.cpu().numpy(), ref.p_up, rep)
    return ref, out, rep


def check_verify(draft_cpu, target_cpu, tokens, flag, u_accept, u_resample, window, mode,
                 valid_begin=0, valid_count=None, device="cuda", draft_stats=None,
                 draft_dev=None, target_dev=None, threads=0):
    """flag: numpy uint8 (or None in mode ALL), fed to both sides.  draft_stats: optional
    (row_max, sum_exp) CUDA tensors from ciar.quantify; None makes the library recompute them."""
    rows, vocab = draft_cpu.shape
    n = vocab - valid_begin if valid_count is None else valid_count
    ref = oracle.verify(draft_cpu, target_cpu, tokens, flag, u_accept, u_resample, window, mode, valid_begin, n,
                        threads=threads)
    dd = draft_cpu.to(device) if draft_dev is None else draft_dev
    td = target_cpu.to(device) if target_dev is None else target_dev
    as_dev = lambda x, dt: None if x is None else torch.as_tensor(np.asarray(x.cpu() if isinstance(x, torch.Tensor) else x)).to(dt).to(device)
    out = ciar.VerifyOut.allocate(rows, window, device)
    guard = Guarded(out)
    ws = ciar.alloc_workspace(rows, window, device)
    rm, se = draft_stats if draft_stats is not None else (None, None)
    ciar.verify(dd, td, as_dev(tokens, torch.int32), as_dev(flag, torch.uint8), rm, se,
                as_dev(u_accept, torch.float32), as_dev(u_resample, torch.float32), window, mode, out, ws,
                valid_begin, n)
    torch.cuda.synchronize()
    guard.check()
    rep = Report(rows=rows, windows=rows // window)
    assert np.array_equal(out.row_status.cpu().numpy(), ref.row_status), "verify row_status"
    assert np.array_equal(out.first_flag.cpu().numpy(), ref.first_flag), "first_flag"
    assert np.array_equal(out.cloud_call.cpu().numpy(), ref.cloud_call), "cloud_call"
    assert_close("p_draft_tok", out.p_draft_tok.cpu().numpy(), ref.p_draft_tok, rep)
    assert_close("p_target_tok", out.p_target_tok.cpu().numpy(), ref.p_target_tok, rep)
    near_acc = ref.accept_margin < NEAR_TIE
    rep.near_tie_accepts = int(near_acc.sum())
    gacc = out.accept.cpu().numpy()
    # a near-tie row may flip, and then every later row of its window is tested or not accordingly:
    # compare accept bits only in windows without a near-tie row
    win_near = near_acc.reshape(-1, window).any(1)
    near_res = ref.resample_margin < NEAR_TIE
    rep.near_tie_resamples = int(near_res.sum())
    ok_rows = np.repeat(~win_near, window)
    assert np.array_equal(gacc[ok_rows], ref.accept[ok_rows]), "accept bits"
    assert np.array_equal(out.accepted_len.cpu().numpy()[~win_near], ref.accepted_len[~win_near]), "accepted_len"
    ok_win = ~win_near & ~near_res
    rep.excluded_windows = int((~ok_win).sum())
    got_tok, want_tok = out.resampled_token.cpu().numpy(), ref.resampled_token
    bad = (got_tok != want_tok) & ok_win
    assert not bad.any(), "resampled_token differs in %d windows (first %d: got %d want %d, margin %.3g)" % (
        bad.sum(), np.flatnonzero(bad)[0], got_tok[np.flatnonzero(bad)[0]], want_tok[np.flatnonzero(bad)[0]],
        ref.resample_margin[np.flatnonzero(bad)[0]])
    return ref, out, rep
