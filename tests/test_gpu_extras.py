"""GPU parity of the entry points beyond the quantify / verify / decode path -- the discrete top-k quantifier,
the score variants, soft and hard voting over several Inter-Heads, the Inter-DRO forward value -- against the
CPU oracle on the same seeded inputs, through the C ABI.  Bar: sets, counts, flags and status bit-exact (flags
except rows whose oracle margin is below 1e-6); floating point within 1e-5 relative or 1e-7 absolute."""
import numpy as np
import pytest
import torch

import oracle
import parity_util as pu
from paper_2603_25463_b200 import ciar, synth

pytestmark = pytest.mark.gpu

T_FLOAT = ("mass", "entropy", "S_lo", "S_up", "omega", "sigma", "score")


def _check_topk(logits_cpu, k, prm, valid_begin=0, valid_count=None, indices=True, logits_dev=None):
    rows, vocab = logits_cpu.shape
    n = vocab - valid_begin if valid_count is None else valid_count
    ref = oracle.topk(logits_cpu, k, prm, valid_begin, n, indices=indices)
    out = ciar.TopkOut.allocate(rows, "cuda", k if indices else 0)
    guard = pu.Guarded(out)
    ld = logits_cpu.cuda() if logits_dev is None else logits_dev
    ciar.quantify_topk(ld, k, pu.to_ciar_params(prm, "cuda"), out, valid_begin, n)
    torch.cuda.synchronize()
    guard.check()
    rep = pu.Report(rows=rows)
    assert np.array_equal(out.row_status.cpu().numpy(), ref.row_status), "row_status"
    assert np.array_equal(out.n_above.cpu().numpy(), ref.n_above), "n_above"
    assert np.array_equal(out.kth_logit.cpu().numpy().astype(np.float64), ref.kth_logit, equal_nan=True), "kth_logit"
    if indices:
        assert np.array_equal(out.indices.cpu().numpy(), ref.indices), "the selected set differs"
    for name in T_FLOAT:
        pu.assert_close(name, getattr(out, name).cpu().numpy(), getattr(ref, name), rep)
    near = ref.margin < pu.NEAR_TIE
    mism = out.flag.cpu().numpy() != ref.flag
    assert not (mism & ~near).any(), "flag differs away from the threshold"
    rep.near_tie_flags = int(near.sum())
    return ref, out, rep


def _per_row(rows, seed, lo=0.05, hi=1.5):
    g = torch.Generator().manual_seed(seed)
    return (lo + (hi - lo) * torch.rand(rows, generator=g)).float()


@pytest.mark.parametrize("v,k", [(64, 1), (64, 10), (64, 64), (1000, 100), (1000, 400), (1000, 999)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_topk_small_rows(v, k, dtype):
    g = torch.Generator().manual_seed(v * 7 + k)
    c = (3.0 * torch.randn(37, v, generator=g)).to(dtype)
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=_per_row(37, k), tau=1e-3)
    _check_topk(c, k, prm)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("k", [100, 400])
def test_topk_codebook_rows(dtype, k):
    # the workload's own rows (blob-field scales: near one-hot interiors and flat boundaries), more rows than CTAs
    wl = synth.WORKLOADS["llamagen384"].scaled(images=3)
    inp = synth.make_inputs(wl)
    c = inp.draft.to(dtype)
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=inp.radius_row, tau=wl.tau)
    ref, out, rep = _check_topk(c, k, prm)
    assert c.shape[0] > 3 * 148 and c.shape[1] == 16384
    print("topk k=%d %s: near-tie flags %d of %d, max rel err %s" % (k, dtype, rep.near_tie_flags, rep.rows, rep.max_rel_err))


def test_topk_ties_and_slices():
    # a coarse grid of values (many equal logits, the quota of ties runs out inside a warp's stretch), -0 / +0,
    # -inf stretches, and an unaligned slice inside wider rows
    g = torch.Generator().manual_seed(11)
    c = (torch.randint(-8, 8, (64, 4104), generator=g).float() * 0.25)
    c[3, ::2] = -0.0
    c[3, 1::2] = 0.0
    c[4, 100:3000] = float("-inf")
    c[5, :] = 1.5
    for dtype in (torch.float32, torch.bfloat16):
        cc = c.to(dtype)
        for k in (1, 7, 333, 2048, 4104):
            _check_topk(cc, k, oracle.IntervalParams(r_scalar=0.4, tau=1e-4))
        _check_topk(cc, 50, oracle.IntervalParams(r_scalar=0.4, tau=1e-4), valid_begin=13, valid_count=4001)
        _check_topk(cc, 4001, oracle.IntervalParams(r_scalar=0.4, tau=1e-4), valid_begin=13, valid_count=4001)


def test_topk_wide_rows_and_unusable_rows():
    # rows too wide for the shared-memory copy (read again through L2), k = V on them, and unusable rows
    g = torch.Generator().manual_seed(12)
    c = (2.0 * torch.randn(9, 40000, generator=g)).to(torch.bfloat16)
    c[2, 77] = float("nan")
    c[6, :] = float("-inf")
    prm = oracle.IntervalParams(r_scalar=0.7, tau=1e-5)
    ref, out, _ = _check_topk(c, 400, prm)
    assert ref.row_status[2] == oracle.ROW_NAN and ref.row_status[6] == oracle.ROW_NO_FINITE
    assert (out.indices[2] == -1).all() and out.flag[2] == 1
    _check_topk(c, 40000, prm, indices=False)
    rad = _per_row(9, 5)
    rad[4] = float("nan")
    _check_topk(c.float()[:, :3000].contiguous(), 64, oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=rad, tau=1e-5))


def test_topk_argument_errors():
    c = torch.zeros(4, 64, device="cuda")
    out = ciar.TopkOut.allocate(4, "cuda", 8)
    for k in (0, 65):
        with pytest.raises(ciar.CiarError):
            ciar.quantify_topk(c, k, ciar.IntervalParams(r_scalar=0.1), out)
    with pytest.raises(ciar.CiarError):
        ciar.quantify_topk(c, 8, ciar.IntervalParams(radius_mode=ciar.RADIUS_PER_CODE, radius=c), out)


# ---------------------------------------------------------------- score variants and several heads
def test_rescore_variants():
    wl = synth.WORKLOADS["llamagen384"].scaled(images=2)
    inp = synth.make_inputs(wl)
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=inp.radius_row, tau=wl.tau)
    ref, out, _ = pu.check_quantify(inp.draft, prm)
    n, rows = inp.draft.shape[1], inp.draft.shape[0]
    cases = [(oracle.SCORE_PRODUCT, {}, wl.tau), (oracle.SCORE_PER_N, {}, wl.tau / n),
             (oracle.SCORE_PER_OMEGA2, {}, 3e-3), (oracle.SCORE_SMOOTHED, {"eps": 1e-9}, wl.tau),
             (oracle.SCORE_ADDITIVE, {"lambda1": 1e-3, "lambda2": 2.0}, 2.5 * wl.tau)]
    for variant, kw, tau in cases:
        want, wflag, margin = oracle.score_variant(ref.omega, ref.sigma, n, variant, tau=tau, **kw)
        score = torch.empty(rows, device="cuda")
        flag = torch.empty(rows, dtype=torch.uint8, device="cuda")
        ciar.rescore(out.omega, out.sigma, n, variant, tau=tau, score_out=score, flag_out=flag, **kw)
        torch.cuda.synchronize()
        pu.assert_close("variant %d" % variant, score.cpu().numpy(), want)
        # the inputs are the quantifier's float32 omega / sigma: a decision closer to tau than their rounding is a near tie
        near = margin < 1e-5
        mism = flag.cpu().numpy() != wflag
        assert not (mism & ~near).any(), "variant %d: flag differs away from the threshold" % variant
        assert 0 < wflag.sum() < rows
    # an unusable row carries NaN through and is flagged
    om = torch.tensor([float("nan"), 0.5], device="cuda")
    sg = torch.tensor([0.1, 0.1], device="cuda")
    sc = torch.empty(2, device="cuda")
    fl = torch.empty(2, dtype=torch.uint8, device="cuda")
    ciar.rescore(om, sg, 16, ciar.SCORE_PER_N, tau=1.0, score_out=sc, flag_out=fl)
    assert torch.isnan(sc[0]) and fl.tolist() == [1, 0]
    with pytest.raises(ciar.CiarError):
        ciar.rescore(om, sg, 16, 9, score_out=sc, flag_out=fl)


E_FLOAT = ("p_max", "entropy", "S_lo", "S_up", "omega", "sigma", "score")


def _check_ensemble(heads_cpu, prm, valid_begin=0, valid_count=None, dense=False):
    n_heads, rows, vocab = heads_cpu.shape
    n = vocab - valid_begin if valid_count is None else valid_count
    ref = oracle.ensemble(heads_cpu, prm, valid_begin, n, dense=dense)
    out = ciar.QuantifyOut()
    for name in E_FLOAT:
        setattr(out, name, torch.empty(rows, device="cuda"))
    out.flag = torch.empty(rows, dtype=torch.uint8, device="cuda")
    out.row_status = torch.empty(rows, dtype=torch.uint8, device="cuda")
    if dense:
        out.dense_p = torch.empty((rows, n), device="cuda")
    guard = pu.Guarded(out)
    ciar.quantify_ensemble(heads_cpu.cuda().contiguous(), pu.to_ciar_params(prm, "cuda"), out, valid_begin, n)
    torch.cuda.synchronize()
    guard.check()
    rep = pu.Report(rows=rows)
    assert np.array_equal(out.row_status.cpu().numpy(), ref.row_status), "row_status"
    for name in E_FLOAT:
        pu.assert_close(name, getattr(out, name).cpu().numpy(), getattr(ref, name), rep)
    if dense:
        pu.assert_close("pbar", out.dense_p.cpu().numpy(), ref.pbar, rep)
    near = ref.margin < pu.NEAR_TIE
    mism = out.flag.cpu().numpy() != ref.flag
    assert not (mism & ~near).any(), "flag differs away from the threshold"
    return ref, out, rep


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("n_heads", [1, 2, 3, 5])
def test_ensemble_small_rows(dtype, n_heads):
    g = torch.Generator().manual_seed(40 + n_heads)
    rows, v = 29, 1000
    base = 3.0 * torch.randn(rows, v, generator=g)
    heads = torch.stack([base + 0.3 * torch.randn(rows, v, generator=g) for _ in range(n_heads)]).to(dtype)
    heads[:, 3, :] *= 6.0  # a dominant code in every head
    rad = torch.stack([_per_row(rows, 50 + h) for h in range(n_heads)])
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=rad, tau=2e-4)
    _check_ensemble(heads, prm, dense=True)
    _check_ensemble(heads, oracle.IntervalParams(r_scalar=-0.3, radius_is_raw=True, tau=2e-4), valid_begin=5, valid_count=900)


def test_ensemble_codebook_rows_and_degenerate_rows():
    wl = synth.WORKLOADS["llamagen384"].scaled(images=2)
    inp = synth.make_inputs(wl)
    g = torch.Generator().manual_seed(7)
    c = inp.draft.float()
    heads = torch.stack([c, c + 0.2 * torch.randn(c.shape, generator=g), c + 0.2 * torch.randn(c.shape, generator=g)]).to(torch.bfloat16)
    heads[0, 5, :] = 0.0                    # a constant row in one head
    heads[:, 6, :] = 2.0                    # constant in every head: equal widths, Sigma = 0
    heads[1, 7, 100] = float("nan")         # unusable
    heads[:, 8, 50:9000] = float("-inf")    # a masked stretch
    rad = torch.stack([inp.radius_row, inp.radius_row * 1.5, inp.radius_row * 0.5])
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=rad, tau=wl.tau)
    ref, out, rep = _check_ensemble(heads, prm)
    assert ref.row_status[7] == oracle.ROW_NAN and out.flag[7] == 1
    assert heads.shape[1] > 148 * 7
    print("ensemble: max rel err %s" % rep.max_rel_err)


def test_vote():
    g = torch.Generator().manual_seed(3)
    for n_heads in (1, 2, 3, 5, 8):
        flags = (torch.rand(n_heads, 5000, generator=g) < 0.4).to(torch.uint8)
        want, wvotes = oracle.vote(flags.numpy())
        fo = torch.empty(5000, dtype=torch.uint8, device="cuda")
        vo = torch.empty(5000, dtype=torch.int32, device="cuda")
        ciar.vote(flags.cuda(), fo, vo)
        assert np.array_equal(fo.cpu().numpy(), want) and np.array_equal(vo.cpu().numpy(), wvotes)


# ---------------------------------------------------------------- Inter-DRO forward value
def _check_interdro(c, rho, t, valid_begin=0, valid_count=None, **kw):
    rows = c.shape[0]
    ref = oracle.interdro(c, rho, t, valid_begin=valid_begin, valid_count=valid_count, **kw)
    out = ciar.InterDroOut.allocate(rows, "cuda")
    guard = pu.Guarded(out)
    ws = torch.empty(ciar.interdro_workspace_bytes(rows), dtype=torch.uint8, device="cuda")
    ciar.interdro_forward(c.cuda(), rho.cuda(), t.cuda(), out, ws, valid_begin=valid_begin, valid_count=valid_count, **kw)
    torch.cuda.synchronize()
    guard.check()
    rep = pu.Report(rows=rows)
    pu.assert_close("l1", out.l1.cpu().numpy(), ref.l1, rep)
    pu.assert_close("ce", out.ce.cpu().numpy(), ref.ce, rep)
    pu.assert_close("kl", out.kl.cpu().numpy(), ref.kl, rep)
    pu.assert_close("weights", out.weights.cpu().numpy(), ref.weights, rep)
    pu.assert_close("loss", out.loss.cpu().numpy(), ref.loss, rep)
    return ref, out, rep


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_interdro_small_rows(dtype):
    g = torch.Generator().manual_seed(21)
    rows, v = 45, 1000
    c = (3.0 * torch.randn(rows, v, generator=g)).to(dtype)
    rho = (torch.randn(rows, v, generator=g) - 1.0).to(dtype)
    t = (c.float() + 0.5 * torch.randn(rows, v, generator=g)).to(dtype)
    _check_interdro(c, rho, t, radius_is_raw=True, lambda_v=0.7, lambda_p=1.3, lambda_beta=0.4, alpha=0.5)
    _check_interdro(c, rho.abs(), t, radius_is_raw=False, r_max=0.8, alpha=0.0)
    _check_interdro(c, rho, t, valid_begin=3, valid_count=990, alpha=0.25)


def test_interdro_codebook_rows():
    # the bench batch's rows with one raw radius per code, more rows than CTAs; the stage holds the three tensors
    wl = synth.WORKLOADS["llamagen384"].scaled(images=2)
    inp = synth.make_inputs(wl, per_code_radius=True)
    ref, out, rep = _check_interdro(inp.draft, inp.radius_code, inp.target, radius_is_raw=True, alpha=0.1)
    assert inp.draft.shape[0] > 148 * 2 * 3
    print("interdro: loss %s, max rel err %s" % (ref.loss, rep.max_rel_err))
    # a masked stretch and rows wider than the stage (read again through L2)
    g = torch.Generator().manual_seed(22)
    c = (2.0 * torch.randn(6, 20000, generator=g)).to(torch.bfloat16)
    t = (c.float() + 0.3 * torch.randn(6, 20000, generator=g)).to(torch.bfloat16)
    rho = (0.5 * torch.randn(6, 20000, generator=g)).to(torch.bfloat16)
    c[1, 300:15000] = float("-inf")
    t[1, 300:15000] = float("-inf")
    _check_interdro(c, rho, t, alpha=0.3)


def test_interdro_argument_errors():
    c = torch.zeros(4, 64, device="cuda")
    out = ciar.InterDroOut.allocate(4, "cuda")
    small = torch.empty(8, dtype=torch.uint8, device="cuda")
    with pytest.raises(ciar.CiarError):
        ciar.interdro_forward(c, c, c, out, small)
    with pytest.raises(ciar.CiarError):
        ciar.interdro_forward(c[:0], c[:0], c[:0], out, torch.empty(256, dtype=torch.uint8, device="cuda"))
