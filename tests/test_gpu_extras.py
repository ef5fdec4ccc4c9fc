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
    c = (torch.randint(-8, 8, (64, 4100), generator=g).float() * 0.25)
    c[3, ::2] = -0.0
    c[3, 1::2] = 0.0
    c[4, 100:3000] = float("-inf")
    c[5, :] = 1.5
    for dtype in (torch.float32, torch.bfloat16):
        cc = c.to(dtype)
        for k in (1, 7, 333, 2048, 4100):
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
