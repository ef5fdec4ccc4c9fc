"""GPU parity: the CUDA path, called through the C ABI binding, against the CPU oracle on the
same seeded input bytes.  Integer results bit-exact (near-tie rows reported separately), floating
point within 1e-5 relative / 1e-7 absolute."""
import numpy as np
import pytest
import torch

import oracle
import parity_util as pu
from paper_2603_25463_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ciar(ciar_lib):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    return ciar_lib


def _logits(rows, v, dtype, scale=3.0, seed=0):
    g = torch.Generator().manual_seed(seed)
    return (scale * torch.randn(rows, v, generator=g)).to(dtype)


def _row_params(rows, seed=0, tau=None, **kw):
    g = torch.Generator().manual_seed(seed + 77)
    r = torch.rand(rows, generator=g) * 1.5
    return oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=r, tau=1e-4 if tau is None else tau, **kw)


# ---------------------------------------------------------------- quantify

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("v", [1, 2, 3, 7, 32, 33, 64, 1000, 2048, 16384])
def test_quantify_small_shapes_dense(ciar, v, dtype):
    rows = 24
    stride = (v + 7) // 8 * 8
    full = torch.full((rows, stride), float("nan"), dtype=dtype)
    full[:, :v] = _logits(rows, v, dtype, seed=v)
    logits = full[:, :v]  # row stride > vocab, padding holds NaN that must never be read
    prm = _row_params(rows, seed=v)
    dev = full.cuda()[:, :v]
    ref, out, rep = pu.check_quantify(logits.contiguous(), prm, dense=True, logits_dev=dev)
    assert rep.near_tie_flags <= 1


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("vb,n", [(0, 77), (3, 77), (5, 8), (8, 1), (13, 999), (1, 1030)])
def test_quantify_unaligned_valid_slice(ciar, vb, n, dtype):
    rows, vocab = 9, 1040
    logits = _logits(rows, vocab, dtype, seed=vb + n)
    logits[:, :vb] = float("nan")  # outside the slice: never read
    logits[:, vb + n:] = float("inf")
    pu.check_quantify(logits, _row_params(rows, seed=n), valid_begin=vb, valid_count=n, dense=True)


@pytest.mark.parametrize("mode", ["scalar", "scalar_raw", "per_code", "per_code_raw"])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_quantify_radius_modes(ciar, mode, dtype):
    rows, v = 16, 1500 if dtype == torch.float32 else 1504
    logits = _logits(rows, v, dtype, scale=4.0, seed=3)
    g = torch.Generator().manual_seed(5)
    if mode == "scalar":
        prm = oracle.IntervalParams(r_scalar=0.35, tau=1e-3)
    elif mode == "scalar_raw":
        prm = oracle.IntervalParams(r_scalar=-0.7, radius_is_raw=True, tau=1e-3)
    elif mode == "per_code":
        prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_CODE, radius=(torch.rand(rows, v, generator=g) * 2).to(dtype),
                                    tau=1e-3)
    else:
        prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_CODE, radius_is_raw=True, r_max=1.5,
                                    radius=torch.randn(rows, v, generator=g).to(dtype), tau=1e-3)
    pu.check_quantify(logits, prm, dense=True)


@pytest.mark.parametrize("raw", [False, True])
@pytest.mark.parametrize("dtype,v", [(torch.bfloat16, 2048), (torch.bfloat16, 5000), (torch.bfloat16, 16384),
                                     (torch.float32, 2052), (torch.float32, 8192)])
def test_quantify_per_code_radius_streaming_rows(ciar, dtype, v, raw):
    """Rows of 2048 codes and more with one radius per code (logits and radii streamed together): ordinary
    rows of several sharpnesses, more rows than a CTA parks, a constant row with constant radii (Sigma = 0),
    nearly uniform widths, ties of the maximum, -inf stretches, a near one-hot row, unusable rows, radii from
    tiny to beyond the clamp, stored and raw."""
    g = torch.Generator().manual_seed(v + int(raw))
    rows = []
    for scale in (8.0, 1.0, 3.0, 0.3) * 9:  # 36 ordinary rows
        rows.append(torch.randn(v, generator=g) * scale)
    n_ord = len(rows)
    rows.append(torch.full((v,), -0.75))                        # constant row
    rows.append(torch.randn(v, generator=g) * 1e-3)             # nearly uniform widths
    ties = torch.zeros(v); ties[40:44] = 5.0; ties[v - 1] = 5.0; rows.append(ties)
    holes = torch.randn(v, generator=g); holes[100:1700] = float("-inf"); rows.append(holes)
    near = torch.full((v,), -30.0); near[v - 9] = 20.0; rows.append(near)
    nan_row = torch.randn(v, generator=g); nan_row[v - 2] = float("nan"); rows.append(nan_row)
    rows.append(torch.full((v,), float("-inf")))
    inf_row = torch.randn(v, generator=g); inf_row[9] = float("inf"); rows.append(inf_row)
    rows.append(torch.randn(v, generator=g) * 2.0)              # an ordinary row after the unusable ones
    logits = torch.stack(rows).to(dtype)
    n = logits.shape[0]
    if raw:
        radius = torch.randn(n, v, generator=g) * 1.5 - 1.0     # Softplus -> about 0.03 .. 3
        radius[1] = -12.0 + torch.randn(v, generator=g)         # tiny radii
        radius[2] = 6.0 + torch.randn(v, generator=g)           # all beyond the clamp
    else:
        radius = torch.rand(n, v, generator=g) * 2.0
        radius[1] = torch.rand(v, generator=g) * 1e-3
        radius[2] = 4.0 + torch.rand(v, generator=g)
        radius[3] = torch.rand(v, generator=g) * 0.6            # both sides of the series / exponential switch
    radius[n_ord] = 0.4                                         # constant row, constant radius
    radius[n_ord + 1] = 0.4
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_CODE, radius=radius.to(dtype), radius_is_raw=raw,
                                r_max=2.5, tau=1e-4)
    ref, out, rep = pu.check_quantify(logits, prm)
    st = out.row_status.cpu().numpy()
    assert st[n_ord + 5] == oracle.ROW_NAN and st[n_ord + 6] == oracle.ROW_NO_FINITE and st[n_ord + 7] == oracle.ROW_NAN
    assert out.argmax.cpu().numpy()[n_ord + 2] == 40
    assert rep.near_tie_flags <= 1


@pytest.mark.parametrize("raw", [False, True])
@pytest.mark.parametrize("dtype,v", [(torch.bfloat16, 4096), (torch.float32, 2048), (torch.bfloat16, 520), (torch.float32, 100)])
def test_quantify_per_code_radius_nan_marks_the_row(ciar, dtype, v, raw):
    """A NaN among a row's per-code radii makes the row unusable (status bit, flag 1, NaN scores), on the streaming
    per-code kernel's rows and on the short rows of the general kernel; the rows around it are untouched."""
    g = torch.Generator().manual_seed(v)
    rows = 40
    logits = _logits(rows, v, dtype, scale=3.0, seed=v + 1)
    radius = (torch.randn(rows, v, generator=g) - 1.0) if raw else torch.rand(rows, v, generator=g)
    for i, j in ((3, 0), (17, v - 1), (18, v // 2), (39, 7)):
        radius[i, j] = float("nan")
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_CODE, radius=radius.to(dtype), radius_is_raw=raw, tau=1e-4)
    ref, out, rep = pu.check_quantify(logits, prm)
    st = out.row_status.cpu().numpy()
    bad = np.zeros(rows, bool); bad[[3, 17, 18, 39]] = True
    assert (st[bad] == oracle.ROW_NAN).all() and (st[~bad] == 0).all()
    assert out.flag.cpu().numpy()[bad].all() and np.isnan(out.score.cpu().numpy()[bad]).all()


def test_quantify_per_code_radius_streaming_slice(ciar):
    """The same kernel on a valid slice inside wider rows with a row stride beyond the vocabulary; what lies
    outside the slice (NaN logits, NaN radii) must never be read."""
    g = torch.Generator().manual_seed(77)
    rows, vocab, stride, vb, n = 40, 8192, 8200, 1024, 4096
    full = torch.full((rows, stride), float("nan"))
    rfull = torch.full((rows, stride), float("nan"))
    full[:, vb:vb + n] = torch.randn(rows, n, generator=g) * torch.tensor([8.0, 1.0] * (rows // 2))[:, None]
    rfull[:, vb:vb + n] = torch.randn(rows, n, generator=g) - 1.0
    logits = full.to(torch.bfloat16)
    radius = rfull.to(torch.bfloat16)
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_CODE, radius=radius[:, :vocab].contiguous(),
                                radius_is_raw=True, tau=1e-4)
    dev = logits.cuda()[:, :vocab]
    rdev = radius.cuda()[:, :vocab]
    pu.check_quantify(logits[:, :vocab].contiguous(), prm, valid_begin=vb, valid_count=n, logits_dev=dev, radius_dev=rdev)


@pytest.mark.parametrize("r", [0.0, 1e-4, 0.05, 1.0, 5.0, 10.0, 40.0])
def test_quantify_radius_extremes_and_closed_forms(ciar, r):
    rows, v = 12, 4096
    logits = _logits(rows, v, torch.float32, scale=6.0, seed=11)
    ref, out, _ = pu.check_quantify(logits, oracle.IntervalParams(r_scalar=r, r_max=80.0, tau=1e-5), dense=True)
    if r == 0.0:  # delta = 0.02 p: Omega = 0.02 exactly
        np.testing.assert_allclose(out.omega.cpu().numpy(), 0.02, rtol=1e-6)


def test_quantify_degenerate_rows(ciar):
    v = 520
    g = torch.Generator().manual_seed(520)
    rows = []
    one_hot = torch.full((v,), float("-inf")); one_hot[17] = 2.5; rows.append(one_hot)
    rows.append(torch.full((v,), -0.75))  # constant row: Sigma = 0
    near = torch.full((v,), -30.0); near[100] = 20.0; rows.append(near)  # p_max = 1 - 5e-20
    two = torch.full((v,), float("-inf")); two[3] = 1.0; two[400] = 1.0; rows.append(two)
    ties = torch.zeros(v); ties[40:44] = 5.0; rows.append(ties)  # arg-max tie -> lowest index
    nan_row = torch.randn(v, generator=g); nan_row[7] = float("nan"); rows.append(nan_row)
    rows.append(torch.full((v,), float("-inf")))  # no finite code
    inf_row = torch.randn(v, generator=g); inf_row[9] = float("inf"); rows.append(inf_row)
    big = torch.randn(v, generator=g) * 1e4; rows.append(big)  # huge dynamic range
    flat_small = torch.randn(v, generator=g) * 1e-3; rows.append(flat_small)  # nearly uniform widths (low CV)
    logits = torch.stack(rows)
    for dtype in (torch.float32, torch.bfloat16):
        for r in (0.0, 0.3, 2.0):
            ref, out, _ = pu.check_quantify(logits.to(dtype), oracle.IntervalParams(r_scalar=r, tau=1e-4), dense=True)
            st = out.row_status.cpu().numpy()
            assert st[5] == oracle.ROW_NAN and st[6] == oracle.ROW_NO_FINITE and st[7] == oracle.ROW_NAN
            assert out.flag.cpu().numpy()[5:8].all()
            assert out.argmax.cpu().numpy()[4] == 40


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_quantify_streaming_rows_with_many_large_codes(ciar, dtype):
    """Rows of the streaming quantifier (>= 2048 codes) in which tens to hundreds of codes sit above
    the probability level that is treated exactly, several such rows in a row, mixed with ordinary
    ones, for radii on both sides of 1 (series and direct routes)."""
    v = 4096
    g = torch.Generator().manual_seed(123)
    rows = []
    for tops in (1, 40, 200, 600, 3, 650, 650, 33, 32, 31, 0, 256):
        row = torch.randn(v, generator=g) * 0.5 - 6.0
        idx = torch.randperm(v, generator=g)[:tops]
        row[idx] = 5.0 + 0.01 * torch.randn(tops, generator=g)
        rows.append(row)
    logits = torch.stack(rows * 3).to(dtype)  # 36 rows: more than one batch of parked rows
    n = logits.shape[0]
    radius = torch.tensor([0.05, 1.0, 0.3, 0.9, 2.5, 1.0] * (n // 6))
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=radius, tau=1e-3)
    ref, out, rep = pu.check_quantify(logits, prm)
    assert rep.near_tie_flags <= 1


def _sm_count():
    return torch.cuda.get_device_properties(0).multi_processor_count


def _edge_rows(v, g, with_many_large=True):
    """The rows that exercise every special path of the streaming quantifiers, for a row of v codes: ordinary
    rows of several sharpnesses, degenerate rows (one-hot, constant, near one-hot, two equal maxima far apart,
    ties of the maximum, a long -inf stretch, a huge dynamic range, nearly uniform rows), rows with tens to
    hundreds of codes above the exactly treated level, and unusable rows (NaN, no finite code, +inf)."""
    rows, kinds = [], []
    def add(kind, row):
        rows.append(row); kinds.append(kind)
    for scale in (8.0, 1.0, 3.0, 0.3, 0.05):
        add("ordinary", torch.randn(v, generator=g) * scale)
    one_hot = torch.full((v,), float("-inf")); one_hot[v // 3] = 2.5; add("one_hot", one_hot)
    add("constant", torch.full((v,), -0.75))
    near = torch.full((v,), -30.0); near[v - 9] = 20.0; add("near_one_hot", near)
    two = torch.full((v,), float("-inf")); two[3] = 1.0; two[v - 400] = 1.0; add("two_hot", two)
    ties = torch.zeros(v); ties[40:44] = 5.0; ties[v - 1] = 5.0; add("ties", ties)
    holes = torch.randn(v, generator=g); holes[100:v // 2 + 600] = float("-inf"); add("holes", holes)
    add("huge_range", torch.randn(v, generator=g) * 1e4)
    add("flat_small", torch.randn(v, generator=g) * 1e-3)
    add("flat_offset", 7.0 + torch.randn(v, generator=g) * 0.02)
    if with_many_large:
        for tops in (1, 40, 200, 650, 33, 31):
            row = torch.randn(v, generator=g) * 0.5 - 6.0
            row[torch.randperm(v, generator=g)[:tops]] = 5.0 + 0.01 * torch.randn(tops, generator=g)
            add("tops%d" % tops, row)
    nan_row = torch.randn(v, generator=g); nan_row[v - 2] = float("nan"); add("nan", nan_row)
    add("no_finite", torch.full((v,), float("-inf")))
    inf_row = torch.randn(v, generator=g); inf_row[9] = float("inf"); add("pos_inf", inf_row)
    return torch.stack(rows), kinds


def _tile(base, total, g):
    """`total` rows drawn from `base` in a seeded shuffled order in which every kind of row follows every other."""
    idx = torch.randint(0, base.shape[0], (total,), generator=g)
    idx[:base.shape[0]] = torch.arange(base.shape[0])
    return idx


@pytest.mark.parametrize("dtype,v", [(torch.bfloat16, 16384), (torch.bfloat16, 8192), (torch.bfloat16, 5000),
                                     (torch.bfloat16, 2048), (torch.float32, 16384), (torch.float32, 3000)])
def test_quantify_streaming_edge_rows_many_per_cta(ciar, dtype, v):
    """Every kind of special row next to every other inside one CTA's walk of the streaming quantifier: far more
    rows than the persistent grid has CTAs, in a shuffled order, with radii on both sides of the series / direct
    switch (and a NaN radius), so that the ring's stages, the slots the sweep warps fill, and the batches of the
    finishing warps are reused many times by rows of different kinds."""
    g = torch.Generator().manual_seed(v + (1 if dtype == torch.float32 else 0))
    base, kinds = _edge_rows(v, g)
    cap = _sm_count() * 2
    total = 20 * cap + 7 if v <= 8192 else 16 * cap + 7
    idx = _tile(base, total, g)
    logits = base.to(dtype)[idx].contiguous()
    assert logits.shape[0] > 16 * cap
    rad_choices = torch.tensor([0.05, 1.0, 0.3, 0.9, 2.5, 0.0, 1.0000001, 7.0])
    radius = rad_choices[torch.randint(0, len(rad_choices), (total,), generator=g)]
    radius[total // 2] = float("nan")
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=radius, tau=1e-4)
    ref, out, rep = pu.check_quantify(logits, prm)
    st = out.row_status.cpu().numpy()
    k = np.array(kinds, dtype=object)[idx.numpy()]
    ok_radius = ~np.isnan(radius.numpy())
    assert (st[(k == "nan") | (k == "pos_inf")] & oracle.ROW_NAN).all()
    assert (st[k == "no_finite"] == oracle.ROW_NO_FINITE).all()
    assert (st[(k == "ordinary") & ok_radius] == 0).all() and st[total // 2] & oracle.ROW_NAN
    assert (out.argmax.cpu().numpy()[(k == "ties") & ok_radius] == 40).all()
    print("near-tie flags: %d of %d rows" % (rep.near_tie_flags, total))
    assert rep.near_tie_flags <= 4


@pytest.mark.parametrize("raw", [False, True])
@pytest.mark.parametrize("dtype,v", [(torch.bfloat16, 2048), (torch.bfloat16, 16384), (torch.float32, 4096)])
def test_quantify_per_code_edge_rows_many_per_cta(ciar, dtype, v, raw):
    """The per-code streaming quantifier on far more rows than its grid has CTAs: special rows of every kind in a
    shuffled order, so that its parked-row batches fill and its stages are reused by rows of different kinds."""
    g = torch.Generator().manual_seed(3 * v + int(raw))
    base, kinds = _edge_rows(v, g, with_many_large=False)
    cap = _sm_count()
    total = 21 * cap + 5
    idx = _tile(base, total, g)
    logits = base.to(dtype)[idx].contiguous()
    assert logits.shape[0] > 16 * cap
    nb = 12  # a dozen radius rows, drawn like the logit rows
    if raw:
        rbase = torch.randn(nb, v, generator=g) * 1.5 - 1.0
        rbase[1] = -12.0 + torch.randn(v, generator=g)
        rbase[2] = 6.0 + torch.randn(v, generator=g)
    else:
        rbase = torch.rand(nb, v, generator=g) * 2.0
        rbase[1] = torch.rand(v, generator=g) * 1e-3
        rbase[2] = 4.0 + torch.rand(v, generator=g)
        rbase[3] = torch.rand(v, generator=g) * 0.6
    rbase[4] = 0.4
    ridx = torch.randint(0, nb, (total,), generator=g)
    ridx[idx == kinds.index("constant")] = 4  # constant row with constant radius: Sigma = 0
    radius = rbase.to(dtype)[ridx].contiguous()
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_CODE, radius=radius, radius_is_raw=raw, r_max=2.5, tau=1e-4)
    ref, out, rep = pu.check_quantify(logits, prm)
    print("near-tie flags: %d of %d rows" % (rep.near_tie_flags, total))
    assert rep.near_tie_flags <= 4


@pytest.mark.parametrize("dtype,v", [(torch.bfloat16, 16392), (torch.bfloat16, 20480), (torch.float32, 17000)])
def test_quantify_wide_edge_rows_many_per_cta(ciar, dtype, v):
    """The chunked quantifier for rows that do not fit a stage, on far more rows than its grid has CTAs."""
    g = torch.Generator().manual_seed(5 * v)
    base, kinds = _edge_rows(v, g)
    extra = []
    late = torch.randn(v, generator=g); late[v - 3] = 30.0; extra.append(late)
    rising = torch.randn(v, generator=g) + torch.linspace(0.0, 40.0, v); extra.append(rising)
    ties = torch.zeros(v); ties[[16390, 300, v - 1, 9000]] = 5.0; extra.append(ties)
    base = torch.cat([base, torch.stack(extra)])
    cap = _sm_count()
    total = 21 * cap + 3
    idx = _tile(base, total, g)
    logits = base.to(dtype)[idx].contiguous()
    assert logits.shape[0] > 16 * cap
    rad_choices = torch.tensor([0.05, 1.0, 0.3, 2.5, 0.9])
    radius = rad_choices[torch.randint(0, len(rad_choices), (total,), generator=g)]
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=radius, tau=1e-3)
    ref, out, rep = pu.check_quantify(logits, prm)
    print("near-tie flags: %d of %d rows" % (rep.near_tie_flags, total))
    assert rep.near_tie_flags <= 4


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("v", [16392, 40000, 65536 + 4096])
def test_quantify_wide_rows(ciar, v, dtype):
    """Rows wider than the on-chip kernel takes (two passes, chunk by chunk; the last chunk ragged): ordinary
    rows of several sharpnesses, many codes above the exactly treated level, the maximum early / late / tied
    across chunks, -inf stretches longer than a chunk, unusable rows; radii on both sides of 1."""
    g = torch.Generator().manual_seed(v)
    rows = []
    for scale in (8.0, 1.0, 0.01, 3.0):
        rows.append(torch.randn(v, generator=g) * scale)
    for tops in (40, 300, 650):
        row = torch.randn(v, generator=g) * 0.5 - 6.0
        row[torch.randperm(v, generator=g)[:tops]] = 5.0 + 0.01 * torch.randn(tops, generator=g)
        rows.append(row)
    early = torch.randn(v, generator=g); early[5] = 30.0; rows.append(early)
    late = torch.randn(v, generator=g); late[v - 3] = 30.0; rows.append(late)
    rising = torch.randn(v, generator=g) + torch.linspace(0.0, 40.0, v); rows.append(rising)  # the running maximum keeps moving
    ties = torch.zeros(v); ties[[16390, 300, v - 1, 9000]] = 5.0; rows.append(ties)  # arg-max tie across chunks -> lowest index
    masked = torch.full((v,), float("-inf")); masked[v - 5000:] = torch.randn(5000, generator=g) * 4.0; rows.append(masked)
    one_hot = torch.full((v,), float("-inf")); one_hot[16388] = 2.5; rows.append(one_hot)
    rows.append(torch.full((v,), -0.75))  # constant row
    nan_row = torch.randn(v, generator=g); nan_row[v - 2] = float("nan"); rows.append(nan_row)
    rows.append(torch.full((v,), float("-inf")))  # no finite code
    inf_row = torch.randn(v, generator=g); inf_row[20000 % v] = float("inf"); rows.append(inf_row)
    logits = torch.stack(rows * 2).to(dtype)  # 34 rows: more than one batch of parked rows
    n = logits.shape[0]
    radius = torch.tensor(([0.05, 1.0, 0.3, 2.5, 0.9] * n)[:n])
    prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=radius, tau=1e-3)
    ref, out, rep = pu.check_quantify(logits, prm)
    st = out.row_status.cpu().numpy()[:17]
    assert st[14] == oracle.ROW_NAN and st[15] == oracle.ROW_NO_FINITE and st[16] == oracle.ROW_NAN
    assert out.argmax.cpu().numpy()[10] == 300
    assert rep.near_tie_flags <= 1


def test_quantify_wide_rows_valid_slice(ciar):
    """A wide valid slice inside a wider row (aligned to 16 bytes), scalar radius."""
    rows, stride, vb, n = 5, 70000, 1024, 50000
    logits = _logits(rows, stride, torch.bfloat16, scale=4.0, seed=5)
    ref, out, rep = pu.check_quantify(logits, oracle.IntervalParams(r_scalar=0.4, tau=1e-4), valid_begin=vb, valid_count=n)


def test_quantify_policies(ciar):
    rows, v = 64, 1024
    logits = _logits(rows, v, torch.bfloat16, scale=2.0, seed=21)
    base = oracle.quantify(logits, oracle.IntervalParams(r_scalar=0.5))
    u = torch.rand(rows, generator=torch.Generator().manual_seed(1))
    for policy, tau in ((oracle.POLICY_INTERVAL, float(np.median(base.score))),
                        (oracle.POLICY_ENTROPY, float(np.median(base.entropy))),
                        (oracle.POLICY_MAXPROB, float(np.median(base.p_max))),
                        (oracle.POLICY_RANDOM, 0.4), (oracle.POLICY_ALL, 0.0)):
        prm = oracle.IntervalParams(r_scalar=0.5, policy=policy, tau=tau, u_flag=u)
        ref, out, rep = pu.check_quantify(logits, prm)
        assert 0 < ref.flag.sum() <= rows


def test_quantify_empty_and_optional_outputs(ciar):
    empty = torch.empty((0, 64), dtype=torch.float32, device="cuda")
    before = ciar.launch_count()
    ciar.quantify(empty, ciar.IntervalParams(r_scalar=0.1), ciar.QuantifyOut.allocate(0, "cuda"))
    assert ciar.launch_count() == before
    logits = _logits(8, 256, torch.float32).cuda()
    out = ciar.QuantifyOut(score=torch.empty(8, device="cuda"), flag=torch.empty(8, dtype=torch.uint8, device="cuda"))
    ciar.quantify(logits, ciar.IntervalParams(r_scalar=0.1, tau=1e-4), out)
    ref = oracle.quantify(logits.cpu(), oracle.IntervalParams(r_scalar=0.1, tau=1e-4))
    pu.assert_close("score", out.score.cpu().numpy(), ref.score)


def test_quantify_is_deterministic(ciar):
    logits = _logits(64, 16384, torch.bfloat16, seed=5).cuda()
    prm = ciar.IntervalParams(r_scalar=0.4, tau=1e-4)
    a = ciar.QuantifyOut.allocate(64, "cuda")
    b = ciar.QuantifyOut.allocate(64, "cuda")
    ciar.quantify(logits, prm, a)
    ciar.quantify(logits, prm, b)
    torch.cuda.synchronize()
    for name in pu.Q_FLOAT_FIELDS:
        assert torch.equal(getattr(a, name), getattr(b, name)), name


def test_quantify_bounded_wait_runs_out_without_a_fault(ciar):
    """A row whose copy is never asked for (test hook: nothing is left in flight) makes the waits for it run out after a
    millisecond: the kernel returns, the rows that CTA had not finished carry ROW_TIMEOUT (flag 1, NaN scores), every other
    row is right, and the next call on the same context works as if nothing had happened."""
    rows, v = 20 * _sm_count() + 3, 4096
    logits = _logits(rows, v, torch.bfloat16, seed=31)
    prm = oracle.IntervalParams(r_scalar=0.3, tau=1e-4)
    ref = oracle.quantify(logits, prm)
    dev = logits.cuda()
    grid = min(rows, _sm_count())
    cta, k = 5, 7
    out = ciar.QuantifyOut.allocate(rows, "cuda")
    ciar.stall_hook(cta, k, 2_000_000)
    try:
        ciar.quantify(dev, pu.to_ciar_params(prm, "cuda"), out)
        torch.cuda.synchronize()
    finally:
        ciar.stall_hook(-1, -1, 0)
    st = out.row_status.cpu().numpy()
    lost = np.flatnonzero(st & ciar.ROW_TIMEOUT)
    walk = np.arange(cta, rows, grid)  # the rows of that CTA's walk
    assert len(lost) > 0 and np.isin(lost, walk[k:]).all() and walk[k] in lost
    assert np.array_equal(lost, walk[-len(lost):])  # from some row of the walk on, every row
    assert out.flag.cpu().numpy()[lost].all() and np.isnan(out.score.cpu().numpy()[lost]).all()
    ok = np.ones(rows, bool); ok[lost] = False
    assert (st[ok] == 0).all()
    for name in pu.Q_FLOAT_FIELDS:
        pu.assert_close(name, getattr(out, name).cpu().numpy()[ok], getattr(ref, name)[ok])
    assert np.array_equal(out.flag.cpu().numpy()[ok & (ref.margin >= pu.NEAR_TIE)], ref.flag[ok & (ref.margin >= pu.NEAR_TIE)])
    pu.check_quantify(logits, prm, logits_dev=dev)  # the hook is off again: the same call is whole


def test_binding_errors_are_loud(ciar):
    logits = _logits(8, 256, torch.float32).cuda()
    with pytest.raises(ciar.CiarError) as e:
        ciar.quantify(logits.half(), ciar.IntervalParams(r_scalar=0.1), ciar.QuantifyOut.allocate(8, "cuda"))
    assert e.value.status == 2
    with pytest.raises(ciar.CiarError) as e:
        ciar.quantify(logits[:, 1:], ciar.IntervalParams(r_scalar=0.1), ciar.QuantifyOut.allocate(8, "cuda"))
    assert e.value.status == 3
    with pytest.raises(ValueError):
        ciar.quantify(logits.cpu(), ciar.IntervalParams(r_scalar=0.1), ciar.QuantifyOut.allocate(8, "cuda"))


# ---------------------------------------------------------------- verify

def _verify_case(rows, v, dtype, window, seed, sigma=0.7, scale=2.0):
    g = torch.Generator().manual_seed(seed)
    draft = (scale * torch.randn(rows, v, generator=g)).to(dtype)
    target = (draft.float() + sigma * torch.randn(rows, v, generator=g)).to(dtype)
    gum = -torch.log(-torch.log(torch.rand(rows, v, generator=g).clamp(1e-9, 1 - 1e-7)))
    tokens = torch.argmax(draft.float() + gum, dim=1).to(torch.int32)
    flag = (torch.rand(rows, generator=g) < 0.3).to(torch.uint8).numpy()
    ua = torch.rand(rows, generator=g).numpy().astype(np.float32)
    ur = torch.rand(rows, generator=g).numpy().astype(np.float32)
    return draft, target, tokens.numpy(), flag, ua, ur


@pytest.mark.parametrize("mode", [oracle.VERIFY_ANCHORED, oracle.VERIFY_PER_TOKEN, oracle.VERIFY_ALL])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("v,window", [(1, 1), (2, 2), (7, 4), (33, 8), (1000, 8), (2056, 16), (16384, 8)])
def test_verify_small_shapes(ciar, v, window, dtype, mode):
    rows = window * 12
    draft, target, tok, flag, ua, ur = _verify_case(rows, v, dtype, window, seed=v * 7 + mode)
    stride = (v + 7) // 8 * 8  # device rows padded to a 16-byte multiple; the padding is never read
    pad = lambda t: torch.cat([t, torch.full((rows, stride - v), float("nan"), dtype=dtype)], 1).cuda()[:, :v]
    ref, out, rep = pu.check_verify(draft, target, tok, flag, ua, ur, window, mode,
                                    draft_dev=pad(draft), target_dev=pad(target))
    assert rep.excluded_windows <= 2
    if v >= 33 and mode == oracle.VERIFY_ALL:
        assert (ref.resampled_token >= 0).any()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_verify_with_quantify_stats_and_slice(ciar, dtype):
    rows, vocab, vb, n, window = 64, 2080, 37, 1999, 8
    draft, target, tok, flag, ua, ur = _verify_case(rows, vocab, dtype, window, seed=99)
    draft[:, :vb] = float("nan"); target[:, :vb] = float("nan")
    draft[:, vb + n:] = 50.0; target[:, vb + n:] = 50.0
    tok = np.clip(tok, vb, vb + n - 1).astype(np.int32)
    tok[5] = 3  # a drafted code outside the valid slice has probability 0 under both models: rejected
    flag[0] = 1
    dd, td = draft.cuda(), target.cuda()
    qo = ciar.QuantifyOut.allocate(rows, "cuda")
    ciar.quantify(dd, ciar.IntervalParams(r_scalar=0.2, tau=1e-4), qo, vb, n)
    ref, out, rep = pu.check_verify(draft, target, tok, flag, ua, ur, window, oracle.VERIFY_ANCHORED, vb, n,
                                    draft_stats=(qo.row_max, qo.sum_exp), draft_dev=dd, target_dev=td)
    assert ref.accept[5] == 0 and ref.p_draft_tok[5] == 0.0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("vocab,vb,n", [(40000, 0, 40000), (70000, 1024, 50008)])
def test_verify_wide_rows(ciar, vocab, vb, n, dtype):
    """The streaming verifier on rows wider than its on-chip sweep takes (one pass, chunk by chunk, last chunk
    ragged), draft statistics from the quantifier; degenerate target rows among ordinary ones."""
    rows, window = 48, 8
    draft, target, tok, flag, ua, ur = _verify_case(rows, vocab, dtype, window, seed=vocab + 3, sigma=0.7)
    tok = np.clip(tok, vb, vb + n - 1).astype(np.int32)
    flag[0] = 1
    target[3] = draft[3]  # identical rows: always accepted
    target[9] = float("-inf")  # target without a finite code
    target[17, vb + n - 1] = float("nan")
    target[20, vb: vb + n - 4000] = float("-inf")  # the first chunks hold nothing finite
    target[26, vb + 5] = 60.0  # maximum in the first chunk
    target[27, vb + n - 2] = 60.0  # maximum in the last one
    target[30, [vb + 7, vb + 20000, vb + n - 1]] = 40.0  # equal maxima in three chunks
    dd, td = draft.cuda(), target.cuda()
    qo = ciar.QuantifyOut.allocate(rows, "cuda")
    ciar.quantify(dd, ciar.IntervalParams(r_scalar=0.2, tau=1e-4), qo, vb, n)
    for mode in (oracle.VERIFY_ANCHORED, oracle.VERIFY_ALL):
        ref, out, rep = pu.check_verify(draft, target, tok, flag, ua, ur, window, mode, vb, n,
                                        draft_stats=(qo.row_max, qo.sum_exp), draft_dev=dd, target_dev=td)
    st = out.row_status.cpu().numpy()  # of the run that tests every row
    assert st[9] & oracle.ROW_NO_FINITE and st[17] & oracle.ROW_NAN


@pytest.mark.parametrize("dtype,v,window", [(torch.bfloat16, 4096, 8), (torch.bfloat16, 16384, 16), (torch.float32, 2056, 4),
                                            (torch.bfloat16, 20480, 8)])
def test_verify_edge_rows_many_per_cta(ciar, dtype, v, window):
    """The streaming verifier (and, at 20480 codes, its chunked accept sweep) on far more tested rows than its persistent
    grid has CTAs, with degenerate target rows of every kind scattered among ordinary ones: identical rows, targets
    without a finite code, NaN and +inf targets, equal maxima far apart, one-hot targets, a -inf stretch."""
    cap = _sm_count() * 2
    rows = -(-(21 * cap) // window) * window
    draft, target, tok, flag, ua, ur = _verify_case(rows, v, dtype, window, seed=v + window, sigma=0.7)
    g = torch.Generator().manual_seed(v)
    kinds = torch.randint(0, 40, (rows,), generator=g)  # 0..6: a special target row; the rest stay ordinary
    for i in torch.nonzero(kinds < 7).flatten().tolist():
        kd = int(kinds[i])
        if kd == 0: target[i] = draft[i]
        elif kd == 1: target[i] = float("-inf")
        elif kd == 2: target[i, (i * 7) % v] = float("nan")
        elif kd == 3: target[i, (i * 5) % v] = float("inf")
        elif kd == 4: target[i, [3, v // 2, v - 1]] = 40.0
        elif kd == 5: target[i] = float("-inf"); target[i, (i * 3) % v] = 1.5
        else: target[i, 100:v - 300] = float("-inf")
    dd, td = draft.cuda(), target.cuda()
    qo = ciar.QuantifyOut.allocate(rows, "cuda")
    ciar.quantify(dd, ciar.IntervalParams(r_scalar=0.2, tau=1e-4), qo)
    for mode in (oracle.VERIFY_ALL, oracle.VERIFY_ANCHORED):
        ref, out, rep = pu.check_verify(draft, target, tok, flag, ua, ur, window, mode,
                                        draft_stats=(qo.row_max, qo.sum_exp), draft_dev=dd, target_dev=td)
        print("verify %d rows of %d codes, mode %d: near-tie accepts %d, windows left out %d" % (rows, v, mode, rep.near_tie_accepts,
                                                                                               rep.excluded_windows))
        assert rep.excluded_windows <= 4 + rep.windows // 50
    assert rows > 16 * cap and (ref.accepted_len < window).any()
    st = out.row_status.cpu().numpy()
    tested = np.repeat(ref.first_flag, window) <= np.tile(np.arange(window), rows // window)
    assert (st[tested & (kinds.numpy() == 1)] & oracle.ROW_NO_FINITE).all() and (st[tested & (kinds.numpy() == 2)] & oracle.ROW_NAN).all()


def test_verify_degenerate_rows(ciar):
    v, window = 264, 4
    draft, target, tok, flag, ua, ur = _verify_case(16, v, torch.float32, window, seed=4)
    target[1] = draft[1]  # identical rows: always accepted
    draft[2] = float("-inf"); draft[2, 5] = 0.0; target[2] = float("-inf"); target[2, 9] = 0.0; tok[2] = 5  # disjoint one-hots
    ua[2] = 0.0
    draft[6, 3] = float("nan")  # NaN draft row -> status, rejected, no token
    target[9] = float("-inf")  # target without a finite code
    tok[13] = v + 5  # token id out of range
    tok[14] = -2
    # identical distributions but the token has zero mass -> rejected with zero residual -> mode of q
    draft[12] = target[12]; draft[12, 7] = float("-inf"); target[12, 7] = float("-inf"); tok[12] = 7
    ref, out, rep = pu.check_verify(draft, target, tok, None, ua, ur, window, oracle.VERIFY_ALL)
    assert ref.accept[1] == 1 and ref.accept[2] == 0
    assert ref.resampled_token[0] >= 0
    st = out.row_status.cpu().numpy()
    assert st[6] & oracle.ROW_NAN and st[9] & oracle.ROW_NO_FINITE and st[13] & oracle.ROW_BAD_TOKEN and st[14]
    assert out.resampled_token.cpu().numpy()[3] == int(torch.argmax(target[12]))


def test_verify_endpoints_of_the_inverse_cdf(ciar):
    rows, v, window = 32, 4096, 1
    draft, target, tok, flag, ua, ur = _verify_case(rows, v, torch.bfloat16, window, seed=8, sigma=1.0)
    ua[:] = 1 - 2.0 ** -24
    p = torch.softmax(draft.double(), 1); q = torch.softmax(target.double(), 1)
    tok = torch.argmin(q / p, dim=1).to(torch.int32).numpy()  # always rejected
    for u in (0.0, 1 - 2.0 ** -24):
        ur[:] = u
        ref, out, rep = pu.check_verify(draft, target, tok, None, ua, ur, window, oracle.VERIFY_ALL)
        assert (ref.accept == 0).all()


def test_verify_errors(ciar):
    draft, target, tok, flag, ua, ur = _verify_case(16, 64, torch.float32, 8, seed=1)
    d, t = draft.cuda(), target.cuda()
    args = lambda: (torch.as_tensor(tok).cuda(), torch.as_tensor(flag).cuda(), None, None,
                    torch.as_tensor(ua).cuda(), torch.as_tensor(ur).cuda())
    out = ciar.VerifyOut.allocate(16, 8, "cuda")
    ws = ciar.alloc_workspace(16, 8, "cuda")
    with pytest.raises(ciar.CiarError) as e:
        ciar.verify(d, t, *args(), 5, ciar.VERIFY_ANCHORED, out, ws)
    assert e.value.status == 1
    with pytest.raises(ciar.CiarError) as e:
        ciar.verify(d, t, *args(), 8, ciar.VERIFY_ANCHORED, out, ws[:16])
    assert e.value.status == 4
    ciar.verify(d, t, *args(), 8, ciar.VERIFY_ANCHORED, out, ws)  # the context is still healthy
    torch.cuda.synchronize()


# ---------------------------------------------------------------- the five workloads

def _pipeline(ciar, wl, inp_cpu, inp_dev=None, per_code=False, threads=0):
    """quantify -> verify on both sides (each side uses ITS OWN flags), reports near ties."""
    dev = inp_dev if inp_dev is not None else None
    dd = inp_cpu.draft.cuda() if dev is None else dev.draft
    td = inp_cpu.target.cuda() if dev is None else dev.target
    if per_code:
        prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_CODE, radius=inp_cpu.radius_code, radius_is_raw=True,
                                    tau=wl.tau)
    else:
        prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=inp_cpu.radius_row, tau=wl.tau)
    ref_q, out_q, rep = pu.check_quantify(inp_cpu.draft, prm, wl.valid_begin, wl.n_valid, logits_dev=dd, threads=threads)
    assert rep.near_tie_flags == 0  # tau sits in the gap between the two token classes
    flags = ref_q.flag
    assert np.array_equal(out_q.flag.cpu().numpy(), flags)
    ref_v, out_v, rep_v = pu.check_verify(inp_cpu.draft, inp_cpu.target, inp_cpu.tokens.numpy(), flags,
                                          inp_cpu.u_accept.numpy(), inp_cpu.u_resample.numpy(), wl.window,
                                          oracle.VERIFY_ANCHORED, wl.valid_begin, wl.n_valid,
                                          draft_stats=(out_q.row_max, out_q.sum_exp), draft_dev=dd, target_dev=td,
                                          threads=threads)
    rep.merge(rep_v)
    print("%s: %d rows, %d windows; near ties reported separately: %d flags, %d accept tests, %d inverse-CDF draws; "
          "%d windows left out of the bit-exact comparison" % (wl.name, rep.rows // 2, rep.windows, rep.near_tie_flags,
                                                                  rep.near_tie_accepts, rep.near_tie_resamples, rep.excluded_windows))
    return ref_q, ref_v, rep


def test_workload_llamagen256_full(ciar):
    wl = synth.WORKLOADS["llamagen256"]
    inp = synth.make_inputs(wl)
    ref_q, ref_v, rep = _pipeline(ciar, wl, inp)
    assert abs(ref_q.flag.mean() - 0.30) < 0.02
    assert rep.excluded_windows <= 2


def test_workload_llamagen384_full(ciar):
    wl = synth.WORKLOADS["llamagen384"]
    inp = synth.make_inputs(wl)
    ref_q, ref_v, rep = _pipeline(ciar, wl, inp)
    assert abs(ref_q.flag.mean() - 0.30) < 0.01
    assert rep.excluded_windows <= 12  # 7 of the 576 windows have an inverse-CDF draw within 1e-6 of a bin edge


def test_workload_llamagen384_per_code_radius(ciar):
    wl = synth.WORKLOADS["llamagen384"].scaled(images=2)
    inp = synth.make_inputs(wl, per_code_radius=True)
    _pipeline(ciar, wl, inp, per_code=True)


def test_workload_anole_full(ciar):
    wl = synth.WORKLOADS["anole"]
    inp = synth.make_inputs(wl)
    ref_q, ref_v, rep = _pipeline(ciar, wl, inp)
    assert abs(ref_q.flag.mean() - 0.30) < 0.01
    assert (ref_q.argmax >= wl.valid_begin).all() and (ref_q.argmax < wl.valid_begin + wl.n_valid).all()


def test_workload_largevocab_sample(ciar):
    """The stress workload at full width (V = 2^18) on a bounded number of rows."""
    wl = synth.WORKLOADS["largevocab"].scaled(images=1, grid_h=8, grid_w=16)
    inp = synth.make_inputs(wl)
    ref_q, ref_v, rep = _pipeline(ciar, wl, inp)
    assert ref_q.flag.any() and not ref_q.flag.all()


def test_workload_largevocab_full_set_flags_and_stratified_sample(ciar):
    """The stress workload at its full size (65536 rows of 2^18 codes, generated on the device: 69 GB of logits) through
    quantify and verify in one launch each, as the benchmark runs it.  Whole set: the flags equal the generator's token
    classes (tau sits between them), no row is unusable, the windows' results are consistent with the flags.  A stratified
    sample -- every 16th window, 4096 rows, both classes -- is copied to the host and compared with the oracle element
    by element."""
    wl = synth.WORKLOADS["largevocab"]
    need = 2 * wl.rows * wl.vocab * wl.elem_bytes + (8 << 30)
    if torch.cuda.mem_get_info()[0] < need:
        pytest.skip("needs %.0f GB of free device memory" % (need / 1e9))
    inp = synth.make_inputs(wl, device="cuda")
    rows, W = wl.rows, wl.window
    qo = ciar.QuantifyOut.allocate(rows, "cuda")
    gq = pu.Guarded(qo)
    prm_dev = ciar.IntervalParams(radius_mode=ciar.RADIUS_PER_ROW, radius=inp.radius_row, tau=wl.tau)
    ciar.quantify(inp.draft, prm_dev, qo, wl.valid_begin, wl.n_valid)
    vo = ciar.VerifyOut.allocate(rows, W, "cuda")
    gv = pu.Guarded(vo)
    ws = ciar.alloc_workspace(rows, W, "cuda")
    ciar.verify(inp.draft, inp.target, inp.tokens, qo.flag, qo.row_max, qo.sum_exp, inp.u_accept, inp.u_resample, W,
                ciar.VERIFY_ANCHORED, vo, ws, wl.valid_begin, wl.n_valid)
    torch.cuda.synchronize()
    gq.check(); gv.check()
    # ---- whole set
    assert torch.equal(qo.flag.bool(), inp.boundary) and abs(float(qo.flag.float().mean()) - 0.30) < 0.01
    assert int(qo.row_status.sum()) == 0 and int(vo.row_status.sum()) == 0
    flag_w = qo.flag.view(-1, W)
    first = torch.where(flag_w.bool().any(1), flag_w.int().argmax(1), torch.full((rows // W,), W, device="cuda")).int()
    assert torch.equal(vo.first_flag, first) and torch.equal(vo.cloud_call.bool(), first < W)
    assert bool((vo.accepted_len >= first).all()) and bool((vo.accepted_len <= W).all())
    assert torch.equal(vo.resampled_token >= 0, vo.accepted_len < W)
    # ---- stratified sample against the oracle
    sel_w = torch.arange(0, rows // W, 16, device="cuda")
    total = pu.Report()
    for c0 in range(0, len(sel_w), 128):  # 1024 rows (0.5 GB per tensor) at a time
        wsel = sel_w[c0:c0 + 128]
        ridx = (wsel[:, None] * W + torch.arange(W, device="cuda")[None, :]).reshape(-1)
        draft_c, target_c = inp.draft[ridx].cpu(), inp.target[ridx].cpu()
        assert inp.boundary[ridx].any() and not inp.boundary[ridx].all()  # both classes in every chunk
        prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=inp.radius_row[ridx].cpu(), tau=wl.tau)
        ref_q = oracle.quantify(draft_c, prm, wl.valid_begin, wl.n_valid)
        rep = pu.Report(rows=len(ridx), windows=len(wsel))
        for name in pu.Q_FLOAT_FIELDS:
            pu.assert_close(name, getattr(qo, name)[ridx].cpu().numpy(), getattr(ref_q, name), rep)
        assert np.array_equal(qo.argmax[ridx].cpu().numpy(), ref_q.argmax)
        assert (ref_q.margin >= pu.NEAR_TIE).all() and np.array_equal(qo.flag[ridx].cpu().numpy(), ref_q.flag)
        ref_v = oracle.verify(draft_c, target_c, inp.tokens[ridx].cpu().numpy(), ref_q.flag, inp.u_accept[ridx].cpu().numpy(),
                              inp.u_resample[ridx].cpu().numpy(), W, oracle.VERIFY_ANCHORED, wl.valid_begin, wl.n_valid)
        near_acc = ref_v.accept_margin < pu.NEAR_TIE
        win_near = near_acc.reshape(-1, W).any(1)
        ok_win = ~win_near & ~(ref_v.resample_margin < pu.NEAR_TIE)
        rep.near_tie_accepts, rep.excluded_windows = int(near_acc.sum()), int((~ok_win).sum())
        ok_rows = np.repeat(~win_near, W)
        assert np.array_equal(vo.accept[ridx].cpu().numpy()[ok_rows], ref_v.accept[ok_rows])
        pu.assert_close("p_draft_tok", vo.p_draft_tok[ridx].cpu().numpy(), ref_v.p_draft_tok, rep)
        pu.assert_close("p_target_tok", vo.p_target_tok[ridx].cpu().numpy(), ref_v.p_target_tok, rep)
        assert np.array_equal(vo.first_flag[wsel].cpu().numpy(), ref_v.first_flag)
        assert np.array_equal(vo.accepted_len[wsel].cpu().numpy()[~win_near], ref_v.accepted_len[~win_near])
        assert np.array_equal(vo.resampled_token[wsel].cpu().numpy()[ok_win], ref_v.resampled_token[ok_win])
        total.merge(rep)
    print("largevocab sample: %d rows, %d windows, near-tie accepts %d, windows left out of the token comparison %d" % (
        total.rows, total.windows, total.near_tie_accepts, total.excluded_windows))
    # (2^18 codes: a flat row's bins are 4e-6 of the mass wide, so a draw within 1e-6 of an edge is common)
    assert total.rows == 4096 and total.excluded_windows <= 40


# ---------------------------------------------------------------- decode loop

def _decode_compare(ciar, wl, mode=oracle.VERIFY_ANCHORED, pos0=0, max_steps=None, per_code=False):
    """Runs the decode loop on both sides to the end.  After a step in which one of the oracle's decisions sat within
    the near-tie margin (the device may legitimately have gone the other way) the device state takes the oracle's
    and the comparison goes on; such steps are counted and returned.  Positions are compared after every other
    step, emitted tokens and counters at the end."""
    inp = synth.make_inputs(wl, per_code_radius=per_code)
    seq, req = wl.tokens_per_image, wl.images
    if per_code:
        prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_CODE, radius=inp.radius_code, radius_is_raw=True,
                                    tau=wl.tau)
    else:
        prm = oracle.IntervalParams(radius_mode=oracle.RADIUS_PER_ROW, radius=inp.radius_row, tau=wl.tau)
    ost = oracle.DecodeState(req, seq, pos0)
    gst = ciar.DecodeState.allocate(req, seq, "cuda")
    ciar.decode_init(gst, pos0)
    dd, td = inp.draft.cuda(), inp.target.cuda()
    tok, ua, ur = inp.tokens.cuda(), inp.u_accept.cuda(), inp.u_resample.cuda()
    gp = pu.to_ciar_params(prm, "cuda")
    ws = ciar.alloc_workspace(req * wl.window, wl.window, "cuda")
    steps = near_steps = 0
    while (ost.pos < seq).any():
        ost.min_margin[:] = np.inf
        oracle.decode_step(ost, inp.draft, inp.target, inp.tokens, inp.u_accept, inp.u_resample, prm, wl.window, mode,
                           wl.valid_begin, wl.n_valid)
        ciar.decode_step(gst, dd, td, tok, ua, ur, gp, wl.window, mode, ws, wl.valid_begin, wl.n_valid)
        steps += 1
        if ost.min_margin.min() < pu.NEAR_TIE:
            near_steps += 1
            torch.cuda.synchronize()
            gst.pos.copy_(torch.from_numpy(ost.pos))
            gst.tokens_out.copy_(torch.from_numpy(ost.tokens_out))
            gst.counters.copy_(torch.from_numpy(ost.counters))
        else:
            assert np.array_equal(gst.pos.cpu().numpy(), ost.pos), "pos after step %d" % steps
        if max_steps and steps >= max_steps:
            break
    torch.cuda.synchronize()
    assert np.array_equal(gst.tokens_out.cpu().numpy(), ost.tokens_out)
    assert np.array_equal(gst.counters.cpu().numpy(), ost.counters)
    print("decode loop: %d steps, %d of them with a near-tie decision (state taken from the oracle)" % (steps, near_steps))
    return steps, ost, near_steps


@pytest.mark.parametrize("mode", [oracle.VERIFY_ANCHORED, oracle.VERIFY_PER_TOKEN, oracle.VERIFY_ALL])
def test_decode_loop_small(ciar, mode):
    wl = synth.Workload("dec", 6, 5, 8, 512, "bf16", 8, 0.5, seed=13, decode=True, tau=2e-3)
    steps, ost, near = _decode_compare(ciar, wl, mode)
    assert (ost.pos == wl.tokens_per_image).all() and (ost.tokens_out >= 0).all()


def test_decode_loop_prefix_and_ragged_tail(ciar):
    wl = synth.Workload("dec2", 5, 3, 9, 1000, "f32", 8, 0.5, seed=14, decode=True, tau=1e-3)  # 27 tokens: ragged windows
    _decode_compare(ciar, wl, pos0=2)


def test_decode_workload_to_the_end(ciar):
    """The serving workload (V = 16384, bf16, window 8, 32 x 32 = 1024 positions per request) on 64 concurrent requests,
    run to the last token of the last request."""
    wl = synth.WORKLOADS["decode"].scaled(images=64)
    steps, ost, near = _decode_compare(ciar, wl)
    assert (ost.pos == wl.tokens_per_image).all() and (ost.tokens_out >= 0).all()
    # (a step has 64 windows; a draw of the inverse CDF falls within 1e-6 of a bin edge of a flat 16384-code row about once in 30)
    assert steps >= wl.tokens_per_image // wl.window and near <= steps // 2
    assert ost.counters[6] >= wl.images * wl.tokens_per_image  # every position was quantified at least once


def test_decode_loop_many_requests_finishing_at_different_steps(ciar):
    """More rows than three per streaming CTA, requests ending at different steps: a CTA's walk then has runs of
    three and more positions past a sequence end before a live row, whose copy has not been asked for yet."""
    wl = synth.Workload("dec3", 168, 4, 5, 2048, "bf16", 8, 0.5, seed=15, decode=True, tau=1e-3)  # 1344 rows per step, 20 tokens
    steps, ost, near = _decode_compare(ciar, wl)
    assert steps >= 3 and (ost.pos == wl.tokens_per_image).all()


def test_decode_loop_per_code_radius(ciar):
    """The decode loop with a pool of raw per-code radii indexed like the logit pools."""
    wl = synth.Workload("dec6", 12, 4, 6, 2048, "bf16", 8, 0.5, seed=17, decode=True, tau=1e-3)  # 24 tokens
    steps, ost, near = _decode_compare(ciar, wl, per_code=True)
    assert (ost.pos == wl.tokens_per_image).all() and near <= 2


def test_decode_loop_wide_rows(ciar):
    """The decode loop on rows wider than the on-chip kernels take (chunked quantifier and accept sweep behind the
    decode row map), ragged last window, requests ending at different steps."""
    wl = synth.Workload("dec5", 40, 3, 5, 20480, "bf16", 4, 0.5, seed=16, decode=True, tau=1e-3)  # 15 tokens, windows of 4
    steps, ost, near = _decode_compare(ciar, wl)
    assert (ost.pos == wl.tokens_per_image).all()

