"""The input generators: Philox known answers, the blob field's exact boundary fraction, the
layout of the masked workload, and that drafted tokens really are samples of the draft row."""
import numpy as np
import scipy.special
import scipy.stats
import torch

from paper_2603_25463_b200 import synth


def _run(counter, key):
    out = synth.philox4x32_10([torch.tensor([x]) for x in counter], key)
    return [int(o) for o in out]


def test_philox_known_answer_vectors():
    # known-answer vectors published with the Philox4x32-10 generator
    assert _run((0, 0, 0, 0), (0, 0)) == [0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8]
    assert _run((0xFFFFFFFF,) * 4, (0xFFFFFFFF,) * 2) == [0x408F276D, 0x41C83B0E, 0xA20BC7C6, 0x6D5451FD]
    assert _run((0x243F6A88, 0x85A308D3, 0x13198A2E, 0x03707344), (0xA4093822, 0x299F31D0)) == \
        [0xD16CFE09, 0x94FDCCEB, 0x5001E420, 0x24126EA1]


def test_uniforms_in_unit_interval_and_offset_consistent():
    ua, ur, uf = synth.philox_uniforms(4096, 0)
    for u in (ua, ur, uf):
        assert u.dtype == torch.float32 and float(u.min()) >= 0.0 and float(u.max()) < 1.0
        assert abs(float(u.mean()) - 0.5) < 0.03
    ub = synth.philox_uniforms(96, 0, row_offset=4000)[0]
    assert torch.equal(ub, ua[4000:])
    assert ua[0].item() == (0x6627E8D5 >> 8) / 2 ** 24


def test_blob_field_boundary_fraction_is_exact_and_structured():
    wl = synth.WORKLOADS["llamagen384"]
    m = synth.blob_boundary_mask(wl)
    assert m.shape == (16, 576)
    assert (m.sum(1) == round(0.3 * 576)).all()
    # spatially smooth: a boundary cell's right neighbour is a boundary cell far more often than 30 %
    g = m.view(16, 24, 24)
    both = (g[:, :, :-1] & g[:, :, 1:]).sum().item() / g[:, :, :-1].sum().item()
    assert both > 0.5


def test_masked_workload_layout_and_dtype():
    wl = synth.WORKLOADS["anole"].scaled(images=1, grid_h=4, grid_w=4, vocab=1024, valid_begin=512, valid_count=128)
    inp = synth.make_inputs(wl)
    assert inp.draft.dtype == torch.bfloat16 and inp.draft.shape == (16, 1024)
    d = inp.draft.float()
    assert torch.isinf(d[:, :512]).all() and torch.isinf(d[:, 640:]).all() and torch.isfinite(d[:, 512:640]).all()
    t = inp.target.float()
    assert torch.isinf(t[:, :512]).all() and torch.isfinite(t[:, 512:640]).all()
    assert ((inp.tokens >= 512) & (inp.tokens < 640)).all()
    assert torch.equal(inp.radius_row == wl.r_boundary, inp.boundary)


def test_zipf_rows_are_a_permuted_power_law():
    wl = synth.WORKLOADS["largevocab"].scaled(images=1, grid_h=2, grid_w=4, vocab=1024)
    inp = synth.make_inputs(wl)
    d = inp.draft.float()
    for r in range(wl.rows):
        s = float(wl.scale_boundary if inp.boundary[r] else wl.scale_interior)
        expect = (-1.1 * s * torch.log(torch.arange(1, 1025, dtype=torch.float32))).to(torch.bfloat16).float()
        assert torch.equal(torch.sort(d[r], descending=True).values, torch.sort(expect, descending=True).values)
    assert not torch.equal(d[0].argsort(), d[1].argsort())


def test_gumbel_tokens_follow_the_draft_row():
    wl = synth.Workload("tok", 1, 100, 100, 8, "f32", 8, 0.5, seed=3, boundary_frac=1.0)
    inp = synth.make_inputs(wl)
    # every row has its own logits; compare the mean assigned probability with its expectation
    p = scipy.special.softmax(inp.draft.double().numpy(), axis=1)
    picked = p[np.arange(wl.rows), inp.tokens.numpy()]
    expect = (p ** 2).sum(1)  # E[p_x] for x ~ p
    z = (picked - expect).sum() / np.sqrt(((p ** 3).sum(1) - expect ** 2).sum())
    assert abs(z) < 4.5


def test_tau_sits_between_the_two_token_classes():
    """tests/golden/tau_calibration.txt (written from the CPU oracle by the script beside it): the
    frozen threshold of every workload lies strictly between the highest interior score and the
    lowest boundary score, so no flag decision of the parity workloads is a near tie."""
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "tau_calibration.txt")
    seen = set()
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        name, rows, hi_int, lo_bnd, mid, tau, frac = line.split()
        assert float(hi_int) * 2 < float(tau) < float(lo_bnd) / 2, name
        assert float(tau) == synth.WORKLOADS[name].tau
        seen.add(name)
    assert seen == set(synth.WORKLOADS)
