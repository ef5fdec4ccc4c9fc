"""ciar_verify_static: the verification entry point for callers that cannot allocate.

A host that runs this library inside someone else's fixed memory arena, inside a stream capture or
in a latency-critical loop may not call cudaMalloc and may have no buffer to lend, so it cannot
give ciar_verify its workspace.  ciar_verify_static takes the same inputs and outputs and keeps its
scratch in a fixed array inside the library instead.  This test calls it through the C ABI twice
in a row, on different inputs (the second call finds the first call's leftovers in the shared
scratch), and checks every output against ciar_verify with an ordinary workspace: integer outputs
bit for bit, floating point outputs within the tolerance of the other GPU tests.

The file name makes pytest collect it last, so a run that stops at the first failure has already
run every other test.  It does not depend on them: it also passes alone in a fresh process."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-5, 1e-7  # the floating-point bar of the parity tests


def _case(rows, v, window, seed, dtype):
    g = torch.Generator().manual_seed(seed)
    draft = (2.0 * torch.randn(rows, v, generator=g)).to(dtype)
    target = (draft.float() + 0.7 * torch.randn(rows, v, generator=g)).to(dtype)
    gum = -torch.log(-torch.log(torch.rand(rows, v, generator=g).clamp(1e-9, 1 - 1e-7)))
    tokens = torch.argmax(draft.float() + gum, dim=1).to(torch.int32)
    flag = (torch.rand(rows, generator=g) < 0.3).to(torch.uint8)
    ua = torch.rand(rows, generator=g)
    ur = torch.rand(rows, generator=g)
    return [t.cuda() for t in (draft, target, tokens, flag, ua, ur)]


def _compare(ciar, got, want):
    for name in ("accept", "row_status", "first_flag", "accepted_len", "resampled_token", "cloud_call"):
        assert torch.equal(getattr(got, name), getattr(want, name)), name
    for name in ("p_draft_tok", "p_target_tok"):
        a, b = getattr(got, name).cpu().numpy().astype(np.float64), getattr(want, name).cpu().numpy().astype(np.float64)
        assert np.all(np.abs(a - b) <= ATOL + RTOL * np.abs(b)), name


def test_verify_static_matches_verify_on_two_calls_in_a_row(ciar_lib):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    ciar = ciar_lib
    cases = [(64, 2056, 8, 11, torch.bfloat16, ciar.VERIFY_ANCHORED), (96, 1000, 16, 12, torch.float32, ciar.VERIFY_ALL)]
    for rows, v, window, seed, dtype, mode in cases:
        draft, target, tokens, flag, ua, ur = _case(rows, v, window, seed, dtype)
        want = ciar.VerifyOut.allocate(rows, window, "cuda")
        ws = ciar.alloc_workspace(rows, window, "cuda")
        ciar.verify(draft, target, tokens, flag, None, None, ua, ur, window, mode, want, ws)
        got = ciar.VerifyOut.allocate(rows, window, "cuda")
        ciar.verify_static(draft, target, tokens, flag, None, None, ua, ur, window, mode, got)
        torch.cuda.synchronize()
        _compare(ciar, got, want)
        assert (want.accepted_len < window).any()  # some window was rejected, so the resampling path ran


def test_verify_static_streaming_path_on_used_scratch_matches_verify_and_oracle(ciar_lib):
    """The path production takes (draft statistics from ciar_quantify, rows of 2048 codes and more: plan, accept sweep and
    window kernels working out of the scratch) through the shared array, twice in a row with different row counts and
    windows, so that the second call finds the first one's counters and lists where it reads.  Checked against
    ciar_verify with an ordinary workspace and against the CPU oracle."""
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import oracle
    import parity_util as pu
    ciar = ciar_lib
    cases = [(8 * 40, 4096, 8, 21, torch.bfloat16, ciar.VERIFY_ANCHORED), (16 * 9, 2048, 16, 22, torch.float32, ciar.VERIFY_ALL),
             (4 * 50, 2056, 4, 23, torch.bfloat16, ciar.VERIFY_PER_TOKEN)]
    for rows, v, window, seed, dtype, mode in cases:
        draft, target, tokens, flag, ua, ur = _case(rows, v, window, seed, dtype)
        qo = ciar.QuantifyOut.allocate(rows, "cuda")
        ciar.quantify(draft, ciar.IntervalParams(r_scalar=0.2, tau=1e-4), qo)
        want = ciar.VerifyOut.allocate(rows, window, "cuda")
        ws = ciar.alloc_workspace(rows, window, "cuda")
        ciar.verify(draft, target, tokens, flag, qo.row_max, qo.sum_exp, ua, ur, window, mode, want, ws)
        got = ciar.VerifyOut.allocate(rows, window, "cuda")
        ciar.verify_static(draft, target, tokens, flag, qo.row_max, qo.sum_exp, ua, ur, window, mode, got)
        torch.cuda.synchronize()
        _compare(ciar, got, want)
        ref = oracle.verify(draft.cpu(), target.cpu(), tokens.cpu().numpy(), flag.cpu().numpy(), ua.cpu().numpy(),
                            ur.cpu().numpy(), window, mode)
        win_ok = ~((ref.accept_margin < pu.NEAR_TIE).reshape(-1, window).any(1) | (ref.resample_margin < pu.NEAR_TIE))
        assert np.array_equal(got.first_flag.cpu().numpy(), ref.first_flag)
        assert np.array_equal(got.accepted_len.cpu().numpy()[win_ok], ref.accepted_len[win_ok])
        assert np.array_equal(got.resampled_token.cpu().numpy()[win_ok], ref.resampled_token[win_ok])
        assert np.array_equal(got.accept.cpu().numpy()[np.repeat(win_ok, window)], ref.accept[np.repeat(win_ok, window)])
        assert win_ok.sum() >= 0.9 * len(win_ok) and (ref.accepted_len < window).any()


def test_verify_static_refuses_more_rows_than_its_scratch_serves(ciar_lib):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    ciar = ciar_lib
    rows, window = 160000, 8  # workspace_bytes(rows, window) is above the fixed 2 MiB
    assert ciar.workspace_bytes(rows, window) > ciar.STATIC_SCRATCH_BYTES
    logits = torch.zeros((rows, 8), dtype=torch.float32, device="cuda")
    tok = torch.zeros(rows, dtype=torch.int32, device="cuda")
    u = torch.zeros(rows, dtype=torch.float32, device="cuda")
    before = ciar.launch_count()
    with pytest.raises(ciar.CiarError) as e:
        ciar.verify_static(logits, logits, tok, None, None, None, u, u, window, ciar.VERIFY_ALL,
                           ciar.VerifyOut.allocate(rows, window, "cuda"))
    assert e.value.status == 4 and ciar.launch_count() == before
