"""CIAR oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Python face of ``ciar_oracle.c``: builds it with gcc on first use and wraps its three
entry points for numpy / CPU torch inputs.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this package; the CUDA library and its binding
never do, and this package imports nothing from them.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ciar_oracle.c")
_LIB = os.path.join(_HERE, "libciar_oracle.so")

F32, BF16 = 0, 1
RADIUS_SCALAR, RADIUS_PER_ROW, RADIUS_PER_CODE = 0, 1, 2
POLICY_INTERVAL, POLICY_ENTROPY, POLICY_MAXPROB, POLICY_RANDOM, POLICY_ALL = 0, 1, 2, 3, 4
VERIFY_ANCHORED, VERIFY_PER_TOKEN, VERIFY_ALL = 0, 1, 2
ROW_NAN, ROW_NO_FINITE, ROW_BAD_TOKEN = 1, 2, 4
SCORE_PRODUCT, SCORE_PER_N, SCORE_PER_OMEGA2, SCORE_SMOOTHED, SCORE_ADDITIVE = 0, 1, 2, 3, 4

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle shared object next to its source (gcc -O2, OpenMP, no fast-math)."""
    stale = force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if stale:
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.run(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-Wall", _SRC, "-o", tmp, "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_quantify.restype = ctypes.c_int
        _lib.orc_verify.restype = ctypes.c_int
        _lib.orc_decode_step.restype = ctypes.c_int
        _lib.orc_max_threads.restype = ctypes.c_int
        for name in ("orc_topk", "orc_score_variant", "orc_ensemble", "orc_vote", "orc_interdro"):
            getattr(_lib, name).restype = ctypes.c_int
    return _lib


def max_threads() -> int:
    return int(lib().orc_max_threads())


def as_host(x):
    """numpy view of a logits / radius tensor: float32 stays, bf16 becomes uint16 bit patterns."""
    try:
        import torch
    except ImportError:  # pragma: no cover
        torch = None
    if torch is not None and isinstance(x, torch.Tensor):
        x = x.detach().cpu().contiguous()
        if x.dtype == torch.bfloat16:
            return x.view(torch.int16).numpy().view(np.uint16), BF16
        if x.dtype == torch.float32:
            return x.numpy(), F32
        raise TypeError("logits must be float32 or bfloat16, got %s" % x.dtype)
    x = np.ascontiguousarray(x)
    if x.dtype == np.uint16:
        return x, BF16
    if x.dtype == np.float32:
        return x, F32
    raise TypeError("logits must be float32 or uint16 (bf16 bits), got %s" % x.dtype)


def _plain(x, dtype):
    try:
        import torch
        if isinstance(x, torch.Tensor):
            x = x.detach().cpu().numpy()
    except ImportError:  # pragma: no cover
        pass
    return np.ascontiguousarray(x, dtype=dtype)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


@dataclass
class IntervalParams:
    """Interval and threshold parameters (radius of the Inter-Head equation, the 0.99 / 1.01
    caps of the normalisation step, the threshold tau of Algorithm 1)."""
    radius_mode: int = RADIUS_SCALAR
    radius: object = None  # PER_ROW: float32[rows]; PER_CODE: tensor shaped like the logits
    radius_is_raw: bool = False
    r_scalar: float = 0.0
    r_max: float = 10.0
    lo_cap: float = 0.99
    hi_cap: float = 1.01
    policy: int = POLICY_INTERVAL
    tau: float = 0.30
    u_flag: object = None  # float32[rows], RANDOM policy only


def _radius_host(params: IntervalParams, dtype_code: int):
    if params.radius_mode == RADIUS_PER_ROW:
        return _plain(params.radius, np.float32)
    if params.radius_mode == RADIUS_PER_CODE:
        r, code = as_host(params.radius)
        if code != dtype_code:
            raise TypeError("per-code radius must have the logits' dtype")
        return r
    return None


@dataclass
class QuantifyResult:
    row_max: np.ndarray
    sum_exp: np.ndarray
    lse: np.ndarray
    p_max: np.ndarray
    entropy: np.ndarray
    S_lo: np.ndarray
    S_up: np.ndarray
    scale_lo: np.ndarray
    scale_up: np.ndarray
    omega: np.ndarray
    sigma: np.ndarray
    score: np.ndarray
    argmax: np.ndarray
    flag: np.ndarray
    row_status: np.ndarray
    margin: np.ndarray
    p: Optional[np.ndarray] = None
    p_lo: Optional[np.ndarray] = None
    p_up: Optional[np.ndarray] = None


def quantify(logits, params: IntervalParams, valid_begin: int = 0, valid_count: Optional[int] = None,
             dense: bool = False, threads: int = 0) -> QuantifyResult:
    """Rows of ``logits`` ([rows, vocab], row stride = vocab) through the device-side quantifier."""
    c, code = as_host(logits)
    rows, vocab = c.shape
    n = vocab - valid_begin if valid_count is None else valid_count
    rad = _radius_host(params, code)
    uf = _plain(params.u_flag, np.float32) if params.u_flag is not None else None
    d = lambda: np.empty(rows, dtype=np.float64)
    out = QuantifyResult(d(), d(), d(), d(), d(), d(), d(), d(), d(), d(), d(), d(),
                         np.empty(rows, np.int32), np.empty(rows, np.uint8), np.empty(rows, np.uint8), d())
    if dense:
        out.p = np.empty((rows, n), np.float64)
        out.p_lo = np.empty((rows, n), np.float64)
        out.p_up = np.empty((rows, n), np.float64)
    rc = lib().orc_quantify(
        _ptr(c), ctypes.c_int(code), ctypes.c_int64(rows), ctypes.c_int32(vocab), ctypes.c_int64(vocab),
        ctypes.c_int32(valid_begin), ctypes.c_int32(n),
        ctypes.c_int(params.radius_mode), _ptr(rad), ctypes.c_int(int(params.radius_is_raw)),
        ctypes.c_double(params.r_scalar), ctypes.c_double(params.r_max),
        ctypes.c_double(params.lo_cap), ctypes.c_double(params.hi_cap),
        ctypes.c_int(params.policy), ctypes.c_double(params.tau), _ptr(uf),
        _ptr(out.row_max), _ptr(out.sum_exp), _ptr(out.lse), _ptr(out.p_max), _ptr(out.entropy),
        _ptr(out.S_lo), _ptr(out.S_up), _ptr(out.scale_lo), _ptr(out.scale_up),
        _ptr(out.omega), _ptr(out.sigma), _ptr(out.score),
        _ptr(out.argmax), _ptr(out.flag), _ptr(out.row_status), _ptr(out.margin),
        _ptr(out.p), _ptr(out.p_lo), _ptr(out.p_up), ctypes.c_int(threads))
    if rc != 0:
        raise ValueError("orc_quantify: invalid arguments (code %d)" % rc)
    return out


@dataclass
class VerifyResult:
    accept: np.ndarray
    p_draft_tok: np.ndarray
    p_target_tok: np.ndarray
    accept_margin: np.ndarray
    row_status: np.ndarray
    first_flag: np.ndarray
    accepted_len: np.ndarray
    resampled_token: np.ndarray
    cloud_call: np.ndarray
    residual_mass: np.ndarray
    resample_margin: np.ndarray


def verify(draft_logits, target_logits, draft_tokens, flag, u_accept, u_resample, window: int,
           mode: int = VERIFY_ANCHORED, valid_begin: int = 0, valid_count: Optional[int] = None,
           threads: int = 0) -> VerifyResult:
    """Cloud-side test of every draft window of ``window`` consecutive rows."""
    c, code = as_host(draft_logits)
    t, code_t = as_host(target_logits)
    if code != code_t or c.shape != t.shape:
        raise TypeError("draft and target logits must share dtype and shape")
    rows, vocab = c.shape
    n = vocab - valid_begin if valid_count is None else valid_count
    if window < 1 or rows % window:
        raise ValueError("rows must be a multiple of the window")
    nw = rows // window
    tok = _plain(draft_tokens, np.int32)
    fl = _plain(flag, np.uint8) if flag is not None else None
    ua = _plain(u_accept, np.float32)
    ur = _plain(u_resample, np.float32)
    out = VerifyResult(np.empty(rows, np.uint8), np.empty(rows, np.float64), np.empty(rows, np.float64),
                       np.empty(rows, np.float64), np.empty(rows, np.uint8),
                       np.empty(nw, np.int32), np.empty(nw, np.int32), np.empty(nw, np.int32),
                       np.empty(nw, np.uint8), np.empty(nw, np.float64), np.empty(nw, np.float64))
    rc = lib().orc_verify(
        _ptr(c), _ptr(t), ctypes.c_int(code), ctypes.c_int64(rows), ctypes.c_int32(vocab), ctypes.c_int64(vocab),
        ctypes.c_int32(valid_begin), ctypes.c_int32(n),
        _ptr(tok), _ptr(fl), _ptr(ua), _ptr(ur), ctypes.c_int32(window), ctypes.c_int(mode),
        _ptr(out.accept), _ptr(out.p_draft_tok), _ptr(out.p_target_tok), _ptr(out.accept_margin),
        _ptr(out.row_status),
        _ptr(out.first_flag), _ptr(out.accepted_len), _ptr(out.resampled_token), _ptr(out.cloud_call),
        _ptr(out.residual_mass), _ptr(out.resample_margin), ctypes.c_int(threads))
    if rc != 0:
        raise ValueError("orc_verify: invalid arguments (code %d)" % rc)
    return out


class DecodeState:
    """Per-request position and emitted tokens, advanced by :func:`decode_step`."""

    def __init__(self, requests: int, seq_len: int, pos0: int = 0):
        self.requests, self.seq_len = requests, seq_len
        self.pos = np.full(requests, pos0, np.int32)
        self.tokens_out = np.full((requests, seq_len), -1, np.int32)
        self.counters = np.zeros(8, np.int64)
        self.min_margin = np.full(3, np.inf, np.float64)


def decode_step(state: DecodeState, draft_pool, target_pool, draft_token_pool, u_accept_pool, u_resample_pool,
                params: IntervalParams, window: int, mode: int = VERIFY_ANCHORED,
                valid_begin: int = 0, valid_count: Optional[int] = None, threads: int = 0) -> None:
    """One trip of Algorithm 1's device loop for every unfinished request (pools are
    [requests * seq_len, vocab] and [requests * seq_len])."""
    c, code = as_host(draft_pool)
    t, code_t = as_host(target_pool)
    if code != code_t or c.shape != t.shape:
        raise TypeError("draft and target pools must share dtype and shape")
    rows, vocab = c.shape
    if rows != state.requests * state.seq_len:
        raise ValueError("pool rows must equal requests * seq_len")
    n = vocab - valid_begin if valid_count is None else valid_count
    rad = _radius_host(params, code)
    uf = _plain(params.u_flag, np.float32) if params.u_flag is not None else None
    tok = _plain(draft_token_pool, np.int32)
    ua = _plain(u_accept_pool, np.float32)
    ur = _plain(u_resample_pool, np.float32)
    rc = lib().orc_decode_step(
        _ptr(c), _ptr(t), ctypes.c_int(code), ctypes.c_int32(state.requests), ctypes.c_int32(state.seq_len),
        ctypes.c_int32(vocab), ctypes.c_int64(vocab), ctypes.c_int32(valid_begin), ctypes.c_int32(n),
        _ptr(tok), _ptr(ua), _ptr(ur),
        ctypes.c_int(params.radius_mode), _ptr(rad), ctypes.c_int(int(params.radius_is_raw)),
        ctypes.c_double(params.r_scalar), ctypes.c_double(params.r_max),
        ctypes.c_double(params.lo_cap), ctypes.c_double(params.hi_cap),
        ctypes.c_int(params.policy), ctypes.c_double(params.tau), _ptr(uf),
        ctypes.c_int32(window), ctypes.c_int(mode),
        _ptr(state.pos), _ptr(state.tokens_out), _ptr(state.counters), _ptr(state.min_margin),
        ctypes.c_int(threads))
    if rc != 0:
        raise ValueError("orc_decode_step: invalid arguments (code %d)" % rc)


@dataclass
class TopkResult:
    kth_logit: np.ndarray
    n_above: np.ndarray
    mass: np.ndarray
    entropy: np.ndarray
    S_lo: np.ndarray
    S_up: np.ndarray
    omega: np.ndarray
    sigma: np.ndarray
    score: np.ndarray
    flag: np.ndarray
    row_status: np.ndarray
    margin: np.ndarray
    indices: Optional[np.ndarray] = None


def topk(logits, k: int, params: IntervalParams, valid_begin: int = 0, valid_count: Optional[int] = None,
         indices: bool = False, threads: int = 0) -> TopkResult:
    """Discrete top-k quantifier: full sort of every row, the interval score of the k kept codes."""
    c, code = as_host(logits)
    rows, vocab = c.shape
    n = vocab - valid_begin if valid_count is None else valid_count
    rad = _radius_host(params, code)
    d = lambda: np.empty(rows, dtype=np.float64)
    out = TopkResult(d(), np.empty(rows, np.int32), d(), d(), d(), d(), d(), d(), d(),
                     np.empty(rows, np.uint8), np.empty(rows, np.uint8), d())
    if indices:
        out.indices = np.empty((rows, k), np.int32)
    rc = lib().orc_topk(
        _ptr(c), ctypes.c_int(code), ctypes.c_int64(rows), ctypes.c_int32(vocab), ctypes.c_int64(vocab),
        ctypes.c_int32(valid_begin), ctypes.c_int32(n), ctypes.c_int32(k),
        ctypes.c_int(params.radius_mode), _ptr(rad), ctypes.c_int(int(params.radius_is_raw)),
        ctypes.c_double(params.r_scalar), ctypes.c_double(params.r_max),
        ctypes.c_double(params.lo_cap), ctypes.c_double(params.hi_cap), ctypes.c_double(params.tau),
        _ptr(out.kth_logit), _ptr(out.n_above), _ptr(out.mass), _ptr(out.entropy),
        _ptr(out.S_lo), _ptr(out.S_up), _ptr(out.omega), _ptr(out.sigma), _ptr(out.score),
        _ptr(out.flag), _ptr(out.row_status), _ptr(out.margin), _ptr(out.indices), ctypes.c_int(threads))
    if rc != 0:
        raise ValueError("orc_topk: invalid arguments (code %d)" % rc)
    return out


def score_variant(omega, sigma, n: int, variant: int, eps: float = 0.0, lambda1: float = 0.0,
                  lambda2: float = 1.0, tau: float = 0.0):
    """Score variants of the uncertainty appendix's practical remarks; returns (value, flag, margin)."""
    om = _plain(omega, np.float64)
    sg = _plain(sigma, np.float64)
    rows = om.shape[0]
    out, flag, margin = np.empty(rows, np.float64), np.empty(rows, np.uint8), np.empty(rows, np.float64)
    rc = lib().orc_score_variant(
        ctypes.c_int64(rows), ctypes.c_int32(n), _ptr(om), _ptr(sg), ctypes.c_int(variant),
        ctypes.c_double(eps), ctypes.c_double(lambda1), ctypes.c_double(lambda2), ctypes.c_double(tau),
        _ptr(out), _ptr(flag), _ptr(margin))
    if rc != 0:
        raise ValueError("orc_score_variant: invalid arguments (code %d)" % rc)
    return out, flag, margin


@dataclass
class EnsembleResult:
    p_max: np.ndarray
    entropy: np.ndarray
    S_lo: np.ndarray
    S_up: np.ndarray
    omega: np.ndarray
    sigma: np.ndarray
    score: np.ndarray
    flag: np.ndarray
    row_status: np.ndarray
    margin: np.ndarray
    pbar: Optional[np.ndarray] = None


def ensemble(heads, params: IntervalParams, valid_begin: int = 0, valid_count: Optional[int] = None,
             dense: bool = False, threads: int = 0) -> EnsembleResult:
    """Soft voting over ``heads`` ([H, rows, vocab]); ``params.radius`` is float32[H, rows] for PER_ROW."""
    c, code = as_host(heads)
    n_heads, rows, vocab = c.shape
    n = vocab - valid_begin if valid_count is None else valid_count
    rad = _plain(params.radius, np.float32) if params.radius_mode == RADIUS_PER_ROW else None
    d = lambda: np.empty(rows, dtype=np.float64)
    out = EnsembleResult(d(), d(), d(), d(), d(), d(), d(), np.empty(rows, np.uint8), np.empty(rows, np.uint8), d())
    if dense:
        out.pbar = np.empty((rows, n), np.float64)
    rc = lib().orc_ensemble(
        _ptr(c), ctypes.c_int(code), ctypes.c_int32(n_heads), ctypes.c_int64(rows * vocab), ctypes.c_int64(rows),
        ctypes.c_int32(vocab), ctypes.c_int64(vocab), ctypes.c_int32(valid_begin), ctypes.c_int32(n),
        ctypes.c_int(params.radius_mode), _ptr(rad), ctypes.c_int(int(params.radius_is_raw)),
        ctypes.c_double(params.r_scalar), ctypes.c_double(params.r_max),
        ctypes.c_double(params.lo_cap), ctypes.c_double(params.hi_cap), ctypes.c_double(params.tau),
        _ptr(out.p_max), _ptr(out.entropy), _ptr(out.S_lo), _ptr(out.S_up),
        _ptr(out.omega), _ptr(out.sigma), _ptr(out.score), _ptr(out.flag), _ptr(out.row_status),
        _ptr(out.margin), _ptr(out.pbar), ctypes.c_int(threads))
    if rc != 0:
        raise ValueError("orc_ensemble: invalid arguments (code %d)" % rc)
    return out


def vote(flags):
    """Hard voting: flags uint8[H, rows] -> (flag uint8[rows], votes int32[rows])."""
    f = _plain(flags, np.uint8)
    n_heads, rows = f.shape
    out, votes = np.empty(rows, np.uint8), np.empty(rows, np.int32)
    rc = lib().orc_vote(ctypes.c_int32(n_heads), ctypes.c_int64(rows), _ptr(f), _ptr(out), _ptr(votes))
    if rc != 0:
        raise ValueError("orc_vote: invalid arguments (code %d)" % rc)
    return out, votes


@dataclass
class InterDroResult:
    l1: np.ndarray       # [3, rows]: mid, up, lo
    ce: np.ndarray       # [3, rows]
    kl: np.ndarray       # [rows]
    weights: np.ndarray  # [rows]
    loss: np.ndarray     # total, centre, upper, lower, dro, align


def interdro(center, radius, cloud, radius_is_raw: bool = True, r_max: float = 10.0, lambda_v: float = 1.0,
             lambda_p: float = 1.0, lambda_beta: float = 1.0, alpha: float = 1.0, valid_begin: int = 0,
             valid_count: Optional[int] = None, threads: int = 0) -> InterDroResult:
    """Forward value of the Inter-DRO loss over a batch of rows (one radius per code)."""
    c, code = as_host(center)
    r, code_r = as_host(radius)
    t, code_t = as_host(cloud)
    if not (code == code_r == code_t) or not (c.shape == r.shape == t.shape):
        raise TypeError("centre, radius and cloud logits must share dtype and shape")
    rows, vocab = c.shape
    n = vocab - valid_begin if valid_count is None else valid_count
    out = InterDroResult(np.empty((3, rows), np.float64), np.empty((3, rows), np.float64),
                         np.empty(rows, np.float64), np.empty(rows, np.float64), np.empty(6, np.float64))
    rc = lib().orc_interdro(
        _ptr(c), _ptr(r), _ptr(t), ctypes.c_int(code), ctypes.c_int64(rows), ctypes.c_int32(vocab),
        ctypes.c_int64(vocab), ctypes.c_int32(valid_begin), ctypes.c_int32(n),
        ctypes.c_int(int(radius_is_raw)), ctypes.c_double(r_max),
        ctypes.c_double(lambda_v), ctypes.c_double(lambda_p), ctypes.c_double(lambda_beta), ctypes.c_double(alpha),
        _ptr(out.l1), _ptr(out.ce), _ptr(out.kl), _ptr(out.weights), _ptr(out.loss), ctypes.c_int(threads))
    if rc != 0:
        raise ValueError("orc_interdro: invalid arguments (code %d)" % rc)
    return out
