"""ctypes binding of ``libciar.so``: the same entry points as ``include/ciar.h``, taking torch
CUDA tensors.  This layer only marshals arguments (pointers, sizes, the current stream); every
step of the path runs in the library's kernels.  There is no CPU or PyTorch fallback: if the
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field
from typing import Optional

import torch

from . import build as _build

F32, BF16 = 0, 1
RADIUS_SCALAR, RADIUS_PER_ROW, RADIUS_PER_CODE = 0, 1, 2
POLICY_INTERVAL, POLICY_ENTROPY, POLICY_MAXPROB, POLICY_RANDOM, POLICY_ALL = 0, 1, 2, 3, 4
VERIFY_ANCHORED, VERIFY_PER_TOKEN, VERIFY_ALL = 0, 1, 2
ROW_NAN, ROW_NO_FINITE, ROW_BAD_TOKEN, ROW_TIMEOUT = 1, 2, 4, 8
MAX_WINDOW = 64

_vp = ctypes.c_void_p


class LogitsDesc(ctypes.Structure):
    _fields_ = [("rows", ctypes.c_int64), ("row_stride", ctypes.c_int64), ("vocab", ctypes.c_int32),
                ("valid_begin", ctypes.c_int32), ("valid_count", ctypes.c_int32), ("dtype", ctypes.c_int32)]


class IntervalParamsC(ctypes.Structure):
    _fields_ = [("radius_mode", ctypes.c_int32), ("radius_is_raw", ctypes.c_int32), ("radius", _vp),
                ("r_scalar", ctypes.c_float), ("r_max", ctypes.c_float), ("lo_cap", ctypes.c_float),
                ("hi_cap", ctypes.c_float), ("policy", ctypes.c_int32), ("tau", ctypes.c_float), ("u_flag", _vp)]


class QuantifyOutC(ctypes.Structure):
    _fields_ = [(n, _vp) for n in ("row_max", "sum_exp", "lse", "p_max", "entropy", "S_lo", "S_up", "omega",
                                   "sigma", "score", "argmax", "flag", "row_status", "dense_p", "dense_lo",
                                   "dense_up")]


class VerifyParamsC(ctypes.Structure):
    _fields_ = [("window", ctypes.c_int32), ("mode", ctypes.c_int32)]


class VerifyOutC(ctypes.Structure):
    _fields_ = [(n, _vp) for n in ("accept", "p_draft_tok", "p_target_tok", "row_status", "first_flag",
                                   "accepted_len", "resampled_token", "cloud_call")]


class DecodeStateC(ctypes.Structure):
    _fields_ = [("requests", ctypes.c_int32), ("seq_len", ctypes.c_int32), ("pos", _vp), ("tokens_out", _vp),
                ("counters", _vp)]


class CiarError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__("%s failed: %s (status %d)" % (fn, status_string(status), status))


_lib = None


def load() -> ctypes.CDLL:
    """Load libciar.so from the package directory; raises if it has not been built."""
    global _lib
    if _lib is None:
        path = _build.LIB_PATH
        if not os.path.exists(path):
            raise RuntimeError("libciar.so is missing at %s: build it with __graft_entry__.build() "
                               "(there is no fallback path)" % path)
        lib = ctypes.CDLL(path)
        lib.ciar_status_string.restype = ctypes.c_char_p
        lib.ciar_status_string.argtypes = [ctypes.c_int]
        lib.ciar_version.restype = ctypes.c_int
        lib.ciar_launch_count.restype = ctypes.c_int64
        lib.ciar_workspace_bytes.restype = ctypes.c_size_t
        lib.ciar_workspace_bytes.argtypes = [ctypes.c_int64, ctypes.c_int32]
        lib.ciar_quantify.restype = ctypes.c_int
        lib.ciar_quantify.argtypes = [ctypes.POINTER(LogitsDesc), _vp, ctypes.POINTER(IntervalParamsC),
                                      ctypes.POINTER(QuantifyOutC), _vp]
        lib.ciar_verify.restype = ctypes.c_int
        lib.ciar_verify.argtypes = [ctypes.POINTER(LogitsDesc), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                                    ctypes.POINTER(VerifyParamsC), ctypes.POINTER(VerifyOutC), _vp,
                                    ctypes.c_size_t, _vp]
        lib.ciar_verify_static.restype = ctypes.c_int
        lib.ciar_verify_static.argtypes = [ctypes.POINTER(LogitsDesc), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                                           ctypes.POINTER(VerifyParamsC), ctypes.POINTER(VerifyOutC), _vp]
        lib.ciar_test_stall.restype = ctypes.c_int
        lib.ciar_test_stall.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int64]
        lib.ciar_decode_init.restype = ctypes.c_int
        lib.ciar_decode_init.argtypes = [ctypes.POINTER(DecodeStateC), ctypes.c_int32, _vp]
        lib.ciar_decode_step.restype = ctypes.c_int
        lib.ciar_decode_step.argtypes = [ctypes.POINTER(DecodeStateC), ctypes.POINTER(LogitsDesc), _vp, _vp, _vp,
                                         _vp, _vp, ctypes.POINTER(IntervalParamsC), ctypes.POINTER(VerifyParamsC),
                                         _vp, ctypes.c_size_t, _vp]
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load().ciar_status_string(int(status)).decode()


def version() -> int:
    return int(load().ciar_version())


def launch_count() -> int:
    return int(load().ciar_launch_count())


def stall_hook(cta: int, row_in_walk: int, wait_cycles: int) -> None:
    """Test hook: CTA `cta` of the streaming quantifier never asks for the `row_in_walk`-th row of its walk and every
    device-side wait is bounded by `wait_cycles` SM clocks (cta < 0: off; wait_cycles <= 0: default bound)."""
    load().ciar_test_stall(int(cta), int(row_in_walk), int(wait_cycles))


def workspace_bytes(rows: int, window: int) -> int:
    return int(load().ciar_workspace_bytes(rows, window))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    return -1  # rejected by the library as unsupported


def _require_cuda(*tensors):
    for t in tensors:
        if t is not None and not t.is_cuda:
            raise ValueError("the CIAR library takes CUDA tensors only (no CPU path exists)")


def make_desc(logits: torch.Tensor, valid_begin: int = 0, valid_count: Optional[int] = None) -> LogitsDesc:
    if logits.dim() != 2 or logits.stride(1) != 1:
        raise ValueError("logits must be a 2-D tensor with unit stride along the vocabulary")
    rows, vocab = logits.shape
    n = vocab - valid_begin if valid_count is None else valid_count
    stride = logits.stride(0) if rows > 1 else max(vocab, logits.stride(0))
    return LogitsDesc(rows, stride, vocab, valid_begin, n, _dtype_code(logits))


@dataclass
class IntervalParams:
    """Interval and threshold parameters; see ciar_interval_params in ciar.h."""
    radius_mode: int = RADIUS_SCALAR
    radius: Optional[torch.Tensor] = None
    radius_is_raw: bool = False
    r_scalar: float = 0.0
    r_max: float = 10.0
    lo_cap: float = 0.99
    hi_cap: float = 1.01
    policy: int = POLICY_INTERVAL
    tau: float = 0.30
    u_flag: Optional[torch.Tensor] = None

    def to_c(self) -> IntervalParamsC:
        _require_cuda(self.radius, self.u_flag)
        return IntervalParamsC(self.radius_mode, int(self.radius_is_raw), _ptr(self.radius), self.r_scalar,
                               self.r_max, self.lo_cap, self.hi_cap, self.policy, self.tau, _ptr(self.u_flag))


_Q_F32 = ("row_max", "sum_exp", "lse", "p_max", "entropy", "S_lo", "S_up", "omega", "sigma", "score")


@dataclass
class QuantifyOut:
    """Output tensors of ciar_quantify; allocate() makes all of them."""
    row_max: Optional[torch.Tensor] = None
    sum_exp: Optional[torch.Tensor] = None
    lse: Optional[torch.Tensor] = None
    p_max: Optional[torch.Tensor] = None
    entropy: Optional[torch.Tensor] = None
    S_lo: Optional[torch.Tensor] = None
    S_up: Optional[torch.Tensor] = None
    omega: Optional[torch.Tensor] = None
    sigma: Optional[torch.Tensor] = None
    score: Optional[torch.Tensor] = None
    argmax: Optional[torch.Tensor] = None
    flag: Optional[torch.Tensor] = None
    row_status: Optional[torch.Tensor] = None
    dense_p: Optional[torch.Tensor] = None
    dense_lo: Optional[torch.Tensor] = None
    dense_up: Optional[torch.Tensor] = None

    @classmethod
    def allocate(cls, rows: int, device, dense_width: int = 0) -> "QuantifyOut":
        o = cls()
        for n in _Q_F32:
            setattr(o, n, torch.empty(rows, dtype=torch.float32, device=device))
        o.argmax = torch.empty(rows, dtype=torch.int32, device=device)
        o.flag = torch.empty(rows, dtype=torch.uint8, device=device)
        o.row_status = torch.empty(rows, dtype=torch.uint8, device=device)
        if dense_width:
            for n in ("dense_p", "dense_lo", "dense_up"):
                setattr(o, n, torch.empty((rows, dense_width), dtype=torch.float32, device=device))
        return o

    def to_c(self) -> QuantifyOutC:
        names = [f[0] for f in QuantifyOutC._fields_]
        _require_cuda(*[getattr(self, n) for n in names])
        return QuantifyOutC(*[_ptr(getattr(self, n)) for n in names])


def quantify(logits: torch.Tensor, params: IntervalParams, out: QuantifyOut, valid_begin: int = 0,
             valid_count: Optional[int] = None, stream=None) -> QuantifyOut:
    """ciar_quantify: device-side uncertainty quantification of every row of ``logits``."""
    _require_cuda(logits)
    desc = make_desc(logits, valid_begin, valid_count)
    pc, oc = params.to_c(), out.to_c()
    st = load().ciar_quantify(ctypes.byref(desc), _ptr(logits), ctypes.byref(pc), ctypes.byref(oc), _stream(stream))
    if st != 0:
        raise CiarError("ciar_quantify", st)
    return out


@dataclass
class VerifyOut:
    accept: Optional[torch.Tensor] = None
    p_draft_tok: Optional[torch.Tensor] = None
    p_target_tok: Optional[torch.Tensor] = None
    row_status: Optional[torch.Tensor] = None
    first_flag: Optional[torch.Tensor] = None
    accepted_len: Optional[torch.Tensor] = None
    resampled_token: Optional[torch.Tensor] = None
    cloud_call: Optional[torch.Tensor] = None

    @classmethod
    def allocate(cls, rows: int, window: int, device) -> "VerifyOut":
        nw = rows // window
        return cls(torch.empty(rows, dtype=torch.uint8, device=device),
                   torch.empty(rows, dtype=torch.float32, device=device),
                   torch.empty(rows, dtype=torch.float32, device=device),
                   torch.empty(rows, dtype=torch.uint8, device=device),
                   torch.empty(nw, dtype=torch.int32, device=device),
                   torch.empty(nw, dtype=torch.int32, device=device),
                   torch.empty(nw, dtype=torch.int32, device=device),
                   torch.empty(nw, dtype=torch.uint8, device=device))

    def to_c(self) -> VerifyOutC:
        names = [f[0] for f in VerifyOutC._fields_]
        _require_cuda(*[getattr(self, n) for n in names])
        return VerifyOutC(*[_ptr(getattr(self, n)) for n in names])


def alloc_workspace(rows: int, window: int, device) -> torch.Tensor:
    return torch.empty(max(16, workspace_bytes(rows, window)), dtype=torch.uint8, device=device)


def verify(draft: torch.Tensor, target: torch.Tensor, draft_tokens: torch.Tensor, flag: Optional[torch.Tensor],
           draft_row_max: Optional[torch.Tensor], draft_sum_exp: Optional[torch.Tensor],
           u_accept: torch.Tensor, u_resample: torch.Tensor, window: int, mode: int, out: VerifyOut,
           workspace: torch.Tensor, valid_begin: int = 0, valid_count: Optional[int] = None,
           stream=None) -> VerifyOut:
    """ciar_verify: cloud-side accept / resample test of every draft window."""
    _require_cuda(draft, target, draft_tokens, flag, draft_row_max, draft_sum_exp, u_accept, u_resample, workspace)
    if target.shape != draft.shape or target.dtype != draft.dtype or target.stride() != draft.stride():
        raise ValueError("draft and target logits must share shape, dtype and strides")
    desc = make_desc(draft, valid_begin, valid_count)
    vp, oc = VerifyParamsC(window, mode), out.to_c()
    st = load().ciar_verify(ctypes.byref(desc), _ptr(draft), _ptr(target), _ptr(draft_tokens), _ptr(flag),
                            _ptr(draft_row_max), _ptr(draft_sum_exp), _ptr(u_accept), _ptr(u_resample),
                            ctypes.byref(vp), ctypes.byref(oc), _ptr(workspace), workspace.numel(), _stream(stream))
    if st != 0:
        raise CiarError("ciar_verify", st)
    return out


STATIC_SCRATCH_BYTES = 2 * 1024 * 1024


def verify_static(draft: torch.Tensor, target: torch.Tensor, draft_tokens: torch.Tensor, flag: Optional[torch.Tensor],
                  draft_row_max: Optional[torch.Tensor], draft_sum_exp: Optional[torch.Tensor],
                  u_accept: torch.Tensor, u_resample: torch.Tensor, window: int, mode: int, out: VerifyOut,
                  valid_begin: int = 0, valid_count: Optional[int] = None, stream=None) -> VerifyOut:
    """ciar_verify_static: ciar_verify for callers that cannot provide a workspace (they may not
    allocate device memory where they run).  The scratch is a fixed 2 MiB array inside the library,
    shared by all calls on a device: calls that could overlap on the GPU must be ordered, and
    batches whose workspace_bytes() exceeds STATIC_SCRATCH_BYTES are refused (status 4)."""
    _require_cuda(draft, target, draft_tokens, flag, draft_row_max, draft_sum_exp, u_accept, u_resample)
    if target.shape != draft.shape or target.dtype != draft.dtype or target.stride() != draft.stride():
        raise ValueError("draft and target logits must share shape, dtype and strides")
    desc = make_desc(draft, valid_begin, valid_count)
    vp, oc = VerifyParamsC(window, mode), out.to_c()
    st = load().ciar_verify_static(ctypes.byref(desc), _ptr(draft), _ptr(target), _ptr(draft_tokens), _ptr(flag),
                                   _ptr(draft_row_max), _ptr(draft_sum_exp), _ptr(u_accept), _ptr(u_resample),
                                   ctypes.byref(vp), ctypes.byref(oc), _stream(stream))
    if st != 0:
        raise CiarError("ciar_verify_static", st)
    return out


@dataclass
class DecodeState:
    """Device-resident state of a batch of requests (see ciar_decode_state in ciar.h)."""
    requests: int
    seq_len: int
    pos: torch.Tensor = field(default=None)
    tokens_out: torch.Tensor = field(default=None)
    counters: torch.Tensor = field(default=None)

    @classmethod
    def allocate(cls, requests: int, seq_len: int, device) -> "DecodeState":
        return cls(requests, seq_len,
                   torch.empty(requests, dtype=torch.int32, device=device),
                   torch.empty((requests, seq_len), dtype=torch.int32, device=device),
                   torch.empty(8, dtype=torch.int64, device=device))

    def to_c(self) -> DecodeStateC:
        _require_cuda(self.pos, self.tokens_out, self.counters)
        return DecodeStateC(self.requests, self.seq_len, _ptr(self.pos), _ptr(self.tokens_out), _ptr(self.counters))


def decode_init(state: DecodeState, pos0: int = 0, stream=None) -> None:
    sc = state.to_c()
    st = load().ciar_decode_init(ctypes.byref(sc), pos0, _stream(stream))
    if st != 0:
        raise CiarError("ciar_decode_init", st)


def decode_step(state: DecodeState, draft_pool: torch.Tensor, target_pool: torch.Tensor,
                draft_token_pool: torch.Tensor, u_accept_pool: torch.Tensor, u_resample_pool: torch.Tensor,
                params: IntervalParams, window: int, mode: int, workspace: torch.Tensor,
                valid_begin: int = 0, valid_count: Optional[int] = None, stream=None) -> None:
    """ciar_decode_step: one trip of the device loop for every unfinished request."""
    _require_cuda(draft_pool, target_pool, draft_token_pool, u_accept_pool, u_resample_pool, workspace)
    if target_pool.shape != draft_pool.shape or target_pool.dtype != draft_pool.dtype:
        raise ValueError("draft and target pools must share shape and dtype")
    desc = make_desc(draft_pool, valid_begin, valid_count)
    sc, pc, vp = state.to_c(), params.to_c(), VerifyParamsC(window, mode)
    st = load().ciar_decode_step(ctypes.byref(sc), ctypes.byref(desc), _ptr(draft_pool), _ptr(target_pool),
                                 _ptr(draft_token_pool), _ptr(u_accept_pool), _ptr(u_resample_pool),
                                 ctypes.byref(pc), ctypes.byref(vp), _ptr(workspace), workspace.numel(),
                                 _stream(stream))
    if st != 0:
        raise CiarError("ciar_decode_step", st)


# ---------------------------------------------------------------- discrete top-k, score variants, several heads, Inter-DRO
SCORE_PRODUCT, SCORE_PER_N, SCORE_PER_OMEGA2, SCORE_SMOOTHED, SCORE_ADDITIVE = 0, 1, 2, 3, 4
MAX_HEADS = 8


class TopkOutC(ctypes.Structure):
    _fields_ = [(n, _vp) for n in ("kth_logit", "n_above", "mass", "entropy", "S_lo", "S_up", "omega", "sigma",
                                   "score", "flag", "row_status", "indices")]


class ScoreParamsC(ctypes.Structure):
    _fields_ = [("variant", ctypes.c_int32), ("eps", ctypes.c_float), ("lambda1", ctypes.c_float),
                ("lambda2", ctypes.c_float), ("tau", ctypes.c_float)]


class InterDroParamsC(ctypes.Structure):
    _fields_ = [("radius_is_raw", ctypes.c_int32), ("r_max", ctypes.c_float), ("lambda_v", ctypes.c_float),
                ("lambda_p", ctypes.c_float), ("lambda_beta", ctypes.c_float), ("alpha", ctypes.c_float)]


class InterDroOutC(ctypes.Structure):
    _fields_ = [(n, _vp) for n in ("l1", "ce", "kl", "weights", "loss")]


_extras_ready = False


def _load_extras() -> ctypes.CDLL:
    global _extras_ready
    lib = load()
    if not _extras_ready:
        lib.ciar_quantify_topk.restype = ctypes.c_int
        lib.ciar_quantify_topk.argtypes = [ctypes.POINTER(LogitsDesc), _vp, ctypes.c_int32,
                                           ctypes.POINTER(IntervalParamsC), ctypes.POINTER(TopkOutC), _vp]
        lib.ciar_rescore.restype = ctypes.c_int
        lib.ciar_rescore.argtypes = [ctypes.c_int64, ctypes.c_int32, _vp, _vp, ctypes.POINTER(ScoreParamsC), _vp, _vp, _vp]
        lib.ciar_quantify_ensemble.restype = ctypes.c_int
        lib.ciar_quantify_ensemble.argtypes = [ctypes.POINTER(LogitsDesc), _vp, ctypes.c_int32, ctypes.c_int64,
                                               ctypes.POINTER(IntervalParamsC), ctypes.POINTER(QuantifyOutC), _vp]
        lib.ciar_vote.restype = ctypes.c_int
        lib.ciar_vote.argtypes = [ctypes.c_int32, ctypes.c_int64, _vp, _vp, _vp, _vp]
        lib.ciar_interdro_workspace_bytes.restype = ctypes.c_size_t
        lib.ciar_interdro_workspace_bytes.argtypes = [ctypes.c_int64]
        lib.ciar_interdro_forward.restype = ctypes.c_int
        lib.ciar_interdro_forward.argtypes = [ctypes.POINTER(LogitsDesc), _vp, _vp, _vp, ctypes.POINTER(InterDroParamsC),
                                              ctypes.POINTER(InterDroOutC), _vp, ctypes.c_size_t, _vp]
        _extras_ready = True
    return lib


_T_F32 = ("kth_logit", "mass", "entropy", "S_lo", "S_up", "omega", "sigma", "score")


@dataclass
class TopkOut:
    """Output tensors of ciar_quantify_topk; allocate() makes all of them."""
    kth_logit: Optional[torch.Tensor] = None
    n_above: Optional[torch.Tensor] = None
    mass: Optional[torch.Tensor] = None
    entropy: Optional[torch.Tensor] = None
    S_lo: Optional[torch.Tensor] = None
    S_up: Optional[torch.Tensor] = None
    omega: Optional[torch.Tensor] = None
    sigma: Optional[torch.Tensor] = None
    score: Optional[torch.Tensor] = None
    flag: Optional[torch.Tensor] = None
    row_status: Optional[torch.Tensor] = None
    indices: Optional[torch.Tensor] = None

    @classmethod
    def allocate(cls, rows: int, device, k: int = 0) -> "TopkOut":
        o = cls()
        for n in _T_F32:
            setattr(o, n, torch.empty(rows, dtype=torch.float32, device=device))
        o.n_above = torch.empty(rows, dtype=torch.int32, device=device)
        o.flag = torch.empty(rows, dtype=torch.uint8, device=device)
        o.row_status = torch.empty(rows, dtype=torch.uint8, device=device)
        if k:
            o.indices = torch.empty((rows, k), dtype=torch.int32, device=device)
        return o

    def to_c(self) -> TopkOutC:
        names = [f[0] for f in TopkOutC._fields_]
        _require_cuda(*[getattr(self, n) for n in names])
        return TopkOutC(*[_ptr(getattr(self, n)) for n in names])


def quantify_topk(logits: torch.Tensor, k: int, params: IntervalParams, out: TopkOut, valid_begin: int = 0,
                  valid_count: Optional[int] = None, stream=None) -> TopkOut:
    """ciar_quantify_topk: the discrete top-k quantifier of every row of ``logits``."""
    _require_cuda(logits)
    desc = make_desc(logits, valid_begin, valid_count)
    pc, oc = params.to_c(), out.to_c()
    st = _load_extras().ciar_quantify_topk(ctypes.byref(desc), _ptr(logits), int(k), ctypes.byref(pc), ctypes.byref(oc),
                                           _stream(stream))
    if st != 0:
        raise CiarError("ciar_quantify_topk", st)
    return out


def rescore(omega: torch.Tensor, sigma: torch.Tensor, n: int, variant: int, eps: float = 0.0, lambda1: float = 0.0,
            lambda2: float = 1.0, tau: float = 0.0, score_out: Optional[torch.Tensor] = None,
            flag_out: Optional[torch.Tensor] = None, stream=None) -> None:
    """ciar_rescore: a score variant and its flag from the omega / sigma arrays of ciar_quantify."""
    _require_cuda(omega, sigma, score_out, flag_out)
    pc = ScoreParamsC(int(variant), eps, lambda1, lambda2, tau)
    st = _load_extras().ciar_rescore(omega.numel(), int(n), _ptr(omega), _ptr(sigma), ctypes.byref(pc), _ptr(score_out),
                                     _ptr(flag_out), _stream(stream))
    if st != 0:
        raise CiarError("ciar_rescore", st)


def quantify_ensemble(heads: torch.Tensor, params: IntervalParams, out: QuantifyOut, valid_begin: int = 0,
                      valid_count: Optional[int] = None, stream=None) -> QuantifyOut:
    """ciar_quantify_ensemble: soft voting over ``heads`` ([H, rows, vocab], contiguous)."""
    _require_cuda(heads)
    if heads.dim() != 3 or not heads.is_contiguous():
        raise ValueError("heads must be a contiguous [H, rows, vocab] tensor")
    desc = make_desc(heads[0], valid_begin, valid_count)
    pc, oc = params.to_c(), out.to_c()
    st = _load_extras().ciar_quantify_ensemble(ctypes.byref(desc), _ptr(heads), heads.shape[0], heads.stride(0),
                                               ctypes.byref(pc), ctypes.byref(oc), _stream(stream))
    if st != 0:
        raise CiarError("ciar_quantify_ensemble", st)
    return out


def vote(flags: torch.Tensor, flag_out: torch.Tensor, votes_out: Optional[torch.Tensor] = None, stream=None) -> None:
    """ciar_vote: hard voting over flags uint8[H, rows]."""
    _require_cuda(flags, flag_out, votes_out)
    if flags.dim() != 2 or not flags.is_contiguous() or flags.dtype != torch.uint8:
        raise ValueError("flags must be a contiguous uint8 [H, rows] tensor")
    st = _load_extras().ciar_vote(flags.shape[0], flags.shape[1], _ptr(flags), _ptr(flag_out), _ptr(votes_out),
                                  _stream(stream))
    if st != 0:
        raise CiarError("ciar_vote", st)


@dataclass
class InterDroOut:
    l1: Optional[torch.Tensor] = None       # float32[3, rows]: mid, up, lo
    ce: Optional[torch.Tensor] = None       # float32[3, rows]
    kl: Optional[torch.Tensor] = None       # float32[rows]
    weights: Optional[torch.Tensor] = None  # float32[rows]
    loss: Optional[torch.Tensor] = None     # float32[6]: total, centre, upper, lower, dro, align

    @classmethod
    def allocate(cls, rows: int, device) -> "InterDroOut":
        f = lambda *s: torch.empty(s, dtype=torch.float32, device=device)
        return cls(f(3, rows), f(3, rows), f(rows), f(rows), f(6))


def interdro_workspace_bytes(rows: int) -> int:
    return int(_load_extras().ciar_interdro_workspace_bytes(rows))


def interdro_forward(center: torch.Tensor, radius: torch.Tensor, cloud: torch.Tensor, out: InterDroOut,
                     workspace: torch.Tensor, radius_is_raw: bool = True, r_max: float = 10.0, lambda_v: float = 1.0,
                     lambda_p: float = 1.0, lambda_beta: float = 1.0, alpha: float = 1.0, valid_begin: int = 0,
                     valid_count: Optional[int] = None, stream=None) -> InterDroOut:
    """ciar_interdro_forward: forward value of the Inter-DRO loss over the batch of rows."""
    _require_cuda(center, radius, cloud, workspace, out.l1, out.ce, out.kl, out.weights, out.loss)
    desc = make_desc(center, valid_begin, valid_count)
    pc = InterDroParamsC(int(radius_is_raw), r_max, lambda_v, lambda_p, lambda_beta, alpha)
    oc = InterDroOutC(_ptr(out.l1), _ptr(out.ce), _ptr(out.kl), _ptr(out.weights), _ptr(out.loss))
    st = _load_extras().ciar_interdro_forward(ctypes.byref(desc), _ptr(center), _ptr(radius), _ptr(cloud), ctypes.byref(pc),
                                              ctypes.byref(oc), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                              _stream(stream))
    if st != 0:
        raise CiarError("ciar_interdro_forward", st)
    return out
