"""Seeded synthetic inputs shaped like the paper's LlamaGen / Anole workloads.

This module only MAKES inputs (logits, radii, drafted tokens, uniforms).  It holds none of
the method's arithmetic: no softmax, no interval, no score, no acceptance test.  Both the
CUDA path's tests / benchmark and the CPU oracle's tests read the tensors produced here,
byte for byte, so neither side ever sees an input the other made.

Recipe (every workload):
  * blob field: per image an h x w grid g(y,x) = sum of 6 Gaussian bumps (centres uniform
    in the grid, widths in [h/8, h/3], amplitudes in [0.5, 1]); the 30 % of cells whose g
    is closest to the image's median level are "boundary" tokens (scale 1, flat logits,
    radius 1.0); the rest are "interior" tokens (scale 8, peaked logits, radius 0.05).
  * draft logits: scale * N(0,1) per code (Zipf-shaped -1.1*scale*ln(rank) under a per-row
    affine permutation for the large-vocabulary stress workload), cast to the dtype.
  * target logits: draft (as stored) + N(0, sigma^2), cast to the dtype.
  * drafted tokens: a sample of the draft distribution drawn with the Gumbel-max trick
    (argmax of logits + Gumbel noise), which needs no softmax.
  * uniforms: Philox4x32-10, key = seed, counter = row; lanes 0,1,2 -> u_accept,
    u_resample, u_flag; u = (bits >> 8) * 2^-24, so u is in [0, 1).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Optional

import torch

_M32 = 0xFFFFFFFF
_PHILOX_M0, _PHILOX_M1 = 0xD2511F53, 0xCD9E8D57
_PHILOX_W0, _PHILOX_W1 = 0x9E3779B9, 0xBB67AE85


def _mulhilo(a: torch.Tensor, m: int):
    """32x32 -> (hi, lo) product of uint32 values held in int64 tensors."""
    m_lo, m_hi = m & 0xFFFF, m >> 16
    a_lo, a_hi = a & 0xFFFF, a >> 16
    ll = a_lo * m_lo
    lh = a_lo * m_hi
    hl = a_hi * m_lo
    hh = a_hi * m_hi
    mid = (ll >> 16) + (lh & 0xFFFF) + (hl & 0xFFFF)
    lo = ((mid & 0xFFFF) << 16) | (ll & 0xFFFF)
    hi = hh + (lh >> 16) + (hl >> 16) + (mid >> 16)
    return hi & _M32, lo & _M32


def philox4x32_10(counter, key):
    """Philox4x32 with 10 rounds (Salmon et al., 'Parallel random numbers: as easy as 1, 2, 3').
    counter: four int64 tensors holding uint32 words; key: two Python ints (uint32).
    Returns four int64 tensors holding uint32 words."""
    c0, c1, c2, c3 = [c.to(torch.int64) & _M32 for c in counter]
    k0, k1 = key[0] & _M32, key[1] & _M32
    for _ in range(10):
        hi0, lo0 = _mulhilo(c0, _PHILOX_M0)
        hi1, lo1 = _mulhilo(c2, _PHILOX_M1)
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & _M32, lo1, (hi0 ^ c3 ^ k1) & _M32, lo0
        k0, k1 = (k0 + _PHILOX_W0) & _M32, (k1 + _PHILOX_W1) & _M32
    return c0, c1, c2, c3


def philox_uniforms(rows: int, seed: int, device="cpu", row_offset: int = 0):
    """u_accept, u_resample, u_flag: float32[rows] in [0, 1), identical on every device."""
    idx = torch.arange(row_offset, row_offset + rows, dtype=torch.int64, device=device)
    zero = torch.zeros_like(idx)
    w = philox4x32_10((idx & _M32, idx >> 32, zero, zero), (seed & _M32, (seed >> 32) & _M32))
    return tuple(((x >> 8).to(torch.float32) * (1.0 / 16777216.0)) for x in w[:3])


@dataclass(frozen=True)
class Workload:
    """One synthetic workload.  rows = images * grid_h * grid_w; a draft window never
    straddles two images (grid_h * grid_w is a multiple of the window)."""
    name: str
    images: int
    grid_h: int
    grid_w: int
    vocab: int  # row stride in codes
    dtype: str  # "f32" | "bf16"
    window: int
    sigma_target: float = 0.5
    valid_begin: int = 0
    valid_count: Optional[int] = None  # None = whole row
    zipf: bool = False
    seed: int = 0
    boundary_frac: float = 0.30
    scale_interior: float = 8.0
    scale_boundary: float = 1.0
    r_interior: float = 0.05
    r_boundary: float = 1.0
    tau: float = 1e-4  # interval-score threshold frozen for this workload (between the two classes)
    decode: bool = False  # rows are a [requests, seq_len] pool for the decode loop
    philox_seed: int = 0  # key of the Philox stream the uniforms come from

    @property
    def rows(self) -> int:
        return self.images * self.grid_h * self.grid_w

    @property
    def tokens_per_image(self) -> int:
        return self.grid_h * self.grid_w

    @property
    def n_valid(self) -> int:
        return self.vocab - self.valid_begin if self.valid_count is None else self.valid_count

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five workloads of the build's problem statement.  tau values were frozen from the CPU
# oracle's scores on these recipes (geometric middle of the gap between the interior and the
# boundary class; see tests/golden/tau_calibration.txt and the script beside it).
WORKLOADS = {
    "llamagen256": Workload("llamagen256", 1, 16, 16, 16384, "f32", 8, 0.5, seed=1),
    "llamagen384": Workload("llamagen384", 16, 24, 24, 16384, "bf16", 16, 0.5, seed=2),
    "anole": Workload("anole", 8, 32, 32, 65536, "bf16", 8, 0.3, valid_begin=32768, valid_count=8192, seed=3),
    "largevocab": Workload("largevocab", 64, 32, 32, 262144, "bf16", 8, 0.5, zipf=True, seed=4),
    "decode": Workload("decode", 256, 32, 32, 16384, "bf16", 8, 0.5, seed=5, decode=True),
}


def blob_boundary_mask(wl: Workload) -> torch.Tensor:
    """bool[images, h*w]: True on boundary tokens (exactly round(frac*h*w) per image). CPU tensor."""
    g = torch.Generator(device="cpu")
    g.manual_seed(1000003 * wl.seed + 17)
    h, w = wl.grid_h, wl.grid_w
    nb = 6
    cy = torch.rand(wl.images, nb, generator=g, dtype=torch.float64) * h
    cx = torch.rand(wl.images, nb, generator=g, dtype=torch.float64) * w
    sg = (h / 8.0) + torch.rand(wl.images, nb, generator=g, dtype=torch.float64) * (h / 3.0 - h / 8.0)
    am = 0.5 + 0.5 * torch.rand(wl.images, nb, generator=g, dtype=torch.float64)
    yy = torch.arange(h, dtype=torch.float64).view(1, 1, h, 1) + 0.5
    xx = torch.arange(w, dtype=torch.float64).view(1, 1, 1, w) + 0.5
    d2 = (yy - cy.view(-1, nb, 1, 1)) ** 2 + (xx - cx.view(-1, nb, 1, 1)) ** 2
    field = (am.view(-1, nb, 1, 1) * torch.exp(-d2 / (2.0 * sg.view(-1, nb, 1, 1) ** 2))).sum(1)
    field = field.reshape(wl.images, h * w)
    level = field.median(dim=1, keepdim=True).values
    dist = (field - level).abs()
    k = max(0, min(h * w, int(round(wl.boundary_frac * h * w))))
    mask = torch.zeros(wl.images, h * w, dtype=torch.bool)
    if k > 0:
        idx = torch.argsort(dist, dim=1, stable=True)[:, :k]
        mask.scatter_(1, idx, True)
    return mask


@dataclass
class Inputs:
    workload: Workload
    draft: torch.Tensor  # [rows, vocab]
    target: torch.Tensor  # [rows, vocab]
    tokens: torch.Tensor  # int32[rows], global code ids
    boundary: torch.Tensor  # bool[rows]
    radius_row: torch.Tensor  # float32[rows]
    u_accept: torch.Tensor  # float32[rows]
    u_resample: torch.Tensor
    u_flag: torch.Tensor
    radius_code: Optional[torch.Tensor] = None  # [rows, vocab] raw (pre-softplus) radii, logits' dtype


def _rows_per_chunk(wl: Workload, budget_bytes: int = 1 << 29) -> int:
    return max(1, min(wl.rows, budget_bytes // (wl.vocab * 8)))


def make_inputs(wl: Workload, device="cpu", per_code_radius: bool = False, row_limit: Optional[int] = None) -> Inputs:
    """Generate a workload's tensors on ``device``.  ``row_limit`` keeps only the first rows
    (a whole number of windows) -- used for bounded samples of a large workload."""
    dev = torch.device(device)
    rows = wl.rows
    if row_limit is not None:
        rows = min(rows, row_limit)
        rows -= rows % wl.window
    gen = torch.Generator(device=dev)
    gen.manual_seed(7919 * wl.seed + 3)
    boundary = blob_boundary_mask(wl).reshape(-1)[:rows].to(dev)
    scale = torch.where(boundary, torch.tensor(wl.scale_boundary), torch.tensor(wl.scale_interior)).to(dev)
    scale = scale.to(torch.float32)
    radius_row = torch.where(boundary, torch.tensor(wl.r_boundary), torch.tensor(wl.r_interior)).to(torch.float32)
    radius_row = radius_row.to(dev)
    dt = wl.torch_dtype
    vb, n = wl.valid_begin, wl.n_valid
    neg_inf = float("-inf")
    draft = torch.full((rows, wl.vocab), neg_inf, dtype=dt, device=dev)
    target = torch.full((rows, wl.vocab), neg_inf, dtype=dt, device=dev)
    tokens = torch.empty(rows, dtype=torch.int32, device=dev)
    radius_code = torch.zeros((rows, wl.vocab), dtype=dt, device=dev) if per_code_radius else None
    step = _rows_per_chunk(wl)
    if wl.zipf:
        # per-row affine permutation of the ranks: rank(j) = ((a*j + b) mod n) + 1, a odd, n a power of two
        assert n & (n - 1) == 0, "the Zipf recipe needs a power-of-two valid width"
        a_row = (torch.randint(0, n // 2, (rows,), generator=gen, device=dev, dtype=torch.int64) * 2 + 1)
        b_row = torch.randint(0, n, (rows,), generator=gen, device=dev, dtype=torch.int64)
        code = torch.arange(n, device=dev, dtype=torch.int64)
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        if wl.zipf:
            rank = ((a_row[r0:r1, None] * code[None, :] + b_row[r0:r1, None]) & (n - 1)) + 1
            c = scale[r0:r1, None] * (-1.1 * torch.log(rank.to(torch.float32)))
            del rank
        else:
            c = scale[r0:r1, None] * torch.randn((r1 - r0, n), generator=gen, device=dev, dtype=torch.float32)
        c_st = c.to(dt)
        draft[r0:r1, vb:vb + n] = c_st
        c = c_st.to(torch.float32)
        t = c + wl.sigma_target * torch.randn((r1 - r0, n), generator=gen, device=dev, dtype=torch.float32)
        target[r0:r1, vb:vb + n] = t.to(dt)
        del t
        u = torch.rand((r1 - r0, n), generator=gen, device=dev, dtype=torch.float32).clamp_(1e-12, 1.0 - 1e-7)
        gumbel = -torch.log(-torch.log(u))
        tokens[r0:r1] = (torch.argmax(c + gumbel, dim=1) + vb).to(torch.int32)
        del u, gumbel, c
        if per_code_radius:
            base = torch.log(torch.expm1(radius_row[r0:r1]))  # inverse softplus of the row's radius
            rho = base[:, None] + 0.25 * torch.randn((r1 - r0, n), generator=gen, device=dev, dtype=torch.float32)
            radius_code[r0:r1, vb:vb + n] = rho.to(dt)
            del rho
    ua, ur, uf = philox_uniforms(rows, wl.philox_seed, device=dev)
    return Inputs(wl, draft, target, tokens, boundary, radius_row, ua, ur, uf, radius_code)


def algorithmic_bytes(wl: Workload, rows: int, sent_rows: int, resample_rows: int, per_code_radius: bool = False) -> int:
    """Bytes the method must move for one quantify+verify pass: every draft row once (twice the
    width with per-code radii), the target row of every row sent to the cloud, and draft + target
    once more for each resampled row; plus the small per-row / per-window outputs."""
    row_bytes = wl.n_valid * wl.elem_bytes
    q = rows * row_bytes * (2 if per_code_radius else 1)
    v = sent_rows * row_bytes + resample_rows * 2 * row_bytes
    small = rows * 64 + (rows // wl.window) * 16
    return q + v + small
