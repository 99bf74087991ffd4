"""Seeded synthetic inputs for the SALAD attention path.

This module only *generates inputs* (tensors, scale parameters, irregular block lists, trivial
all-kept lists).  It contains none of the method's arithmetic, and it is the one
module that both the CPU oracle's callers and the GPU library's callers may use, so that
both sides see bit-identical operands.  It needs numpy and torch (CPU) only.

The tensors stand in for the Q/K/V activations of a Wan2.1-style video DiT (Sec. 5.1
setup: 1.3B model, 12 heads of 128 channels, 21 x 30 x 52 latent tokens at 480p; 14B-shaped
layer with 40 heads), which are not available offline.  "Local blocks dominate" is modelled
by adding to i.i.d. N(0,1) noise a smooth spatio-temporal field that Q and K share.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Optional, Sequence, Tuple

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    d: int
    grid: Tuple[int, int, int]          # (T, Hs, Ws); tokens row-major, time slowest
    Bq: int
    Bk: int
    windows: Tuple[Tuple[int, int, int], ...]  # one (wt, wh, ww) per mask head (Hm = len)
    seed: int
    smooth: bool = True                 # add the shared low-frequency field
    noise_scale: float = 1.0
    irregular: bool = False             # per-head random block lists instead of windows

    @property
    def N(self) -> int:
        T, Hs, Ws = self.grid
        return T * Hs * Ws

    @property
    def nQb(self) -> int:
        return -(-self.N // self.Bq)

    @property
    def nKb(self) -> int:
        return -(-self.N // self.Bk)

    @property
    def Hm(self) -> int:
        return self.H if self.irregular else len(self.windows)


# The five configurations of the benchmark spec.  Window sizes were chosen so that the
# block sparsity 1 - nnz/(nQb*nKb) lands on the stated percentages.
C1 = Workload("tiny", 1, 2, 64, (4, 16, 16), 64, 64, ((0, 15, 15), (3, 0, 0)), 1001,
              smooth=False, noise_scale=0.5)
C2 = Workload("wan1.3b-90", 1, 12, 128, (21, 30, 52), 128, 64, ((2, 5, 24),), 1002)
C3 = Workload("wan1.3b-irregular", 1, 12, 128, (21, 30, 52), 128, 64, (), 1003, irregular=True)
C4 = Workload("wan14b-90", 1, 40, 128, (21, 45, 80), 128, 64, ((2, 10, 36),), 1004)
C5_80 = Workload("cfg-80", 2, 12, 128, (21, 30, 52), 128, 64, ((5, 5, 24),), 1005)
C5_90 = replace(C5_80, name="cfg-90", windows=((2, 5, 24),))
C5_95 = replace(C5_80, name="cfg-95", windows=((1, 4, 24),))
C5_DENSE = replace(C5_80, name="cfg-dense", windows=((21, 30, 52),))
# Not one of the five: the 1.3B model at the higher resolution the paper also reports (Sec. 5.1), i.e.
# its 12 heads on the 21 x 45 x 80 latent grid (75 600 tokens), same window as the 14B-shaped config.
C6 = Workload("wan1.3b-720p-90", 1, 12, 128, (21, 45, 80), 128, 64, ((2, 10, 36),), 1006)
ALL = {w.name: w for w in (C1, C2, C3, C4, C5_80, C5_90, C5_95, C5_DENSE, C6)}


def _smooth_field(rng: np.random.Generator, grid, d: int) -> np.ndarray:
    """[N, d] field  S_c(t,h,w) = 1/4 sum_{m<4} sin(2 pi (ft t/T + fh h/Hs + fw w/Ws) + psi_{c,m})."""
    T, Hs, Ws = grid
    N = T * Hs * Ws
    n = np.arange(N)
    t, h, w = n // (Hs * Ws), (n // Ws) % Hs, n % Ws
    basis = np.empty((N, 8), dtype=np.float32)
    mix = np.empty((8, d), dtype=np.float32)
    for m in range(4):
        while True:
            f = rng.integers(0, 4, size=3)
            if f.any():
                break
        ang = 2.0 * np.pi * (f[0] * t / T + f[1] * h / Hs + f[2] * w / Ws)
        psi = rng.uniform(0.0, 2.0 * np.pi, size=d)
        # sin(a + psi) = sin a cos psi + cos a sin psi
        basis[:, 2 * m] = np.sin(ang); basis[:, 2 * m + 1] = np.cos(ang)
        mix[2 * m] = np.cos(psi); mix[2 * m + 1] = np.sin(psi)
    return 0.25 * (basis @ mix)


def make_qkv(wl: Workload, heads: Optional[Sequence[int]] = None):
    """Q, K, V as bf16 CPU tensors [B, H', N, d] (H' = len(heads) if given, else H).

    Every (batch, head) slice is drawn from its own child generator, so a subset of heads
    reproduces exactly the corresponding slices of the full tensor.
    """
    hs = list(range(wl.H)) if heads is None else list(heads)
    N, d = wl.N, wl.d
    out = [torch.empty((wl.B, len(hs), N, d), dtype=torch.bfloat16) for _ in range(3)]
    for b in range(wl.B):
        for hi, h in enumerate(hs):
            rng = np.random.default_rng([wl.seed, b, h])
            qkv = [rng.standard_normal((N, d), dtype=np.float32) * np.float32(wl.noise_scale)
                   for _ in range(3)]
            if wl.smooth:
                s_qk = _smooth_field(rng, wl.grid, d)
                s_v = _smooth_field(rng, wl.grid, d)
                qkv[0] += s_qk; qkv[1] += s_qk; qkv[2] += s_v
            for t, a in zip(out, qkv):
                t[b, hi] = torch.from_numpy(a).to(torch.bfloat16)
    return tuple(out)


def make_scales(wl: Workload):
    """(lambda_h [H] ~ U(0,1), s_b [B] = sigmoid(N(0,1))) as float32 numpy arrays."""
    rng = np.random.default_rng([wl.seed, 777])
    lam = rng.uniform(0.0, 1.0, size=wl.H).astype(np.float32)
    s = (1.0 / (1.0 + np.exp(-rng.standard_normal(wl.B)))).astype(np.float32)
    return lam, s


def irregular_csr(wl: Workload, lo_frac: float = 0.05, hi_frac: float = 0.15):
    """Per-head random block lists: each query block keeps the key blocks that overlap its
    own tokens plus uniformly sampled others; the row length is uniform in
    [lo_frac, hi_frac] * nKb.  Returns (row_ptr [H*nQb+1], col_idx) int32, ascending rows."""
    rng = np.random.default_rng([wl.seed, 333])
    nQb, nKb = wl.nQb, wl.nKb
    lo, hi = int(round(lo_frac * nKb)), int(round(hi_frac * nKb))
    row_ptr = [0]
    cols = []
    for h in range(wl.H):
        for i in range(nQb):
            first = (i * wl.Bq) // wl.Bk
            last = min(wl.N, (i + 1) * wl.Bq) - 1
            diag = np.arange(first, last // wl.Bk + 1)
            c = int(rng.integers(lo, hi + 1))
            others = np.setdiff1d(np.arange(nKb), diag)
            extra = rng.choice(others, size=max(0, min(c, nKb) - diag.size), replace=False)
            row = np.sort(np.concatenate([diag, extra]))
            cols.append(row)
            row_ptr.append(row_ptr[-1] + row.size)
    return np.asarray(row_ptr, dtype=np.int32), np.concatenate(cols).astype(np.int32)


def dense_csr(nQb: int, nKb: int, Hm: int = 1):
    """All-kept lists (0 % sparsity): every query block keeps every key block."""
    row_ptr = (np.arange(Hm * nQb + 1, dtype=np.int64) * nKb).astype(np.int32)
    col_idx = np.tile(np.arange(nKb, dtype=np.int32), Hm * nQb)
    return row_ptr, col_idx


def sample_rows(wl: Workload, count: int, seed: int = 0, H: Optional[int] = None) -> np.ndarray:
    """Flat output-row indices (b*H + h)*N + n for sampled parity checks: always the first
    and last query block's edge rows of every head, the rest uniform."""
    H = wl.H if H is None else H
    rng = np.random.default_rng([wl.seed, 555, seed])
    N = wl.N
    fixed = []
    for bh in range(wl.B * H):
        for n in (0, wl.Bq - 1, wl.Bq, N - 1, (wl.nQb - 1) * wl.Bq):
            fixed.append(bh * N + min(max(n, 0), N - 1))
    rest = rng.integers(0, wl.B * H * N, size=max(0, count - len(fixed)))
    return np.unique(np.concatenate([np.asarray(fixed, dtype=np.int64), rest.astype(np.int64)]))
