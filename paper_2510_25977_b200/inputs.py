"""Seeded synthetic input generators shared by the tests, the benchmark and the oracle harness.

This module holds no arithmetic of the factored-MLP method itself: it only produces the
tensors the method consumes.  Every value is a pure function of (seed, tensor_id, flat index)
through a counter-based generator, so any slice can be regenerated on any device in any order:

    key   = splitmix64(seed * GOLDEN + tensor_id)
    bits  = splitmix64(key + (index + 1) * GOLDEN)                    (64 random bits)
    u1    = (bits >> 32) + 1) / 2^32   in (0, 1],   u2 = (bits & 0xffffffff) / 2^32
    g     = sqrt(-2 ln u1) * cos(2 pi u2)                             (Box-Muller, fp64)
    value = bf16_round_nearest_even(float32(g) * float32(scale))

Recipes (the value distributions named by the benchmark configurations):
  * "direct" factors (Llama-shaped configs):  V[r, in] ~ N(0, variance 1/in),
    U[out, r] ~ N(0, variance 1/r) * sigma_i with sigma_i = i^-1/2, i = 1..r along the rank axis.
  * "svd" factors (the tiny config): dense W ~ N(0, std 0.02) in fp32, LAPACK SVD on the host in
    fp64, keep the top r triplets, store U*diag(sigma) and V as bf16.
  * activations X ~ N(0, 1), bf16.
Tensor ids: Vg=0 Ug=1 Vu=2 Uu=3 Vd=4 Ud=5 X=6 Wg=7 Wu=8 Wd=9.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np
import torch

GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_MASK64 = (1 << 64) - 1

TID = {"Vg": 0, "Ug": 1, "Vu": 2, "Uu": 3, "Vd": 4, "Ud": 5, "X": 6, "Wg": 7, "Wu": 8, "Wd": 9}


def _s64(v: int) -> int:
    """Reinterpret an unsigned 64-bit constant as the signed value torch.int64 stores."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right on int64 (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _s64(_M1)
    z = (z ^ _lsr(z, 27)) * _s64(_M2)
    return z ^ _lsr(z, 31)


def _mix_int(z: int) -> int:
    z &= _MASK64
    z = ((z ^ (z >> 30)) * _M1) & _MASK64
    z = ((z ^ (z >> 27)) * _M2) & _MASK64
    return z ^ (z >> 31)


def random_bits(seed: int, tensor_id: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """64 random bits (as int64) for flat indices start .. start+count-1."""
    key = _mix_int(seed * GOLDEN + tensor_id)
    idx = torch.arange(start + 1, start + count + 1, dtype=torch.int64, device=device)
    return _mix(idx * _s64(GOLDEN) + _s64(key))


def standard_normal(seed: int, tensor_id: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """fp32 standard normal draws for a flat index range."""
    bits = random_bits(seed, tensor_id, start, count, device)
    hi = _lsr(bits, 32).to(torch.float64)
    lo = (bits & 0xFFFFFFFF).to(torch.float64)
    u1 = (hi + 1.0) * (1.0 / 4294967296.0)
    u2 = lo * (1.0 / 4294967296.0)
    g = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
    return g.to(torch.float32)


def normal_tensor(seed: int, tensor_id: int, shape, scale=1.0, col_scale: torch.Tensor | None = None,
                  dtype=torch.bfloat16, device="cpu", chunk: int = 1 << 24) -> torch.Tensor:
    """Row-major tensor of N(0, scale^2) draws (optionally times a per-column fp32 factor)."""
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=dtype, device=device)
    ncol = int(shape[-1])
    if col_scale is not None:
        col_scale = col_scale.to(device=device, dtype=torch.float32)
        chunk = max(ncol, (chunk // ncol) * ncol)
    for s in range(0, n, chunk):
        c = min(chunk, n - s)
        g = standard_normal(seed, tensor_id, s, c, device) * torch.tensor(scale, dtype=torch.float32, device=device)
        if col_scale is not None:
            g = (g.view(-1, ncol) * col_scale).view(-1)
        out[s:s + c] = g.to(dtype)
    return out.view(*shape)


@dataclass
class Factors:
    """The six row-major bf16 factor tensors of one SVD-factored SwiGLU MLP."""
    d: int
    ffn: int
    r_gate: int
    r_up: int
    r_down: int
    Ug: torch.Tensor  # [ffn, r_gate]
    Vg: torch.Tensor  # [r_gate, d]
    Uu: torch.Tensor  # [ffn, r_up]
    Vu: torch.Tensor  # [r_up, d]
    Ud: torch.Tensor  # [d, r_down]
    Vd: torch.Tensor  # [r_down, ffn]

    def tensors(self):
        return (self.Ug, self.Vg, self.Uu, self.Vu, self.Ud, self.Vd)

    def nbytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in self.tensors())


def _sigma(r: int) -> torch.Tensor:
    i = torch.arange(1, r + 1, dtype=torch.float64)
    return (i ** -0.5).to(torch.float32)


def direct_factors(d: int, ffn: int, r: int, seed: int = 0, device="cpu",
                   r_down: int | None = None) -> Factors:
    """Factors drawn directly from the seed (the Llama-shaped configurations)."""
    rd = r if r_down is None else r_down

    def V(tid, rr, n_in):
        return normal_tensor(seed, tid, (rr, n_in), scale=n_in ** -0.5, device=device)

    def U(tid, n_out, rr):
        return normal_tensor(seed, tid, (n_out, rr), scale=rr ** -0.5, col_scale=_sigma(rr), device=device)

    return Factors(d, ffn, r, r, rd,
                   Ug=U(TID["Ug"], ffn, r), Vg=V(TID["Vg"], r, d),
                   Uu=U(TID["Uu"], ffn, r), Vu=V(TID["Vu"], r, d),
                   Ud=U(TID["Ud"], d, rd), Vd=V(TID["Vd"], rd, ffn))


def dense_weights(d: int, ffn: int, seed: int = 0, std: float = 0.02):
    """Dense fp32 W_gate, W_up [ffn, d] and W_down [d, ffn] ~ N(0, std^2)."""
    Wg = normal_tensor(seed, TID["Wg"], (ffn, d), scale=std, dtype=torch.float32)
    Wu = normal_tensor(seed, TID["Wu"], (ffn, d), scale=std, dtype=torch.float32)
    Wd = normal_tensor(seed, TID["Wd"], (d, ffn), scale=std, dtype=torch.float32)
    return Wg, Wu, Wd


def svd_factors(d: int, ffn: int, r: int, seed: int = 0, std: float = 0.02, device="cpu") -> Factors:
    """Tiny-config recipe: dense weights -> host LAPACK SVD (fp64) -> top-r, stored as
    U*diag(sigma) and V in bf16."""
    out = {}
    for name, W in zip(("g", "u", "d"), dense_weights(d, ffn, seed, std)):
        Uf, S, Vt = np.linalg.svd(W.numpy().astype(np.float64), full_matrices=False)
        out["U" + name] = torch.from_numpy((Uf[:, :r] * S[:r]).astype(np.float32)).to(torch.bfloat16).to(device)
        out["V" + name] = torch.from_numpy(Vt[:r, :].astype(np.float32)).to(torch.bfloat16).to(device)
    return Factors(d, ffn, r, r, r, out["Ug"], out["Vg"], out["Uu"], out["Vu"], out["Ud"], out["Vd"])


def activations(T: int, d: int, seed: int = 0, device="cpu") -> torch.Tensor:
    """X[T, d] ~ N(0, 1), bf16."""
    return normal_tensor(seed, TID["X"], (T, d), scale=1.0, device=device)


# The five benchmark configurations (shapes only; values come from the recipes above).
CONFIGS = {
    "cfg1": dict(d=256, ffn=688, r=(32,), T=(16,), recipe="svd", layers=1),
    "cfg2": dict(d=4096, ffn=11008, r=(256,), T=(1, 4, 8, 32), recipe="direct", layers=1),
    "cfg3": dict(d=4096, ffn=11008, r=(256,), T=(512, 2048, 4096), recipe="direct", layers=1),
    "cfg4": dict(d=4096, ffn=14336, r=(128, 512, 1024), T=(1, 8, 128, 2048, 8192), recipe="direct", layers=1),
    "cfg5": dict(d=5120, ffn=13824, r=(320,), T=(1, 1024), recipe="direct", layers=40),
}


def sample_rows(T: int, tile: int = 128, max_rows: int = 64) -> list[int]:
    """Token rows for sampled parity at large T: first/last row of several tiles plus the tail."""
    rows = {0, T - 1}
    ntile = (T + tile - 1) // tile
    picks = sorted({0, 1, ntile // 2, ntile - 2, ntile - 1} & set(range(ntile)))
    for m in picks:
        lo, hi = m * tile, min(T, (m + 1) * tile) - 1
        rows.update({lo, hi, (lo + hi) // 2, min(hi, lo + 37)})
    rows = sorted(r for r in rows if 0 <= r < T)
    return rows[:max_rows]


def rows_of_every_tile(T: int, tile: int = 128, per_tile: int = 2) -> list[int]:
    """Token rows for sampled parity at the largest T: `per_tile` rows of EVERY `tile`-row tile (a position
    that moves from tile to tile, plus the tile's last row), so that a fault tied to the n-th tile a
    persistent CTA walks cannot hide between samples."""
    rows = set()
    for m in range((T + tile - 1) // tile):
        lo, hi = m * tile, min(T, (m + 1) * tile) - 1
        rows.add(hi)
        for j in range(per_tile - 1):
            rows.add(lo + (m * 37 + j * 53) % (hi - lo + 1))
    return sorted(rows)
