"""Seeded synthetic HGEMM inputs, shared by the tests, the bench and the smoke check.

This module holds no GEMM arithmetic: it only draws fp16 matrices.  The paper's
workload is itself synthetic random matrices over a grid of (M, N, K) (abstract;
section 2.3 "Exact Match"; appendix Listing 8 draws fresh random inputs per round),
so nothing here stands in for a dataset.

The generator is stateless and counter-based: element (r, c) of a matrix depends
only on (seed, tag, r * cols + c), so any subset of rows can be drawn on its own
(the sampled checks of large shapes draw only the rows they need).  All integer
work is wrapping int64 arithmetic and every floating-point intermediate of the
uniform and integer draws is exact in fp32, so CPU and CUDA devices produce the
same bits.  The normal draw uses log/cos and is therefore host-only.

Distributions (value distributions of the five workload families):
  "uniform": 24 random bits k -> k * 2^-23 - 1 in [-1, 1), rounded to fp16 (RNE)
  "int5"   : uniform over {-2, -1, 0, 1, 2}      (sums exact in fp32 -> bit-exact checks)
  "binary" : Bernoulli(p) over {0, 1}            (the paper's exact-match inputs)
  "normal" : N(0, 1) * cols^-1/2 by Box-Muller in fp64, rounded to fp16 (host only)
"""
from __future__ import annotations

import math

import numpy as np
import torch

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_MUL1 = 0xBF58476D1CE4E5B9
_MUL2 = 0x94D049BB133111EB

TAG_A = 0xA
TAG_B = 0xB


def _s64(x: int) -> int:
    """Python int (mod 2^64) as the signed value int64 tensors hold."""
    x &= _MASK64
    return x - (1 << 64) if x >> 63 else x


def _splitmix64_int(x: int) -> int:
    x = (x + _GOLDEN) & _MASK64
    z = x
    z = ((z ^ (z >> 30)) * _MUL1) & _MASK64
    z = ((z ^ (z >> 27)) * _MUL2) & _MASK64
    return z ^ (z >> 31)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    return (z >> s) & ((1 << (64 - s)) - 1)


def _splitmix64(x: torch.Tensor) -> torch.Tensor:
    z = x + _s64(_GOLDEN)
    z = (z ^ _lsr(z, 30)) * _s64(_MUL1)
    z = (z ^ _lsr(z, 27)) * _s64(_MUL2)
    return z ^ _lsr(z, 31)


def shape_seed(M: int, N: int, K: int) -> int:
    """Seed of a grid shape ("seeded by shape")."""
    return _splitmix64_int(0x4847454D4D ^ (M << 42) ^ (N << 21) ^ K)


def draw(seed: int, tag: int, rows: int, cols: int, dist: str = "uniform", device="cpu",
         row_index=None, p: float = 0.5, chunk_rows: int | None = None) -> torch.Tensor:
    """fp16 matrix of shape (rows, cols) -- or (len(row_index), cols) holding those rows of it.

    ``tag`` separates the A and B streams of one seed.  Generated in row chunks so that
    the int64 temporaries stay small next to the result.
    """
    device = torch.device(device)
    if dist == "normal" and device.type != "cpu":
        raise ValueError("the normal draw is host-only (log/cos differ between devices)")
    base = _s64(_splitmix64_int((seed ^ (tag * 0xD1B54A32D192ED03)) & _MASK64))
    if row_index is None:
        ridx = torch.arange(rows, dtype=torch.int64, device=device)
    else:
        ridx = torch.as_tensor(row_index, dtype=torch.int64, device=device)
        if ridx.numel() and (int(ridx.min()) < 0 or int(ridx.max()) >= rows):
            raise IndexError("row_index out of range")
    nrow = ridx.numel()
    out = torch.empty((nrow, cols), dtype=torch.float16, device=device)
    if nrow == 0 or cols == 0:
        return out
    if chunk_rows is None:
        chunk_rows = max(1, (1 << 22) // max(cols, 1))
    cidx = torch.arange(cols, dtype=torch.int64, device=device)
    for r0 in range(0, nrow, chunk_rows):
        rr = ridx[r0:r0 + chunk_rows]
        ctr = rr[:, None] * cols + cidx[None, :]
        x = _splitmix64(ctr + base)
        if dist == "uniform":
            k = _lsr(x, 40).to(torch.float32)
            v = (k * (2.0 ** -23) - 1.0).to(torch.float16)
        elif dist == "int5":
            v = (_lsr(x, 40) % 5 - 2).to(torch.float16)
        elif dist == "binary":
            thr = int(round(p * (1 << 24)))
            v = (_lsr(x, 40) < thr).to(torch.float16)
        elif dist == "normal":
            x2 = _splitmix64(x)
            u1 = (_lsr(x, 11).to(torch.float64) + 1.0) * (2.0 ** -53)
            u2 = _lsr(x2, 11).to(torch.float64) * (2.0 ** -53)
            z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos(2.0 * math.pi * u2) / math.sqrt(cols)
            v = torch.from_numpy(z.numpy().astype(np.float16))  # numpy rounds fp64 -> fp16 once, RNE
        else:
            raise ValueError(f"unknown distribution {dist!r}")
        out[r0:r0 + chunk_rows] = v
    return out


def make_ab(M: int, N: int, K: int, dist: str = "uniform", device="cpu", seed: int | None = None, **kw):
    """(A, B): A is M x K row-major, B is N x K K-contiguous, both fp16, seeded by the shape."""
    s = shape_seed(M, N, K) if seed is None else seed
    return (draw(s, TAG_A, M, K, dist, device, **kw), draw(s, TAG_B, N, K, dist, device, **kw))


def binary_p(K: int) -> float:
    """Bernoulli parameter of the paper-style {0,1} test: keeps E[c_ij] = K p^2 near 1024 for
    large K, so that most outputs are positive and below the fp16 exact-integer limit."""
    return min(0.5, math.sqrt(1024.0 / K))


def bits(t: torch.Tensor) -> np.ndarray:
    """uint16 bit patterns of an fp16 tensor, on the host."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def sample_indices(seed: int, M: int, N: int, n: int = 4096):
    """The sampled check of a large shape: n seeded (i, j) pairs, one seeded row, one seeded column."""
    rng = np.random.Generator(np.random.Philox(key=seed & _MASK64))
    ii = rng.integers(0, M, size=n, dtype=np.int64)
    jj = rng.integers(0, N, size=n, dtype=np.int64)
    row = int(rng.integers(0, M))
    col = int(rng.integers(0, N))
    return ii, jj, row, col
