"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds no arithmetic of the verifier: it only draws operands,
forms a CPU stand-in for the FP32-output GEMM under test, and writes faults
into a finished product.  Both the CUDA path's tests and the CPU oracle's tests
draw their inputs here so that they see the same arrays.

Data recipes (seeded, numpy PCG64):
  "uniform"      A, B ~ U(-1, 1)                       (square FP16 products)
  "gauss_scaled" A ~ N(0,1), B ~ N(0, sd 1/sqrt(n2))   (square BF16 product, rms(C) ~ 1)
  "transformer"  A ~ N(0,1), B ~ N(0, sd 0.02)         (Llama-2-7B-like layer shapes)
  "gauss"        A, B ~ N(0,1)                         (noise / probe-cost sweep)
  "integer"      A, B integers in [-lim, lim]          (exact-arithmetic brute-force cases)
Operands are rounded to FP16 / BF16 with round-to-nearest-even.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass
from typing import List, Sequence, Tuple

import numpy as np
import torch

FP16, BF16 = 0, 1
TORCH_DTYPE = {FP16: torch.float16, BF16: torch.bfloat16}

# (tokens, n2, n3) of the Llama-2-7B-like layer set: Q/K/V/O, gate/up, down
TRANSFORMER_SHAPES = [(t, k, n) for t in (2048, 4096)
                      for (k, n) in ((4096, 4096), (4096, 11008), (11008, 4096))]


def _rng(tag: str, seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([zlib.crc32(tag.encode()), seed & 0xFFFFFFFF, seed >> 32]))


def operands(kind: str, n1: int, n2: int, n3: int, dtype: int, seed: int,
             lim: int = 4) -> Tuple[torch.Tensor, torch.Tensor]:
    """A (n1 x n2) and B (n2 x n3) as CPU tensors of the half-precision operand type."""
    ga, gb = _rng(kind + "/A", seed), _rng(kind + "/B", seed)
    if kind == "uniform":
        a = ga.uniform(-1.0, 1.0, (n1, n2)).astype(np.float32)
        b = gb.uniform(-1.0, 1.0, (n2, n3)).astype(np.float32)
    elif kind == "gauss_scaled":
        a = ga.standard_normal((n1, n2), dtype=np.float32)
        b = gb.standard_normal((n2, n3), dtype=np.float32) * np.float32(1.0 / np.sqrt(n2))
    elif kind == "transformer":
        a = ga.standard_normal((n1, n2), dtype=np.float32)
        b = gb.standard_normal((n2, n3), dtype=np.float32) * np.float32(0.02)
    elif kind == "gauss":
        a = ga.standard_normal((n1, n2), dtype=np.float32)
        b = gb.standard_normal((n2, n3), dtype=np.float32)
    elif kind == "integer":
        a = ga.integers(-lim, lim + 1, (n1, n2)).astype(np.float32)
        b = gb.integers(-lim, lim + 1, (n2, n3)).astype(np.float32)
    else:
        raise ValueError(kind)
    td = TORCH_DTYPE[dtype]
    return torch.from_numpy(a).to(td), torch.from_numpy(b).to(td)


def cpu_fp32_product(A: torch.Tensor, B: torch.Tensor) -> torch.Tensor:
    """CPU stand-in for the GEMM under test: half operands, FP32 accumulation and delivery."""
    return A.float() @ B.float()


def rms(C: torch.Tensor) -> float:
    return float(torch.sqrt(torch.mean(C.double() ** 2)))


@dataclass
class InjectedFault:
    i: int
    j: int
    kind: str          # "add" (C_ij += value) or "scale" (C_ij *= 2^value)
    value: float
    population: str    # "typical", "small", "expflip"


def _distinct_coords(g: np.random.Generator, n1: int, n3: int, count: int, taken=()) -> List[Tuple[int, int]]:
    seen = set(taken)
    out = []
    while len(out) < count:
        c = (int(g.integers(0, n1)), int(g.integers(0, n3)))
        if c not in seen:
            seen.add(c)
            out.append(c)
    return out


def faults_additive(n1: int, n3: int, rms_c: float, seed: int, count: int,
                    lo: float, hi: float, population: str, taken=()) -> List[InjectedFault]:
    """`count` additive faults at distinct seeded coordinates, |delta| ~ U[lo,hi] * rms(C),
    seeded sign."""
    g = _rng("faults/" + population, seed)
    coords = _distinct_coords(g, n1, n3, count, taken)
    out = []
    for (i, j) in coords:
        mag = float(g.uniform(lo, hi)) * rms_c
        sgn = 1.0 if g.integers(0, 2) == 0 else -1.0
        out.append(InjectedFault(i, j, "add", sgn * mag, population))
    return out


def faults_shared_lines(n1: int, n3: int, seed: int, total: int = 16,
                        share_row: int = 4, share_col: int = 3) -> List[Tuple[int, int]]:
    """`total` distinct coordinates of which `share_row` lie on one row and `share_col`
    on one column (simultaneous faults forced to share a line)."""
    g = _rng("faults/shared", seed)
    coords: List[Tuple[int, int]] = []
    row = int(g.integers(0, n1))
    cols = g.choice(n3, size=share_row, replace=False)
    coords += [(row, int(c)) for c in cols]
    col = int(g.integers(0, n3))
    while any(c[1] == col for c in coords):
        col = int(g.integers(0, n3))
    rows = []
    while len(rows) < share_col:
        r_ = int(g.integers(0, n1))
        if r_ != row and r_ not in rows:
            rows.append(r_)
    coords += [(r_, col) for r_ in rows]
    coords += _distinct_coords(g, n1, n3, total - len(coords), coords)
    return coords


def faults_mixed16(C: torch.Tensor, rms_c: float, seed: int) -> List[InjectedFault]:
    """16 simultaneous faults: 4 share a row, 3 share a column, 9 free; every other one an
    exponent-bit-flip size (C_ij * 2^e, e in 1..8, re-drawn until the change is at least
    2 % of rms(C)), the rest additive upsets of 2-9 % of rms(C)."""
    n1, n3 = C.shape
    g = _rng("faults/mixed16", seed)
    coords = faults_shared_lines(n1, n3, seed)
    out = []
    for idx, (i, j) in enumerate(coords):
        if idx % 2 == 0:
            cij = float(C[i, j])
            e = int(g.integers(1, 9))
            while e < 8 and abs(cij * (2.0 ** e) - cij) < 0.02 * rms_c:
                e += 1
            if abs(cij * (2.0 ** e) - cij) >= 0.02 * rms_c:
                out.append(InjectedFault(i, j, "scale", float(e), "expflip"))
                continue
        mag = float(g.uniform(0.02, 0.09)) * rms_c
        sgn = 1.0 if g.integers(0, 2) == 0 else -1.0
        out.append(InjectedFault(i, j, "add", sgn * mag, "small"))
    return out


def inject(C: torch.Tensor, faults: Sequence[InjectedFault]) -> Tuple[torch.Tensor, List[float]]:
    """A copy of C with the faults written in (FP32 arithmetic on the stored value);
    also the change actually made to each entry, new - old, in FP64."""
    out = C.clone()
    changes = []
    for f in faults:
        old = out[f.i, f.j].clone()
        if f.kind == "add":
            new = (old + torch.tensor(f.value, dtype=torch.float32, device=old.device))
        elif f.kind == "scale":
            new = old * torch.tensor(2.0 ** f.value, dtype=torch.float32, device=old.device)
        else:
            raise ValueError(f.kind)
        out[f.i, f.j] = new
        changes.append(float(new.double() - old.double()))
    return out, changes
