"""Seeded synthetic inputs for the ternary mpGEMM path.

This module only draws numbers: it holds none of the method's arithmetic (no
quantiser, no packing, no dot products).  Both the CUDA path's callers and the
CPU oracle's tests take their inputs from here, so the two sides see the same
bytes.

Generator: counter based and order free.  A stream is keyed by
``key = mix64(seed * 2**32 + tensor_id)``; element ``i`` of the stream draws
``u = mix64(key + i)``, where ``mix64`` is the splitmix64 finaliser (add the
golden-ratio constant, two xor-shift-multiply rounds, a last xor-shift).  The
integer part runs identically on CPU and CUDA tensors, so a weight matrix can
be produced directly in device memory and any row of it re-drawn on the host.

* ternary weights: ``r = u >> 32``; ``w = 0`` if ``r < floor(p0 * 2**32)``,
  ``+1`` if ``r < floor((p0 + p_plus) * 2**32)``, else ``-1``.
* weights of cardinality C (the formats beyond ternary): ``w = -(C // 2) +
  ((u >> 32) * C >> 32)``, uniform over the C consecutive integers from -(C // 2).
* normal activations: Box-Muller in float64 on the two 32-bit halves of ``u``
  (always evaluated on the host so that libm differences cannot split the two
  sides), cast to float32.
* the "outlier" recipe overwrites ``ceil(frac * K)`` seeded positions of each
  token with +-20.

The shapes, seeds and weight laws of the five workloads are in ``CONFIGS``.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch

_M64 = (1 << 64) - 1


def _s64(v: int) -> int:
    """Python int (mod 2**64) -> the int64 with the same bit pattern."""
    v &= _M64
    return v - (1 << 64) if v >= (1 << 63) else v


_GOLD = _s64(0x9E3779B97F4A7C15)
_MUL1 = _s64(0xBF58476D1CE4E5B9)
_MUL2 = _s64(0x94D049BB133111EB)


def _mix64_int(z: int) -> int:
    z = (z + 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64(z: torch.Tensor) -> torch.Tensor:
    z = z + _GOLD
    z = (z ^ _lsr(z, 30)) * _MUL1
    z = (z ^ _lsr(z, 27)) * _MUL2
    return z ^ _lsr(z, 31)


def stream_key(seed: int, tensor_id: int) -> int:
    return _mix64_int((seed << 32) + tensor_id)


def draw_u64(seed: int, tensor_id: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """``count`` draws of the stream, elements ``start .. start+count-1``, as int64 bit patterns."""
    key = _s64(stream_key(seed, tensor_id))
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return _mix64(idx + key)


def ternary(seed: int, tensor_id: int, rows: int, cols: int, p0: float, p_plus: float,
            device="cpu", row_start: int = 0, total_cols: int | None = None,
            chunk_elems: int = 1 << 27) -> torch.Tensor:
    """int8 matrix [rows][cols] over {-1,0,+1}.

    ``row_start`` re-draws rows ``row_start .. row_start+rows-1`` of a larger
    matrix whose row length is ``total_cols`` (default ``cols``), bit for bit.
    """
    total_cols = cols if total_cols is None else total_cols
    assert total_cols == cols, "column windows are not needed by any workload"
    t0 = int(math.floor(p0 * 4294967296.0))
    t1 = int(math.floor((p0 + p_plus) * 4294967296.0))
    out = torch.empty(rows * cols, dtype=torch.int8, device=device)
    n = rows * cols
    base = row_start * cols
    for s in range(0, n, chunk_elems):
        c = min(chunk_elems, n - s)
        r = _lsr(draw_u64(seed, tensor_id, base + s, c, device), 32)
        w = torch.where(r < t0, 0, torch.where(r < t1, 1, -1))
        out[s:s + c] = w.to(torch.int8)
    return out.view(rows, cols)


def uniform_alphabet(seed: int, tensor_id: int, rows: int, cols: int, card: int, device="cpu",
                     chunk_elems: int = 1 << 27) -> torch.Tensor:
    """int8 matrix [rows][cols], uniform over the ``card`` consecutive integers from -(card // 2)."""
    out = torch.empty(rows * cols, dtype=torch.int8, device=device)
    n = rows * cols
    for s in range(0, n, chunk_elems):
        c = min(chunk_elems, n - s)
        r = _lsr(draw_u64(seed, tensor_id, s, c, device), 32)
        out[s:s + c] = (_lsr(r * card, 32) - (card // 2)).to(torch.int8)
    return out.view(rows, cols)


def normal(seed: int, tensor_id: int, rows: int, cols: int) -> torch.Tensor:
    """float32 matrix [rows][cols] ~ N(0,1), evaluated on the host in float64."""
    u = draw_u64(seed, tensor_id, 0, rows * cols, "cpu")
    hi = _lsr(u, 32).to(torch.float64)
    lo = (u & 0xFFFFFFFF).to(torch.float64)
    u1 = (hi + 1.0) / 4294967296.0
    u2 = lo / 4294967296.0
    z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos(2.0 * math.pi * u2)
    return z.to(torch.float32).view(rows, cols)


def add_outliers(x: torch.Tensor, seed: int, tensor_id: int, frac: float = 0.001,
                 magnitude: float = 20.0) -> torch.Tensor:
    """Overwrite ceil(frac*K) seeded, distinct positions of every row with +-magnitude."""
    rows, cols = x.shape
    n_out = int(math.ceil(frac * cols))
    x = x.clone()
    for t in range(rows):
        key = stream_key(seed, (tensor_id << 20) + 0x80000 + t)
        seen: set[int] = set()
        j = 0
        while len(seen) < n_out:
            pos = _mix64_int((key + 2 * j) & _M64) % cols
            sgn = _mix64_int((key + 2 * j + 1) & _M64) & 1
            j += 1
            if pos in seen:
                continue
            seen.add(pos)
            x[t, pos] = magnitude if sgn == 0 else -magnitude
    return x


def absmean_scale(w: torch.Tensor) -> float:
    """Per-tensor scale of a ternary matrix: the mean of |w| (count of non-zeros / size), as float32."""
    nnz = int(torch.count_nonzero(w).item())
    return float(torch.tensor(nnz / w.numel(), dtype=torch.float32).item())


@dataclass(frozen=True)
class Linear:
    name: str
    K: int
    M: int


@dataclass(frozen=True)
class Workload:
    """One of the five synthetic workloads (stand-ins for the paper's 700M-100B checkpoints)."""
    name: str
    seed: int
    linears: tuple
    tokens: tuple
    p0: float
    p_plus: float
    layers: int = 1
    outlier_frac: float = 0.0
    formats: tuple = ("i2s", "tl2")
    note: str = field(default="", compare=False)

    def weight_id(self, layer: int, j: int) -> int:
        return layer * 8 + j

    def act_id(self, layer: int, j: int) -> int:
        return layer * 8 + 4 + j

    def weights(self, layer: int, j: int, device="cpu", row_start=0, rows=None) -> torch.Tensor:
        lin = self.linears[j]
        rows = lin.M if rows is None else rows
        return ternary(self.seed, self.weight_id(layer, j), rows, lin.K, self.p0, self.p_plus,
                       device=device, row_start=row_start)

    def activations(self, layer: int, j: int, T: int) -> torch.Tensor:
        lin = self.linears[j]
        x = normal(self.seed, self.act_id(layer, j), T, lin.K)
        if self.outlier_frac > 0:
            x = add_outliers(x, self.seed, self.act_id(layer, j), self.outlier_frac)
        return x


THIRD = 1.0 / 3.0

CONFIGS = {
    # single GEMV, hidden size of the 700M class; activations carry 0.1% outliers at +-20
    "gemv1536": Workload("gemv1536", 0, (Linear("proj", 1536, 1536),), (1,), THIRD, THIRD,
                         outlier_frac=0.001, formats=("i2s", "tl1", "tl2")),
    # 3B-shaped decoder layer at batch 1
    "layer3b": Workload("layer3b", 1, (Linear("qkv", 3200, 9600), Linear("o", 3200, 3200),
                                       Linear("gate_up", 3200, 17280), Linear("down", 8640, 3200)),
                        (1,), THIRD, THIRD),
    # 8B Llama-shaped layer at batch 1 and 8
    "layer8b": Workload("layer8b", 2, (Linear("qkv", 4096, 6144), Linear("o", 4096, 4096),
                                       Linear("gate_up", 4096, 28672), Linear("down", 14336, 4096)),
                        (1, 8), 0.4, 0.3),
    # prefill GEMM
    "prefill": Workload("prefill", 3, (Linear("up", 4096, 14336),), (2048,), THIRD, THIRD,
                        formats=("i2s",)),
    # 100B-shaped decode sweep, 80 layers
    "sweep100b": Workload("sweep100b", 4, (Linear("qkv", 8192, 10240), Linear("o", 8192, 8192),
                                           Linear("gate_up", 8192, 57344), Linear("down", 28672, 8192)),
                          (1,), THIRD, THIRD, layers=80),
}
