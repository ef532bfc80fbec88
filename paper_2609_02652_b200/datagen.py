"""Seeded synthetic inputs: 48-bit block codes, per-row scales, activations, and the layer shapes.

This module serves both the CUDA path's tests/bench and the CPU oracle's tests.  It holds none
of the method's arithmetic: it draws integers and normals from a counter-based generator and
knows the *sizes* of the shells of the ball (the Leech theta series, a closed form) so that an
index can be drawn uniformly inside a shell.  It never decodes an index.

Recipe (stands in for the paper's quantised model files, which are not available): per block a
shell m is drawn uniformly from 2..12, then an index uniformly among that shell's points (shells
occupy consecutive index ranges in ascending m); the gain bit is a fair coin; the code word is
index | gain << 47.  Row scales are fp16(0.02 * |N(0,1)|), activations fp16(N(0,1)) with the
zero padding of the in-dimension up to a multiple of 24 left at zero.
"""
from __future__ import annotations

import dataclasses
import math

import torch

MASK64 = (1 << 64) - 1
SHELLS = tuple(range(2, 13))
GAIN = (0.75, 1.5)  # the two per-tensor gain centroids used by every synthetic tensor


def _sigma11(n: int) -> int:
    return sum(d**11 for d in range(1, n + 1) if n % d == 0)


def _ramanujan_tau(nmax: int) -> list[int]:
    # coefficients of q * prod (1 - q^n)^24
    poly = [0] * (nmax + 1)
    poly[0] = 1
    for n in range(1, nmax + 1):
        for _ in range(24):
            for k in range(nmax, n - 1, -1):
                poly[k] -= poly[k - n]
    return [0] + poly[:nmax]  # tau[1] = poly[0]


def shell_sizes() -> dict[int, int]:
    """Points of the Leech lattice on shell m (norm 2m in the standard scaling), m = 2..12."""
    tau = _ramanujan_tau(13)
    return {m: 65520 * (_sigma11(m) - tau[m]) // 691 for m in SHELLS}


def shell_bases() -> dict[int, int]:
    sizes, base, acc = shell_sizes(), {}, 0
    for m in SHELLS:
        base[m] = acc
        acc += sizes[m]
    base[13] = acc  # one past the last valid index
    return base


def _s64(v: int) -> int:
    v &= MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix(counter: torch.Tensor, key: int) -> torch.Tensor:
    """splitmix64 finaliser of (counter + key), on int64 tensors with wrap-around arithmetic."""
    z = counter + _s64(key)
    z = (z ^ _lsr(z, 30)) * _s64(0xBF58476D1CE4E5B9)
    z = (z ^ _lsr(z, 27)) * _s64(0x94D049BB133111EB)
    return z ^ _lsr(z, 31)


def _key(seed: int, tensor_id: int, stream: int) -> int:
    k = (seed * 0x9E3779B97F4A7C15 + tensor_id * 0xD1B54A32D192ED03 + stream * 0x8CB92BA72F3D8DD7 + 0x1234567) & MASK64
    # one scalar round of the same finaliser
    k = ((k ^ (k >> 30)) * 0xBF58476D1CE4E5B9) & MASK64
    k = ((k ^ (k >> 27)) * 0x94D049BB133111EB) & MASK64
    return k ^ (k >> 31)


def make_codes(rows: int, nb: int, seed: int, tensor_id: int = 0, device="cpu", start: int = 0, count: int | None = None) -> torch.Tensor:
    """int64 tensor of rows*nb code words (or the slice [start, start+count) of it), integer-only."""
    n = rows * nb if count is None else count
    i = torch.arange(start, start + n, dtype=torch.int64, device=device) * _s64(0x9E3779B97F4A7C15)
    sizes, bases = shell_sizes(), shell_bases()
    size_t = torch.tensor([sizes[m] for m in SHELLS], dtype=torch.int64, device=device)
    base_t = torch.tensor([bases[m] for m in SHELLS], dtype=torch.int64, device=device)
    shell = _lsr(_mix(i, _key(seed, tensor_id, 1)), 40) % len(SHELLS)
    u = _lsr(_mix(i, _key(seed, tensor_id, 2)), 2)
    idx = base_t[shell] + u % size_t[shell]
    gain = _lsr(_mix(i, _key(seed, tensor_id, 3)), 63)
    return idx | (gain << 47)


def make_indices(n: int, seed: int, stream: int = 9) -> torch.Tensor:
    """n extra random valid indices (no gain bit), same shell-uniform draw."""
    return make_codes(n, 1, seed, tensor_id=1 << 20 | stream) & ((1 << 47) - 1)


def _normals(n: int, seed: int, tensor_id: int, stream: int) -> torch.Tensor:
    # Box-Muller in f64 on the host, so that every caller sees the same bits
    i = torch.arange(n, dtype=torch.int64) * _s64(0x9E3779B97F4A7C15)
    u1 = (_lsr(_mix(i, _key(seed, tensor_id, stream)), 11).double() + 1.0) / 9007199254740992.0
    u2 = _lsr(_mix(i, _key(seed, tensor_id, stream + 100)), 11).double() / 9007199254740992.0
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos(2.0 * math.pi * u2)


def make_row_scale(rows: int, seed: int, tensor_id: int = 0) -> torch.Tensor:
    return (0.02 * _normals(rows, seed, tensor_id, 4).abs()).to(torch.float16)


def make_x(k: int, k_padded: int, seed: int, tensor_id: int = 0) -> torch.Tensor:
    x = torch.zeros(k_padded, dtype=torch.float16)
    x[:k] = _normals(k, seed, tensor_id, 5).to(torch.float16)
    return x


@dataclasses.dataclass(frozen=True)
class Matrix:
    name: str
    rows: int
    k: int          # in-dimension before padding
    tensor_id: int
    group: int = -1  # matrices with the same non-negative group share x and may run as one launch

    @property
    def nb(self) -> int:
        return (self.k + 23) // 24

    @property
    def k_padded(self) -> int:
        return self.nb * 24

    @property
    def blocks(self) -> int:
        return self.rows * self.nb


def _decoder_layer(hidden: int, inter: int, q_heads: int, kv_heads: int, head_dim: int, layer: int) -> list[Matrix]:
    t = layer * 7
    g = layer * 4
    return [
        Matrix(f"L{layer}.q", q_heads * head_dim, hidden, t + 0, g + 0),
        Matrix(f"L{layer}.k", kv_heads * head_dim, hidden, t + 1, g + 0),
        Matrix(f"L{layer}.v", kv_heads * head_dim, hidden, t + 2, g + 0),
        Matrix(f"L{layer}.o", hidden, q_heads * head_dim, t + 3, g + 1),
        Matrix(f"L{layer}.gate", inter, hidden, t + 4, g + 2),
        Matrix(f"L{layer}.up", inter, hidden, t + 5, g + 2),
        Matrix(f"L{layer}.down", hidden, inter, t + 6, g + 3),
    ]


@dataclasses.dataclass(frozen=True)
class Workload:
    config: int
    name: str
    seed: int
    matrices: tuple
    head: tuple | None = None  # (rows, k) of the fp16 output head, if any

    @property
    def blocks(self) -> int:
        return sum(m.blocks for m in self.matrices)


def workload(config: int, layers: int | None = None) -> Workload:
    """The five workloads; `layers` truncates the two multi-layer stacks (for tests)."""
    if config == 0:
        return Workload(0, "single 3072x3072", 0, (Matrix("w", 3072, 3072, 0),))
    if config == 1:
        return Workload(1, "4B-like decoder layer", 1, tuple(_decoder_layer(2560, 9728, 32, 8, 128, 0)))
    if config == 2:
        n = 36 if layers is None else layers
        mats = [m for l in range(n) for m in _decoder_layer(4096, 12288, 32, 8, 128, l)]
        return Workload(2, f"8B-like stack x{n}", 2, tuple(mats), (151936, 4096))
    if config == 3:
        n = 40 if layers is None else layers
        mats = [m for l in range(n) for m in _decoder_layer(5120, 17408, 40, 8, 128, l)]
        return Workload(3, f"14B-like stack x{n}", 3, tuple(mats), (151936, 5120))
    if config == 4:
        return Workload(4, "layout sweep 8192x8192", 4, (Matrix("w", 8192, 8192, 0),))
    raise ValueError(f"unknown config {config}")
