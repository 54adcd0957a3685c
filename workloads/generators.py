"""Counter-based generators for graphs and node tensors (torch tensors, CPU or CUDA).

Hashing is SplitMix64's finaliser applied to (seed, stream, counter); all of it is int64
arithmetic with wrap-around, so CPU and CUDA agree bit for bit.  Uniforms use the top 53
bits.  Power-law endpoints are drawn by inverse CDF on a float64 cumulative-weight table
that is always computed with numpy on the host (one fixed summation order), and looked up
with exact comparisons, so ranks agree across devices too.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np
import torch

_MASK64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Python int -> the int64 with the same low 64 bits."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_M1 = _s64(0xBF58476D1CE4E5B9)
_M2 = _s64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of int64 lanes."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def hash64(counter: torch.Tensor, seed: int, stream: int = 0) -> torch.Tensor:
    """SplitMix64 finaliser of (counter + 1) * golden + f(seed, stream); int64 in, int64 out."""
    assert counter.dtype == torch.int64
    key = _s64((seed * 0xD1342543DE82EF95 + stream * 0xA0761D6478BD642F + 0x2545F4914F6CDD1D) & _MASK64)
    z = (counter + 1) * _GOLDEN + key
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def uniform01(counter: torch.Tensor, seed: int, stream: int = 0) -> torch.Tensor:
    """float64 uniforms in [0,1) from the top 53 bits of hash64."""
    return _lsr(hash64(counter, seed, stream), 11).to(torch.float64) * (1.0 / (1 << 53))


def normal_tensor(shape, seed: int, stream: int, device="cpu", dtype=torch.float32,
                  chunk: int = 1 << 26) -> torch.Tensor:
    """N(0,1) values by Box-Muller in float64, then rounded once to `dtype` (float32 or bfloat16).

    Element c of the flattened tensor uses counters 2c and 2c+1 of (seed, stream)."""
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=dtype, device=device)
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        c = torch.arange(lo, hi, dtype=torch.int64, device=device)
        u1 = uniform01(2 * c, seed, stream)
        u2 = uniform01(2 * c + 1, seed, stream)
        z = torch.sqrt(-2.0 * torch.log1p(-u1)) * torch.cos((2.0 * math.pi) * u2)
        out[lo:hi] = z.to(torch.float32).to(dtype)
    return out.reshape(shape)


def uniform_edges(n: int, e: int, seed: int, self_loops: bool, device="cpu"):
    """e directed edges with src uniform and dst uniform over the other n-1 nodes (duplicates
    allowed), followed, when asked, by one self-loop per node.  Returns (src, dst) int32."""
    c = torch.arange(e, dtype=torch.int64, device=device)
    src = _lsr(hash64(c, seed, 1), 1) % n
    off = _lsr(hash64(c, seed, 2), 1) % (n - 1)
    dst = (src + 1 + off) % n
    if self_loops:
        loop = torch.arange(n, dtype=torch.int64, device=device)
        src = torch.cat([src, loop])
        dst = torch.cat([dst, loop])
    return src.to(torch.int32), dst.to(torch.int32)


# --------------------------------------------------------------------------------------
# Chung-Lu style power-law graphs
# --------------------------------------------------------------------------------------

@dataclass(frozen=True)
class ChungLuSpec:
    n: int
    e: int
    gamma: float      # degree exponent; weights w_r = (r + 1 + r0)^(-1/(gamma-1))
    d_max: float      # expected degree of the heaviest node (sets r0)
    seed: int
    permute: bool = True  # map ranks to node ids through a seeded random permutation


def _weight_sum(n: int, r0: float, a: float) -> float:
    """sum_{r<n} (r+1+r0)^-a by Euler-Maclaurin (integral + end-point terms); a != 1."""
    lo, hi = 1.0 + r0, n + r0
    integral = (hi ** (1.0 - a) - lo ** (1.0 - a)) / (1.0 - a)
    return integral + 0.5 * (lo ** -a + hi ** -a) + (a / 12.0) * (lo ** (-a - 1.0) - hi ** (-a - 1.0))


def chung_lu_r0(n: int, e: int, gamma: float, d_max: float) -> float:
    """Offset r0 >= 0 such that e * w_0 / sum(w) = d_max (60 bisection steps on the closed form)."""
    a = 1.0 / (gamma - 1.0)

    def top_degree(r0):
        return e * (1.0 + r0) ** -a / _weight_sum(n, r0, a)

    lo, hi = 0.0, float(n)
    if top_degree(lo) <= d_max:
        return 0.0
    for _ in range(60):
        mid = 0.5 * (lo + hi)
        if top_degree(mid) > d_max:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def _cumulative_weights(spec: ChungLuSpec) -> np.ndarray:
    a = 1.0 / (spec.gamma - 1.0)
    r0 = chung_lu_r0(spec.n, spec.e, spec.gamma, spec.d_max)
    w = (np.arange(spec.n, dtype=np.float64) + (1.0 + r0)) ** -a
    cum = np.cumsum(w)
    cum /= cum[-1]
    return cum


def chung_lu_edges(spec: ChungLuSpec, device="cpu", chunk: int = 1 << 26):
    """e directed edges whose source rank and destination rank are independent draws with
    probability proportional to w_rank; duplicates and self-loops stay as drawn.  Both the
    in- and the out-degree sequence are power laws.  Returns (src, dst) int32 on `device`."""
    cum = torch.from_numpy(_cumulative_weights(spec)).to(device)
    if spec.permute:
        keys = hash64(torch.arange(spec.n, dtype=torch.int64, device=device), spec.seed, 7)
        perm = torch.sort(keys, stable=True).indices.to(torch.int32)
    src = torch.empty(spec.e, dtype=torch.int32, device=device)
    dst = torch.empty(spec.e, dtype=torch.int32, device=device)
    for lo in range(0, spec.e, chunk):
        hi = min(spec.e, lo + chunk)
        c = torch.arange(lo, hi, dtype=torch.int64, device=device)
        for stream, target in ((3, src), (4, dst)):
            rank = torch.searchsorted(cum, uniform01(c, spec.seed, stream), right=True)
            rank.clamp_(max=spec.n - 1)
            target[lo:hi] = perm[rank] if spec.permute else rank.to(torch.int32)
    return src, dst
