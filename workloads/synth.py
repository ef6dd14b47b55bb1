"""Counter-based seeded generator of Q/K/V for a workload.

Every element is a pure function of (seed, stream, head, token, dim), so any
part can be regenerated independently and on any torch device: the integer
hash is exact everywhere; the Box-Muller transform runs in fp64 and the result
is rounded to the storage dtype.  The same bits then go to the CPU oracle (by
host copy) and to the CUDA path.

Structure (stands in for real late-scale activations, which need the trained
backbone):
  * base: i.i.d. N(0,1) for Q, K and V;
  * locality: every visual token belongs to a coarse (time, height) cell of
    its own grid; per (head, cell) an offset vector alpha*N(0,1) is added to the
    Q and K tokens of that cell - the same vector for queries, current-scale
    keys and (by normalised position) reference/image keys.  V gets none, so
    it stays unit-variance;
  * sinks: the first n_sink key rows are multiplied by 4.
"""
from __future__ import annotations

import math
from typing import Dict, Optional, Tuple

import torch

from .configs import Workload

_M64 = (1 << 64) - 1


def _s64(c: int) -> int:
    c &= _M64
    return c - (1 << 64) if c >= (1 << 63) else c


_C1 = _s64(0x9E3779B97F4A7C15)
_C2 = _s64(0xBF58476D1CE4E5B9)
_C3 = _s64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix(x: torch.Tensor) -> torch.Tensor:
    """64-bit finaliser on int64 tensors (two's-complement wraparound)."""
    x = x + _C1
    x = (x ^ _lsr(x, 30)) * _C2
    x = (x ^ _lsr(x, 27)) * _C3
    return x ^ _lsr(x, 31)


def _mix_int(x: int) -> int:
    x = (x + 0x9E3779B97F4A7C15) & _M64
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & _M64
    return x ^ (x >> 31)


def _stream_key(seed: int, *ids: int) -> int:
    k = _mix_int(seed)
    for i in ids:
        k = _mix_int(k ^ ((i + 1) * 0xD6E8FEB86659FD93 & _M64))
    return _s64(k)


def normal_pairs(key: int, first: int, count: int, device) -> torch.Tensor:
    """2*count standard normals (fp64) for counters first..first+count-1 of
    stream `key`; counter c yields elements 2c and 2c+1."""
    c = torch.arange(first, first + count, dtype=torch.int64, device=device)
    a = _mix(c ^ key)
    b = _mix(a + _C1)
    u1 = (_lsr(a, 11).to(torch.float64) + 0.5) * (1.0 / 9007199254740992.0)
    u2 = (_lsr(b, 11).to(torch.float64) + 0.5) * (1.0 / 9007199254740992.0)
    r = torch.sqrt(-2.0 * torch.log(u1))
    th = (2.0 * math.pi) * u2
    return torch.stack((r * torch.cos(th), r * torch.sin(th)), dim=-1).reshape(-1)


_KIND_ID = {"text": 1, "ref": 2, "image": 3, "cur": 4}
_TENSOR_ID = {"q": 1, "k": 2, "v": 3, "mu": 4}


def _cells(grid: Tuple[int, int, int], cells: Tuple[int, int], device) -> torch.Tensor:
    """Locality cell id of every token of a raster (t, h, w) grid."""
    T, Hh, W = grid
    n = torch.arange(T * Hh * W, dtype=torch.int64, device=device)
    t = n // (Hh * W)
    h = (n // W) % Hh
    return (t * cells[0] // T) * cells[1] + (h * cells[1] // Hh)


def _segment_stream(w: Workload, tensor: str, kind: str) -> int:
    tag = w.scale_tag if kind == "cur" else 0
    return _stream_key(w.seed, _TENSOR_ID[tensor], _KIND_ID[kind], tag)


def generate(w: Workload, device="cpu", heads: Optional[Tuple[int, int]] = None) -> Dict[str, torch.Tensor]:
    """Returns q [B,H,L_q,D], k, v [B,H,L_k,D] in the workload's dtype on
    `device` (contiguous).  `heads` = (h0, h1) generates only heads h0..h1-1 of
    the workload (tensors of h1-h0 heads holding exactly the bits those heads
    have in the full tensors): a rank of a head-sharded run makes its own shard."""
    dt = torch.float32 if w.dtype == "f32" else torch.bfloat16
    dev = torch.device(device)
    B, D = w.B, w.D
    h0, h1 = (0, w.H) if heads is None else (int(heads[0]), int(heads[1]))
    if not (0 <= h0 < h1 <= w.H):
        raise ValueError(f"head range {heads} outside 0..{w.H}")
    H = h1 - h0
    n_cells = w.cells[0] * w.cells[1]
    q = torch.empty((B, H, w.L_q, D), dtype=dt, device=dev)
    k = torch.empty((B, H, w.L_k, D), dtype=dt, device=dev)
    v = torch.empty((B, H, w.L_k, D), dtype=dt, device=dev)
    mu_key = _stream_key(w.seed, _TENSOR_ID["mu"])
    q_cells = _cells(w.q_grid, w.cells, dev)
    for b in range(B):
        for h in range(H):
            bh = b * w.H + h0 + h
            mu = w.alpha * normal_pairs(mu_key, bh * n_cells * D // 2, n_cells * D // 2, dev).reshape(n_cells, D)
            # queries: the current-scale tokens
            L = w.L_q
            x = normal_pairs(_segment_stream(w, "q", "cur"), bh * L * D // 2, L * D // 2, dev).reshape(L, D)
            q[b, h] = (x + mu[q_cells]).to(dt)
            pos = 0
            for s in w.segments:
                L = s.length
                xk = normal_pairs(_segment_stream(w, "k", s.kind), bh * L * D // 2, L * D // 2, dev).reshape(L, D)
                xv = normal_pairs(_segment_stream(w, "v", s.kind), bh * L * D // 2, L * D // 2, dev).reshape(L, D)
                if s.grid is not None:
                    xk = xk + mu[_cells(s.grid, w.cells, dev)]
                if pos < w.n_sink:
                    ns = min(w.n_sink - pos, L)
                    xk[:ns] *= 4.0
                k[b, h, pos:pos + L] = xk.to(dt)
                v[b, h, pos:pos + L] = xv.to(dt)
                pos += L
    return {"q": q, "k": k, "v": v}
