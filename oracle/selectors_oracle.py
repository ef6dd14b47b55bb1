"""CPU twins of the library's comparison selectors (sliding window, random blocks, cross-scale
reuse through nearest-position maps): the selectors of the paper's selection-strategy ablation.

TEST INFRASTRUCTURE, NOT PRODUCT.  The paper names these selectors without defining them, so
there is nothing of the paper's to pin them to ("parity unpinned by the paper"); the definitions
are the library's own (include/sparstar.h) and this module restates them in plain Python / numpy:
integer index sums, IEEE double operations in a fixed order, one rounding to fp32.  Pins in
tests/test_selectors.py are closed forms of those definitions.  It shares no code with the CUDA
library and never calls it.
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple

import numpy as np

Segment = Tuple[int, Optional[Tuple[int, int, int]]]      # (length, (T, H, W) or None for text)


def block_centres(segs: Sequence[Segment], block: int) -> np.ndarray:
    """[n_blocks, 3] centres: per coordinate the mean over the block's tokens of index / extent;
    tokens without a position sit at 1/2.  Partial sums are formed per segment (integer index
    sums, one division), added in segment order, divided by the token count."""
    L = sum(s[0] for s in segs)
    n = -(-L // block)
    out = np.zeros((n, 3), dtype=np.float64)
    for blk in range(n):
        lo, hi = blk * block, blk * block + block
        st = sh = sw = 0.0
        cnt = 0
        pos = 0
        for (length, grid) in segs:
            a, e = max(lo, pos), pos + length
            b = min(hi, e)
            if a < b:
                m = b - a
                if grid is None:
                    st = st + 0.5 * float(m); sh = sh + 0.5 * float(m); sw = sw + 0.5 * float(m)
                else:
                    T, H, W = grid
                    it = ih = iw = 0
                    for u in range(a - pos, b - pos):
                        it += u // (H * W)
                        ih += (u // W) % H
                        iw += u % W
                    st = st + float(it) / float(T)
                    sh = sh + float(ih) / float(H)
                    sw = sw + float(iw) / float(W)
                cnt += m
            pos = e
        d = float(cnt) if cnt > 0 else 1.0
        out[blk] = (st / d, sh / d, sw / d)
    return out


def nearest_block_map(fine: np.ndarray, coarse: np.ndarray) -> np.ndarray:
    """map[i] = argmin_j of the squared distance between fine centre i and coarse centre j; ties go
    to the lower index."""
    out = np.zeros(len(fine), dtype=np.int32)
    for i in range(len(fine)):
        best, bd = 0, math.inf
        for j in range(len(coarse)):
            dt, dh, dw = (float(fine[i][c]) - float(coarse[j][c]) for c in range(3))
            d2 = (dt * dt + dh * dh) + dw * dw
            if d2 < bd:
                best, bd = j, d2
        out[i] = best
    return out


def window_scores(q_segs: Sequence[Segment], k_segs: Sequence[Segment], block: int) -> np.ndarray:
    """[n_q, n_k] fp32: minus the Euclidean distance between block centres (fp64, rounded once)."""
    cq, ck = block_centres(q_segs, block), block_centres(k_segs, block)
    d = cq[:, None, :] - ck[None, :, :]
    d2 = (d[..., 0] * d[..., 0] + d[..., 1] * d[..., 1]) + d[..., 2] * d[..., 2]
    return (-np.sqrt(d2)).astype(np.float32)


def random_scores(seed: int, shape: Tuple[int, ...]) -> np.ndarray:
    """Uniform numbers in [0, 1) from a 64-bit mixing function of (seed, linear index)."""
    n = int(np.prod(shape))
    with np.errstate(over="ignore"):
        idx = np.arange(1, n + 1, dtype=np.uint64)
        z = np.uint64(seed % (1 << 64)) + idx * np.uint64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
    return ((z >> np.uint64(40)).astype(np.float32) * np.float32(2.0 ** -24)).reshape(shape)


def remap_scores(coarse: np.ndarray, q_map: np.ndarray, k_map: np.ndarray) -> np.ndarray:
    """out[..., i, j] = coarse[..., q_map[i], k_map[j]]."""
    return coarse[..., q_map, :][..., k_map]
