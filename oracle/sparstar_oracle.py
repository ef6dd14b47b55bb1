"""CPU oracle for per-head dynamic block-sparse attention (SparSTAR).

TEST INFRASTRUCTURE, NOT PRODUCT.  Only the test-suite, the smoke check and the
benchmark's CPU-baseline leg may import this module.  It shares no code with
the CUDA library and never calls it.

Everything is numpy float64 on exactly-widened inputs, one head at a time,
following the paper's steps in the paper's order and notation:

  pool_blocks      block means over the nominal block length b, final partial
                   block zero-padded          (Sec. "Aggregated Query-Key Block
                                               Selector", block partition and
                                               per-head score paragraphs)
  block_scores     S_ij = tau * qbar_i . kbar_j                       (Eq. 2)
  forced_blocks    J_text / J_ref by token-range intersection   (same section)
  budget           k = min(n_sel, max(1, ceil(rho * n_sel)))          (Eq. 5)
  select_topk      A_i = J_keep U TopKIdx_{j in J_sel}(S_ij, k)    (Eq. 3,4,6)
  select_mass      cumulative block-score mass selection - NOT in the paper;
                   defined by the benchmark (softmax of S over J_sel, smallest
                   prefix of the descending order whose mass reaches p)
  sparse_attention softmax attention under M_tu = 1[pi_k(u) in A_{pi_q(t)}]
                                                                      (Eq. 7)
  dense_attention  the same with every block visible        (Sec. "Complexity")

Pins: every function is checked by tests/test_oracle_pins.py against closed
forms, brute force in pure Python, the bilinearity identity stated under Eq. 2,
hand-enumerated block sets, a library softmax-attention, and a hand-worked
example stored under tests/golden/.  select_mass has no counterpart in the
paper: it is pinned by its own definition's invariants and by exhaustive subset
search on tiny inputs only ("paper-unpinned, benchmark-defined").
"""
from __future__ import annotations

import math
from typing import List, Sequence, Tuple

import numpy as np


# --------------------------------------------------------------------------- partition
def num_blocks(L: int, b: int) -> int:
    """n = ceil(L / b): contiguous blocks of b tokens from token 0."""
    return -(-int(L) // int(b))


def pool_blocks(x: np.ndarray, b: int) -> np.ndarray:
    """x [L, D] -> [n, D]; xbar_i = (1/b) * sum of the block's tokens, the final
    partial block padded with zeros and still divided by the nominal b."""
    x = np.asarray(x, dtype=np.float64)
    L, D = x.shape
    n = num_blocks(L, b)
    out = np.zeros((n, D), dtype=np.float64)
    for i in range(n):
        out[i] = x[i * b:min((i + 1) * b, L)].sum(axis=0) / b
    return out


def block_scores(qbar: np.ndarray, kbar: np.ndarray, tau: float) -> np.ndarray:
    """Eq. 2: S_ij = tau * qbar_i^T kbar_j."""
    return tau * (np.asarray(qbar, np.float64) @ np.asarray(kbar, np.float64).T)


def forced_blocks(L_k: int, b: int, ranges: Sequence[Tuple[int, int]]) -> np.ndarray:
    """Boolean [n_k]: block j is forced iff its token set [j*b, min((j+1)*b, L_k))
    intersects one of the half-open token ranges (covers blocks that straddle a
    segment boundary)."""
    n_k = num_blocks(L_k, b)
    f = np.zeros(n_k, dtype=bool)
    for j in range(n_k):
        lo, hi = j * b, min((j + 1) * b, L_k)
        for (rb, re) in ranges:
            if max(lo, rb) < min(hi, re):
                f[j] = True
    return f


def budget(n_sel: int, rho: float) -> int:
    """Eq. 5.  The product is formed in double; a guard of 1e-9 keeps a ratio
    such as 0.3 * 10 from rounding up past its exact value."""
    if n_sel <= 0:
        return 0
    return min(n_sel, max(1, int(math.ceil(rho * n_sel - 1e-9))))


# --------------------------------------------------------------------------- selection
def _descending_order(s: np.ndarray) -> np.ndarray:
    """Positions sorted by (score descending, position ascending)."""
    return np.argsort(-s, kind="stable")


def select_topk_row(S_row: np.ndarray, forced: np.ndarray, k: int) -> np.ndarray:
    """Eq. 6 for one query block: forced blocks plus the k best selectable
    blocks; equal scores resolve to the lower block index.  Sorted ascending."""
    sel = np.nonzero(~forced)[0]
    order = _descending_order(S_row[sel])
    taken = sel[order[:k]]
    return np.sort(np.concatenate([np.nonzero(forced)[0], taken])).astype(np.int32)


def mass_prefix_length(S_sel: np.ndarray, p: float) -> Tuple[int, np.ndarray, np.ndarray]:
    """Softmax of the selectable scores, descending order, r* = the smallest r >= 1
    whose cumulative mass reaches p.  Returns (r*, order, cumulative mass)."""
    if S_sel.size == 0:
        return 0, np.zeros(0, dtype=np.int64), np.zeros(0)
    e = np.exp(S_sel - S_sel.max())
    P = e / e.sum()
    order = _descending_order(S_sel)
    c = np.cumsum(P[order])
    hit = np.nonzero(c >= p)[0]
    r = int(hit[0]) + 1 if hit.size else int(S_sel.size)
    return r, order, c


def select_mass_row(S_row: np.ndarray, forced: np.ndarray, p: float) -> np.ndarray:
    """Benchmark-defined variant: forced blocks plus the shortest descending
    prefix of the selectable blocks whose softmax mass (over selectable blocks
    only) is >= p."""
    sel = np.nonzero(~forced)[0]
    r, order, _ = mass_prefix_length(S_row[sel], p)
    taken = sel[order[:r]]
    return np.sort(np.concatenate([np.nonzero(forced)[0], taken])).astype(np.int32)


def select(S: np.ndarray, forced: np.ndarray, mode: str, ratio: float = 0.0,
           count: int = 0, mass: float = 0.0) -> List[np.ndarray]:
    """Per query block i the ascending list A_i (the forward BlockMask fields
    are len(A_i) and A_i)."""
    n_sel = int((~forced).sum())
    if mode == "topk_ratio":
        k = budget(n_sel, ratio)
        return [select_topk_row(S[i], forced, k) for i in range(S.shape[0])]
    if mode == "topk_count":
        k = min(n_sel, max(0, int(count)))
        return [select_topk_row(S[i], forced, k) for i in range(S.shape[0])]
    if mode == "mass":
        return [select_mass_row(S[i], forced, mass) for i in range(S.shape[0])]
    raise ValueError(mode)


def select_head(Q: np.ndarray, K: np.ndarray, b: int, tau: float,
                ranges: Sequence[Tuple[int, int]], mode: str, ratio: float = 0.0,
                count: int = 0, mass: float = 0.0):
    """pool -> score -> forced sets -> select for one head.  Returns
    (lists, S, forced)."""
    qbar = pool_blocks(Q, b)
    kbar = pool_blocks(K, b)
    S = block_scores(qbar, kbar, tau)
    forced = forced_blocks(K.shape[0], b, ranges)
    return select(S, forced, mode, ratio, count, mass), S, forced


# --------------------------------------------------------------------------- attention
def attention_block(Qi: np.ndarray, K: np.ndarray, V: np.ndarray, blocks: Sequence[int],
                    b: int, tau: float) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 7 for the queries of one block: keys u with pi_k(u) in `blocks` and
    u < L_k.  Two passes (max, then sum).  Returns (O [m, D], LSE [m]) with
    LSE = log sum_u exp(tau q.k_u)."""
    L_k = K.shape[0]
    idx = np.concatenate([np.arange(j * b, min((j + 1) * b, L_k)) for j in blocks]) \
        if len(blocks) else np.zeros(0, dtype=np.int64)
    logits = tau * (np.asarray(Qi, np.float64) @ np.asarray(K[idx], np.float64).T)
    m = logits.max(axis=1, keepdims=True)
    w = np.exp(logits - m)
    z = w.sum(axis=1, keepdims=True)
    O = (w @ np.asarray(V[idx], np.float64)) / z
    return O, (m + np.log(z))[:, 0]


def sparse_attention(Q: np.ndarray, K: np.ndarray, V: np.ndarray, lists: Sequence[Sequence[int]],
                     b: int, tau: float) -> Tuple[np.ndarray, np.ndarray]:
    """One head: O [L_q, D], LSE [L_q] under the block lists."""
    L_q, D = Q.shape
    O = np.zeros((L_q, V.shape[1]), dtype=np.float64)
    lse = np.zeros(L_q, dtype=np.float64)
    for i in range(num_blocks(L_q, b)):
        r0, r1 = i * b, min((i + 1) * b, L_q)
        O[r0:r1], lse[r0:r1] = attention_block(Q[r0:r1], K, V, lists[i], b, tau)
    return O, lse


def dense_attention(Q: np.ndarray, K: np.ndarray, V: np.ndarray, tau: float) -> Tuple[np.ndarray, np.ndarray]:
    """softmax(tau Q K^T) V over every key."""
    logits = tau * (np.asarray(Q, np.float64) @ np.asarray(K, np.float64).T)
    m = logits.max(axis=1, keepdims=True)
    w = np.exp(logits - m)
    z = w.sum(axis=1, keepdims=True)
    return (w @ np.asarray(V, np.float64)) / z, (m + np.log(z))[:, 0]


# --------------------------------------------------------------------------- acceptance band
def near_cutoff_exempt(S_row: np.ndarray, forced: np.ndarray, mode: str, k: int = 0,
                       mass: float = 0.0, rel: float = 1e-5, mass_rel: float = None) -> Tuple[np.ndarray, bool]:
    """Blocks of one row whose membership may legitimately differ from the
    oracle's list: selectable blocks whose score lies within rel*|c| of the
    cutoff score c (top-k: the k-th best; mass: the r*-th).  In mass mode the
    second value tells whether the cumulative mass just before or just after
    the r*-th block is within mass_rel*p of p (mass_rel defaults to rel); then
    the prefix may end one block earlier or later, so the blocks of ranks r*
    and r*+1 are exempt and the count may differ by one.  (Rank r*-1 is never
    exempt on this account: a prefix that stops before it has a mass further
    from p than the one that stops before r*.)"""
    sel = np.nonzero(~forced)[0]
    ex = np.zeros(S_row.shape[0], dtype=bool)
    if sel.size == 0:
        return ex, False
    s = S_row[sel]
    mass_edge = False
    if mode == "mass":
        width = (rel if mass_rel is None else mass_rel) * mass
        r, order, c = mass_prefix_length(s, mass)
        cut = s[order[r - 1]]
        before = c[r - 2] if r >= 2 else 0.0
        if abs(c[r - 1] - mass) <= width or abs(before - mass) <= width:
            mass_edge = True
            ex[sel[order[r - 1:r + 1]]] = True
    else:
        if k <= 0:
            return ex, False
        order = _descending_order(s)
        cut = s[order[min(k, s.size) - 1]]
    ex[sel[np.abs(s - cut) <= rel * abs(cut)]] = True
    return ex, mass_edge


# --------------------------------------------------------------------------- clip policy
def keep_ranges(clip: int, text_range: Tuple[int, int], ref_range: Tuple[int, int]) -> List[Tuple[int, int]]:
    """Eq. 3: the token ranges whose blocks are always retained.  Clip 1: text and the final
    image-pyramid (reference) range; clip c >= 2: text only."""
    if clip < 1:
        raise ValueError("clips are numbered from 1")
    out = [tuple(text_range)]
    if clip == 1:
        out.append(tuple(ref_range))
    return [r for r in out if r[1] > r[0]]


def density_lookup(table: Sequence[Tuple[int, float]], L_q: int):
    """rho_c(L_q): the density of the clip group's table for this query length, None when the
    scale is not sparsified (density-schedule paragraph of Sec. "Clip-Dependent Retained and
    Selectable Blocks": scales with the same token count share a fixed density)."""
    for (L, rho) in table:
        if L == L_q:
            return rho
    return None


# --------------------------------------------------------------------------- attention-mass analysis
def block_mass(Q: np.ndarray, K: np.ndarray, b: int, tau: float) -> np.ndarray:
    """Exact post-softmax attention mass per (query block, key block): M_ij = mean over the
    queries t of block i of sum over the keys u of block j of softmax_u(tau q_t . k_u), the
    quantity the paper's analysis calls retained attention mass when summed over a kept set
    (Sec. "Analysis").  Rows of M sum to 1."""
    L_q, L_k = Q.shape[0], K.shape[0]
    logits = tau * (np.asarray(Q, np.float64) @ np.asarray(K, np.float64).T)
    logits -= logits.max(axis=1, keepdims=True)
    P = np.exp(logits)
    P /= P.sum(axis=1, keepdims=True)
    n_q, n_k = num_blocks(L_q, b), num_blocks(L_k, b)
    M = np.zeros((n_q, n_k), dtype=np.float64)
    for i in range(n_q):
        rows = P[i * b:min((i + 1) * b, L_q)]
        for j in range(n_k):
            M[i, j] = rows[:, j * b:min((j + 1) * b, L_k)].sum(axis=1).mean()
    return M


def retained_mass(M: np.ndarray, lists: Sequence[Sequence[int]]) -> np.ndarray:
    """Per query block the attention mass that the kept set A_i retains: sum_{j in A_i} M_ij."""
    return np.array([M[i, np.asarray(l, dtype=np.int64)].sum() for i, l in enumerate(lists)])
