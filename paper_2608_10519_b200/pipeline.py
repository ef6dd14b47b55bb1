"""Convenience layer over the binding: owns a context and allocates outputs with torch.
Every step still runs in the library's kernels; this file only sizes buffers."""
from __future__ import annotations

from typing import Optional, Sequence, Tuple

import torch

from . import binding as sp

_MODES = {"topk_ratio": sp.SEL_TOPK_RATIO, "topk_count": sp.SEL_TOPK_COUNT, "mass": sp.SEL_MASS}


class SparstarAttention:
    def __init__(self, device: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (no CPU fallback exists)")
        self.device = torch.device("cuda", device)
        with torch.cuda.device(self.device):
            self.ctx = sp.sparstar_create(device)

    def close(self):
        if self.ctx:
            sp.sparstar_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def check(self) -> None:
        st, site = sp.sparstar_check(self.ctx)
        if st != sp.OK:
            raise sp.SparstarError(st, f"device status (site {site})")

    def pool(self, x: torch.Tensor, block: int) -> torch.Tensor:
        B, H, L, D = x.shape
        out = torch.empty((B, H, sp.sparstar_num_blocks(L, block), D), dtype=torch.float32, device=x.device)
        sp.sparstar_pool_blocks(self.ctx, x, block, out)
        return out

    def select(self, q: torch.Tensor, k: torch.Tensor, block: int, mode: str, ratio: float = 0.0,
               count: int = 0, mass: float = 0.0, forced: Sequence[Tuple[int, int]] = (),
               scale: Optional[float] = None, cap: Optional[int] = None, want_scores: bool = False):
        """pool(Q), pool(K), score + select.  Returns (kv_num_blocks, kv_indices, scores|None)."""
        scale = q.shape[3] ** -0.5 if scale is None else scale
        qbar, kbar = self.pool(q, block), self.pool(k, block)
        B, H, n_q, _ = qbar.shape
        n_k = kbar.shape[2]
        cap = n_k if cap is None else cap
        num = torch.empty((B, H, n_q), dtype=torch.int32, device=q.device)
        idx = torch.empty((B, H, n_q, cap), dtype=torch.int32, device=q.device)
        scores = torch.empty((B, H, n_q, n_k), dtype=torch.float32, device=q.device) if want_scores else None
        sp.sparstar_score_select(self.ctx, qbar, kbar, block, k.shape[2], scale, _MODES[mode], num, idx,
                                 ratio=ratio, count=count, mass=mass, forced=forced, scores_out=scores)
        return num, idx, scores

    def select_fused(self, q: torch.Tensor, k: torch.Tensor, block: int, mode: str, ratio: float = 0.0,
                     count: int = 0, mass: float = 0.0, forced: Sequence[Tuple[int, int]] = (),
                     scale: Optional[float] = None, cap: Optional[int] = None,
                     k_cond_pooled: Optional[torch.Tensor] = None):
        """pool(Q), pool(K), score + select in ONE launch.  Returns (kv_num_blocks, kv_indices)."""
        scale = q.shape[3] ** -0.5 if scale is None else scale
        B, H, L_q, D = q.shape
        n_q, n_k = sp.sparstar_num_blocks(L_q, block), sp.sparstar_num_blocks(k.shape[2], block)
        cap = n_k if cap is None else cap
        qbar = torch.empty((B, H, n_q, D), dtype=torch.float32, device=q.device)
        kbar = torch.empty((B, H, n_k, D), dtype=torch.float32, device=q.device)
        num = torch.empty((B, H, n_q), dtype=torch.int32, device=q.device)
        idx = torch.empty((B, H, n_q, cap), dtype=torch.int32, device=q.device)
        sp.sparstar_select_fused(self.ctx, q, k, block, scale, _MODES[mode], qbar, kbar, num, idx, ratio=ratio,
                                 count=count, mass=mass, forced=forced, k_cond_pooled=k_cond_pooled)
        return num, idx

    def sparse_forward(self, q, k, v, block: int, kv_num_blocks, kv_indices, scale: Optional[float] = None,
                       want_lse: bool = False):
        scale = q.shape[3] ** -0.5 if scale is None else scale
        o = torch.empty_like(q)
        lse = torch.empty(q.shape[:3], dtype=torch.float32, device=q.device) if want_lse else None
        sp.sparstar_sparse_attn_fwd(self.ctx, q, k, v, o, block, scale, kv_num_blocks, kv_indices, lse)
        return (o, lse) if want_lse else o

    def dense_forward(self, q, k, v, block: int, scale: Optional[float] = None, want_lse: bool = False):
        scale = q.shape[3] ** -0.5 if scale is None else scale
        o = torch.empty_like(q)
        lse = torch.empty(q.shape[:3], dtype=torch.float32, device=q.device) if want_lse else None
        sp.sparstar_attn_fwd(self.ctx, q, k, v, o, block, scale, lse)
        return (o, lse) if want_lse else o

    def block_mass(self, q, k, v, block: int, scale: Optional[float] = None):
        """Exact attention mass per (query block, key block): a dense pass for the log-sum-exp,
        then the mass kernel.  Returns (mass [B,H,n_q,n_k], lse_dense)."""
        scale = q.shape[3] ** -0.5 if scale is None else scale
        _, lse = self.dense_forward(q, k, v, block, scale=scale, want_lse=True)
        B, H = q.shape[:2]
        n_q, n_k = sp.sparstar_num_blocks(q.shape[2], block), sp.sparstar_num_blocks(k.shape[2], block)
        mass = torch.empty((B, H, n_q, n_k), dtype=torch.float32, device=q.device)
        sp.sparstar_block_mass(self.ctx, q, k, block, scale, lse, mass)
        return mass, lse

    def select_from_scores(self, scores, block: int, L_k: int, mode: str, ratio: float = 0.0, count: int = 0,
                           mass: float = 0.0, forced: Sequence[Tuple[int, int]] = ()):
        B, H, n_q, n_k = scores.shape
        num = torch.empty((B, H, n_q), dtype=torch.int32, device=scores.device)
        idx = torch.empty((B, H, n_q, n_k), dtype=torch.int32, device=scores.device)
        sp.sparstar_select_from_scores(self.ctx, scores, block, L_k, _MODES[mode], num, idx, ratio=ratio, count=count,
                                       mass=mass, forced=forced)
        return num, idx

    def retained_mass(self, mass, kv_num_blocks, kv_indices):
        out = torch.empty(mass.shape[:3], dtype=torch.float32, device=mass.device)
        sp.sparstar_retained_mass(self.ctx, mass, kv_num_blocks, kv_indices, out)
        return out

    def forward(self, q, k, v, block: int, mode: str, **sel):
        """The whole hot path: pool -> score -> select -> sparse attention."""
        num, idx, _ = self.select(q, k, block, mode, **sel)
        return self.sparse_forward(q, k, v, block, num, idx, scale=sel.get("scale"))

    def forward_host(self, hq, hk, hv, ho, block: int, mode: str, chunk_heads: int = 4, **sel):
        """The whole hot path for Q, K, V in pinned host memory, O written to pinned host memory.
        Heads are independent, so they are streamed in chunks of at most `chunk_heads` heads: the
        host-to-device copy of chunk c+1 and the device-to-host copy of chunk c-1 overlap the
        kernels of chunk c (three streams, two device buffer sets).  Returns after everything has
        landed in `ho`."""
        B, H, L_q, D = hq.shape
        L_k = hk.shape[2]
        dev = self.device
        compute = torch.cuda.current_stream(dev)
        s_in, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        ch = max(1, min(chunk_heads, H))
        bufs = []
        for _ in range(2):
            bufs.append({
                "q": torch.empty((B, ch, L_q, D), dtype=hq.dtype, device=dev),
                "k": torch.empty((B, ch, L_k, D), dtype=hq.dtype, device=dev),
                "v": torch.empty((B, ch, L_k, D), dtype=hq.dtype, device=dev),
                "o": torch.empty((B, ch, L_q, D), dtype=hq.dtype, device=dev),
                "in": torch.cuda.Event(), "done": torch.cuda.Event(), "out": torch.cuda.Event(),
            })
        s_in.wait_stream(compute)
        s_out.wait_stream(compute)
        # The copies in are the bottleneck (PCIe), so the call ends one chunk's kernels and copy out
        # after the last byte has arrived: the last chunks are made small (.., ch, ch/2, ch/4, .., 1, 1).
        sizes, left = [], H
        while left > ch:
            sizes.append(ch)
            left -= ch
        while left > 1:
            sizes.append((left + 1) // 2)
            left -= sizes[-1]
        if left:
            sizes.append(left)
        starts = [sum(sizes[:i]) for i in range(len(sizes))]
        chunks = [(h0, h0 + n) for h0, n in zip(starts, sizes)]
        for c, (h0, h1) in enumerate(chunks):
            b = bufs[c % 2]
            n = h1 - h0
            with torch.cuda.stream(s_in):
                if c >= 2:
                    s_in.wait_event(b["done"])           # the kernels of chunk c-2 have read these inputs
                b["q"][:, :n].copy_(hq[:, h0:h1], non_blocking=True)
                b["k"][:, :n].copy_(hk[:, h0:h1], non_blocking=True)
                b["v"][:, :n].copy_(hv[:, h0:h1], non_blocking=True)
                b["in"].record(s_in)
            compute.wait_event(b["in"])
            if c >= 2:
                compute.wait_event(b["out"])             # O of chunk c-2 has left the buffer
            q, k, v = b["q"][:, :n], b["k"][:, :n], b["v"][:, :n]
            num, idx, _ = self.select(q, k, block, mode, **sel)
            sp.sparstar_sparse_attn_fwd(self.ctx, q, k, v, b["o"][:, :n], block,
                                        sel.get("scale") or D ** -0.5, num, idx)
            b["done"].record(compute)
            with torch.cuda.stream(s_out):
                s_out.wait_event(b["done"])
                ho[:, h0:h1].copy_(b["o"][:, :n], non_blocking=True)
                b["out"].record(s_out)
        compute.wait_stream(s_out)
        compute.wait_stream(s_in)
        torch.cuda.current_stream(dev).synchronize()


class ClipPyramid:
    """The clip-level policy around the operators: clip-dependent retained ranges (Eq. 3), the
    density schedule rho_c(L_q), and the block means of the conditioning keys computed once per
    clip.  Key order is (text, reference, current scale); the text + reference part is the same
    at every scale of a clip, so the means of the blocks that lie wholly inside it are cached and
    only the blocks from the first one that holds a current-scale token are pooled per scale."""

    def __init__(self, eng: SparstarAttention, clip: int, text_len: int, ref_len: int, block: int,
                 schedule: Sequence[Tuple[int, float]], extra_forced: Sequence[Tuple[int, int]] = ()):
        self.eng, self.block = eng, block
        self.cond_len = text_len + ref_len
        self.forced = sp.sparstar_keep_ranges(clip, (0, text_len), (text_len, self.cond_len)) + list(extra_forced)
        self.schedule = list(schedule)
        self.full_blocks = self.cond_len // block          # blocks with no current-scale token
        self.cond_pool = None

    def set_conditioning(self, k_cond: torch.Tensor) -> None:
        """k_cond [B,H,cond_len,D]: pools the blocks that never change within the clip."""
        assert k_cond.shape[2] == self.cond_len
        if self.full_blocks > 0:
            self.cond_pool = self.eng.pool(k_cond[:, :, :self.full_blocks * self.block], self.block)

    def density(self, L_q: int) -> Optional[float]:
        return sp.sparstar_density_lookup(self.schedule, L_q)

    def select(self, q, k):
        """Lists for one scale (k = conditioning + current keys)."""
        B, H, L_k, D = k.shape
        rho = self.density(q.shape[2])
        assert rho is not None, "this scale is not in the schedule (run it dense)"
        cond = self.cond_pool if (self.cond_pool is not None and self.full_blocks > 0) else None
        return self.eng.select_fused(q, k, self.block, "topk_ratio", ratio=rho, forced=self.forced, k_cond_pooled=cond)

    def forward(self, q, k, v):
        """One scale: sparse when the schedule lists its query length, dense otherwise."""
        if self.density(q.shape[2]) is None:
            return self.eng.dense_forward(q, k, v, self.block)
        num, idx = self.select(q, k)
        return self.eng.sparse_forward(q, k, v, self.block, num, idx)

    def capture(self, scales):
        """Chains the scales of a clip into one CUDA graph.  `scales` = list of (q, k, v) device
        tensors that stay alive and are refilled in place between replays.  Every scale is run
        once eagerly first (first-use set-up of the library: kernel attributes, scratch growth),
        then the same calls are captured.  Returns (graph, outputs); `graph.replay()` re-runs
        selection and attention of all scales on the tensors' current contents."""
        for (q, k, v) in scales:
            self.forward(q, k, v)
        torch.cuda.current_stream(self.eng.device).synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            outs = [self.forward(q, k, v) for (q, k, v) in scales]
        return graph, outs
