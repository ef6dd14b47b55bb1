"""ctypes binding of libsparstar.so: argument marshalling only.

Each function has the name of the C entry point it calls (see include/sparstar.h);
torch supplies device memory and the current stream, nothing else.  There is no
fallback: if the library is missing or a call returns a non-zero status, an
exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsparstar.so")

F32, BF16 = 0, 1
SEL_TOPK_RATIO, SEL_TOPK_COUNT, SEL_MASS = 0, 1, 2
ATTN_AUTO, ATTN_SIMT, ATTN_TCGEN05, ATTN_TCGEN05_2STREAM, ATTN_TCGEN05_PAIR = 0, 1, 2, 3, 4
SCORE_FP64, SCORE_TCGEN05 = 0, 1
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CAPACITY, ERR_BAD_INDEX, ERR_TIMEOUT, ERR_CUDA, ERR_TOO_LARGE, ERR_CAPTURE = range(9)

EXPORTS = (
    "sparstar_create", "sparstar_destroy", "sparstar_check", "sparstar_set_attn_impl", "sparstar_set_score_impl",
    "sparstar_launch_count", "sparstar_set_trace", "sparstar_set_debug", "sparstar_reserve_scratch",
    "sparstar_scratch_bytes", "sparstar_status_string", "sparstar_num_blocks", "sparstar_budget",
    "sparstar_forced_count", "sparstar_keep_ranges", "sparstar_density_lookup", "sparstar_schedule_preset",
    "sparstar_pool_blocks", "sparstar_pool_blocks_range", "sparstar_score_select", "sparstar_select_fused",
    "sparstar_sparse_attn_fwd", "sparstar_attn_fwd", "sparstar_sparse_attn_fwd_static",
    "sparstar_block_mass", "sparstar_select_from_scores", "sparstar_retained_mass",
    "sparstar_block_centres", "sparstar_nearest_block_map", "sparstar_window_scores", "sparstar_random_scores",
    "sparstar_remap_scores",
)


class SparstarError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


class _Range(C.Structure):
    _fields_ = [("begin", C.c_int64), ("end", C.c_int64)]


class _DensityEntry(C.Structure):
    _fields_ = [("L_q", C.c_int64), ("rho", C.c_double)]


class _Segment(C.Structure):
    _fields_ = [("length", C.c_int64), ("T", C.c_int32), ("H", C.c_int32), ("W", C.c_int32)]


class _Tensor(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("dtype", C.c_int32), ("B", C.c_int32), ("H", C.c_int32),
                ("L", C.c_int32), ("D", C.c_int32), ("sB", C.c_int64), ("sH", C.c_int64), ("sL", C.c_int64)]


class _SelectParams(C.Structure):
    _fields_ = [("mode", C.c_int32), ("count", C.c_int32), ("ratio", C.c_double), ("mass", C.c_double),
                ("forced", C.POINTER(_Range)), ("n_forced", C.c_int32)]


_lib = None


def load() -> C.CDLL:
    """Loads the shared library (built in-tree by build.py)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2608_10519_b200.build` "
                           "(there is no CPU or PyTorch fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, dbl, flt = C.c_void_p, C.c_int32, C.c_int64, C.c_double, C.c_float
    tp = C.POINTER(_Tensor)
    lib.sparstar_create.argtypes = [C.POINTER(vp), C.c_int]
    lib.sparstar_destroy.argtypes = [vp]
    lib.sparstar_check.argtypes = [vp, vp, C.POINTER(i32)]
    lib.sparstar_set_attn_impl.argtypes = [vp, i32]
    lib.sparstar_set_score_impl.argtypes = [vp, i32]
    lib.sparstar_set_trace.argtypes = [vp, vp, i32, i32]
    lib.sparstar_set_debug.argtypes = [vp, i32, i32]
    lib.sparstar_reserve_scratch.argtypes = [vp, i64, vp]
    lib.sparstar_scratch_bytes.argtypes = [vp]
    lib.sparstar_scratch_bytes.restype = i64
    lib.sparstar_launch_count.argtypes = [vp]
    lib.sparstar_launch_count.restype = i64
    lib.sparstar_status_string.argtypes = [C.c_int]
    lib.sparstar_status_string.restype = C.c_char_p
    lib.sparstar_num_blocks.argtypes = [i64, i32]
    lib.sparstar_num_blocks.restype = i32
    lib.sparstar_budget.argtypes = [i32, dbl]
    lib.sparstar_budget.restype = i32
    lib.sparstar_forced_count.argtypes = [i64, i32, C.POINTER(_Range), i32]
    lib.sparstar_forced_count.restype = i32
    lib.sparstar_pool_blocks.argtypes = [vp, tp, i32, vp, vp]
    lib.sparstar_pool_blocks_range.argtypes = [vp, tp, i32, i32, i32, vp, vp]
    lib.sparstar_keep_ranges.argtypes = [i32, _Range, _Range, C.POINTER(_Range)]
    lib.sparstar_keep_ranges.restype = i32
    lib.sparstar_density_lookup.argtypes = [C.POINTER(_DensityEntry), i32, i64, C.POINTER(dbl)]
    lib.sparstar_density_lookup.restype = i32
    lib.sparstar_schedule_preset.argtypes = [i32, C.POINTER(_DensityEntry)]
    lib.sparstar_schedule_preset.restype = i32
    lib.sparstar_score_select.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, i64, dbl,
                                          C.POINTER(_SelectParams), vp, vp, i32, vp, vp]
    lib.sparstar_select_fused.argtypes = [vp, tp, tp, i32, dbl, C.POINTER(_SelectParams), vp, i32, vp, vp, vp, vp, i32, vp]
    lib.sparstar_sparse_attn_fwd.argtypes = [vp, tp, tp, tp, tp, i32, flt, vp, vp, i32, vp, vp]
    lib.sparstar_attn_fwd.argtypes = [vp, tp, tp, tp, tp, i32, flt, vp, vp]
    lib.sparstar_block_mass.argtypes = [vp, tp, tp, i32, flt, vp, vp, vp]
    lib.sparstar_select_from_scores.argtypes = [vp, vp, i32, i32, i32, i32, i32, i64, C.POINTER(_SelectParams), vp, vp, i32, vp]
    lib.sparstar_retained_mass.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, vp]
    sp_ = C.POINTER(_Segment)
    lib.sparstar_block_centres.argtypes = [sp_, i32, i32, C.POINTER(dbl)]
    lib.sparstar_block_centres.restype = i32
    lib.sparstar_nearest_block_map.argtypes = [C.POINTER(dbl), i32, C.POINTER(dbl), i32, C.POINTER(i32)]
    lib.sparstar_nearest_block_map.restype = i32
    lib.sparstar_window_scores.argtypes = [vp, sp_, i32, sp_, i32, i32, i32, i32, vp, vp]
    lib.sparstar_random_scores.argtypes = [vp, C.c_uint64, i32, i32, i32, i32, vp, vp]
    lib.sparstar_remap_scores.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, i32, i32, vp, vp]
    lib.sparstar_sparse_attn_fwd_static.argtypes = [tp, tp, tp, tp, i32, flt, vp, vp, i32, vp, vp, vp]
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().sparstar_status_string(int(status)).decode()


def _raise(status: int, where: str):
    if status != OK:
        raise SparstarError(status, where)


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _tensor(t: torch.Tensor) -> _Tensor:
    if t.dim() != 4 or t.stride(3) != 1:
        raise ValueError("expected a [B,H,L,D] tensor with contiguous D")
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    dt = {torch.float32: F32, torch.bfloat16: BF16}[t.dtype]
    B, H, L, D = t.shape
    return _Tensor(t.data_ptr(), dt, B, H, L, D, t.stride(0), t.stride(1), t.stride(2))


def _ranges(ranges: Sequence[Tuple[int, int]]):
    arr = (_Range * max(1, len(ranges)))()
    for i, (b, e) in enumerate(ranges):
        arr[i].begin, arr[i].end = int(b), int(e)
    return arr


# ---- the C entry points, same names ------------------------------------------------------
def sparstar_create(device: int = 0) -> int:
    h = C.c_void_p()
    _raise(load().sparstar_create(C.byref(h), int(device)), "sparstar_create")
    return h.value


def sparstar_destroy(ctx: int) -> None:
    _raise(load().sparstar_destroy(ctx), "sparstar_destroy")


def sparstar_check(ctx: int, stream=None) -> Tuple[int, int]:
    """Synchronises the stream; returns (device status, site) and clears them."""
    site = C.c_int32(0)
    st = load().sparstar_check(ctx, _stream(stream), C.byref(site))
    return st, site.value


def sparstar_set_attn_impl(ctx: int, impl: int) -> None:
    _raise(load().sparstar_set_attn_impl(ctx, int(impl)), "sparstar_set_attn_impl")


def sparstar_set_score_impl(ctx: int, impl: int) -> None:
    _raise(load().sparstar_set_score_impl(ctx, int(impl)), "sparstar_set_score_impl")


def sparstar_set_debug(ctx: int, work_order_on: bool = True, drop_stage: int = -1) -> None:
    """Test aid (see the header): work order on/off, and the list position whose copy the TMA
    producer of the tensor-core attention skips so that a bounded wait runs out (-1 = off)."""
    _raise(load().sparstar_set_debug(ctx, 1 if work_order_on else 0, int(drop_stage)), "sparstar_set_debug")


def sparstar_reserve_scratch(ctx: int, nbytes: int, stream=None) -> None:
    _raise(load().sparstar_reserve_scratch(ctx, int(nbytes), _stream(stream)), "sparstar_reserve_scratch")


def sparstar_scratch_bytes(ctx: int) -> int:
    return int(load().sparstar_scratch_bytes(ctx))


def sparstar_launch_count(ctx: int) -> int:
    return int(load().sparstar_launch_count(ctx))


def sparstar_set_trace(ctx: int, buf: Optional[torch.Tensor], skip: int = 0) -> None:
    """buf: int64 CUDA tensor of shape [4, capacity, 2] (zero it first), or None to switch off."""
    if buf is None:
        _raise(load().sparstar_set_trace(ctx, None, 0, 0), "sparstar_set_trace")
        return
    assert buf.dtype == torch.int64 and buf.is_contiguous() and buf.dim() == 3 and buf.shape[0] == 4 and buf.shape[2] == 2
    _raise(load().sparstar_set_trace(ctx, buf.data_ptr(), buf.shape[1], int(skip)), "sparstar_set_trace")


def sparstar_num_blocks(L: int, block: int) -> int:
    return int(load().sparstar_num_blocks(int(L), int(block)))


def sparstar_budget(n_sel: int, ratio: float) -> int:
    return int(load().sparstar_budget(int(n_sel), float(ratio)))


def sparstar_forced_count(L_k: int, block: int, ranges: Sequence[Tuple[int, int]]) -> int:
    return int(load().sparstar_forced_count(int(L_k), int(block), _ranges(ranges), len(ranges)))


SCHEDULE_480P, SCHEDULE_720P_PYRAMID = 0, 1


def sparstar_keep_ranges(clip: int, text: Tuple[int, int], ref: Tuple[int, int]):
    out = (_Range * 2)()
    n = load().sparstar_keep_ranges(int(clip), _Range(*map(int, text)), _Range(*map(int, ref)), out)
    if n < 0:
        raise ValueError("sparstar_keep_ranges: invalid arguments")
    return [(out[i].begin, out[i].end) for i in range(n)]


def sparstar_density_lookup(table: Sequence[Tuple[int, float]], L_q: int) -> Optional[float]:
    """rho for this query length, or None when the scale is not in the table (stays dense)."""
    arr = (_DensityEntry * max(1, len(table)))()
    for i, (L, r) in enumerate(table):
        arr[i].L_q, arr[i].rho = int(L), float(r)
    rho = C.c_double(0.0)
    st = load().sparstar_density_lookup(arr, len(table), int(L_q), C.byref(rho))
    if st < 0:
        raise ValueError("sparstar_density_lookup: invalid arguments")
    return rho.value if st == 1 else None


def sparstar_schedule_preset(preset: int):
    arr = (_DensityEntry * 4)()
    n = load().sparstar_schedule_preset(int(preset), arr)
    if n < 0:
        raise ValueError("unknown schedule preset")
    return [(arr[i].L_q, arr[i].rho) for i in range(n)]


def sparstar_pool_blocks_range(ctx: int, x: torch.Tensor, block: int, first_block: int, n_blocks: int,
                               pooled: torch.Tensor, stream=None) -> None:
    nb = sparstar_num_blocks(x.shape[2], block)
    assert pooled.dtype == torch.float32 and pooled.is_contiguous()
    assert tuple(pooled.shape) == (x.shape[0], x.shape[1], nb, x.shape[3])
    t = _tensor(x)
    _raise(load().sparstar_pool_blocks_range(ctx, C.byref(t), int(block), int(first_block), int(n_blocks),
                                             pooled.data_ptr(), _stream(stream)), "sparstar_pool_blocks_range")


def sparstar_pool_blocks(ctx: int, x: torch.Tensor, block: int, pooled: torch.Tensor, stream=None) -> None:
    nb = sparstar_num_blocks(x.shape[2], block)
    assert pooled.dtype == torch.float32 and pooled.is_contiguous()
    assert tuple(pooled.shape) == (x.shape[0], x.shape[1], nb, x.shape[3])
    t = _tensor(x)
    _raise(load().sparstar_pool_blocks(ctx, C.byref(t), int(block), pooled.data_ptr(), _stream(stream)),
           "sparstar_pool_blocks")


def sparstar_score_select(ctx: int, q_pooled: torch.Tensor, k_pooled: torch.Tensor, block: int, L_k: int,
                          scale: float, mode: int, kv_num_blocks: torch.Tensor, kv_indices: torch.Tensor,
                          ratio: float = 0.0, count: int = 0, mass: float = 0.0,
                          forced: Sequence[Tuple[int, int]] = (), scores_out: Optional[torch.Tensor] = None,
                          stream=None) -> None:
    B, H, n_q, D = q_pooled.shape
    n_k = k_pooled.shape[2]
    assert q_pooled.is_contiguous() and k_pooled.is_contiguous()
    assert kv_num_blocks.dtype == torch.int32 and kv_indices.dtype == torch.int32
    assert kv_num_blocks.is_contiguous() and kv_indices.is_contiguous()
    assert tuple(kv_num_blocks.shape) == (B, H, n_q) and tuple(kv_indices.shape[:3]) == (B, H, n_q)
    cap = kv_indices.shape[3]
    if scores_out is not None:
        assert scores_out.dtype == torch.float32 and scores_out.is_contiguous()
        assert tuple(scores_out.shape) == (B, H, n_q, n_k)
    arr = _ranges(forced)
    p = _SelectParams(int(mode), int(count), float(ratio), float(mass), arr, len(forced))
    _raise(load().sparstar_score_select(
        ctx, q_pooled.data_ptr(), k_pooled.data_ptr(), B, H, n_q, n_k, D, int(block), int(L_k), float(scale),
        C.byref(p), kv_num_blocks.data_ptr(), kv_indices.data_ptr(), cap,
        None if scores_out is None else scores_out.data_ptr(), _stream(stream)), "sparstar_score_select")


def sparstar_select_fused(ctx: int, q: torch.Tensor, k: torch.Tensor, block: int, scale: float, mode: int,
                          q_pooled: torch.Tensor, k_pooled: torch.Tensor, kv_num_blocks: torch.Tensor,
                          kv_indices: torch.Tensor, ratio: float = 0.0, count: int = 0, mass: float = 0.0,
                          forced: Sequence[Tuple[int, int]] = (), k_cond_pooled: Optional[torch.Tensor] = None,
                          stream=None) -> None:
    """Pooling + scores + selection of one scale in one launch (see the header)."""
    B, H, L_q, D = q.shape
    n_q, n_k = sparstar_num_blocks(L_q, block), sparstar_num_blocks(k.shape[2], block)
    for t, n in ((q_pooled, n_q), (k_pooled, n_k)):
        assert t.dtype == torch.float32 and t.is_contiguous() and tuple(t.shape) == (B, H, n, D)
    assert kv_num_blocks.dtype == torch.int32 and kv_indices.dtype == torch.int32
    assert kv_num_blocks.is_contiguous() and kv_indices.is_contiguous()
    assert tuple(kv_num_blocks.shape) == (B, H, n_q) and tuple(kv_indices.shape[:3]) == (B, H, n_q)
    n_cond = 0
    if k_cond_pooled is not None:
        assert k_cond_pooled.dtype == torch.float32 and k_cond_pooled.is_contiguous()
        assert tuple(k_cond_pooled.shape[:2]) == (B, H) and k_cond_pooled.shape[3] == D
        n_cond = k_cond_pooled.shape[2]
    tq, tk = _tensor(q), _tensor(k)
    arr = _ranges(forced)
    p = _SelectParams(int(mode), int(count), float(ratio), float(mass), arr, len(forced))
    _raise(load().sparstar_select_fused(
        ctx, C.byref(tq), C.byref(tk), int(block), float(scale), C.byref(p),
        None if k_cond_pooled is None else k_cond_pooled.data_ptr(), n_cond, q_pooled.data_ptr(), k_pooled.data_ptr(),
        kv_num_blocks.data_ptr(), kv_indices.data_ptr(), kv_indices.shape[3], _stream(stream)), "sparstar_select_fused")


def sparstar_sparse_attn_fwd(ctx: int, q, k, v, o, block: int, scale: float, kv_num_blocks: torch.Tensor,
                             kv_indices: torch.Tensor, lse: Optional[torch.Tensor] = None, stream=None) -> None:
    tq, tk, tv, to = _tensor(q), _tensor(k), _tensor(v), _tensor(o)
    assert kv_num_blocks.dtype == torch.int32 and kv_indices.dtype == torch.int32
    assert kv_num_blocks.is_contiguous() and kv_indices.is_contiguous()
    if lse is not None:
        assert lse.dtype == torch.float32 and lse.is_contiguous() and tuple(lse.shape) == tuple(q.shape[:3])
    _raise(load().sparstar_sparse_attn_fwd(
        ctx, C.byref(tq), C.byref(tk), C.byref(tv), C.byref(to), int(block), float(scale),
        kv_num_blocks.data_ptr(), kv_indices.data_ptr(), kv_indices.shape[3],
        None if lse is None else lse.data_ptr(), _stream(stream)), "sparstar_sparse_attn_fwd")


def sparstar_attn_fwd(ctx: int, q, k, v, o, block: int, scale: float, lse: Optional[torch.Tensor] = None,
                      stream=None) -> None:
    tq, tk, tv, to = _tensor(q), _tensor(k), _tensor(v), _tensor(o)
    if lse is not None:
        assert lse.dtype == torch.float32 and lse.is_contiguous() and tuple(lse.shape) == tuple(q.shape[:3])
    _raise(load().sparstar_attn_fwd(
        ctx, C.byref(tq), C.byref(tk), C.byref(tv), C.byref(to), int(block), float(scale),
        None if lse is None else lse.data_ptr(), _stream(stream)), "sparstar_attn_fwd")


def sparstar_sparse_attn_fwd_static(q, k, v, o, block: int, scale: float, kv_num_blocks: torch.Tensor,
                                    kv_indices: torch.Tensor, lse: Optional[torch.Tensor] = None,
                                    status_out: Optional[torch.Tensor] = None, stream=None) -> None:
    """The sparse forward for callers that may not allocate device memory: no context, the
    scratch is a fixed array inside the library (see the header for its limits).  `status_out`:
    optional int32 CUDA tensor of 2 elements that receives {status, site}."""
    tq, tk, tv, to = _tensor(q), _tensor(k), _tensor(v), _tensor(o)
    assert kv_num_blocks.dtype == torch.int32 and kv_indices.dtype == torch.int32
    assert kv_num_blocks.is_contiguous() and kv_indices.is_contiguous()
    if lse is not None:
        assert lse.dtype == torch.float32 and lse.is_contiguous() and tuple(lse.shape) == tuple(q.shape[:3])
    if status_out is not None:
        assert status_out.dtype == torch.int32 and status_out.is_contiguous() and status_out.numel() >= 2
    _raise(load().sparstar_sparse_attn_fwd_static(
        C.byref(tq), C.byref(tk), C.byref(tv), C.byref(to), int(block), float(scale),
        kv_num_blocks.data_ptr(), kv_indices.data_ptr(), kv_indices.shape[3],
        None if lse is None else lse.data_ptr(), None if status_out is None else status_out.data_ptr(),
        _stream(stream)), "sparstar_sparse_attn_fwd_static")


def sparstar_block_mass(ctx: int, q, k, block: int, scale: float, lse_dense: torch.Tensor, mass_out: torch.Tensor,
                        stream=None) -> None:
    tq, tk = _tensor(q), _tensor(k)
    B, H, L_q, _ = q.shape
    n_q, n_k = sparstar_num_blocks(L_q, block), sparstar_num_blocks(k.shape[2], block)
    assert lse_dense.dtype == torch.float32 and lse_dense.is_contiguous() and tuple(lse_dense.shape) == (B, H, L_q)
    assert mass_out.dtype == torch.float32 and mass_out.is_contiguous() and tuple(mass_out.shape) == (B, H, n_q, n_k)
    _raise(load().sparstar_block_mass(ctx, C.byref(tq), C.byref(tk), int(block), float(scale), lse_dense.data_ptr(),
                                      mass_out.data_ptr(), _stream(stream)), "sparstar_block_mass")


def sparstar_select_from_scores(ctx: int, scores: torch.Tensor, block: int, L_k: int, mode: int,
                                kv_num_blocks: torch.Tensor, kv_indices: torch.Tensor, ratio: float = 0.0,
                                count: int = 0, mass: float = 0.0, forced: Sequence[Tuple[int, int]] = (),
                                stream=None) -> None:
    B, H, n_q, n_k = scores.shape
    assert scores.dtype == torch.float32 and scores.is_contiguous()
    assert kv_num_blocks.dtype == torch.int32 and kv_indices.dtype == torch.int32
    assert kv_num_blocks.is_contiguous() and kv_indices.is_contiguous()
    arr = _ranges(forced)
    p = _SelectParams(int(mode), int(count), float(ratio), float(mass), arr, len(forced))
    _raise(load().sparstar_select_from_scores(ctx, scores.data_ptr(), B, H, n_q, n_k, int(block), int(L_k), C.byref(p),
                                              kv_num_blocks.data_ptr(), kv_indices.data_ptr(), kv_indices.shape[3],
                                              _stream(stream)), "sparstar_select_from_scores")


def sparstar_retained_mass(ctx: int, mass: torch.Tensor, kv_num_blocks: torch.Tensor, kv_indices: torch.Tensor,
                           out: torch.Tensor, stream=None) -> None:
    B, H, n_q, n_k = mass.shape
    assert mass.dtype == torch.float32 and mass.is_contiguous() and out.dtype == torch.float32 and out.is_contiguous()
    assert tuple(out.shape) == (B, H, n_q) and tuple(kv_num_blocks.shape) == (B, H, n_q)
    _raise(load().sparstar_retained_mass(ctx, mass.data_ptr(), kv_num_blocks.data_ptr(), kv_indices.data_ptr(),
                                         B * H * n_q, n_k, kv_indices.shape[3], out.data_ptr(), _stream(stream)),
           "sparstar_retained_mass")


# ---- comparison selectors -----------------------------------------------------------------
def _segments(segs):
    """segs: sequence of (length, grid) with grid = (T, H, W) or None for tokens without a position."""
    arr = (_Segment * max(1, len(segs)))()
    for i, (length, grid) in enumerate(segs):
        arr[i].length = int(length)
        arr[i].T, arr[i].H, arr[i].W = (0, 0, 0) if grid is None else tuple(int(x) for x in grid)
    return arr


def sparstar_block_centres(segs, block: int):
    """Host helper: list of (t, h, w) centres of the blocks over the concatenated segments."""
    arr = _segments(segs)
    n = load().sparstar_block_centres(arr, len(segs), int(block), None)
    if n < 0:
        raise ValueError("sparstar_block_centres: invalid arguments")
    out = (C.c_double * (3 * n))()
    load().sparstar_block_centres(arr, len(segs), int(block), out)
    return [(out[3 * i], out[3 * i + 1], out[3 * i + 2]) for i in range(n)]


def sparstar_nearest_block_map(fine, coarse):
    """Host helper: for every fine centre the index of the nearest coarse centre (ties: lower index)."""
    nf, nc = len(fine), len(coarse)
    f = (C.c_double * (3 * nf))(*[x for c in fine for x in c])
    c = (C.c_double * (3 * nc))(*[x for cc in coarse for x in cc])
    out = (C.c_int32 * nf)()
    if load().sparstar_nearest_block_map(f, nf, c, nc, out) < 0:
        raise ValueError("sparstar_nearest_block_map: invalid arguments")
    return list(out)


def sparstar_window_scores(ctx: int, q_segs, k_segs, block: int, scores_out: torch.Tensor, stream=None) -> None:
    B, H = scores_out.shape[:2]
    assert scores_out.dtype == torch.float32 and scores_out.is_contiguous() and scores_out.is_cuda
    _raise(load().sparstar_window_scores(ctx, _segments(q_segs), len(q_segs), _segments(k_segs), len(k_segs), int(block),
                                         B, H, scores_out.data_ptr(), _stream(stream)), "sparstar_window_scores")


def sparstar_random_scores(ctx: int, seed: int, scores_out: torch.Tensor, stream=None) -> None:
    B, H, n_q, n_k = scores_out.shape
    assert scores_out.dtype == torch.float32 and scores_out.is_contiguous() and scores_out.is_cuda
    _raise(load().sparstar_random_scores(ctx, int(seed), B, H, n_q, n_k, scores_out.data_ptr(), _stream(stream)),
           "sparstar_random_scores")


def sparstar_remap_scores(ctx: int, coarse_scores: torch.Tensor, q_map: torch.Tensor, k_map: torch.Tensor,
                          scores_out: torch.Tensor, stream=None) -> None:
    B, H, n_qc, n_kc = coarse_scores.shape
    n_q, n_k = scores_out.shape[2:]
    assert coarse_scores.dtype == torch.float32 and coarse_scores.is_contiguous() and coarse_scores.is_cuda
    assert scores_out.dtype == torch.float32 and scores_out.is_contiguous() and tuple(scores_out.shape[:2]) == (B, H)
    assert q_map.dtype == torch.int32 and k_map.dtype == torch.int32 and q_map.is_cuda and k_map.is_cuda
    assert q_map.is_contiguous() and k_map.is_contiguous() and q_map.numel() == n_q and k_map.numel() == n_k
    _raise(load().sparstar_remap_scores(ctx, coarse_scores.data_ptr(), B, H, n_qc, n_kc, q_map.data_ptr(),
                                        k_map.data_ptr(), n_q, n_k, scores_out.data_ptr(), _stream(stream)),
           "sparstar_remap_scores")
