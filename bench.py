#!/usr/bin/env python
"""Benchmark of the SparSTAR hot path on B200: one step = pool(Q), pool(K), score+select,
sparse attention forward over one synthetic 720p final-scale workload (72,000 queries,
144,512 keys, 32 heads, D = 128, blocks of 128, cumulative mass 0.90).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl reference]

Prints one JSON line (rank 0).  `value` = kept-block attention FLOPs of the whole job divided
by the time of the whole step (selection included), inputs resident in HBM.  For N > 1 launch
with torch.distributed.run; every rank runs the same-shaped workload on its own seed (the
path has no exchange step), timing is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "sparse_attn_effective_tflops_kept_blocks"
UNIT = "TFLOP/s"
# dram__bytes_read.sum / dram__bytes_write.sum of one sparse attention launch, as taken from the latest ncu capture
# of the small (few-head) case of config c2: a small data file kept beside the capture's summary
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "attn_tc_kernel_c2_traffic.json")
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS, source="fallback")


def measured_traffic(workload_name: str, heads: int, batch: int):
    """DRAM bytes of one sparse attention launch from the recorded ncu capture, scaled by heads (every
    head streams its own K/V, so the traffic grows in proportion).  None when no capture of this
    workload shape is on record."""
    if not workload_name.startswith("c2") or not os.path.exists(TRAFFIC_FILE):
        return None, None
    d = json.load(open(TRAFFIC_FILE))
    per_head = (float(d["dram_bytes_read"]) + float(d["dram_bytes_write"])) / float(d["heads"])
    return per_head * heads * batch, d.get("source")


def dense_library_times(q, k, v, scale, reps=2):
    """The dense comparison on library kernels (context for the repo's own dense kernel): torch
    scaled_dot_product_attention per available backend and FlashAttention-2 if importable, on the
    same tensors in this GPU's memory.  Returns {name: ms}."""
    import torch
    out = {}
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        a, b = ev(), ev()
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    try:
        from torch.nn.attention import SDPBackend, sdpa_kernel
        import torch.nn.functional as F
        for name, be in (("sdpa_flash", SDPBackend.FLASH_ATTENTION), ("sdpa_cudnn", SDPBackend.CUDNN_ATTENTION)):
            try:
                def run():
                    with sdpa_kernel([be]):
                        return F.scaled_dot_product_attention(q, k, v, scale=scale)
                out[name] = timed(run)
            except Exception:
                torch.cuda.synchronize()
    except Exception:
        pass
    try:
        from flash_attn import flash_attn_func
        qt, kt, vt = (t.transpose(1, 2) for t in (q, k, v))            # [B, L, H, D] views
        out["flash_attn2"] = timed(lambda: flash_attn_func(qt, kt, vt, softmax_scale=scale))
    except Exception:
        torch.cuda.synchronize()
    return out


def workload_config(w, in_gb: float, sharding: str):
    """The `config` object of the JSON line: the same keys and values in the CUDA arm and in the
    reference arm (static facts of the workload only)."""
    return {"workload": w.name, "L_q": w.L_q, "L_k": w.L_k, "H": w.H, "D": w.D, "block": w.block, "batch": w.B,
            "select": w.mode, "mass": w.mass, "ratio": w.ratio,
            "l2": (f"inputs ({in_gb:.2f} GB) exceed L2; no flush between steps" if in_gb > 0.2 else
                   f"inputs ({in_gb:.2f} GB) fit L2 and are not flushed: a profiling-size run, not a bench value"),
            "sharding": sharding}


def input_gb(w) -> float:
    esz = 2 if w.dtype == "bf16" else 4
    return (w.L_q + 2 * w.L_k) * w.D * w.H * w.B * esz / 1e9


def kept_flops(w, num, idx) -> float:
    """4*D*|B_i^q|*|B_j^k| summed over kept (query block, key block) pairs, valid tokens only."""
    import torch
    b = w.block
    qv = torch.full((w.n_q,), b, dtype=torch.float64, device=num.device)
    qv[-1] = w.L_q - (w.n_q - 1) * b
    tail = w.L_k - (w.n_k - 1) * b
    cnt = num.to(torch.float64)                                    # [B,H,n_q]
    ar = torch.arange(idx.shape[-1], device=idx.device)
    has_last = ((idx == w.n_k - 1) & (ar < num.unsqueeze(-1))).any(dim=-1).to(torch.float64)
    keys = cnt * b - has_last * (b - tail)
    return float((4.0 * w.D * keys * qv).sum().item())


SHARDING = {"weak": "one same-shaped workload per GPU, no collective",
            "strong": "the heads of ONE workload split across the GPUs, no collective"}


def rank_workload(w0, rank: int):
    """Weak scaling: rank r runs the same-shaped workload on its own seed (the path has no exchange step)."""
    from dataclasses import replace
    return replace(w0, seed=w0.seed + 1000 * rank) if rank else w0


def head_shard(H: int, rank: int, world: int):
    """Strong scaling: heads [h0, h1) of the one workload that rank `rank` of `world` owns.  Heads are
    independent (scores, selection and attention are per head), so the shards need no exchange.  The
    ranges tile 0..H-1 in rank order; the first H % world ranks hold one head more."""
    base, extra = divmod(H, world)
    h0 = rank * base + min(rank, extra)
    return h0, h0 + base + (1 if rank < extra else 0)


def reduce_over_ranks(times_ms, flops: float, device, dist=None):
    """Timing = maximum over ranks, work = sum over ranks.  `dist` is torch.distributed when more
    than one rank runs, else None."""
    if dist is None:
        return list(times_ms), float(flops)
    import torch
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    f = torch.tensor([flops], dtype=torch.float64, device=device)
    dist.all_reduce(f, op=dist.ReduceOp.SUM)
    return t.tolist(), float(f.item())


class ClockSampler:
    """Samples SM clock, power and clock-event reasons of one GPU every few ms on a host thread
    (NVML, read-only) while the timed region runs."""
    _REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, uuid: str, period_s: float = 0.005):
        import threading
        self.samples, self.stop_flag, self.thread, self.max_mhz = [], False, None, None
        try:
            import pynvml
            pynvml.nvmlInit()
            try:
                h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if isinstance(uuid, str) else uuid)
            except Exception:
                h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))

            def reasons():
                fn = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                    pynvml.nvmlDeviceGetCurrentClocksThrottleReasons
                return int(fn(h))

            def loop():
                while not self.stop_flag:
                    try:
                        self.samples.append((pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM),
                                             pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0, reasons()))
                    except Exception:
                        pass
                    time.sleep(period_s)

            self.thread = threading.Thread(target=loop, daemon=True)
            self.thread.start()
        except Exception:
            self.thread = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "power_w": None}
        if self.thread is None:
            return out
        self.stop_flag = True
        self.thread.join(timeout=2)
        if not self.samples:
            return out
        sm = sorted(s[0] for s in self.samples)
        out["sm_mhz"] = float(sm[len(sm) // 2])
        out["power_w"] = round(sum(s[1] for s in self.samples) / len(self.samples), 1)
        bits = 0
        for s_ in self.samples:
            bits |= s_[2]
        out["reasons"] = sorted(name for bit, name in self._REASONS.items() if bits & bit)
        out["samples"] = len(self.samples)
        return out


# --------------------------------------------------------------------------- oracle arm
def oracle_sample(w, n_units: int = 24, heads=(0, 1), host=None):
    """One bounded sample of the workload for the CPU oracle: for each head in `heads` the whole
    selection (pool, score, select for every query block) plus the attention of `n_units` evenly
    spaced query blocks.  `host` maps head -> (q, k, v) float64 arrays (the bits the GPU holds);
    missing heads are generated on the CPU.  Returns times and the throughput extrapolated to
    whole heads by kept-tile count."""
    import numpy as np
    from oracle import sparstar_oracle as orc
    from workloads import generate
    from workloads.configs import shrink
    tau = w.D ** -0.5
    t_sel = t_att = 0.0
    tiles_s = tiles_h = 0
    units_done = 0
    for h in heads:
        if h >= w.H:
            continue
        x = (host or {}).get(h) or oracle_sample.cache.get((w.name, w.seed, h))
        if x is None:
            # head h of the full workload = head 0 of the single-head workload shifted by h streams
            full = generate(shrink(w, h + 1), "cpu")
            x = tuple(full[n][0, h].double().numpy() for n in ("q", "k", "v"))
            oracle_sample.cache[(w.name, w.seed, h)] = x
        q, k, v = x
        t0 = time.perf_counter()
        lists, S, forced = orc.select_head(q, k, w.block, tau, w.forced_ranges(), w.mode, ratio=w.ratio, mass=w.mass)
        t_sel += time.perf_counter() - t0
        units = sorted({int(round(i * (w.n_q - 1) / max(n_units - 1, 1))) for i in range(n_units)})
        t0 = time.perf_counter()
        for i in units:
            r0, r1 = i * w.block, min((i + 1) * w.block, w.L_q)
            orc.attention_block(q[r0:r1], k, v, lists[i], w.block, tau)
        t_att += time.perf_counter() - t0
        tiles_s += sum(len(lists[i]) for i in units)
        tiles_h += sum(len(l) for l in lists)
        units_done += len(units)
    flops = 4.0 * w.D * w.block * w.block * tiles_h              # tile-nominal count for the sampled heads
    t_heads = t_sel + t_att * tiles_h / max(tiles_s, 1)
    return {"t_select_s": t_sel, "t_attn_sample_s": t_att, "units": units_done, "tiles_sample": tiles_s,
            "tiles_heads": tiles_h, "t_heads_extrapolated_s": t_heads, "tflops": flops / t_heads / 1e12,
            "heads": [h for h in heads if h < w.H]}


oracle_sample.cache = {}


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def resolve_workload(args):
    """The workload both arms run: the named configuration with the profiling overrides applied."""
    from dataclasses import replace
    from workloads import get_config
    w0 = get_config(args.workload)
    if args.heads:
        w0 = replace(w0, H=args.heads, name=f"{w0.name}_h{args.heads}")
    if args.block:
        w0 = replace(w0, block=args.block, name=f"{w0.name}_b{args.block}")
    return w0


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    w = resolve_workload(args)
    import numpy as np  # noqa: F401  (loads BLAS before counting threads)
    for _ in range(args.warmup):
        oracle_sample(w, n_units=2, heads=(0,))
    t0 = time.perf_counter()
    vals = [oracle_sample(w, n_units=8, heads=(0,)) for _ in range(args.steps)]
    dt = time.perf_counter() - t0
    v = sum(s["tflops"] for s in vals) / len(vals)
    sample = ("per step: oracle selection of 1 of %d heads in full + attention of 8 of its %d query blocks; "
              "throughput extrapolated to the head by kept-tile count" % (w.H, w.n_q))
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, input_gb(w), SHARDING[args.scaling]),
            "achieved_density": sum(s["tiles_heads"] for s in vals) / (len(vals) * w.n_q * w.n_k),
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# --------------------------------------------------------------------------- clip pyramid
def run_pyramid(args):
    """The four late scales of one later clip (c >= 2) with the paper's density schedule
    (0.625, 0.1875, 0.1875, 0.09375): text forced, preceding-clip keys ranked jointly, selection
    recomputed at every scale, conditioning block means pooled once per clip.  Prints one JSON
    line with per-scale and per-clip times against dense on the same GPU."""
    import torch
    import __graft_entry__ as ge
    ge.build()
    import paper_2608_10519_b200 as sp
    from paper_2608_10519_b200.pipeline import SparstarAttention, ClipPyramid
    from workloads import generate, pyramid_sweep
    eng = SparstarAttention(0)
    scales = pyramid_sweep(0)                      # shapes and shared conditioning streams; densities come from the schedule
    schedule = sp.sparstar_schedule_preset(sp.SCHEDULE_720P_PYRAMID)
    w0 = scales[0]
    text_len, ref_len = w0.segments[0].length, w0.segments[1].length
    pyr = ClipPyramid(eng, 2, text_len, ref_len, w0.block, schedule, extra_forced=[(0, w0.n_sink)])
    ev = lambda: torch.cuda.Event(enable_timing=True)
    out, tot_s, tot_d = [], 0.0, 0.0
    for w in scales:
        x = generate(w, "cuda")
        q, k, v = x["q"], x["k"], x["v"]
        pyr.set_conditioning(k[:, :, :text_len + ref_len])
        for _ in range(2):
            pyr.forward(q, k, v)
        torch.cuda.synchronize()
        reps = max(3, args.steps)
        l0 = sp.sparstar_launch_count(eng.ctx)
        e0, e1 = ev(), ev()
        e0.record()
        for _ in range(reps):
            pyr.forward(q, k, v)
        e1.record()
        torch.cuda.synchronize()
        launches = (sp.sparstar_launch_count(eng.ctx) - l0) // reps     # fused selection, work order, attention
        t_sparse = e0.elapsed_time(e1) / reps
        eng.dense_forward(q, k, v, w.block)
        torch.cuda.synchronize()
        d0, d1 = ev(), ev()
        d0.record()
        for _ in range(2):
            eng.dense_forward(q, k, v, w.block)
        d1.record()
        torch.cuda.synchronize()
        t_dense = d0.elapsed_time(d1) / 2
        num, idx = pyr.select(q, k)
        eng.check()
        out.append({"L_q": w.L_q, "L_k": w.L_k, "rho": pyr.density(w.L_q), "kept_density": float(num.double().mean()) / w.n_k,
                    "sparse_step_ms": t_sparse, "dense_ms": t_dense, "speedup": t_dense / t_sparse,
                    "launches_per_scale": int(launches)})
        tot_s += t_sparse
        tot_d += t_dense
        del x, q, k, v
    print(json.dumps({"metric": "clip_pyramid_attention_ms", "unit": "ms", "clip": 2, "schedule": schedule,
                      "scales": out, "clip_sparse_ms": tot_s, "clip_dense_ms": tot_d, "clip_speedup": tot_d / tot_s,
                      "data": "synthetic", "dtype": "bf16"}))


# --------------------------------------------------------------------------- block-size sweep
def run_block_sweep(args):
    """The whole path at the 72k scale for selection blocks of 32, 64, 128 and 256 tokens at the
    same keep ratio of selectable blocks (the block-size ablation's operating points): per block
    size the step time, the kept density, the attention mass the selection retains and the
    throughput on kept blocks, against dense."""
    import torch
    from dataclasses import replace
    import __graft_entry__ as ge
    ge.build()
    from paper_2608_10519_b200.pipeline import SparstarAttention
    from workloads import generate, get_config
    eng = SparstarAttention(0)
    w0 = get_config("c3")
    if args.heads:
        w0 = replace(w0, H=args.heads)
    x = generate(w0, "cuda")
    q, k, v = x["q"], x["k"], x["v"]
    ev = lambda: torch.cuda.Event(enable_timing=True)
    _, lse_dense = eng.dense_forward(q, k, v, 128, want_lse=True)
    torch.cuda.synchronize()
    d0, d1 = ev(), ev()
    d0.record()
    eng.dense_forward(q, k, v, 128)
    d1.record()
    torch.cuda.synchronize()
    t_dense = d0.elapsed_time(d1)
    rows = []
    for block in (32, 64, 128, 256):
        w = replace(w0, block=block)
        kw = dict(ratio=w.ratio, forced=w.forced_ranges())
        for _ in range(2):
            eng.forward(q, k, v, block, w.mode, **kw)
        torch.cuda.synchronize()
        reps = max(3, args.steps)
        e0, e1 = ev(), ev()
        e0.record()
        for _ in range(reps):
            eng.forward(q, k, v, block, w.mode, **kw)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        num, idx, _ = eng.select(q, k, block, w.mode, **kw)
        eng.check()
        flops = kept_flops(w, num, idx)
        # attention mass the selection retains = mean over queries of exp(LSE_sparse - LSE_dense)
        _, lse = eng.sparse_forward(q, k, v, block, num, idx, want_lse=True)
        retained = float(torch.exp(lse.double() - lse_dense.double()).mean().item())
        rows.append({"block": block, "n_q": w.n_q, "n_k": w.n_k, "kept_density": float(num.double().mean()) / w.n_k,
                     "retained_mass": retained, "step_ms": ms, "tflops_kept": flops / ms / 1e9,
                     "speedup_vs_dense": t_dense / ms})
    print(json.dumps({"metric": "block_size_sweep_step_ms", "unit": "ms", "workload": w0.name, "H": w0.H,
                      "ratio": w0.ratio, "dense_ms": t_dense, "blocks": rows, "data": "synthetic", "dtype": "bf16"}))


# --------------------------------------------------------------------------- attention-mass analysis
def run_mass_analysis(args):
    """Retained attention mass versus kept density on synthetic inputs: the aggregated-QK
    selector (the method) against the block-wise oracle selector (top-k on exact block masses)
    and a random selection of the same size.  Prints one JSON line."""
    import torch
    from dataclasses import replace
    import __graft_entry__ as ge
    ge.build()
    from paper_2608_10519_b200.pipeline import SparstarAttention
    from workloads import generate, get_config
    eng = SparstarAttention(0)
    w = replace(get_config(args.workload), H=args.heads or 4)
    x = generate(w, "cuda")
    q, k, v = x["q"], x["k"], x["v"]
    forced = w.forced_ranges()
    mass, _ = eng.block_mass(q, k, v, w.block)
    rows = []
    import paper_2608_10519_b200 as sp

    # comparison selectors of the paper's ablation (the library's own definitions; analysis only): score
    # arrays from the library's generators, turned into lists by sparstar_select_from_scores
    q_segs = [(w.segments[-1].length, w.segments[-1].grid)]
    k_segs = [(sg.length, sg.grid) for sg in w.segments]
    shape = (w.B, w.H, w.n_q, w.n_k)
    window = torch.empty(shape, dtype=torch.float32, device="cuda")
    sp.sparstar_window_scores(eng.ctx, q_segs, k_segs, w.block, window)
    noise = torch.empty(shape, dtype=torch.float32, device="cuda")
    sp.sparstar_random_scores(eng.ctx, 0, noise)
    # cross-scale reuse: the aggregated-QK scores of 4x coarser blocks carried over by nearest block centre
    cb = 4 * w.block
    _, _, coarse = eng.select(q, k, cb, "topk_ratio", ratio=0.5, forced=forced, want_scores=True)
    cq_f, ck_f = sp.sparstar_block_centres(q_segs, w.block), sp.sparstar_block_centres(k_segs, w.block)
    cq_c, ck_c = sp.sparstar_block_centres(q_segs, cb), sp.sparstar_block_centres(k_segs, cb)
    q_map = torch.tensor(sp.sparstar_nearest_block_map(cq_f, cq_c), dtype=torch.int32, device="cuda")
    k_map = torch.tensor(sp.sparstar_nearest_block_map(ck_f, ck_c), dtype=torch.int32, device="cuda")
    stale = torch.empty(shape, dtype=torch.float32, device="cuda")
    sp.sparstar_remap_scores(eng.ctx, coarse, q_map, k_map, stale)
    # token-wise top-K upper bound (the paper's reference curve): every sampled query keeps its own best
    # rho * L_k keys; plain torch on a sample of rows, analysis only
    rows_s = torch.linspace(0, w.L_q - 1, 512, device="cuda").long()
    logits = (q[0, 0, rows_s].float() @ k[0, 0].float().T) * (w.D ** -0.5)
    probs_sorted = torch.softmax(logits, dim=-1).sort(dim=-1, descending=True).values.cumsum(dim=-1)
    del logits
    for rho in (0.05, 0.09375, 0.1875, 0.3, 0.5):
        num_a, idx_a, _ = eng.select(q, k, w.block, "topk_ratio", ratio=rho, forced=forced)
        r = {}
        for name, sc in (("exact_block", mass), ("random", noise), ("sliding_window", window), ("reuse_of_coarser_blocks", stale)):
            n_, i_ = eng.select_from_scores(sc, w.block, w.L_k, "topk_ratio", ratio=rho, forced=forced)
            r[name] = float(eng.retained_mass(mass, n_, i_).double().mean())
        r["aggregated_qk"] = float(eng.retained_mass(mass, num_a, idx_a).double().mean())
        kept_keys = max(1, int(round(float(num_a.double().mean()) / w.n_k * w.L_k)))
        r["tokenwise_topk_head0_sample"] = float(probs_sorted[:, kept_keys - 1].double().mean())
        eng.check()
        rows.append({"rho": rho, "kept_density": float(num_a.double().mean()) / w.n_k, **r})
    print(json.dumps({"metric": "retained_attention_mass", "workload": w.name, "heads": w.H, "data": "synthetic",
                      "rows": rows}))


# --------------------------------------------------------------------------- CUDA arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--heads", type=int, default=0, help="use only the first HEADS heads (profiling captures)")
    ap.add_argument("--block", type=int, default=0, help="override the workload's selection block size (profiling captures)")
    ap.add_argument("--impl", default="sparstar", choices=["sparstar", "reference"])
    ap.add_argument("--score-impl", type=int, default=0,
                    help="scoring path of the library (sparstar_score_impl; 0 = fp64 MMA fused with the selection, "
                         "1 = tcgen05 split-bf16 pre-score launch + selection with exact re-scoring near the cutoff)")
    ap.add_argument("--attn-impl", type=int, default=0,
                    help="attention implementation of the library (sparstar_attn_impl; 0 = default, 4 = CTA pairs where "
                         "two query tiles share a list: the dense comparison and blocks of 256 / 512 tokens)")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="N > 1: weak = one workload per GPU (default), strong = the heads of one workload split across GPUs")
    ap.add_argument("--no-library-dense", action="store_true", help="skip the torch SDPA / FlashAttention-2 dense timings")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-dense", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--mass-analysis", action="store_true", help="retained attention mass vs density (analysis)")
    ap.add_argument("--pyramid", action="store_true", help="clip-pyramid report with the paper's density schedule")
    ap.add_argument("--block-sweep", action="store_true", help="whole path for selection blocks of 32..256 tokens")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "sparstar" else args.warmup
    if args.impl == "reference":
        return run_reference(args)
    if args.pyramid:
        return run_pyramid(args)
    if args.mass_analysis:
        return run_mass_analysis(args)
    if args.block_sweep:
        return run_block_sweep(args)

    import torch
    import torch.distributed as dist
    from dataclasses import replace
    import __graft_entry__ as ge
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if rank == 0:
        ge.build()
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    torch.cuda.set_device(local)
    import paper_2608_10519_b200 as sp
    from paper_2608_10519_b200.pipeline import SparstarAttention, _MODES
    from workloads import generate, get_config

    w0 = resolve_workload(args)
    dev = torch.device("cuda", local)
    if args.scaling == "strong" and world > 1:
        if w0.H < world:
            raise SystemExit(f"--scaling strong needs at least one head per GPU ({w0.H} heads, {world} GPUs)")
        h0, h1 = head_shard(w0.H, rank, world)
        x = generate(w0, dev, heads=(h0, h1))                 # this rank's heads of the SAME workload
        w = replace(w0, H=h1 - h0)
    else:
        w = rank_workload(w0, rank)
        x = generate(w, dev)
    q, k, v = x["q"], x["k"], x["v"]
    eng = SparstarAttention(local)
    if args.attn_impl:
        sp.sparstar_set_attn_impl(eng.ctx, args.attn_impl)
    if args.score_impl:
        sp.sparstar_set_score_impl(eng.ctx, args.score_impl)
    ctx = eng.ctx
    B, H, D, blk = w.B, w.H, w.D, w.block
    scale = D ** -0.5
    qbar = torch.empty((B, H, w.n_q, D), dtype=torch.float32, device=dev)
    kbar = torch.empty((B, H, w.n_k, D), dtype=torch.float32, device=dev)
    num = torch.empty((B, H, w.n_q), dtype=torch.int32, device=dev)
    idx = torch.empty((B, H, w.n_q, w.n_k), dtype=torch.int32, device=dev)
    o = torch.empty_like(q)
    forced = w.forced_ranges()
    stream = torch.cuda.current_stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def step(evs=None):
        if evs: evs[0].record(stream)
        sp.sparstar_pool_blocks(ctx, q, blk, qbar)
        sp.sparstar_pool_blocks(ctx, k, blk, kbar)
        if evs: evs[1].record(stream)
        sp.sparstar_score_select(ctx, qbar, kbar, blk, w.L_k, scale, _MODES[w.mode], num, idx,
                                 ratio=w.ratio, mass=w.mass, forced=forced)
        if evs: evs[2].record(stream)
        sp.sparstar_sparse_attn_fwd(ctx, q, k, v, o, blk, scale, num, idx)
        if evs: evs[3].record(stream)

    for _ in range(args.warmup):
        step()
    eng.check()
    flops = kept_flops(w, num, idx)
    density = float(num.double().mean().item()) / w.n_k
    in_gb = (q.numel() * q.element_size() + 2 * k.numel() * k.element_size()) / 1e9

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    evs = [[ev() for _ in range(4)] for _ in range(args.steps)]
    uuid = str(torch.cuda.get_device_properties(dev).uuid)
    uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
    sync_all()
    sampler = ClockSampler(uuid) if rank == 0 else None
    l0 = sp.sparstar_launch_count(ctx)
    e0, e1 = ev(), ev()
    e0.record(stream)
    for i in range(args.steps):
        step(evs[i])
    e1.record(stream)
    sync_all()
    launches = sp.sparstar_launch_count(ctx) - l0
    clocks = sampler.stop() if sampler else None
    eng.check()
    total_ms = e0.elapsed_time(e1)
    t_pool = sum(e[0].elapsed_time(e[1]) for e in evs) / args.steps
    t_sel = sum(e[1].elapsed_time(e[2]) for e in evs) / args.steps
    t_att = sum(e[2].elapsed_time(e[3]) for e in evs) / args.steps
    (total_ms, t_pool, t_sel, t_att), flops_all = reduce_over_ranks(
        [total_ms, t_pool, t_sel, t_att], flops, dev, dist if world > 1 else None)
    ms_per_step = total_ms / args.steps
    value = flops_all / (ms_per_step * 1e-3) / 1e12

    # dense comparison on the same GPU (outside the timed steps)
    dense_ms = None
    dense_lib = {}
    if not args.no_dense and not args.no_library_dense and rank == 0 and w.dtype == "bf16":
        dense_lib = dense_library_times(q, k, v, scale)
    if not args.no_dense:
        od = torch.empty_like(q)
        sp.sparstar_attn_fwd(ctx, q, k, v, od, blk, scale)
        torch.cuda.synchronize()
        d0, d1 = ev(), ev()
        d0.record(stream)
        for _ in range(2):
            sp.sparstar_attn_fwd(ctx, q, k, v, od, blk, scale)
        d1.record(stream)
        torch.cuda.synchronize()
        dense_ms = d0.elapsed_time(d1) / 2
        del od

    # end to end: host buffers in, host result out, through the public API, every step
    e2e = None
    if not args.no_e2e:
        hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
        ho = torch.empty(o.shape, dtype=o.dtype).pin_memory()

        def e2e_step():
            # public API with host buffers: head chunks are streamed (copies overlap the kernels)
            eng.forward_host(hq, hk, hv, ho, blk, w.mode, chunk_heads=4, ratio=w.ratio, mass=w.mass, forced=forced)

        e2e_step()
        sync_all()
        n_e2e = min(args.steps, 5)
        a0, a1 = ev(), ev()
        a0.record(stream)
        for _ in range(n_e2e):
            e2e_step()
        a1.record(stream)
        sync_all()
        ms = a0.elapsed_time(a1) / n_e2e
        (ms,), _ = reduce_over_ranks([ms], 0.0, dev, dist if world > 1 else None)
        e2e = {"value": flops_all / (ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms, "steps": n_e2e,
               "h2d_bytes_per_step": sum(t.numel() * t.element_size() for t in (hq, hk, hv)),
               "d2h_bytes_per_step": ho.numel() * ho.element_size()}

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    pk = peaks()
    att_tflops = flops / (t_att * 1e-3) / 1e12
    traffic, traffic_src = measured_traffic(w0.name, H, B)
    esz = q.element_size()
    # bytes one launch must move: Q in, O out, each K/V block once per head (all of them is the upper bound)
    algo_bytes = float((2 * q.numel() + k.numel() + v.numel()) * esz)
    dense_all = dict(dense_lib)
    if dense_ms is not None:
        dense_all["sparstar_attn_fwd"] = dense_ms
    dense_best = min(dense_all, key=dense_all.get) if dense_all else None
    wfull = w0
    pool_bytes = (q.numel() + k.numel()) * q.element_size() + (qbar.numel() + kbar.numel()) * 4
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": args.scaling if world > 1 else "weak",
        "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
        "config": workload_config(wfull, input_gb(w), SHARDING[args.scaling]),
        "achieved_density": density,
        "gpu_launches": int(launches),
        "clocks": clocks,
        "e2e": e2e,
        "roofline": {"bound": "tensor", "kernel": "attn_tc3_kernel (sparse forward)", "achieved": att_tflops,
                     "peak": pk["bf16_tflops"], "unit": "TFLOP/s", "frac": att_tflops / pk["bf16_tflops"],
                     "frac_of_sustained": att_tflops / pk["bf16_tflops_sustained"], "peak_source": pk["source"],
                     "traffic": traffic, "traffic_unit": "bytes per launch", "traffic_source": traffic_src,
                     "algorithmic_bytes": algo_bytes,
                     "traffic_over_algorithmic": None if traffic is None else traffic / algo_bytes,
                     "ms_per_launch": t_att, "flops_per_launch": flops,
                     # the same launch counted per kept tile (4*D*b^2 each, padding of partial blocks included),
                     # and against the nominal dense bf16 figure of the part (2,250 TFLOP/s, from its data sheet)
                     "achieved_tile_nominal": 4.0 * D * blk * blk * float(num.double().sum().item()) / (t_att * 1e-3) / 1e12,
                     "frac_of_nominal_2250": att_tflops / 2250.0},
        "speedup_attention_only_vs_dense": None if dense_ms is None else dense_ms / t_att,
        "breakdown_ms": {"pool": t_pool, "score_select": t_sel, "sparse_attn": t_att, "dense_attn": dense_ms},
        "pool_gbs": pool_bytes / (t_pool * 1e-3) / 1e9, "pool_frac_of_hbm": pool_bytes / (t_pool * 1e-3) / 1e9 / pk["hbm_gbs"],
        "selection_overhead": (t_pool + t_sel) / t_att,
        # the dense comparison: this library's dense kernel and library kernels on the same tensors; the
        # speed-up is taken against the FASTEST of them
        "dense_ms": dense_all, "dense_fastest": dense_best,
        "dense_sdpa_ms": min([v_ for n_, v_ in dense_lib.items() if n_.startswith("sdpa")], default=None),
        "speedup_vs_dense": None if dense_best is None else dense_all[dense_best] / ms_per_step,
        "speedup_vs_own_dense_kernel": None if dense_ms is None else dense_ms / ms_per_step,
        "dense_tflops": None if dense_ms is None else 4.0 * D * w.L_q * w.L_k * H * B / (dense_ms * 1e-3) / 1e12,
    }
    if world == 1 and not args.no_cpu_baseline:
        host = {h: tuple(t[0, h].cpu().double().numpy() for t in (q, k, v)) for h in (0, 1, 2) if h < H}
        s = oracle_sample(w0, n_units=96, heads=(0, 1, 2), host=host)
        line["cpu_baseline"] = {"value": s["tflops"], "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                                "sample": "oracle selection of heads %s in full (%.1f s) + attention of %d query blocks "
                                          "(%d kept tiles, %.1f s); extrapolated to those heads by kept-tile count"
                                          % (s["heads"], s["t_select_s"], s["units"], s["tiles_sample"],
                                             s["t_attn_sample_s"])}
    print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
