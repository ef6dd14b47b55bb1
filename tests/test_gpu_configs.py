"""Parity on the benchmark configurations: config 0 in full (fp32), the bf16 configurations
at full size with the selection compared in full on sampled heads and the attention compared
on sampled (head, query block) units computed with the oracle's lists."""
import numpy as np
import pytest
import torch

from oracle import compare
from oracle import sparstar_oracle as orc
from tests.gpu_util import f64, lists_to_tensors, oracle_selection_head, sample_units
from workloads import generate, get_config, pyramid_sweep

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def eng():
    from paper_2608_10519_b200 import build
    build.build()
    from paper_2608_10519_b200.pipeline import SparstarAttention
    e = SparstarAttention(0)
    yield e
    e.close()


def test_config0_full_parity(eng):
    w = get_config("c0")
    x = generate(w, "cuda")
    q, k, v = x["q"], x["k"], x["v"]
    num, idx, _ = eng.select(q, k, w.block, w.mode, ratio=w.ratio, forced=w.forced_ranges())
    eng.check()
    num_h, idx_h = num.cpu().numpy(), idx.cpu().numpy()
    tau = w.D ** -0.5
    rep = compare.ListReport()
    all_lists = []
    for h in range(w.H):
        lists, S, forced = oracle_selection_head(w, q, k, h)
        all_lists.append(lists)
        compare.compare_lists(num_h[0, h], idx_h[0, h], lists, S, forced, w.mode,
                              k=orc.budget(int((~forced).sum()), w.ratio), tag=f"h{h}", report=rep)
    assert rep.ok and rep.exact == rep.rows, rep.bad[:5]
    on, oi = lists_to_tensors(all_lists, w.n_k, "cuda")
    o, lse = eng.sparse_forward(q, k, v, w.block, on, oi, want_lse=True)
    od = eng.dense_forward(q, k, v, w.block)
    # the whole path in one call gives the same result as its steps
    o2 = eng.forward(q, k, v, w.block, w.mode, ratio=w.ratio, forced=w.forced_ranges())
    eng.check()
    assert torch.equal(o, o2)
    for h in range(w.H):
        want, want_lse = orc.sparse_attention(f64(q[0, h]), f64(k[0, h]), f64(v[0, h]), all_lists[h], w.block, tau)
        compare.check_output(f64(o[0, h]), want, "f32", f"sparse h{h}")
        assert np.abs(f64(lse[0, h]) - want_lse).max() <= 1e-4
        wantd, _ = orc.dense_attention(f64(q[0, h]), f64(k[0, h]), f64(v[0, h]), tau)
        compare.check_output(f64(od[0, h]), wantd, "f32", f"dense h{h}")


ATTN_HEADS = (0, 7, 19, 31)


def _full_size_case(eng, w, sel_heads, n_hashed, attn_heads=None, dense_units=0):
    """Selection on the whole tensor, compared in full on `sel_heads` ("all" = every head); sparse
    attention on the whole tensor in the benchmark's launch configuration with the ORACLE's lists
    on those heads (the CUDA lists elsewhere), compared on sampled (head, query block) units of
    `attn_heads` (default: the selection heads); `dense_units` of those units are also checked
    on the dense comparison kernel."""
    x = generate(w, "cuda")
    q, k, v = x["q"], x["k"], x["v"]
    num, idx, _ = eng.select(q, k, w.block, w.mode, ratio=w.ratio, mass=w.mass, forced=w.forced_ranges())
    eng.check()
    tau = w.D ** -0.5
    sel_heads = tuple(range(w.H)) if sel_heads == "all" else tuple(sel_heads)
    attn_heads = tuple(h for h in (attn_heads or sel_heads) if h in sel_heads)
    rep = compare.ListReport()
    num_h, idx_h = num[0].cpu().numpy(), idx[0].cpu().numpy()
    num_o, idx_o = num_h.copy(), idx_h.copy()
    oracle_lists = {}
    for h in sel_heads:
        lists, S, forced = oracle_selection_head(w, q, k, h)
        if h in attn_heads:
            oracle_lists[h] = lists
        kk = orc.budget(int((~forced).sum()), w.ratio) if w.mode != "mass" else 0
        compare.compare_lists(num_h[h], idx_h[h], lists, S, forced, w.mode,
                              k=kk, mass=w.mass, tag=f"{w.name} h{h}", report=rep)
        # forced blocks present, rows sorted and unique
        f_ids = np.nonzero(forced)[0]
        for i in range(0, w.n_q, max(1, w.n_q // 50)):
            row = idx_h[h, i, :num_h[h, i]]
            assert np.all(np.diff(row) > 0) and set(f_ids) <= set(row)
        for i, l in enumerate(lists):                      # the attention below runs with the oracle's lists
            num_o[h, i] = len(l)
            idx_o[h, i, :len(l)] = l
    print(f"{w.name}: lists on {len(sel_heads)} heads: rows {rep.rows} exact {rep.exact} excused {rep.excused}")
    assert rep.ok, rep.bad[:5]
    assert rep.excused <= max(2, rep.rows // 500), (rep.excused, rep.rows)
    num2, idx2 = torch.from_numpy(num_o)[None].cuda(), torch.from_numpy(idx_o)[None].cuda()
    o, lse = eng.sparse_forward(q, k, v, w.block, num2, idx2, want_lse=True)
    eng.check()
    units = [(h, i) for (h, i) in sample_units(w.n_q, w.H, w.seed, n_hashed, heads=attn_heads)]
    kcache = {h: (f64(k[0, h]), f64(v[0, h])) for h in attn_heads}
    worst = [0.0, 0.0]
    for (h, i) in units:
        r0, r1 = i * w.block, min((i + 1) * w.block, w.L_q)
        Kh, Vh = kcache[h]
        want, want_lse = orc.attention_block(f64(q[0, h, r0:r1]), Kh, Vh, oracle_lists[h][i], w.block, tau)
        compare.check_output(f64(o[0, h, r0:r1]), want, "bf16", f"{w.name} sparse unit h{h} i{i}")
        mx, mean = compare.output_errors(f64(o[0, h, r0:r1]), want)
        worst = [max(worst[0], mx), max(worst[1], mean)]
        assert np.abs(f64(lse[0, h, r0:r1]) - want_lse).max() <= 1e-3
    print(f"{w.name}: sparse attention on {len(units)} units: worst max-abs {worst[0]:.2e}, worst mean-abs {worst[1]:.2e}")
    if dense_units:
        del o, lse
        od = eng.dense_forward(q, k, v, w.block)
        eng.check()
        step = max(1, len(units) // dense_units)
        for (h, i) in units[::step][:dense_units]:
            r0, r1 = i * w.block, min((i + 1) * w.block, w.L_q)
            want, _ = orc.dense_attention(f64(q[0, h, r0:r1]), *kcache[h], tau)
            compare.check_output(f64(od[0, h, r0:r1]), want, "bf16", f"{w.name} dense unit h{h} i{i}")
        print(f"{w.name}: dense attention checked on {min(dense_units, len(units[::step]))} units")
    return q, k, v, kcache, units, rep


def test_config1_mid_scale(eng):
    _full_size_case(eng, get_config("c1"), sel_heads="all", n_hashed=11, attn_heads=ATTN_HEADS, dense_units=2)


def test_config2_final_scale(eng):
    """The headline configuration: lists on all 32 heads, sparse attention on 64 (head, query
    block) units, the dense comparison kernel (the denominator of the speed-up) on 8 of them."""
    _full_size_case(eng, get_config("c2"), sel_heads="all", n_hashed=11, attn_heads=ATTN_HEADS, dense_units=8)


def test_config3_first_clip(eng):
    w = get_config("c3")
    q, k, v, kcache, units, rep = _full_size_case(eng, w, sel_heads="all", n_hashed=11, attn_heads=ATTN_HEADS,
                                                  dense_units=8)
    assert rep.exact + rep.excused == rep.rows


@pytest.mark.parametrize("block", [64, 32])
def test_config3_small_blocks_full_length(eng, block):
    """Selection blocks of 64 / 32 tokens at the 72k scale (four heads): long gathered lists on
    every SM for many waves, where the TMA producer trails the issuing thread the most."""
    from dataclasses import replace
    w = replace(get_config("c3"), H=4, block=block, name=f"c3_b{block}")
    _full_size_case(eng, w, sel_heads=(1,), n_hashed=4)


def test_config4_pyramid_scale(eng):
    # one scale of the sweep at the extreme densities (cutoff near the median score at 0.5): the
    # sparsest on every head, the densest on one
    _full_size_case(eng, pyramid_sweep(0)[1], sel_heads="all", n_hashed=11, attn_heads=ATTN_HEADS)
    _full_size_case(eng, pyramid_sweep(4)[1], sel_heads=(3,), n_hashed=2)


def test_forward_host_streams_head_chunks(eng):
    """Host-resident inputs streamed by head chunks give bit-identical output to the device path."""
    w = get_config("c0")
    x = generate(w, "cuda")
    want = eng.forward(x["q"], x["k"], x["v"], w.block, w.mode, ratio=w.ratio, forced=w.forced_ranges())
    hq, hk, hv = (x[n].cpu().pin_memory() for n in ("q", "k", "v"))
    for chunk in (1, 2, 5):
        ho = torch.zeros(want.shape, dtype=want.dtype).pin_memory()
        eng.forward_host(hq, hk, hv, ho, w.block, w.mode, chunk_heads=chunk, ratio=w.ratio, forced=w.forced_ranges())
        eng.check()
        assert torch.equal(ho, want.cpu())
    # bf16 tensor-core shape, three chunks of unequal size
    g = torch.Generator().manual_seed(9)
    mk = lambda L: torch.randn((1, 5, L, 128), generator=g).to(torch.bfloat16)
    hq, hk, hv = mk(300).pin_memory(), mk(1000).pin_memory(), mk(1000).pin_memory()
    want = eng.forward(hq.cuda(), hk.cuda(), hv.cuda(), 128, "mass", mass=0.8, forced=[(0, 100)])
    ho = torch.zeros(want.shape, dtype=want.dtype).pin_memory()
    eng.forward_host(hq, hk, hv, ho, 128, "mass", chunk_heads=2, mass=0.8, forced=[(0, 100)])
    eng.check()
    assert torch.equal(ho, want.cpu())


@pytest.mark.parametrize("d,s", [(1, 0), (2, 2), (3, 3)])
def test_config4_more_scales(eng, d, s):
    _full_size_case(eng, pyramid_sweep(d)[s], sel_heads=(11,), n_hashed=1)


def test_clip_pyramid_policy(eng):
    """Clip policy on a shrunken pyramid: cached conditioning means + per-scale pooling give the
    lists of the plain path and of the oracle; a scale outside the schedule runs dense."""
    from paper_2608_10519_b200.pipeline import ClipPyramid
    g = torch.Generator().manual_seed(21)
    text_len, ref_len, H = 200, 1500, 2                      # conditioning ends mid-block (1700 = 13.28 blocks)
    mk = lambda L: torch.randn((1, H, L, 128), generator=g).to(torch.bfloat16).cuda()
    k_cond, v_cond = mk(text_len + ref_len), mk(text_len + ref_len)
    schedule = [(640, 0.625), (1000, 0.1875)]
    for clip in (1, 2):
        pyr = ClipPyramid(eng, clip, text_len, ref_len, 128, schedule)
        pyr.set_conditioning(k_cond)
        assert pyr.full_blocks == 13
        for L_q in (640, 1000, 300):
            q, kc, vc = mk(L_q), mk(L_q), mk(L_q)
            k, v = torch.cat([k_cond, kc], dim=2), torch.cat([v_cond, vc], dim=2)
            o = pyr.forward(q, k, v)
            eng.check()
            tau = 128 ** -0.5
            rho = orc.density_lookup(schedule, L_q)
            forced = orc.keep_ranges(clip, (0, text_len), (text_len, text_len + ref_len))
            for h in range(H):
                if rho is None:
                    want, _ = orc.dense_attention(f64(q[0, h]), f64(k[0, h]), f64(v[0, h]), tau)
                else:
                    lists, S, fm = orc.select_head(f64(q[0, h]), f64(k[0, h]), 128, tau, forced, "topk_ratio", ratio=rho)
                    num, idx = pyr.select(q, k)
                    rep = compare.compare_lists(num[0, h].cpu().numpy(), idx[0, h].cpu().numpy(), lists, S, fm,
                                                "topk_ratio", k=orc.budget(int((~fm).sum()), rho))
                    assert rep.ok and rep.exact == rep.rows, rep.bad[:3]
                    want, _ = orc.sparse_attention(f64(q[0, h]), f64(k[0, h]), f64(v[0, h]), lists, 128, tau)
                compare.check_output(f64(o[0, h]), want, "bf16", f"clip {clip} L_q {L_q} h{h}")


@pytest.mark.parametrize("name", ["c2", "c3", "c4_d4_s3"])
def test_full_size_with_tcgen05_prescore(eng, name):
    import paper_2608_10519_b200 as sp
    sp.sparstar_set_score_impl(eng.ctx, sp.SCORE_TCGEN05)
    try:
        _full_size_case(eng, get_config(name), sel_heads=(5,), n_hashed=1)
    finally:
        sp.sparstar_set_score_impl(eng.ctx, sp.SCORE_FP64)


def test_clip_pyramid_graph_replay(eng):
    """Two scales of a clip chained in one CUDA graph: the replay reproduces the eager results and
    follows new contents of the input tensors."""
    from paper_2608_10519_b200.pipeline import ClipPyramid
    g = torch.Generator().manual_seed(31)
    text_len, ref_len, H = 128, 1000, 2
    mk = lambda L: torch.randn((1, H, L, 128), generator=g).to(torch.bfloat16).cuda()
    k_cond, v_cond = mk(text_len + ref_len), mk(text_len + ref_len)
    pyr = ClipPyramid(eng, 2, text_len, ref_len, 128, [(384, 0.5), (700, 0.25)])
    pyr.set_conditioning(k_cond)
    scales = []
    for L_q in (384, 700):
        scales.append((mk(L_q), torch.cat([k_cond, mk(L_q)], dim=2), torch.cat([v_cond, mk(L_q)], dim=2)))
    graph, outs = pyr.capture(scales)
    for rnd in range(2):
        if rnd == 1:                                   # new current-scale content, same buffers
            for (q, k, v) in scales:
                q.copy_(mk(q.shape[2]))
                k[:, :, text_len + ref_len:].copy_(mk(q.shape[2]))
        graph.replay()
        torch.cuda.synchronize()
        for (q, k, v), o in zip(scales, outs):
            want = pyr.forward(q, k, v)
            eng.check()
            assert torch.equal(o, want)


def test_clip_pyramid_full_size_with_the_papers_schedule(eng):
    """The four late scales of a later clip at full size (4,800 / 18,400 / 40,800 / 72,000 queries
    against 72,512 conditioning keys + themselves, 32 heads) with the paper's density schedule
    (0.625, 0.1875, 0.1875, 0.09375; clip >= 2: text kept, preceding-clip keys ranked jointly),
    conditioning block means pooled once, one fused selection launch per scale: lists on sampled
    heads and attention on sampled units against the oracle, then all four scales chained in one
    CUDA graph and replayed."""
    import paper_2608_10519_b200 as sp
    from paper_2608_10519_b200.pipeline import ClipPyramid
    scales = pyramid_sweep(0)
    schedule = sp.sparstar_schedule_preset(sp.SCHEDULE_720P_PYRAMID)
    assert [r for (_, r) in schedule] == [0.625, 0.1875, 0.1875, 0.09375]
    w0 = scales[0]
    text_len, ref_len = w0.segments[0].length, w0.segments[1].length
    pyr = ClipPyramid(eng, 2, text_len, ref_len, w0.block, schedule, extra_forced=[(0, w0.n_sink)])
    forced = orc.keep_ranges(2, (0, text_len), (text_len, text_len + ref_len)) + [(0, w0.n_sink)]
    tau = w0.D ** -0.5
    heads = (0, 31)
    tensors = []
    for w in scales:
        x = generate(w, "cuda")
        q, k, v = x["q"], x["k"], x["v"]
        tensors.append((q, k, v))
        if pyr.cond_pool is None:
            pyr.set_conditioning(k[:, :, :text_len + ref_len])
        else:                                              # the conditioning keys are the same at every scale of the clip
            assert torch.equal(k[:, :, :text_len + ref_len], tensors[0][1][:, :, :text_len + ref_len])
        rho = orc.density_lookup(schedule, w.L_q)
        l0 = sp.sparstar_launch_count(eng.ctx)
        num, idx = pyr.select(q, k)
        assert sp.sparstar_launch_count(eng.ctx) - l0 == 1          # pooling + scores + selection: one launch
        o, lse = eng.sparse_forward(q, k, v, w.block, num, idx, want_lse=True)
        eng.check()
        rep = compare.ListReport()
        for h in heads:
            lists, S, fm = orc.select_head(f64(q[0, h]), f64(k[0, h]), w.block, tau, forced, "topk_ratio", ratio=rho)
            compare.compare_lists(num[0, h].cpu().numpy(), idx[0, h].cpu().numpy(), lists, S, fm, "topk_ratio",
                                  k=orc.budget(int((~fm).sum()), rho), tag=f"{w.name} h{h}", report=rep)
            Kh, Vh = f64(k[0, h]), f64(v[0, h])
            got_lists = idx[0, h].cpu().numpy()
            got_num = num[0, h].cpu().numpy()
            for (_, i) in sample_units(w.n_q, 1, w.seed, 2, heads=(0,)):
                r0, r1 = i * w.block, min((i + 1) * w.block, w.L_q)
                want, want_lse = orc.attention_block(f64(q[0, h, r0:r1]), Kh, Vh, got_lists[i, :got_num[i]], w.block, tau)
                compare.check_output(f64(o[0, h, r0:r1]), want, "bf16", f"{w.name} h{h} i{i}")
                assert np.abs(f64(lse[0, h, r0:r1]) - want_lse).max() <= 1e-3
        print(f"{w.name}: rho {rho}: rows {rep.rows} exact {rep.exact} excused {rep.excused}")
        assert rep.ok and rep.exact == rep.rows, rep.bad[:3]      # exact lists: the outputs above were formed with the oracle's lists
    # the whole clip as one graph
    eager = [pyr.forward(q, k, v) for (q, k, v) in tensors]
    graph, outs = pyr.capture(tensors)
    for o_ in outs:
        o_.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    eng.check()
    for a, b in zip(eager, outs):
        assert torch.equal(a, b)
