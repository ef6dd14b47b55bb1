"""Comparison selectors (sliding window, random blocks, cross-scale reuse): the oracle twins
against closed forms of their definitions, the library's host helpers against the twins, and on
the GPU the score arrays bit for bit against the twins and the lists they select against the
oracle's selection on the twins' scores."""
import numpy as np
import pytest

from oracle import selectors_oracle as so
from oracle import sparstar_oracle as orc


def _segs(w):
    """(length, grid) runs of a workload's keys; the queries are the last ("cur") run."""
    k = [(s.length, s.grid) for s in w.segments]
    return [k[-1]], k


# ----------------------------------------------------------------- twins against closed forms
def test_block_centres_closed_forms():
    T, H, W = 3, 4, 5
    c = so.block_centres([(T * H * W, (T, H, W))], H * W)            # one frame per block
    assert c.shape == (3, 3)
    for t in range(T):
        want = (t / T, ((H - 1) / 2) / H, ((W - 1) / 2) / W)
        assert all(abs(c[t, d] - want[d]) < 1e-15 for d in range(3))
    # tokens without a position sit at the centre
    assert np.all(so.block_centres([(10, None)], 4) == 0.5)
    # a block straddling text and a grid: (2 text tokens + tokens (0,0,0), (0,0,1)) / 4
    c = so.block_centres([(2, None), (8, (2, 2, 2))], 4)
    assert c[0, 0] == (1.0 + 0.0) / 4 and c[0, 1] == (1.0 + 0.0) / 4 and c[0, 2] == (1.0 + 0.5) / 4
    # ragged tail: the last block holds 2 tokens, (1,1,0) and (1,1,1)
    assert tuple(c[2]) == ((1 / 2 + 1 / 2) / 2, (1 / 2 + 1 / 2) / 2, (0 + 1 / 2) / 2)


def test_window_scores_closed_form_and_symmetry():
    seg = [(2 * 4 * 4, (2, 4, 4))]
    S = so.window_scores(seg, seg, 4)                                # blocks = rows of the raster
    assert S.dtype == np.float32 and S.shape == (8, 8)
    assert np.all(np.diag(S) == 0) and np.array_equal(S, S.T)
    assert S[0, 1] == np.float32(-0.25) and S[0, 4] == np.float32(-0.5)   # next row: dh = 1/4; next frame: dt = 1/2
    assert S[0, 5] == np.float32(-math_hypot(0.5, 0.25))


def math_hypot(a, b):
    return float(np.sqrt(np.float64(a) * a + np.float64(b) * b))


def test_random_scores_published_vector_and_range():
    # seed 0, first number: the mixing function's well-known first output 0xE220A8397B1DCDAF
    u = so.random_scores(0, (4,))
    assert u[0] == np.float32((0xE220A8397B1DCDAF >> 40) * 2.0 ** -24)
    r = so.random_scores(7, (2, 3, 50, 40))
    assert r.dtype == np.float32 and r.min() >= 0.0 and r.max() < 1.0 and abs(float(r.mean()) - 0.5) < 0.02
    assert not np.array_equal(r, so.random_scores(8, (2, 3, 50, 40)))
    assert np.array_equal(r.ravel()[:10], so.random_scores(7, (10,)))       # a function of the linear index


def test_nearest_map_and_remap_by_hand():
    fine = so.block_centres([(4 * 4 * 4, (4, 4, 4))], 4)              # 16 blocks: (t, h) rows
    coarse = so.block_centres([(2 * 2 * 4, (2, 2, 4))], 4)            # 4 blocks
    assert np.array_equal(so.nearest_block_map(fine, fine), np.arange(16))
    m = so.nearest_block_map(fine, coarse)
    # fine centres (t/4, h/4, 3/8), coarse centres (tc/2, hc/2, 3/8): t = 0, 1 -> tc = 0 (1/4 ties low), h likewise
    want = [(0 if t <= 1 else 1) * 2 + (0 if h <= 1 else 1) for t in range(4) for h in range(4)]
    assert list(m) == want
    coarse_scores = np.arange(12, dtype=np.float32).reshape(1, 1, 3, 4)
    out = so.remap_scores(coarse_scores, np.array([2, 0]), np.array([3, 3, 1]))
    assert out.shape == (1, 1, 2, 3) and out[0, 0].tolist() == [[11, 11, 9], [3, 3, 1]]


# ----------------------------------------------------------------- host helpers against the twins
@pytest.fixture(scope="module")
def sp():
    from paper_2608_10519_b200 import build
    build.build()
    import paper_2608_10519_b200 as sp
    sp.binding.load()
    return sp


def test_host_helpers_match_twins(sp):
    from workloads import get_config
    for name in ("c0", "c1"):
        w = get_config(name)
        q_segs, k_segs = _segs(w)
        for segs in (q_segs, k_segs):
            got = np.array(sp.sparstar_block_centres(segs, w.block))
            assert np.array_equal(got, so.block_centres(segs, w.block))
    w = get_config("c0")
    q_segs, k_segs = _segs(w)
    fine, coarse = so.block_centres(k_segs, 64), so.block_centres(k_segs, 256)
    got = sp.sparstar_nearest_block_map([tuple(c) for c in fine], [tuple(c) for c in coarse])
    assert np.array_equal(np.array(got), so.nearest_block_map(fine, coarse))
    assert sp.binding.load().sparstar_block_centres(None, 0, 64, None) == -1


# ----------------------------------------------------------------- GPU
def _check_lists(num, idx, S, forced, k, tag):
    """validity + equality with the oracle's top-k on the twin's scores"""
    f_ids = set(np.nonzero(forced)[0].tolist())
    for i in range(S.shape[0]):
        row = idx[i, :num[i]]
        assert np.all(np.diff(row) > 0), (tag, i)                       # ascending, unique
        assert f_ids <= set(row.tolist()) and len(row) == len(f_ids) + k, (tag, i)
        assert np.array_equal(row, orc.select_topk_row(S[i].astype(np.float64), forced, k)), (tag, i)


@pytest.mark.gpu
def test_selectors_scores_and_lists_match_twins():
    import torch
    from paper_2608_10519_b200 import build
    build.build()
    import paper_2608_10519_b200 as sp
    from paper_2608_10519_b200.pipeline import SparstarAttention
    from workloads import generate, get_config
    eng = SparstarAttention(0)
    try:
        w = get_config("c0")
        q_segs, k_segs = _segs(w)
        B, H, n_q, n_k = w.B, w.H, w.n_q, w.n_k
        forced = orc.forced_blocks(w.L_k, w.block, w.forced_ranges())
        k = orc.budget(int((~forced).sum()), w.ratio)
        # sliding window
        s_win = torch.empty((B, H, n_q, n_k), dtype=torch.float32, device="cuda")
        sp.sparstar_window_scores(eng.ctx, q_segs, k_segs, w.block, s_win)
        want = so.window_scores(q_segs, k_segs, w.block)
        assert all(np.array_equal(s_win[0, h].cpu().numpy(), want) for h in range(H))
        num, idx = eng.select_from_scores(s_win, w.block, w.L_k, "topk_ratio", ratio=w.ratio, forced=w.forced_ranges())
        eng.check()
        _check_lists(num[0, 0].cpu().numpy(), idx[0, 0].cpu().numpy(), want, forced, k, "window")
        # random blocks
        s_rnd = torch.empty((B, H, n_q, n_k), dtype=torch.float32, device="cuda")
        sp.sparstar_random_scores(eng.ctx, 1234, s_rnd)
        want = so.random_scores(1234, (B, H, n_q, n_k))
        assert np.array_equal(s_rnd.cpu().numpy(), want)
        num, idx = eng.select_from_scores(s_rnd, w.block, w.L_k, "topk_ratio", ratio=w.ratio, forced=w.forced_ranges())
        eng.check()
        for h in range(H):
            _check_lists(num[0, h].cpu().numpy(), idx[0, h].cpu().numpy(), want[0, h], forced, k, f"random h{h}")
        # cross-scale reuse: the scores of the same inputs partitioned into 4x coarser blocks, carried
        # over to the fine blocks through nearest-centre maps
        x = generate(w, "cuda")
        cb = 4 * w.block
        _, _, s_coarse = eng.select(x["q"], x["k"], cb, "topk_ratio", ratio=w.ratio, forced=w.forced_ranges(),
                                    want_scores=True)
        cq_f, ck_f = so.block_centres(q_segs, w.block), so.block_centres(k_segs, w.block)
        cq_c, ck_c = so.block_centres(q_segs, cb), so.block_centres(k_segs, cb)
        q_map, k_map = so.nearest_block_map(cq_f, cq_c), so.nearest_block_map(ck_f, ck_c)
        lib_q = sp.sparstar_nearest_block_map([tuple(c) for c in cq_f], [tuple(c) for c in cq_c])
        assert np.array_equal(np.array(lib_q), q_map)
        s_re = torch.empty((B, H, n_q, n_k), dtype=torch.float32, device="cuda")
        sp.sparstar_remap_scores(eng.ctx, s_coarse, torch.from_numpy(q_map).cuda(), torch.from_numpy(k_map).cuda(), s_re)
        eng.check()
        want = so.remap_scores(s_coarse.cpu().numpy(), q_map, k_map)
        assert np.array_equal(s_re.cpu().numpy(), want)
        num, idx = eng.select_from_scores(s_re, w.block, w.L_k, "topk_ratio", ratio=w.ratio, forced=w.forced_ranges())
        eng.check()
        for h in range(H):
            _check_lists(num[0, h].cpu().numpy(), idx[0, h].cpu().numpy(), want[0, h], forced, k, f"reuse h{h}")
        # a map entry out of range is flagged, not followed
        bad = torch.from_numpy(q_map.copy()).cuda()
        bad[3] = 10 ** 6
        sp.sparstar_remap_scores(eng.ctx, s_coarse, bad, torch.from_numpy(k_map).cuda(), s_re)
        st, site = sp.sparstar_check(eng.ctx)
        assert st == sp.ERR_BAD_INDEX and site == 3
    finally:
        eng.close()
