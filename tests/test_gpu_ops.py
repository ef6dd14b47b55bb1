"""Per-call parity of the CUDA library against the oracle on small and adversarial shapes
(ragged tails, tiny inputs, forced-only rows, ties, capacity, malformed lists)."""
import numpy as np
import pytest
import torch

from oracle import compare
from oracle import sparstar_oracle as orc
from tests.gpu_util import f64, lists_to_tensors

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def eng():
    from paper_2608_10519_b200 import build
    build.build()
    from paper_2608_10519_b200.pipeline import SparstarAttention
    e = SparstarAttention(0)
    yield e
    e.close()


def _rand(shape, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(shape, generator=g, dtype=torch.float32).to(dtype).cuda()


# ----------------------------------------------------------------- pooling
@pytest.mark.parametrize("dtype,D,block,L", [
    (torch.bfloat16, 128, 128, 128 * 5 + 37), (torch.bfloat16, 128, 128, 1), (torch.bfloat16, 128, 128, 127),
    (torch.bfloat16, 64, 64, 64 * 3), (torch.float32, 64, 64, 64 * 4 + 63), (torch.float32, 128, 128, 300),
    (torch.bfloat16, 128, 256, 1000), (torch.float32, 8, 16, 50),
])
def test_pool_matches_oracle(eng, dtype, D, block, L):
    x = _rand((2, 3, L, D), dtype, 1)
    got = eng.pool(x, block).cpu().numpy()
    for b in range(2):
        for h in range(3):
            want = orc.pool_blocks(f64(x[b, h]), block)
            assert np.abs(got[b, h] - want).max() <= 1e-5


def test_pool_strided_view(eng):
    big = _rand((1, 2, 300, 256), torch.bfloat16, 2)
    x = big[..., :128]                       # row stride 256 elements
    got = eng.pool(x, 128).cpu().numpy()
    want = orc.pool_blocks(f64(x[0, 1]), 128)
    assert np.abs(got[0, 1] - want).max() <= 1e-5


# ----------------------------------------------------------------- score + select
def _check_select(eng, q, k, block, mode, forced, ratio=0.0, count=0, mass=0.0, cap=None):
    import paper_2608_10519_b200 as sp
    num, idx, scores = eng.select(q, k, block, mode, ratio=ratio, count=count, mass=mass, forced=forced,
                                  cap=cap, want_scores=True)
    eng.check()
    num, idx, scores = num.cpu().numpy(), idx.cpu().numpy(), scores.cpu().numpy()
    B, H = q.shape[:2]
    tau = q.shape[3] ** -0.5
    rep = compare.ListReport()
    for b in range(B):
        for h in range(H):
            lists, S, fm = orc.select_head(f64(q[b, h]), f64(k[b, h]), block, tau, forced, mode,
                                           ratio=ratio, count=count, mass=mass)
            assert (np.abs(scores[b, h] - S) <= 1e-5 + 1.2e-7 * np.abs(S)).all()      # fp32 output of fp64 scores
            n_sel = int((~fm).sum())
            kk = orc.budget(n_sel, ratio) if mode == "topk_ratio" else min(n_sel, count)
            compare.compare_lists(num[b, h], idx[b, h], lists, S, fm, mode, k=kk, mass=mass,
                                  tag=f"b{b}h{h}", report=rep)
            for i, l in enumerate(lists):            # forced blocks always present
                assert set(np.nonzero(fm)[0]) <= set(idx[b, h, i, :num[b, h, i]])
    assert rep.ok, rep.bad[:5]
    return rep


@pytest.mark.parametrize("mode,kw", [("topk_ratio", {"ratio": 0.25}), ("topk_ratio", {"ratio": 1.0}),
                                     ("topk_ratio", {"ratio": 0.0}), ("topk_count", {"count": 3}),
                                     ("topk_count", {"count": 0}), ("mass", {"mass": 0.9}),
                                     ("mass", {"mass": 0.5}), ("mass", {"mass": 1.0})])
def test_select_small(eng, mode, kw):
    q = _rand((1, 3, 128 * 9 + 50, 128), torch.bfloat16, 3)
    k = _rand((1, 3, 128 * 40 + 17, 128), torch.bfloat16, 4)
    rep = _check_select(eng, q, k, 128, mode, [(0, 200), (1000, 1001)], **kw)
    assert rep.excused <= 1


def test_select_fp32_block64_unaligned_segments(eng):
    q = _rand((2, 2, 64 * 5, 64), torch.float32, 5)
    k = _rand((2, 2, 64 * 21 + 1, 64), torch.float32, 6)
    # paper key order: (ref, text, cur) puts the text range in the middle, straddling blocks
    _check_select(eng, q, k, 64, "topk_ratio", [(500, 700)], ratio=0.3)
    _check_select(eng, q, k, 64, "mass", [(500, 700)], mass=0.8)
    _check_select(eng, q, k, 64, "topk_ratio", [], ratio=0.3)              # nothing forced
    _check_select(eng, q, k, 64, "topk_ratio", [(0, 64 * 21 + 1)], ratio=0.3)  # everything forced


def test_select_ties_resolve_to_lower_index(eng):
    k = _rand((1, 1, 128 * 12, 128), torch.bfloat16, 7)
    k[0, 0, 128 * 6:128 * 7] = k[0, 0, 128 * 2:128 * 3]          # blocks 2 and 6 identical
    k[0, 0, 128 * 9:128 * 10] = k[0, 0, 128 * 2:128 * 3]         # and 9
    q = _rand((1, 1, 128 * 4, 128), torch.bfloat16, 8)
    for count in range(1, 12):
        _check_select(eng, q, k, 128, "topk_count", [], count=count)
    for mass in (0.2, 0.5, 0.7, 0.9):
        _check_select(eng, q, k, 128, "mass", [], mass=mass)


def test_select_capacity_is_reported_not_overrun(eng):
    import paper_2608_10519_b200 as sp
    q = _rand((1, 1, 128 * 2, 128), torch.bfloat16, 9)
    k = _rand((1, 1, 128 * 20, 128), torch.bfloat16, 10)
    qbar, kbar = eng.pool(q, 128), eng.pool(k, 128)
    num = torch.zeros((1, 1, 2), dtype=torch.int32, device="cuda")
    idx = torch.full((1, 1, 2, 8), -7, dtype=torch.int32, device="cuda")      # 4 live + 4 guard
    view = idx[..., :4].contiguous()
    sp.sparstar_score_select(eng.ctx, qbar, kbar, 128, 128 * 20, 128 ** -0.5, sp.SEL_TOPK_COUNT, num, view,
                             count=10)
    st, _ = sp.sparstar_check(eng.ctx)
    assert st == sp.ERR_CAPACITY
    assert num.cpu().tolist() == [[[10, 10]]]            # full count still reported
    st, _ = sp.sparstar_check(eng.ctx)
    assert st == sp.OK                                   # cleared


# ----------------------------------------------------------------- attention (SIMT family)
def _attn_case(eng, dtype, D, block, L_q, L_k, H, density, seed, impl):
    import paper_2608_10519_b200 as sp
    sp.sparstar_set_attn_impl(eng.ctx, impl)
    try:
        q = _rand((1, H, L_q, D), dtype, seed)
        k = _rand((1, H, L_k, D), dtype, seed + 1)
        v = _rand((1, H, L_k, D), dtype, seed + 2)
        n_q, n_k = orc.num_blocks(L_q, block), orc.num_blocks(L_k, block)
        rng = np.random.default_rng(seed)
        lists = [[np.sort(rng.choice(n_k, size=max(1, int(round(density * n_k))), replace=False)).astype(np.int32)
                  for _ in range(n_q)] for _ in range(H)]
        lists[0][0] = np.array([n_k - 1], dtype=np.int32)            # only the (partial) tail block
        lists[-1][-1] = np.arange(n_k, dtype=np.int32)               # everything
        num, idx = lists_to_tensors(lists, n_k, "cuda")
        tau = D ** -0.5
        o, lse = eng.sparse_forward(q, k, v, block, num, idx, want_lse=True)
        od, lsed = eng.dense_forward(q, k, v, block, want_lse=True)
        eng.check()
        name = "f32" if dtype == torch.float32 else "bf16"
        for h in range(H):
            want, want_lse = orc.sparse_attention(f64(q[0, h]), f64(k[0, h]), f64(v[0, h]), lists[h], block, tau)
            compare.check_output(f64(o[0, h]), want, name, f"sparse O h{h}")
            assert np.abs(f64(lse[0, h]) - want_lse).max() <= 1e-3
            wantd, want_lsed = orc.dense_attention(f64(q[0, h]), f64(k[0, h]), f64(v[0, h]), tau)
            compare.check_output(f64(od[0, h]), wantd, name, f"dense O h{h}")
            assert np.abs(f64(lsed[0, h]) - want_lsed).max() <= 1e-3
    finally:
        sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_AUTO)


@pytest.mark.parametrize("dtype,D,block,L_q,L_k", [
    (torch.float32, 64, 64, 64 * 3 + 5, 64 * 7 + 33), (torch.float32, 64, 64, 17, 40),
    (torch.bfloat16, 128, 128, 128 * 2 + 96, 128 * 6 + 32), (torch.bfloat16, 64, 64, 200, 500),
    (torch.bfloat16, 128, 64, 130, 333), (torch.float32, 128, 64, 100, 200),
])
def test_attention_simt(eng, dtype, D, block, L_q, L_k):
    _attn_case(eng, dtype, D, block, L_q, L_k, 2, 0.4, 11, 1)


@pytest.mark.parametrize("L_q,L_k,H,density", [
    (128, 128, 1, 1.0),                       # one tile: stream 1 stays empty
    (128 * 2 + 96, 128 * 6 + 32, 2, 0.4),     # ragged query and key tails
    (64, 128 * 3 + 1, 1, 0.7),                # fewer queries than a block, one key in the tail block
    (128 * 5, 128 * 33, 3, 0.15),             # long odd/even lists
])
def test_attention_tcgen05(eng, L_q, L_k, H, density):
    _attn_case(eng, torch.bfloat16, 128, 128, L_q, L_k, H, density, 13, 2)


@pytest.mark.parametrize("D,L_q,L_k,H,density", [(128, 128 * 2 + 96, 128 * 6 + 32, 2, 0.4), (128, 128 * 5, 128 * 33, 2, 0.15),
                                                 (64, 128 * 3, 128 * 20, 2, 0.2), (128, 128, 128, 1, 1.0)])
def test_attention_two_stream_kernel_cross_check(eng, D, L_q, L_k, H, density):
    """The older two-stream kernel (two score tiles, two accumulators merged at the end), selectable
    as ATTN_TCGEN05_2STREAM: the same oracle, an independent pipeline."""
    _attn_case(eng, torch.bfloat16, D, 128, L_q, L_k, H, density, 17, 3)


@pytest.mark.parametrize("block,L_q,L_k,H,density", [
    (256, 256 * 2 + 100, 256 * 5 + 130, 2, 0.5),     # odd number of query tiles: the last pair has an empty second CTA
    (512, 512 + 300, 512 * 3 + 129, 2, 0.6),
    (256, 200, 256 * 3 + 7, 1, 0.7),
    (128, 128 * 5, 128 * 11 + 20, 3, 0.3),           # blocks of one tile: the sparse call stays on single CTAs, the dense one pairs
])
def test_attention_cta_pairs(eng, block, L_q, L_k, H, density):
    """ATTN_TCGEN05_PAIR: two adjacent query tiles that walk the same list (dense, blocks of 256 / 512
    tokens) on a pair of CTAs issuing cta_group::2 MMAs, each CTA holding half of every K and V tile.
    Against the oracle, and bit-identical to the single-CTA kernel over repeated runs (same arithmetic in
    the same order; repeated because the hand-over between the two CTAs is timing dependent)."""
    import paper_2608_10519_b200 as sp
    _attn_case(eng, torch.bfloat16, 128, block, L_q, L_k, H, density, 23, sp.ATTN_TCGEN05_PAIR)
    q = _rand((2, H, L_q, 128), torch.bfloat16, 31)
    k = _rand((2, H, L_k, 128), torch.bfloat16, 32)
    v = _rand((2, H, L_k, 128), torch.bfloat16, 33)
    n_q, n_k = orc.num_blocks(L_q, block), orc.num_blocks(L_k, block)
    rng = np.random.default_rng(5)
    lists = [[np.sort(rng.choice(n_k, size=max(1, int(round(density * n_k))), replace=False)).astype(np.int32)
              for _ in range(n_q)] for _ in range(2 * H)]
    num, idx = lists_to_tensors(lists, n_k, "cuda")
    num, idx = num.view(2, H, n_q), idx.view(2, H, n_q, -1)
    want_s = eng.sparse_forward(q, k, v, block, num, idx)
    want_d = eng.dense_forward(q, k, v, block)
    sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_TCGEN05_PAIR)
    try:
        for _ in range(8):
            assert torch.equal(eng.sparse_forward(q, k, v, block, num, idx), want_s)
            assert torch.equal(eng.dense_forward(q, k, v, block), want_d)
        eng.check()
    finally:
        sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_AUTO)


def test_attention_tcgen05_strided_inputs_and_rerun(eng):
    """Non-contiguous views (packed QKV-style buffer) and bit-reproducibility of two runs."""
    import paper_2608_10519_b200 as sp
    g = torch.Generator().manual_seed(3)
    L = 128 * 4 + 17
    qkv = torch.randn((1, L, 2, 3, 128), generator=g).to(torch.bfloat16).cuda()
    q, k, v = (qkv[:, :, :, i].permute(0, 2, 1, 3) for i in range(3))      # [1,2,L,128], row stride 768
    n = orc.num_blocks(L, 128)
    lists = [[np.arange(0, n, 1 + (i + h) % 2, dtype=np.int32) for i in range(n)] for h in range(2)]
    num, idx = lists_to_tensors(lists, n, "cuda")
    o1 = eng.sparse_forward(q, k, v, 128, num, idx)
    o2 = eng.sparse_forward(q, k, v, 128, num, idx)
    eng.check()
    assert torch.equal(o1, o2)
    for h in range(2):
        want, _ = orc.sparse_attention(f64(q[0, h]), f64(k[0, h]), f64(v[0, h]), lists[h], 128, 128 ** -0.5)
        compare.check_output(f64(o1[0, h]), want, "bf16")


def test_attention_tcgen05_strided_output(eng):
    """The output may be a view too (rows of a wider buffer, heads interleaved): the staged row-contiguous stores
    must land where the strides say and leave the gaps alone."""
    import paper_2608_10519_b200 as sp
    L_q, L_k, H = 128 * 2 + 70, 128 * 5 + 9, 2
    q = _rand((1, H, L_q, 128), torch.bfloat16, 41)
    k = _rand((1, H, L_k, 128), torch.bfloat16, 42)
    v = _rand((1, H, L_k, 128), torch.bfloat16, 43)
    n = orc.num_blocks(L_k, 128)
    lists = [[np.arange(i % 2, n, 2, dtype=np.int32) for i in range(orc.num_blocks(L_q, 128))] for _ in range(H)]
    num, idx = lists_to_tensors(lists, n, "cuda")
    buf = torch.full((1, L_q, H, 192), 3.0, dtype=torch.bfloat16, device="cuda")     # [B, L, H, 192]: 64 spare columns
    o = buf[..., :128].permute(0, 2, 1, 3)                                            # [1, H, L_q, 128] view
    sp.sparstar_sparse_attn_fwd(eng.ctx, q, k, v, o, 128, 128 ** -0.5, num, idx)
    eng.check()
    assert torch.all(buf[..., 128:] == 3.0)
    for h in range(H):
        want, _ = orc.sparse_attention(f64(q[0, h]), f64(k[0, h]), f64(v[0, h]), lists[h], 128, 128 ** -0.5)
        compare.check_output(f64(o[0, h]), want, "bf16")
    buf.fill_(3.0)
    sp.sparstar_attn_fwd(eng.ctx, q, k, v, o, 128, 128 ** -0.5)
    eng.check()
    assert torch.all(buf[..., 128:] == 3.0)
    for h in range(H):
        want, _ = orc.dense_attention(f64(q[0, h]), f64(k[0, h]), f64(v[0, h]), 128 ** -0.5)
        compare.check_output(f64(o[0, h]), want, "bf16")


def test_tcgen05_bad_list_entry_is_flagged(eng):
    import paper_2608_10519_b200 as sp
    q = _rand((1, 1, 128, 128), torch.bfloat16, 20)
    k = _rand((1, 1, 128 * 4, 128), torch.bfloat16, 21)
    num = torch.tensor([[[3]]], dtype=torch.int32, device="cuda")
    idx = torch.tensor([[[[1, 9, 2, 0]]]], dtype=torch.int32, device="cuda")
    o = eng.sparse_forward(q, k, k, 128, num, idx)             # stays in bounds, output unspecified
    st, _ = sp.sparstar_check(eng.ctx)
    assert st == sp.ERR_BAD_INDEX
    assert torch.isfinite(o.float()).all()


def test_malformed_list_is_flagged_and_skipped(eng):
    import paper_2608_10519_b200 as sp
    sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_SIMT)
    try:
        q = _rand((1, 1, 128, 128), torch.bfloat16, 20)
        k = _rand((1, 1, 128 * 4, 128), torch.bfloat16, 21)
        v = _rand((1, 1, 128 * 4, 128), torch.bfloat16, 22)
        num = torch.tensor([[[3]]], dtype=torch.int32, device="cuda")
        idx = torch.tensor([[[[1, 9, 2, 0]]]], dtype=torch.int32, device="cuda")     # 9 is out of range
        o = eng.sparse_forward(q, k, v, 128, num, idx)
        st, _ = sp.sparstar_check(eng.ctx)
        assert st == sp.ERR_BAD_INDEX
        want, _ = orc.sparse_attention(f64(q[0, 0]), f64(k[0, 0]), f64(v[0, 0]), [[1, 2]], 128, 128 ** -0.5)
        compare.check_output(f64(o[0, 0]), want, "bf16")
    finally:
        sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_AUTO)


@pytest.mark.parametrize("block", [64, 32])
def test_attention_small_blocks_disjoint_lists_in_a_tile(eng, block):
    """The query blocks that share a 128-row tile keep disjoint key blocks (every union entry is
    masked for all but one of them), one of them keeps a single late block, one keeps only the
    partial tail block: rows of a tile must never see another query block's keys."""
    import paper_2608_10519_b200 as sp
    g = 128 // block
    L_q, L_k, D, H = block * (2 * g) + 7, block * 37 + 5, 128, 1
    q = _rand((1, H, L_q, D), torch.bfloat16, 41)
    k = _rand((1, H, L_k, D), torch.bfloat16, 42)
    v = _rand((1, H, L_k, D), torch.bfloat16, 43)
    n_q, n_k = orc.num_blocks(L_q, block), orc.num_blocks(L_k, block)
    lists = [np.arange(i % g, n_k, g, dtype=np.int32) for i in range(n_q)]       # residue classes: disjoint in a tile
    lists[1] = np.array([n_k - 2], dtype=np.int32)                               # first kept key comes last
    lists[g] = np.array([n_k - 1], dtype=np.int32)                               # only the partial tail block
    num, idx = lists_to_tensors([lists], n_k, "cuda")
    sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_TCGEN05)
    try:
        o, lse = eng.sparse_forward(q, k, v, block, num, idx, want_lse=True)
        eng.check()
    finally:
        sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_AUTO)
    want, want_lse = orc.sparse_attention(f64(q[0, 0]), f64(k[0, 0]), f64(v[0, 0]), lists, block, D ** -0.5)
    compare.check_output(f64(o[0, 0]), want, "bf16", "disjoint lists")
    assert np.abs(f64(lse[0, 0]) - want_lse).max() <= 1e-3


def test_malformed_list_small_blocks_flagged_and_skipped(eng):
    """Blocks of 64 tokens on the tensor-core kernel: an out-of-range entry and a descending one are
    reported and left out when the lists of a tile are merged."""
    import paper_2608_10519_b200 as sp
    q = _rand((1, 1, 128, 128), torch.bfloat16, 24)
    k = _rand((1, 1, 64 * 8, 128), torch.bfloat16, 25)
    v = _rand((1, 1, 64 * 8, 128), torch.bfloat16, 26)
    num = torch.tensor([[[3, 3]]], dtype=torch.int32, device="cuda")
    idx = torch.tensor([[[[1, 19, 2, 0], [4, 3, 6, 0]]]], dtype=torch.int32, device="cuda")   # 19 out of range; 3 descends
    sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_TCGEN05)
    try:
        o = eng.sparse_forward(q, k, v, 64, num, idx)
        st, _ = sp.sparstar_check(eng.ctx)
    finally:
        sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_AUTO)
    assert st == sp.ERR_BAD_INDEX
    want, _ = orc.sparse_attention(f64(q[0, 0]), f64(k[0, 0]), f64(v[0, 0]), [[1], [4, 6]], 64, 128 ** -0.5)
    compare.check_output(f64(o[0, 0]), want, "bf16")


@pytest.mark.parametrize("order", ["rising", "falling"])
def test_attention_tcgen05_reference_follows_large_score_steps(eng, order):
    """Scores that step up (or down) by about 41 binary orders of magnitude from one key block to
    the next: the softmax reference, which normally stays at the first tile's maximum, has to be
    raised twice on the way up (sum of exponentials beyond the safe range), and on the way down
    the later blocks underflow against it, as they do in the exact result."""
    import paper_2608_10519_b200 as sp
    L_q, n_kb, D = 128 * 2 + 40, 8, 128
    q = _rand((1, 1, L_q, D), torch.bfloat16, 140) * 0.25
    k = _rand((1, 1, 128 * n_kb, D), torch.bfloat16, 141) * 0.25
    v = _rand((1, 1, 128 * n_kb, D), torch.bfloat16, 142)
    q[..., 0] = 8.0
    steps = torch.arange(n_kb, device="cuda").repeat_interleave(128).to(torch.bfloat16) * 40.0
    k[0, 0, :, 0] = steps if order == "rising" else steps.flip(0)
    lists = [np.arange(n_kb, dtype=np.int32), np.array([0, 3, 4, 7], dtype=np.int32), np.array([1, 2, 6], dtype=np.int32)]
    num, idx = lists_to_tensors([lists], n_kb, "cuda")
    sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_TCGEN05)
    try:
        o, lse = eng.sparse_forward(q, k, v, 128, num, idx, want_lse=True)
        od, lsed = eng.dense_forward(q, k, v, 128, want_lse=True)
        eng.check()
    finally:
        sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_AUTO)
    tau = D ** -0.5
    want, want_lse = orc.sparse_attention(f64(q[0, 0]), f64(k[0, 0]), f64(v[0, 0]), lists, 128, tau)
    compare.check_output(f64(o[0, 0]), want, "bf16", f"sparse, {order}")
    assert np.abs(f64(lse[0, 0]) - want_lse).max() <= 1e-3 * (1 + np.abs(want_lse).max())
    wantd, want_lsed = orc.dense_attention(f64(q[0, 0]), f64(k[0, 0]), f64(v[0, 0]), tau)
    compare.check_output(f64(od[0, 0]), wantd, "bf16", f"dense, {order}")
    assert np.abs(f64(lsed[0, 0]) - want_lsed).max() <= 1e-3 * (1 + np.abs(want_lsed).max())


def _wide_spread_inputs():
    n_kb, block, D = 70, 128, 128
    q = _rand((1, 2, block * 3 + 9, D), torch.bfloat16, 150) * 0.25
    k = _rand((1, 2, block * n_kb, D), torch.bfloat16, 151) * 0.25
    q[..., 0] = 20.0
    k[..., 0] = (torch.arange(n_kb, device="cuda").repeat_interleave(block) * 10.0).to(torch.bfloat16)
    return q, k, block


@pytest.mark.parametrize("mass", [0.5, 0.999999])
def test_select_mass_with_underflowing_numerators(eng, mass):
    """Block scores spread over more than 1,000 nats: the softmax numerators of most blocks
    underflow to zero in fp64.  Such blocks must stay selectable blocks (not be mistaken for
    kept ones) and stay out of the lists."""
    q, k, block = _wide_spread_inputs()
    rep = _check_select(eng, q, k, block, "mass", [(0, 130)], mass=mass)
    assert rep.excused == 0


def test_select_mass_one_on_a_plateau_is_a_valid_prefix(eng):
    """p = 1 with the same inputs: once the leading blocks are in, the cumulative mass equals 1 in
    fp64 for every longer prefix, so where the prefix ends depends on the order of additions.
    What is unique: the list is the kept blocks plus a prefix of the ranking, and its mass is 1
    to rounding."""
    q, k, block = _wide_spread_inputs()
    forced = [(0, 130)]
    num, idx, _ = eng.select(q, k, block, "mass", mass=1.0, forced=forced)
    eng.check()
    tau = q.shape[3] ** -0.5
    for h in range(q.shape[1]):
        _, S, fm = orc.select_head(f64(q[0, h]), f64(k[0, h]), block, tau, forced, "mass", mass=1.0)
        for i in range(S.shape[0]):
            got = idx[0, h, i, :int(num[0, h, i])].cpu().numpy()
            assert np.all(np.diff(got) > 0) and set(np.nonzero(fm)[0]) <= set(got)
            taken = np.array([j for j in got if not fm[j]], dtype=np.int64)
            sel = np.nonzero(~fm)[0]
            order = sel[np.lexsort((sel, -S[i, sel]))]           # score descending, index ascending
            assert len(taken) >= 1 and set(taken) == set(order[:len(taken)])
            e = np.exp(S[i, sel] - S[i, sel].max())
            assert np.exp(S[i, taken] - S[i, sel].max()).sum() >= e.sum() * (1 - 1e-12)


def test_unsupported_and_invalid_arguments(eng):
    import paper_2608_10519_b200 as sp
    q = _rand((1, 1, 128, 96), torch.bfloat16, 30)
    o = torch.empty_like(q)
    with pytest.raises(sp.SparstarError) as e:
        sp.sparstar_attn_fwd(eng.ctx, q, q, q, o, 128, 0.1)
    assert e.value.status == sp.ERR_UNSUPPORTED
    k = _rand((1, 2, 128, 96), torch.bfloat16, 31)
    with pytest.raises(sp.SparstarError) as e:
        sp.sparstar_attn_fwd(eng.ctx, q, k, k, o, 128, 0.1)
    assert e.value.status == sp.ERR_INVALID_ARG


@pytest.mark.parametrize("block", [128, 64])
def test_batch_two_whole_path(eng, block):
    """B = 2 (e.g. conditional + unconditional branches): every batch entry has its own lists;
    strided inputs (heads sliced out of a wider tensor) with the small-block kernel too."""
    H = 2
    wide = _rand((2, H + 1, block * 3 + 5, 128), torch.bfloat16, 40)
    q = wide[:, 1:]                                              # non-contiguous view
    k = _rand((2, H, block * 10 + 70, 128), torch.bfloat16, 41)
    v = _rand((2, H, block * 10 + 70, 128), torch.bfloat16, 42)
    forced = [(0, 200)]
    num, idx, _ = eng.select(q, k, block, "topk_ratio", ratio=0.3, forced=forced)
    o = eng.sparse_forward(q, k, v, block, num, idx)
    eng.check()
    tau = 128 ** -0.5
    for b in range(2):
        for h in range(H):
            lists, S, fm = orc.select_head(f64(q[b, h]), f64(k[b, h]), block, tau, forced, "topk_ratio", ratio=0.3)
            rep = compare.compare_lists(num[b, h].cpu().numpy(), idx[b, h].cpu().numpy(), lists, S, fm, "topk_ratio",
                                        k=orc.budget(int((~fm).sum()), 0.3))
            assert rep.ok and rep.exact == rep.rows
            want, _ = orc.sparse_attention(f64(q[b, h]), f64(k[b, h]), f64(v[b, h]), lists, block, tau)
            compare.check_output(f64(o[b, h]), want, "bf16", f"b{b} h{h}")


def test_trace_records_role_events(eng):
    """The profiling aid returns (tag, clock) pairs for the four roles of the first CTA."""
    import paper_2608_10519_b200 as sp
    q = _rand((1, 1, 128, 128), torch.bfloat16, 50)
    k = _rand((1, 1, 128 * 12, 128), torch.bfloat16, 51)
    o = torch.empty_like(q)
    buf = torch.zeros((4, 16, 2), dtype=torch.int64, device="cuda")
    sp.sparstar_set_trace(eng.ctx, buf, skip=2)
    try:
        sp.sparstar_attn_fwd(eng.ctx, q, k, k, o, 128, 128 ** -0.5)
        eng.check()
    finally:
        sp.sparstar_set_trace(eng.ctx, None)
    b = buf.cpu()
    assert int((b[:, :, 0] != 0).sum()) >= 12          # every role logged something
    for role in range(4):
        clocks = b[role, b[role, :, 0] != 0, 1]
        assert clocks.numel() >= 2


@pytest.mark.parametrize("D", [128, 64])
@pytest.mark.parametrize("L_q,L_k,density", [(64 * 5 + 20, 64 * 31 + 9, 0.3), (64, 64, 1.0), (50, 64 * 3 + 1, 1.0),
                                             (64 * 3, 64 * 20, 0.05), (64 * 2 + 1, 64 * 9 + 63, 0.5)])
@pytest.mark.parametrize("impl", [2, 3])
def test_attention_tcgen05_block64(eng, D, L_q, L_k, density, impl):
    """Selection blocks of 64 tokens on the tensor-core kernels (impl 2: the three-tile kernel's gathered
    instance; impl 3: the older two-stream kernel's, as a cross-check): two listed blocks are gathered
    into one 128-key tile (odd list lengths leave half a tile unused, the last block may be
    partial) and a CTA's query tile holds two 64-row query blocks."""
    _attn_case(eng, torch.bfloat16, D, 64, L_q, L_k, 2, density, 23, impl)


@pytest.mark.parametrize("D", [128, 64])
@pytest.mark.parametrize("L_q,L_k,density", [(32 * 5 + 20, 32 * 61 + 9, 0.3), (32, 32, 1.0), (20, 32 * 3 + 1, 1.0),
                                             (32 * 3, 32 * 40, 0.05), (32 * 2 + 1, 32 * 18 + 31, 0.5),
                                             (32 * 2, 32 * 7, 0.72), (32 * 2, 32 * 6, 0.99)])
@pytest.mark.parametrize("impl", [2, 3])
def test_attention_tcgen05_block32(eng, D, L_q, L_k, density, impl):
    """Selection blocks of 32 tokens: four listed blocks per 128-key tile, list lengths of every
    residue modulo four, a partial last block (both tensor-core kernels, as above)."""
    _attn_case(eng, torch.bfloat16, D, 32, L_q, L_k, 2, density, 29, impl)


@pytest.mark.parametrize("block,L_q,L_k", [(256, 256 * 2 + 100, 256 * 5 + 130), (256, 200, 256 * 3 + 7), (512, 512 + 300, 512 * 3 + 129)])
def test_attention_tcgen05_larger_selection_blocks(eng, block, L_q, L_k):
    """Selection blocks of 256 / 512 tokens on the tensor-core kernel (walked as 128-token tiles),
    including a last key block with fewer tiles than a full block."""
    _attn_case(eng, torch.bfloat16, 128, block, L_q, L_k, 2, 0.5, 17, 2)


@pytest.mark.parametrize("block", [256, 64, 32])
def test_whole_path_other_block_sizes(eng, block):
    """Pool, select and sparse forward (tensor-core kernel) with selection blocks of 256, 64 and 32 tokens."""
    L_k = block * 13 + (200 if block == 256 else 50)
    q = _rand((1, 2, block * 4 + 33, 128), torch.bfloat16, 60)
    k = _rand((1, 2, L_k, 128), torch.bfloat16, 61)
    v = _rand((1, 2, L_k, 128), torch.bfloat16, 62)
    forced = [(0, 300)]
    num, idx, _ = eng.select(q, k, block, "mass", mass=0.7, forced=forced)
    o = eng.sparse_forward(q, k, v, block, num, idx)
    eng.check()
    tau = 128 ** -0.5
    for h in range(2):
        lists, S, fm = orc.select_head(f64(q[0, h]), f64(k[0, h]), block, tau, forced, "mass", mass=0.7)
        rep = compare.compare_lists(num[0, h].cpu().numpy(), idx[0, h].cpu().numpy(), lists, S, fm, "mass", mass=0.7)
        assert rep.ok, rep.bad[:3]
        got_lists = [idx[0, h, i, :int(num[0, h, i])].cpu().numpy() for i in range(len(lists))]
        want, _ = orc.sparse_attention(f64(q[0, h]), f64(k[0, h]), f64(v[0, h]), got_lists, block, tau)
        compare.check_output(f64(o[0, h]), want, "bf16", f"h{h}")


@pytest.mark.parametrize("impl", [1, 2])
def test_rows_without_blocks_give_zeros(eng, impl):
    import paper_2608_10519_b200 as sp
    sp.sparstar_set_attn_impl(eng.ctx, impl)
    try:
        q = _rand((1, 1, 128 * 3, 128), torch.bfloat16, 70)
        k = _rand((1, 1, 128 * 5, 128), torch.bfloat16, 71)
        num = torch.tensor([[[2, 0, 1]]], dtype=torch.int32, device="cuda")
        idx = torch.tensor([[[[0, 3, 0, 0, 0], [0, 0, 0, 0, 0], [4, 0, 0, 0, 0]]]], dtype=torch.int32, device="cuda")
        o, lse = eng.sparse_forward(q, k, k, 128, num, idx, want_lse=True)
        eng.check()
        assert torch.all(o[0, 0, 128:256] == 0) and torch.all(torch.isinf(lse[0, 0, 128:256]))
        want, _ = orc.sparse_attention(f64(q[0, 0]), f64(k[0, 0]), f64(k[0, 0]), [[0, 3], [0], [4]], 128, 128 ** -0.5)
        compare.check_output(f64(o[0, 0, :128]), want[:128], "bf16")
        compare.check_output(f64(o[0, 0, 256:]), want[256:], "bf16")
    finally:
        sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_AUTO)


@pytest.mark.parametrize("block", [64, 32])
def test_rows_without_blocks_small_blocks(eng, block):
    """Small selection blocks on the tensor-core kernel: a query block without any key block next
    to one with blocks inside the same 128-row tile, and a whole tile without blocks."""
    import paper_2608_10519_b200 as sp
    g = 128 // block
    n_q, n_k = 2 * g + 1, 9
    q = _rand((1, 1, block * n_q, 128), torch.bfloat16, 72)
    k = _rand((1, 1, block * n_k - 3, 128), torch.bfloat16, 73)
    lists = [np.array([], dtype=np.int32) for _ in range(n_q)]
    lists[0] = np.array([1, 8], dtype=np.int32)              # tile 0: first query block only
    lists[2 * g] = np.array([0, 2, 5], dtype=np.int32)       # tile 2; tile 1 has nothing at all
    num, idx = lists_to_tensors([lists], n_k, "cuda")
    sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_TCGEN05)
    try:
        o, lse = eng.sparse_forward(q, k, k, block, num, idx, want_lse=True)
        eng.check()
    finally:
        sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_AUTO)
    for i in range(n_q):
        rows = slice(i * block, (i + 1) * block)
        if len(lists[i]) == 0:
            assert torch.all(o[0, 0, rows] == 0) and torch.all(torch.isinf(lse[0, 0, rows])), i
        else:
            want, want_lse = orc.attention_block(f64(q[0, 0, rows]), f64(k[0, 0]), f64(k[0, 0]), lists[i], block, 128 ** -0.5)
            compare.check_output(f64(o[0, 0, rows]), want, "bf16", f"query block {i}")
            assert np.abs(f64(lse[0, 0, rows]) - want_lse).max() <= 1e-3


def test_bounded_wait_reports_timeout_and_context_stays_usable(eng):
    """Failure detection without a fault: the producer is told to arm one stage barrier and copy
    nothing; the MMA role's bounded wait (about a second) runs out, every role leaves its loop,
    tensor memory is released, the kernel returns and the status word says so."""
    import paper_2608_10519_b200 as sp
    q = _rand((1, 1, 128, 128), torch.bfloat16, 80)
    k = _rand((1, 1, 128 * 6, 128), torch.bfloat16, 81)
    o = torch.empty_like(q)
    sp.sparstar_set_debug(eng.ctx, True, 1)
    try:
        sp.sparstar_attn_fwd(eng.ctx, q, k, k, o, 128, 128 ** -0.5)      # one CTA, six tiles
        st, site = sp.sparstar_check(eng.ctx)
    finally:
        sp.sparstar_set_debug(eng.ctx, True, -1)
    assert st == sp.ERR_TIMEOUT and site != 0
    # several waves of CTAs: once the expiry is on record the remaining CTAs do no work, so the
    # launch ends after about one timeout (one second), not one per wave
    import time
    qw = _rand((1, 1, 128 * 600, 128), torch.bfloat16, 82)
    ow = torch.empty_like(qw)
    sp.sparstar_set_debug(eng.ctx, True, 1)
    try:
        torch.cuda.synchronize()
        t0 = time.time()
        sp.sparstar_attn_fwd(eng.ctx, qw, k, k, ow, 128, 128 ** -0.5)
        st, site = sp.sparstar_check(eng.ctx)
        elapsed = time.time() - t0
    finally:
        sp.sparstar_set_debug(eng.ctx, True, -1)
    assert st == sp.ERR_TIMEOUT and elapsed < 3.0, elapsed
    # the next call on the same context is healthy
    sp.sparstar_attn_fwd(eng.ctx, q, k, k, o, 128, 128 ** -0.5)
    assert sp.sparstar_check(eng.ctx)[0] == sp.OK
    want, _ = orc.dense_attention(f64(q[0, 0]), f64(k[0, 0]), f64(k[0, 0]), 128 ** -0.5)
    compare.check_output(f64(o[0, 0]), want, "bf16")


def test_bounded_wait_in_a_cta_pair(eng):
    """The same without a fault for a pair of CTAs: neither producer copies stage 1, the issuing warp's
    wait runs out in the first CTA, the second CTA's own waits run out beside it, both meet at the
    cluster barrier, tensor memory is released; the next call in pair mode is healthy."""
    import time
    import paper_2608_10519_b200 as sp
    q = _rand((1, 1, 256, 128), torch.bfloat16, 83)
    k = _rand((1, 1, 128 * 6, 128), torch.bfloat16, 84)
    o = torch.empty_like(q)
    sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_TCGEN05_PAIR)
    try:
        sp.sparstar_set_debug(eng.ctx, True, 1)
        try:
            torch.cuda.synchronize()
            t0 = time.time()
            sp.sparstar_attn_fwd(eng.ctx, q, k, k, o, 128, 128 ** -0.5)      # one pair, six tiles
            st, site = sp.sparstar_check(eng.ctx)
            elapsed = time.time() - t0
        finally:
            sp.sparstar_set_debug(eng.ctx, True, -1)
        assert st == sp.ERR_TIMEOUT and site != 0 and elapsed < 5.0, (st, site, elapsed)
        sp.sparstar_attn_fwd(eng.ctx, q, k, k, o, 128, 128 ** -0.5)
        assert sp.sparstar_check(eng.ctx)[0] == sp.OK
    finally:
        sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_AUTO)
    want, _ = orc.dense_attention(f64(q[0, 0]), f64(k[0, 0]), f64(k[0, 0]), 128 ** -0.5)
    compare.check_output(f64(o[0, 0]), want, "bf16")


@pytest.mark.parametrize("L_q,L_k,H,density", [(128, 128, 1, 1.0), (128 * 2 + 50, 128 * 7 + 3, 2, 0.5), (128 * 3, 128 * 20, 2, 0.2)])
def test_attention_tcgen05_head_dim_64(eng, L_q, L_k, H, density):
    _attn_case(eng, torch.bfloat16, 64, 128, L_q, L_k, H, density, 19, 2)


@pytest.mark.parametrize("mode,kw", [("topk_ratio", {"ratio": 0.25}), ("topk_ratio", {"ratio": 0.5}),
                                     ("topk_count", {"count": 1}), ("mass", {"mass": 0.9}), ("mass", {"mass": 0.3})])
def test_select_with_tcgen05_prescore(eng, mode, kw):
    """Scores from the tcgen05 split-bf16 GEMM, made exact next to the cutoff: same lists."""
    import paper_2608_10519_b200 as sp
    sp.sparstar_set_score_impl(eng.ctx, sp.SCORE_TCGEN05)
    try:
        q = _rand((1, 3, 128 * 9 + 50, 128), torch.bfloat16, 3)
        k = _rand((1, 3, 128 * 40 + 17, 128), torch.bfloat16, 4)
        rep = _check_select(eng, q, k, 128, mode, [(0, 200), (1000, 1001)], **kw)
        assert rep.excused <= 1
        # more than one 128 x 128 score tile in both directions, D = 64, duplicated blocks (exact ties)
        q2 = _rand((2, 2, 64 * 150 + 3, 64), torch.bfloat16, 5)
        k2 = _rand((2, 2, 64 * 300 + 9, 64), torch.bfloat16, 6)
        k2[:, :, 64 * 7:64 * 8] = k2[:, :, 64 * 2:64 * 3]
        _check_select(eng, q2, k2, 64, mode, [(0, 70)], **kw)
    finally:
        sp.sparstar_set_score_impl(eng.ctx, sp.SCORE_FP64)


def test_select_randomised_shapes(eng):
    """Random shapes, modes, parameters and forced ranges (both score paths), lists against the oracle."""
    import paper_2608_10519_b200 as sp
    rng = np.random.default_rng(2024)
    try:
        for trial in range(24):
            sp.sparstar_set_score_impl(eng.ctx, trial % 2)
            D = int(rng.choice([64, 128]))
            block = int(rng.choice([64, 128]))
            L_q = int(rng.integers(1, 9 * block))
            L_k = int(rng.integers(block, 60 * block))
            dtype = torch.bfloat16 if rng.random() < 0.7 else torch.float32
            q = _rand((1, 2, L_q, D), dtype, 100 + trial)
            k = _rand((1, 2, L_k, D), dtype, 200 + trial)
            forced = []
            for _ in range(int(rng.integers(0, 4))):
                s0 = int(rng.integers(0, L_k))
                forced.append((s0, s0 + int(rng.integers(0, 3 * block))))
            mode = str(rng.choice(["topk_ratio", "topk_count", "mass"]))
            kw = {"topk_ratio": {"ratio": float(rng.choice([0.0, 0.1, 0.33, 0.5, 1.0]))},
                  "topk_count": {"count": int(rng.integers(0, 70))},
                  "mass": {"mass": float(rng.choice([0.05, 0.5, 0.9, 0.999]))}}[mode]
            _check_select(eng, q, k, block, mode, forced, **kw)
    finally:
        sp.sparstar_set_score_impl(eng.ctx, sp.SCORE_FP64)


def test_attention_tcgen05_randomised(eng):
    """Random sizes, head dimensions, selection block sizes and lists on the tensor-core kernel."""
    import paper_2608_10519_b200 as sp
    rng = np.random.default_rng(77)
    sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_TCGEN05)
    try:
        for trial in range(14):
            D = int(rng.choice([64, 128]))
            block = int(rng.choice([32, 64, 128, 256]))
            H = int(rng.integers(1, 4))
            L_q = int(rng.integers(1, 5 * block))
            L_k = int(rng.integers(1, 24 * block))
            q = _rand((1, H, L_q, D), torch.bfloat16, 300 + trial)
            k = _rand((1, H, L_k, D), torch.bfloat16, 400 + trial)
            v = _rand((1, H, L_k, D), torch.bfloat16, 500 + trial)
            n_q, n_k = orc.num_blocks(L_q, block), orc.num_blocks(L_k, block)
            lists = [[np.sort(rng.choice(n_k, size=int(rng.integers(1, n_k + 1)), replace=False)).astype(np.int32)
                      for _ in range(n_q)] for _ in range(H)]
            num, idx = lists_to_tensors(lists, n_k, "cuda")
            o, lse = eng.sparse_forward(q, k, v, block, num, idx, want_lse=True)
            eng.check()
            tau = D ** -0.5
            for h in range(H):
                want, want_lse = orc.sparse_attention(f64(q[0, h]), f64(k[0, h]), f64(v[0, h]), lists[h], block, tau)
                compare.check_output(f64(o[0, h]), want, "bf16", f"trial {trial} h{h}")
                assert np.abs(f64(lse[0, h]) - want_lse).max() <= 1e-3
    finally:
        sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_AUTO)


def test_size_limits_are_reported(eng):
    """Largest strip the selection kernel holds in shared memory: beyond it the call is refused on
    the host (no launch); just below it the result is still right."""
    import paper_2608_10519_b200 as sp
    block = 128
    for n_k, ok in ((24000, True), (26000, False)):
        L_k = n_k * block
        qb = _rand((1, 1, 2, 128), torch.float32, 90)
        kb = _rand((1, 1, n_k, 128), torch.float32, 91)
        num = torch.zeros((1, 1, 2), dtype=torch.int32, device="cuda")
        idx = torch.zeros((1, 1, 2, 64), dtype=torch.int32, device="cuda")
        if ok:
            sp.sparstar_score_select(eng.ctx, qb, kb, block, L_k, 128 ** -0.5, sp.SEL_TOPK_COUNT, num, idx, count=50)
            eng.check()
            S = (128 ** -0.5) * (f64(qb[0, 0]) @ f64(kb[0, 0]).T)
            for i in range(2):
                want = np.sort(np.argsort(-S[i], kind="stable")[:50])
                assert np.array_equal(idx[0, 0, i, :50].cpu().numpy(), want) and int(num[0, 0, i]) == 50
        else:
            with pytest.raises(sp.SparstarError) as e:
                sp.sparstar_score_select(eng.ctx, qb, kb, block, L_k, 128 ** -0.5, sp.SEL_TOPK_COUNT, num, idx, count=50)
            assert e.value.status == sp.ERR_UNSUPPORTED
    # rows that are not a whole number of 16-byte vectors cannot be pooled
    x = _rand((1, 1, 64, 12), torch.bfloat16, 92)
    with pytest.raises((sp.SparstarError, AssertionError)) as e:
        eng.pool(x, 16)


def _random_lists(n_q, n_k, H, seed):
    rng = np.random.default_rng(seed)
    return [[np.sort(rng.choice(n_k, size=int(rng.integers(1, n_k + 1)), replace=False)).astype(np.int32)
             for _ in range(n_q)] for _ in range(H)]


def test_scratch_growth_keeps_a_captured_graph_valid():
    """A graph captured from a sparse call names the context's scratch (the work order).  A later,
    larger eager call makes the scratch grow; the outgrown buffer must stay alive, so the replay
    still gives the eager result.  A call that would have to grow the scratch DURING capture is
    refused with ERR_CAPTURE and enqueues nothing."""
    import paper_2608_10519_b200 as sp
    from paper_2608_10519_b200.pipeline import SparstarAttention
    e = SparstarAttention(0)
    try:
        H, L_q, L_k = 2, 128 * 5 + 9, 128 * 12 + 70
        q, k, v = (_rand((1, H, L, 128), torch.bfloat16, 700 + i) for i, L in enumerate((L_q, L_k, L_k)))
        num, idx = lists_to_tensors(_random_lists(6, 13, H, 1), 13, "cuda")
        o = torch.empty_like(q)
        # no scratch yet: growth inside a capture is refused
        g0 = torch.cuda.CUDAGraph()
        status = []
        with torch.cuda.graph(g0):
            try:
                sp.sparstar_sparse_attn_fwd(e.ctx, q, k, v, o, 128, 128 ** -0.5, num, idx)
            except sp.SparstarError as err:
                status.append(err.status)
        assert status == [sp.ERR_CAPTURE] and sp.sparstar_scratch_bytes(e.ctx) == 0
        # reserve (or run once eagerly), then capture
        sp.sparstar_reserve_scratch(e.ctx, 1 << 20)
        small = sp.sparstar_scratch_bytes(e.ctx)
        assert small >= 1 << 20
        sp.sparstar_sparse_attn_fwd(e.ctx, q, k, v, o, 128, 128 ** -0.5, num, idx)
        e.check()
        want = o.clone()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            sp.sparstar_sparse_attn_fwd(e.ctx, q, k, v, o, 128, 128 ** -0.5, num, idx)
        # a much larger eager call: the work order of 2 x 4,100 query tiles of 64-token blocks plus
        # its union lists needs more than the reserved megabyte
        Lq2, Lk2 = 64 * 8200, 64 * 40
        q2, k2 = _rand((1, 2, Lq2, 128), torch.bfloat16, 710), _rand((1, 2, Lk2, 128), torch.bfloat16, 711)
        num2 = torch.full((1, 2, 8200), 2, dtype=torch.int32, device="cuda")
        idx2 = torch.zeros((1, 2, 8200, 4), dtype=torch.int32, device="cuda")
        idx2[..., 1] = 7
        sp.sparstar_sparse_attn_fwd(e.ctx, q2, k2, k2, torch.empty_like(q2), 64, 128 ** -0.5, num2, idx2)
        e.check()
        assert sp.sparstar_scratch_bytes(e.ctx) > small
        o.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        e.check()
        assert torch.equal(o, want)
    finally:
        e.close()


def test_context_checks_the_current_device(eng):
    """Every operator call verifies that the context's device is current (one GPU is visible here,
    so only the matching case can run; a mismatch returns ERR_INVALID_ARG before any launch)."""
    import paper_2608_10519_b200 as sp
    assert torch.cuda.current_device() == 0
    x = _rand((1, 1, 256, 128), torch.bfloat16, 95)
    out = eng.pool(x, 128)
    eng.check()
    assert out.shape == (1, 1, 2, 128)


@pytest.mark.parametrize("mode,kw", [("topk_ratio", {"ratio": 0.25}), ("mass", {"mass": 0.9}), ("topk_count", {"count": 3})])
def test_select_fused_gives_the_lists_of_the_separate_calls(eng, mode, kw):
    """Pooling + scores + selection in one cooperative launch: the same bits as pool, pool,
    score_select, with and without cached block means of the leading (conditioning) key blocks."""
    for (dtype, D, block, H, L_q, L_k) in [(torch.bfloat16, 128, 128, 3, 128 * 11 + 70, 128 * 37 + 5),
                                           (torch.float32, 64, 64, 2, 64 * 5 + 1, 64 * 9)]:
        q, k = _rand((1, H, L_q, D), dtype, 900), _rand((1, H, L_k, D), dtype, 901)
        forced = [(0, block + 7)]
        want_num, want_idx, _ = eng.select(q, k, block, mode, forced=forced, **kw)
        num, idx = eng.select_fused(q, k, block, mode, forced=forced, **kw)
        eng.check()
        assert torch.equal(num, want_num)
        for h in range(H):
            for i in range(num.shape[2]):
                c = int(num[0, h, i])
                assert torch.equal(idx[0, h, i, :c], want_idx[0, h, i, :c])
        # the first 5 key blocks from a cache
        cond = eng.pool(k[:, :, :5 * block], block)
        num2, idx2 = eng.select_fused(q, k, block, mode, forced=forced, k_cond_pooled=cond, **kw)
        eng.check()
        assert torch.equal(num2, want_num)
        for h in range(H):
            for i in range(num.shape[2]):
                c = int(num[0, h, i])
                assert torch.equal(idx2[0, h, i, :c], want_idx[0, h, i, :c])
