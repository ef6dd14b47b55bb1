"""Attention-mass analysis calls against the oracle: exact block masses, the block-wise oracle
selector, retained mass (and its identity with the log-sum-exp gap)."""
import numpy as np
import pytest
import torch

from oracle import compare
from oracle import sparstar_oracle as orc
from tests.gpu_util import f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def eng():
    from paper_2608_10519_b200 import build
    build.build()
    from paper_2608_10519_b200.pipeline import SparstarAttention
    e = SparstarAttention(0)
    yield e
    e.close()


def _rand(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (scale * torch.randn(shape, generator=g)).to(torch.bfloat16).cuda()


@pytest.mark.parametrize("L_q,L_k,H", [(128 * 3 + 40, 128 * 7 + 9, 2), (100, 128, 1), (128 * 2, 128 * 11, 3)])
def test_block_mass_matches_oracle(eng, L_q, L_k, H):
    q, k, v = _rand((1, H, L_q, 128), 1, 1.5), _rand((1, H, L_k, 128), 2), _rand((1, H, L_k, 128), 3)
    mass, lse = eng.block_mass(q, k, v, 128)
    eng.check()
    tau = 128 ** -0.5
    for h in range(H):
        want = orc.block_mass(f64(q[0, h]), f64(k[0, h]), 128, tau)
        got = f64(mass[0, h])
        assert np.abs(got - want).max() <= 2e-3                      # bf16 operands, fp32 lse
        assert np.abs(got.sum(axis=1) - 1.0).max() <= 2e-3


def test_exact_selector_and_retained_mass(eng):
    from workloads import generate, get_config
    from workloads.configs import shrink
    w = shrink(get_config("c1"), 2)
    x = generate(w, "cuda")
    q, k, v = x["q"][:, :, :128 * 20], x["k"][:, :, :128 * 150 + 17], x["v"][:, :, :128 * 150 + 17]
    q, k, v = q.contiguous(), k.contiguous(), v.contiguous()
    L_k = k.shape[2]
    forced = [(0, 512)]
    mass, lse_d = eng.block_mass(q, k, v, 128)
    # block-wise oracle selector = top-k on the exact masses (same tie rule, forced blocks kept)
    num_e, idx_e = eng.select_from_scores(mass, 128, L_k, "topk_ratio", ratio=0.2, forced=forced)
    num_a, idx_a, _ = eng.select(q, k, 128, "topk_ratio", ratio=0.2, forced=forced)
    r_e = eng.retained_mass(mass, num_e, idx_e)
    r_a = eng.retained_mass(mass, num_a, idx_a)
    o, lse_s = eng.sparse_forward(q, k, v, 128, num_a, idx_a, want_lse=True)
    eng.check()
    tau = 128 ** -0.5
    for h in range(2):
        M = f64(mass[0, h])
        fm = orc.forced_blocks(L_k, 128, forced)
        kk = orc.budget(int((~fm).sum()), 0.2)
        lists = [orc.select_topk_row(M[i], fm, kk) for i in range(M.shape[0])]     # oracle selection on the same scores
        rep = compare.compare_lists(num_e[0, h].cpu().numpy(), idx_e[0, h].cpu().numpy(), lists, M, fm, "topk_ratio", k=kk)
        assert rep.ok and rep.exact == rep.rows, rep.bad[:3]
        want = orc.retained_mass(M, lists)
        assert np.abs(f64(r_e[0, h]) - want).max() <= 1e-5
        # exact selection never retains less than the aggregated-QK selection of the same size
        assert np.all(f64(r_e[0, h]) >= f64(r_a[0, h]) - 1e-5)
        # identity: retained mass = mean over the block's queries of exp(lse_sparse - lse_dense)
        gap = np.exp(f64(lse_s[0, h]) - f64(lse_d[0, h])).reshape(-1, 128).mean(axis=1)
        assert np.abs(f64(r_a[0, h]) - gap).max() <= 3e-3
        # and the oracle agrees with the GPU's retained mass from first principles
        Mo = orc.block_mass(f64(q[0, h]), f64(k[0, h]), 128, tau)
        la = [idx_a[0, h, i, :int(num_a[0, h, i])].cpu().numpy() for i in range(M.shape[0])]
        assert np.abs(f64(r_a[0, h]) - orc.retained_mass(Mo, la)).max() <= 3e-3


@pytest.mark.parametrize("D,block,L_q,L_k,H", [(64, 128, 128 * 2 + 30, 128 * 5 + 9, 2), (128, 64, 64 * 5 + 11, 64 * 13 + 3, 2),
                                                (128, 256, 256 * 2 + 100, 256 * 4 + 77, 1), (128, 32, 32 * 9 + 5, 32 * 21 + 1, 1),
                                                (64, 64, 64 * 3, 64 * 6 + 40, 1), (128, 512, 512 + 130, 512 * 3 + 5, 1)])
def test_block_mass_other_block_sizes_and_head_dims(eng, D, block, L_q, L_k, H):
    """Exact block masses per selection block of 32 ... 512 tokens and for D = 64 (the attention
    kernel's own shape range), ragged tails on both sides."""
    q, k, v = _rand((1, H, L_q, D), 11, 1.5), _rand((1, H, L_k, D), 12), _rand((1, H, L_k, D), 13)
    mass, lse = eng.block_mass(q, k, v, block)
    eng.check()
    tau = D ** -0.5
    assert tuple(mass.shape) == (1, H, orc.num_blocks(L_q, block), orc.num_blocks(L_k, block))
    for h in range(H):
        want = orc.block_mass(f64(q[0, h]), f64(k[0, h]), block, tau)
        got = f64(mass[0, h])
        assert np.abs(got - want).max() <= 2e-3
        assert np.abs(got.sum(axis=1) - 1.0).max() <= 2e-3


def test_peaked_rows_error_of_bf16_probabilities(eng):
    """Keys scaled by 8: logits of standard deviation 8, rows dominated by one or two keys, outputs
    of magnitude up to 4 - OUTSIDE the unit-variance domain the 2e-2 / 2e-3 tolerance is stated for.
    P enters the second GEMM rounded to bf16 (relative error up to 2^-9 per term) while the row's
    denominator is summed from the unrounded values, so the error grows with |O|.  This test records
    it and pins it below 3e-2 / 2e-3 (measured 1.7e-2 / 1.1e-3 on the tensor-core kernel, 0.8e-2 on
    the fp32 SIMT kernel); on the same rows with unit-scale keys the error is 4e-4."""
    import paper_2608_10519_b200 as sp
    g = torch.Generator().manual_seed(3)
    H, L_q, L_k = 2, 128 * 4, 128 * 24
    out = {}
    for kscale in (1.0, 8.0):
        q = torch.randn((1, H, L_q, 128), generator=g).to(torch.bfloat16).cuda()
        k = (kscale * torch.randn((1, H, L_k, 128), generator=g)).to(torch.bfloat16).cuda()
        v = torch.randn((1, H, L_k, 128), generator=g).to(torch.bfloat16).cuda()
        for impl in (sp.ATTN_TCGEN05, sp.ATTN_SIMT):
            sp.sparstar_set_attn_impl(eng.ctx, impl)
            try:
                o = eng.dense_forward(q, k, v, 128)
                eng.check()
            finally:
                sp.sparstar_set_attn_impl(eng.ctx, sp.ATTN_AUTO)
            mx = mean = 0.0
            for h in range(H):
                want, _ = orc.dense_attention(f64(q[0, h]), f64(k[0, h]), f64(v[0, h]), 128 ** -0.5)
                e = compare.output_errors(f64(o[0, h]), want)
                mx, mean = max(mx, e[0]), max(mean, e[1])
            out[(kscale, impl)] = (mx, mean)
            print(f"keys x{kscale:g}, impl {impl}: max-abs {mx:.3e}, mean-abs {mean:.3e}")
    assert out[(1.0, sp.ATTN_TCGEN05)][0] <= 2e-2 and out[(1.0, sp.ATTN_TCGEN05)][1] <= 2e-3     # the stated tolerance
    assert out[(8.0, sp.ATTN_TCGEN05)][0] <= 3e-2 and out[(8.0, sp.ATTN_TCGEN05)][1] <= 2e-3
    assert out[(8.0, sp.ATTN_SIMT)][0] <= 2e-2
