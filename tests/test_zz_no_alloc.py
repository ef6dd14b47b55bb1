"""The allocation-free sparse forward (fixed scratch inside the library, no context): same
bits as the context-based entry point (same kernel, same work order), both within the bf16
tolerance of the oracle, and no device memory taken.  Collected last on purpose: if it fails, a
run that stops at the first failure has already run every other test.  It passes alone in a
fresh process and after the rest of the suite, and checks two calls in a row because the second
call finds the first one's leftovers in the shared scratch."""
import numpy as np
import pytest
import torch

from oracle import compare
from oracle import sparstar_oracle as orc

pytestmark = pytest.mark.gpu


def _lists(n_q, n_k, H, seed):
    rng = np.random.default_rng(seed)
    lists = [[np.sort(rng.choice(n_k, size=int(rng.integers(1, n_k + 1)), replace=False)).astype(np.int32)
              for _ in range(n_q)] for _ in range(H)]
    num = torch.zeros((1, H, n_q), dtype=torch.int32)
    idx = torch.zeros((1, H, n_q, n_k), dtype=torch.int32)
    for h in range(H):
        for i, l in enumerate(lists[h]):
            num[0, h, i] = len(l)
            idx[0, h, i, :len(l)] = torch.from_numpy(l)
    return lists, num.cuda(), idx.cuda()


def _f64(t):
    return t.detach().cpu().double().numpy()


def test_static_entry_matches_context_entry_and_oracle_twice_in_a_row():
    from paper_2608_10519_b200 import build
    build.build()
    import paper_2608_10519_b200 as sp
    g = torch.Generator().manual_seed(77)
    ctx = sp.sparstar_create(0)
    tau = 128 ** -0.5
    try:
        # two different problems back to back: the second one is smaller, so stale entries of the
        # first remain in the scratch beyond what it rewrites
        for (H, L_q, L_k, seed) in [(3, 128 * 9 + 40, 128 * 21 + 7, 1), (2, 128 * 4 + 1, 128 * 6, 2)]:
            q = torch.randn((1, H, L_q, 128), generator=g).to(torch.bfloat16).cuda()
            k = torch.randn((1, H, L_k, 128), generator=g).to(torch.bfloat16).cuda()
            v = torch.randn((1, H, L_k, 128), generator=g).to(torch.bfloat16).cuda()
            n_q, n_k = sp.sparstar_num_blocks(L_q, 128), sp.sparstar_num_blocks(L_k, 128)
            lists, num, idx = _lists(n_q, n_k, H, seed)
            want = torch.empty_like(q)
            want_lse = torch.empty(q.shape[:3], dtype=torch.float32, device="cuda")
            sp.sparstar_sparse_attn_fwd(ctx, q, k, v, want, 128, tau, num, idx, want_lse)
            assert sp.sparstar_check(ctx)[0] == sp.OK
            got = torch.full_like(q, float("nan"))
            got_lse = torch.empty_like(want_lse)
            got2 = torch.full_like(q, float("nan"))
            status = torch.full((2,), 99, dtype=torch.int32, device="cuda")
            sp.sparstar_sparse_attn_fwd_static(q, k, v, got, 128, tau, num, idx, got_lse, status)
            torch.cuda.synchronize()
            free0 = torch.cuda.mem_get_info()[0]
            alloc0 = torch.cuda.memory_allocated()
            sp.sparstar_sparse_attn_fwd_static(q, k, v, got2, 128, tau, num, idx)       # built-in status word
            torch.cuda.synchronize()
            # the call took no device memory: neither from the driver nor from torch's pool
            assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0
            assert status.cpu().tolist() == [0, 0]
            # same kernel, same inputs, same work order: the same bits
            assert torch.equal(got, want) and torch.equal(got_lse, want_lse) and torch.equal(got2, want)
            # and both within the stated bf16 tolerance of the oracle
            for h in range(H):
                o_ref, lse_ref = orc.sparse_attention(_f64(q[0, h]), _f64(k[0, h]), _f64(v[0, h]), lists[h], 128, tau)
                compare.check_output(_f64(got[0, h]), o_ref, "bf16", f"static h{h}")
                compare.check_output(_f64(want[0, h]), o_ref, "bf16", f"context h{h}")
                assert np.abs(_f64(got_lse[0, h]) - lse_ref).max() <= 1e-3
    finally:
        sp.sparstar_destroy(ctx)


def test_static_entry_reports_a_bad_list_entry_through_status_out():
    """An entry past the last key block is flagged as {ERR_BAD_INDEX, row} in the caller's status
    word; the kernel clamps the index, so no access leaves the tensors."""
    from paper_2608_10519_b200 import build
    build.build()
    import paper_2608_10519_b200 as sp
    g = torch.Generator().manual_seed(78)
    H, L_q, L_k = 1, 128 * 3, 128 * 5
    q = torch.randn((1, H, L_q, 128), generator=g).to(torch.bfloat16).cuda()
    k = torch.randn((1, H, L_k, 128), generator=g).to(torch.bfloat16).cuda()
    num = torch.tensor([[[2, 2, 2]]], dtype=torch.int32, device="cuda")
    idx = torch.tensor([[[[0, 1, 0, 0, 0], [1, 9, 0, 0, 0], [2, 3, 0, 0, 0]]]], dtype=torch.int32, device="cuda")
    o = torch.empty_like(q)
    status = torch.zeros((2,), dtype=torch.int32, device="cuda")
    sp.sparstar_sparse_attn_fwd_static(q, k, k, o, 128, 128 ** -0.5, num, idx, None, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [sp.ERR_BAD_INDEX, 1]
    # the next call starts from a clean status word
    idx[0, 0, 1, 1] = 4
    sp.sparstar_sparse_attn_fwd_static(q, k, k, o, 128, 128 ** -0.5, num, idx, None, status)
    torch.cuda.synchronize()
    assert status.cpu().tolist() == [0, 0]


def test_static_entry_rejects_what_it_cannot_hold():
    from paper_2608_10519_b200 import build
    build.build()
    import paper_2608_10519_b200 as sp
    # 65537 work items: one more than the fixed scratch holds -> refused before any launch
    H, n_q = 257, 255
    q = torch.empty((1, H, n_q * 128 + 128, 128), dtype=torch.bfloat16, device="cuda")      # n_q + 1 = 256 blocks
    assert H * 256 > 65536
    k = torch.empty((1, H, 128, 128), dtype=torch.bfloat16, device="cuda")
    num = torch.ones((1, H, 256), dtype=torch.int32, device="cuda")
    idx = torch.zeros((1, H, 256, 1), dtype=torch.int32, device="cuda")
    with pytest.raises(sp.SparstarError) as e:
        sp.sparstar_sparse_attn_fwd_static(q, k, k, q, 128, 0.1, num, idx)
    assert e.value.status == sp.ERR_TOO_LARGE
    # more query tiles in one (batch, head) than the order kernel sorts in shared memory
    n_big = 51201
    qb = torch.empty((1, 1, n_big * 128, 128), dtype=torch.bfloat16, device="cuda")
    numb = torch.ones((1, 1, n_big), dtype=torch.int32, device="cuda")
    idxb = torch.zeros((1, 1, n_big, 1), dtype=torch.int32, device="cuda")
    with pytest.raises(sp.SparstarError) as e:
        sp.sparstar_sparse_attn_fwd_static(qb, k[:, :1], k[:, :1], qb, 128, 0.1, numb, idxb)
    assert e.value.status == sp.ERR_TOO_LARGE
    # fp32 is outside what this entry point covers
    qf = torch.empty((1, 1, 64, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(sp.SparstarError) as e:
        sp.sparstar_sparse_attn_fwd_static(qf, qf, qf, qf, 64, 0.1, num[:, :1, :1].contiguous(), idx[:, :1, :1].contiguous())
    assert e.value.status == sp.ERR_UNSUPPORTED
