"""Pins for the CPU oracle: each check fixes the oracle to something other
than itself - closed forms, brute force in pure Python, identities the paper
states, hand-enumerated integers, a library routine, a hand-worked example."""
import itertools
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import sparstar_oracle as orc
from workloads import CONFIGS, generate, get_config, pyramid_sweep

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


# ----------------------------------------------------------------- pooling
def test_pool_constant_and_ramp_closed_form():
    b, D = 8, 3
    x = np.full((24, D), 2.5)
    assert np.allclose(orc.pool_blocks(x, b), 2.5)
    # ramp t -> t : mean of block i is i*b + (b-1)/2
    x = np.arange(24, dtype=np.float64)[:, None] * np.ones((1, D))
    want = np.array([i * b + (b - 1) / 2 for i in range(3)])
    assert np.allclose(orc.pool_blocks(x, b)[:, 1], want, rtol=0, atol=1e-12)


def test_pool_tail_is_occupancy_times_mean_of_valid():
    # zero padding then division by nominal b (block-partition paragraph)
    b = 8
    x = rng.normal(size=(8 * 2 + 3, 5))
    p = orc.pool_blocks(x, b)
    assert p.shape == (3, 5)
    assert np.allclose(p[2], (3 / b) * x[16:].mean(axis=0), atol=1e-14)
    assert np.allclose(p[0], x[:8].mean(axis=0), atol=1e-14)


def test_score_bilinearity_brute_force():
    # Under Eq. 2: for full blocks S_ij equals the mean pairwise pre-softmax logit.
    b, D = 4, 6
    Q = rng.normal(size=(2 * b, D))
    K = rng.normal(size=(3 * b, D))
    tau = D ** -0.5
    S = orc.block_scores(orc.pool_blocks(Q, b), orc.pool_blocks(K, b), tau)
    for i in range(2):
        for j in range(3):
            acc = 0.0
            for t in range(i * b, (i + 1) * b):
                for u in range(j * b, (j + 1) * b):
                    acc += tau * sum(Q[t][d] * K[u][d] for d in range(D))
            assert abs(S[i, j] - acc / (b * b)) < 1e-12


def test_score_not_transposed_and_scaled():
    # rectangular, asymmetric: a transposed operand or a dropped tau fails
    qbar = np.array([[1.0, 0.0], [0.0, 2.0], [1.0, 1.0]])
    kbar = np.array([[3.0, 5.0], [7.0, 11.0]])
    S = orc.block_scores(qbar, kbar, 0.5)
    assert S.shape == (3, 2)
    assert np.array_equal(S, 0.5 * np.array([[3.0, 7.0], [10.0, 22.0], [8.0, 18.0]]))


# ----------------------------------------------------------------- forced sets, budget
def _forced_ids(w, ranges=None):
    f = orc.forced_blocks(w.L_k, w.block, ranges if ranges is not None else w.forced_ranges())
    return list(np.nonzero(f)[0])


def test_forced_sets_hand_enumerated():
    # text 0..511 -> blocks 0..3 at b=128; c0: text 0..127 -> blocks 0,1 at b=64
    assert _forced_ids(CONFIGS["c0"]) == [0, 1]
    assert _forced_ids(CONFIGS["c1"]) == [0, 1, 2, 3]
    assert _forced_ids(CONFIGS["c2"]) == [0, 1, 2, 3]
    # c3: text + image tokens 512..4111; 4112/128 = 32.125 -> block 32 straddles image|current
    assert _forced_ids(CONFIGS["c3"]) == list(range(33))
    for w in pyramid_sweep(0):
        assert _forced_ids(w) == [0, 1, 2, 3]


def test_forced_sets_paper_key_order_straddles():
    # Eq. 1 order (ref, text, cur): text = tokens 72000..72511 -> 562.5 .. 566.49 -> 5 blocks
    f = _forced_ids(CONFIGS["c2"], ranges=[(72000, 72512)])
    assert f == [562, 563, 564, 565, 566]
    # empty and touching ranges
    assert list(np.nonzero(orc.forced_blocks(300, 128, [(128, 128)]))[0]) == []
    assert list(np.nonzero(orc.forced_blocks(300, 128, [(127, 129)]))[0]) == [0, 1]
    assert list(np.nonzero(orc.forced_blocks(300, 128, [(256, 1000)]))[0]) == [2]


def test_block_counts():
    want = {"c0": (16, 26), "c1": (144, 711), "c2": (563, 1129), "c3": (563, 595)}
    for n, (nq, nk) in want.items():
        assert (CONFIGS[n].n_q, CONFIGS[n].n_k) == (nq, nk)
    assert [(w.n_q, w.n_k) for w in pyramid_sweep(2)] == [(38, 604), (144, 711), (319, 886), (563, 1129)]


def test_budget_closed_form():
    # Eq. 5 with the configurations' integers
    assert orc.budget(24, 0.25) == 6
    assert orc.budget(562, 0.20) == 113
    assert orc.budget(1125, 0.09375) == 106          # the paper's final-scale density
    assert orc.budget(1125, 0.625) == 704
    assert orc.budget(1125, 0.1875) == 211
    assert orc.budget(10, 0.3) == 3                   # 0.3*10 = 3.0000000000000004 in double
    assert orc.budget(7, 0.0) == 1                    # max(1, .)
    assert orc.budget(7, 1.0) == 7 and orc.budget(7, 5.0) == 7
    assert orc.budget(0, 0.5) == 0


# ----------------------------------------------------------------- top-k
def test_topk_matches_python_sort_and_invariants():
    for trial in range(50):
        n = int(rng.integers(3, 40))
        S = rng.normal(size=n)
        forced = rng.random(n) < 0.2
        n_sel = int((~forced).sum())
        k = int(rng.integers(0, n_sel + 1))
        got = list(orc.select_topk_row(S, forced, k))
        cand = sorted([j for j in range(n) if not forced[j]], key=lambda j: (-S[j], j))[:k]
        want = sorted(set(cand) | {j for j in range(n) if forced[j]})
        assert got == want
        assert got == sorted(set(got))
        assert len(got) == int(forced.sum()) + k
        inc = [S[j] for j in got if not forced[j]]
        exc = [S[j] for j in range(n) if not forced[j] and j not in got]
        if inc and exc:
            assert min(inc) >= max(exc)


def test_topk_ties_lower_index_wins():
    S = np.array([1.0, 5.0, 5.0, 5.0, 0.0, 5.0])
    forced = np.zeros(6, dtype=bool)
    assert list(orc.select_topk_row(S, forced, 2)) == [1, 2]
    assert list(orc.select_topk_row(S, forced, 3)) == [1, 2, 3]
    forced[2] = True    # forced blocks neither compete nor consume budget
    assert list(orc.select_topk_row(S, forced, 2)) == [1, 2, 3]


def test_no_quota_for_reference_blocks():
    # later clips: a row may keep no preceding-clip block at all
    S = np.concatenate([np.zeros(4), -np.ones(10), np.ones(10)])
    forced = np.zeros(24, dtype=bool)
    forced[:4] = True
    got = orc.select_topk_row(S, forced, 5)
    assert all(j < 4 or j >= 14 for j in got)


# ----------------------------------------------------------------- mass (benchmark-defined)
def test_mass_invariants_and_subset_brute_force():
    for trial in range(40):
        n = int(rng.integers(2, 13))
        S = rng.normal(size=n) * 2
        forced = np.zeros(n, dtype=bool)
        forced[rng.integers(0, n)] = True
        p = float(rng.uniform(0.05, 0.99))
        got = [j for j in orc.select_mass_row(S, forced, p) if not forced[j]]
        sel = [j for j in range(n) if not forced[j]]
        e = {j: math.exp(S[j]) for j in sel}
        Z = sum(e.values())
        mass = lambda js: sum(e[j] for j in js) / Z
        assert mass(got) >= p - 1e-12
        # minimal cardinality over ALL subsets, and among those the maximal mass
        best = None
        for r in range(1, len(sel) + 1):
            ok = [c for c in itertools.combinations(sel, r) if mass(c) >= p - 1e-12]
            if ok:
                best = (r, max(ok, key=mass))
                break
        assert len(got) == best[0]
        assert sorted(got) == sorted(best[1])
        # dropping the weakest taken block falls below p
        if len(got) > 1:
            weakest = min(got, key=lambda j: S[j])
            assert mass([j for j in got if j != weakest]) < p


def test_mass_all_when_p_is_one_and_single_when_tiny():
    S = rng.normal(size=9)
    forced = np.zeros(9, dtype=bool)
    assert list(orc.select_mass_row(S, forced, 1.0)) == list(range(9))
    assert list(orc.select_mass_row(S, forced, 1e-9)) == [int(np.argmax(S))]


# ----------------------------------------------------------------- attention
def _sdpa64(Q, K, V, tau):
    q, k, v = (torch.from_numpy(a)[None, None] for a in (Q, K, V))
    return torch.nn.functional.scaled_dot_product_attention(q, k, v, scale=tau)[0, 0].numpy()


def test_dense_matches_library_attention():
    Q, K, V = rng.normal(size=(7, 5)), rng.normal(size=(11, 5)), rng.normal(size=(11, 3))
    O, lse = orc.dense_attention(Q, K, V, 0.4)
    assert np.allclose(O, _sdpa64(Q, K, V, 0.4), atol=1e-13)
    want_lse = torch.logsumexp(torch.from_numpy(0.4 * Q @ K.T), dim=1).numpy()
    assert np.allclose(lse, want_lse, atol=1e-13)


def test_select_all_equals_dense_with_ragged_tails():
    b, D = 4, 6
    Q, K, V = rng.normal(size=(10, D)), rng.normal(size=(15, D)), rng.normal(size=(15, D))
    tau = D ** -0.5
    lists, S, forced = orc.select_head(Q, K, b, tau, [(0, 2)], "topk_ratio", ratio=1.0)
    assert all(list(l) == [0, 1, 2, 3] for l in lists)
    O, lse = orc.sparse_attention(Q, K, V, lists, b, tau)
    Od, lsed = orc.dense_attention(Q, K, V, tau)
    assert np.allclose(O, Od, atol=1e-13) and np.allclose(lse, lsed, atol=1e-13)


def test_sparse_equals_library_attention_on_gathered_keys():
    # Eq. 7: masked softmax == dense softmax over the kept keys only
    b, D = 4, 5
    Q, K, V = rng.normal(size=(6, D)), rng.normal(size=(18, D)), rng.normal(size=(18, D))
    lists = [[0, 3], [1, 2, 4]]     # block 4 is the partial tail (2 keys)
    O, _ = orc.sparse_attention(Q, K, V, lists, b, 0.3)
    for i, l in enumerate(lists):
        idx = np.concatenate([np.arange(j * b, min((j + 1) * b, 18)) for j in l])
        rows = slice(i * b, min((i + 1) * b, 6))
        assert np.allclose(O[rows], _sdpa64(Q[rows], K[idx], V[idx], 0.3), atol=1e-13)


def test_attention_permutation_invariance_and_constant_values():
    b, D = 4, 5
    Q, K, V = rng.normal(size=(4, D)), rng.normal(size=(12, D)), rng.normal(size=(12, D))
    O1, _ = orc.attention_block(Q, K, V, [0, 2], b, 0.3)
    perm = np.concatenate([np.arange(8, 12), np.arange(4, 8), np.arange(0, 4)])   # swap blocks 0 and 2
    O2, _ = orc.attention_block(Q, K[perm], V[perm], [0, 2], b, 0.3)
    assert np.allclose(O1, O2, atol=1e-13)
    V2 = V.copy()
    V2[4:8] = np.array([1.0, 2.0, 3.0, 4.0, 5.0])
    O3, _ = orc.attention_block(Q, K, V2, [1], b, 0.3)
    assert np.allclose(O3, np.array([1.0, 2.0, 3.0, 4.0, 5.0]), atol=1e-13)


# ----------------------------------------------------------------- hand-worked example
def test_hand_worked_example():
    g = json.load(open(os.path.join(GOLDEN, "hand_worked_d1.json")))
    b, tau = g["b"], g["tau"]
    ln2 = math.log(2.0)
    Q = np.array(g["q_over_ln2"])[:, None] * ln2
    K = np.array(g["k"])[:, None]
    V = np.array(g["v"])[:, None]
    kbar = orc.pool_blocks(K, b)
    assert np.allclose(kbar[:, 0], g["kbar"], atol=1e-15)
    S = orc.block_scores(orc.pool_blocks(Q, b), kbar, tau)
    assert np.allclose(S[0] / ln2, g["scores_over_ln2"], atol=1e-14)
    forced = orc.forced_blocks(K.shape[0], b, [tuple(r) for r in g["forced_ranges"]])
    assert list(forced) == [True, False, False, False]
    for k, want in g["topk"].items():
        assert list(orc.select_topk_row(S[0], forced, int(k))) == want
    for p, want in g["mass"].items():
        assert list(orc.select_mass_row(S[0], forced, float(p))) == want
    for key, want in g["attention"].items():
        blocks = [int(x) for x in key.split(",")]
        O, lse = orc.attention_block(Q, K, V, blocks, b, tau)
        assert np.allclose(O, want["O"], atol=1e-13)
        assert np.allclose(lse, math.log(want["sumexp"]), atol=1e-13)


# ----------------------------------------------------------------- whole selection on config 0
def test_config0_lists_invariants():
    w = get_config("c0")
    x = generate(w)
    tau = w.D ** -0.5
    for h in range(w.H):
        Q = x["q"][0, h].double().numpy()
        K = x["k"][0, h].double().numpy()
        lists, S, forced = orc.select_head(Q, K, w.block, tau, w.forced_ranges(), "topk_ratio", ratio=w.ratio)
        assert S.shape == (16, 26) and int((~forced).sum()) == 24
        for l in lists:
            assert len(l) == 8 and l[0] == 0 and l[1] == 1
            assert list(l) == sorted(set(int(j) for j in l))


def test_heads_are_independent():
    w = get_config("c0")
    x = generate(w)
    tau = w.D ** -0.5
    per_head = []
    for h in range(w.H):
        lists, _, _ = orc.select_head(x["q"][0, h].double().numpy(), x["k"][0, h].double().numpy(),
                                      w.block, tau, w.forced_ranges(), "topk_ratio", ratio=w.ratio)
        per_head.append([list(l) for l in lists])
    assert per_head[0] != per_head[1]          # fresh per head, no sharing


def test_near_cutoff_band_helper():
    S = np.array([9.0, 5.0, 4.00001, 4.0, 3.0])
    forced = np.array([True, False, False, False, False])
    ex, _ = orc.near_cutoff_exempt(S, forced, "topk", k=2)
    assert list(np.nonzero(ex)[0]) == [2, 3]
    ex, _ = orc.near_cutoff_exempt(S, forced, "topk", k=1)
    assert list(np.nonzero(ex)[0]) == [1]


def test_near_cutoff_band_mass_branch_hand_built_rows():
    """Scores ln(8, 4, 2, 1, 1) on the selectable blocks 1..5 (block 0 is kept): masses 1/2, 1/4,
    1/8, 1/16, 1/16, cumulative 0.5, 0.75, 0.875, 0.9375, 1."""
    S = np.concatenate([[99.0], np.log([8.0, 4.0, 2.0, 1.0, 1.0])])
    forced = np.array([True, False, False, False, False, False])
    ids = lambda ex: list(np.nonzero(ex)[0])
    # mass just AFTER rank 2 within 1e-5 p of p from above: r* = 2, the prefix may also run to rank 3
    ex, edge = orc.near_cutoff_exempt(S, forced, "mass", mass=0.75 * (1 - 5e-6))
    assert edge and ids(ex) == [2, 3]
    # mass just BEFORE rank 3 within 1e-5 p of p from below: r* = 3, the prefix may also stop at rank 2
    ex, edge = orc.near_cutoff_exempt(S, forced, "mass", mass=0.75 * (1 + 5e-6))
    assert edge and ids(ex) == [3, 4]
    # neither: only the score band around the cutoff block (rank 3 = block 3) - and nothing of rank r*-1
    ex, edge = orc.near_cutoff_exempt(S, forced, "mass", mass=0.8)
    assert not edge and ids(ex) == [3]
    # just outside the edge (2e-5 p away): no edge
    ex, edge = orc.near_cutoff_exempt(S, forced, "mass", mass=0.75 * (1 - 2e-5))
    assert not edge and ids(ex) == [2]
    # a narrower mass edge can be asked for
    ex, edge = orc.near_cutoff_exempt(S, forced, "mass", mass=0.75 * (1 - 5e-6), mass_rel=1e-6)
    assert not edge and ids(ex) == [2]
    # r* = 1: "before" is the empty prefix (mass 0)
    ex, edge = orc.near_cutoff_exempt(S, forced, "mass", mass=0.5 * (1 - 5e-6))
    assert edge and ids(ex) == [1, 2]
    ex, edge = orc.near_cutoff_exempt(S, forced, "mass", mass=0.3)
    assert not edge and ids(ex) == [1]
    # equal scores at the cutoff (blocks 4 and 5 tie): both are in the score band
    ex, edge = orc.near_cutoff_exempt(S, forced, "mass", mass=0.9)
    assert not edge and ids(ex) == [4, 5]
    # r* = last rank: rank r*+1 does not exist
    ex, edge = orc.near_cutoff_exempt(S, forced, "mass", mass=1.0)
    assert ids(ex) == [4, 5]


def test_compare_lists_uses_the_band_and_nothing_wider():
    from oracle import compare
    S = np.concatenate([[99.0], np.log([8.0, 4.0, 2.0, 1.0, 1.0])])[None]
    forced = np.array([True, False, False, False, False, False])
    p = 0.75 * (1 + 5e-6)                                    # oracle: r* = 3 -> blocks {0,1,2,3}
    want = [orc.select_mass_row(S[0], forced, p)]
    assert list(want[0]) == [0, 1, 2, 3]
    def rep(row):
        idx = np.zeros((1, 6), dtype=np.int32)
        idx[0, :len(row)] = row
        return compare.compare_lists(np.array([len(row)]), idx, want, S, forced, "mass", mass=p)
    assert rep([0, 1, 2, 3]).exact == 1
    r = rep([0, 1, 2])                                        # stopped one early at the mass edge: excused
    assert r.ok and r.excused == 1
    assert not rep([0, 1]).ok                                 # two early: not excused
    assert not rep([0, 1, 3]).ok                              # dropped rank 2 (= r*-1): not excused
    assert not rep([0, 1, 2, 3, 4, 5]).ok                     # two more blocks: count off by two
    assert not rep([0, 2, 1, 3]).ok                           # not ascending


# ----------------------------------------------------------------- attention-mass analysis
def test_block_mass_rows_sum_to_one_and_uniform_case():
    b = 4
    Q, K = rng.normal(size=(10, 6)), rng.normal(size=(15, 6))
    M = orc.block_mass(Q, K, b, 0.4)
    assert M.shape == (3, 4) and np.allclose(M.sum(axis=1), 1.0, atol=1e-14)
    # zero queries -> uniform attention -> a block's mass is its share of the keys
    M0 = orc.block_mass(np.zeros((5, 6)), K, b, 0.4)
    assert np.allclose(M0, np.array([4, 4, 4, 3]) / 15.0, atol=1e-15)


def test_block_mass_pure_python_brute_force():
    b, D = 2, 3
    Q, K = rng.normal(size=(3, D)), rng.normal(size=(5, D))
    M = orc.block_mass(Q, K, b, 0.7)
    for i in range(2):
        rows = range(i * b, min((i + 1) * b, 3))
        for j in range(3):
            acc = 0.0
            for t in rows:
                w = [math.exp(0.7 * sum(Q[t][d] * K[u][d] for d in range(D))) for u in range(5)]
                acc += sum(w[j * b:min((j + 1) * b, 5)]) / sum(w)
            assert abs(M[i, j] - acc / len(rows)) < 1e-13


def test_retained_mass_equals_lse_gap():
    # two independent routes: block masses summed over the kept set, and exp(LSE_sparse - LSE_dense)
    b, D = 4, 5
    Q, K, V = rng.normal(size=(10, D)), rng.normal(size=(22, D)), rng.normal(size=(22, D))
    lists = [[0, 3, 5], [1, 2], [0, 1, 2, 3, 4, 5]]
    M = orc.block_mass(Q, K, b, 0.5)
    _, lse_s = orc.sparse_attention(Q, K, V, lists, b, 0.5)
    _, lse_d = orc.dense_attention(Q, K, V, 0.5)
    gap = np.exp(lse_s - lse_d)
    want = np.array([gap[i * b:min((i + 1) * b, 10)].mean() for i in range(3)])
    assert np.allclose(orc.retained_mass(M, lists), want, atol=1e-13)
    assert abs(orc.retained_mass(M, lists)[2] - 1.0) < 1e-13
