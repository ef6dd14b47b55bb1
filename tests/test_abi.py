"""CPU-side checks of the boundary: the library builds/loads, exports every symbol the
header declares, and its host integer helpers agree with the oracle's definitions."""
import os
import re

import numpy as np
import pytest

from oracle import sparstar_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def sp():
    from paper_2608_10519_b200 import build
    build.build()
    import paper_2608_10519_b200 as sp
    sp.binding.load()
    return sp


def test_library_exports_every_declared_symbol(sp):
    hdr = open(os.path.join(ROOT, "include", "sparstar.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(sparstar_[a-z0-9_]+)\s*\(", hdr))
    assert {"sparstar_pool_blocks", "sparstar_score_select", "sparstar_sparse_attn_fwd",
            "sparstar_attn_fwd"} <= declared
    lib = sp.binding.load()
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(sp.binding.EXPORTS)


def test_num_blocks_and_budget_match_oracle(sp):
    for L, b in [(1, 128), (128, 128), (129, 128), (72000, 128), (144512, 128), (1664, 64)]:
        assert sp.sparstar_num_blocks(L, b) == orc.num_blocks(L, b)
    assert sp.sparstar_num_blocks(5, 0) == -1
    rng = np.random.default_rng(0)
    for _ in range(2000):
        n = int(rng.integers(0, 3000))
        rho = float(rng.choice([rng.uniform(0, 1.2), rng.integers(0, 17) / 16.0, rng.integers(0, 11) / 10.0]))
        assert sp.sparstar_budget(n, rho) == orc.budget(n, rho), (n, rho)
    assert sp.sparstar_budget(1125, 0.09375) == 106


def test_forced_count_matches_oracle(sp):
    rng = np.random.default_rng(1)
    for _ in range(500):
        b = int(rng.choice([4, 64, 128]))
        L = int(rng.integers(1, 40 * b))
        ranges = []
        for _ in range(int(rng.integers(0, 6))):
            s = int(rng.integers(-5, L + 5))
            ranges.append((s, s + int(rng.integers(0, 5 * b))))
        clipped = [(max(0, s), min(L, e)) for s, e in ranges]
        want = int(orc.forced_blocks(L, b, clipped).sum())
        assert sp.sparstar_forced_count(L, b, ranges) == want, (L, b, ranges)
    assert sp.sparstar_forced_count(76112, 128, [(0, 512), (512, 4112)]) == 33
    assert sp.sparstar_forced_count(144512, 128, [(72000, 72512)]) == 5


def test_status_strings(sp):
    assert sp.status_string(sp.OK) == "ok"
    assert "cap" in sp.status_string(sp.ERR_CAPACITY)


def test_calls_reject_bad_arguments_without_a_gpu(sp):
    lib = sp.binding.load()
    # null context / null pointers are refused on the host before any CUDA call
    assert lib.sparstar_pool_blocks(None, None, 128, None, None) == sp.ERR_INVALID_ARG
    assert lib.sparstar_attn_fwd(None, None, None, None, None, 128, 1.0, None, None) == sp.ERR_INVALID_ARG
    assert lib.sparstar_set_attn_impl(None, 0) == sp.ERR_INVALID_ARG
    assert lib.sparstar_set_debug(None, 1, -1) == sp.ERR_INVALID_ARG
    assert lib.sparstar_reserve_scratch(None, 1024, None) == sp.ERR_INVALID_ARG
    assert lib.sparstar_scratch_bytes(None) == -1
    assert lib.sparstar_check(None, None, None) == sp.ERR_INVALID_ARG
    assert "captur" in sp.status_string(sp.ERR_CAPTURE)
