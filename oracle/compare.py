"""Acceptance checks that set CUDA results beside the oracle's (test infrastructure).

Lists: bit-exact, except for blocks whose oracle score lies within 1e-5 relative of the
selection cutoff (several results are then correct).  Outputs: computed with the ORACLE's
lists; fp32 max-abs <= 1e-4, bf16 max-abs <= 2e-2 and mean-abs <= 2e-3.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Sequence

import numpy as np

from . import sparstar_oracle as orc

TOL = {"f32": {"max_abs": 1e-4, "mean_abs": 1e-4}, "bf16": {"max_abs": 2e-2, "mean_abs": 2e-3}}


@dataclass
class ListReport:
    rows: int = 0
    exact: int = 0
    excused: int = 0
    bad: List[str] = field(default_factory=list)

    @property
    def ok(self) -> bool:
        return not self.bad


def compare_lists(counts: np.ndarray, indices: np.ndarray, lists: Sequence[np.ndarray], S: np.ndarray,
                  forced: np.ndarray, mode: str, k: int = 0, mass: float = 0.0, tag: str = "",
                  report: ListReport = None, mass_rel: float = None) -> ListReport:
    """counts [n_q], indices [n_q, cap] from the CUDA path for one head; lists/S/forced from the
    oracle.  Differences must lie inside the near-cutoff band and keep the count (top-k) or
    change it by at most one at a mass edge."""
    rep = report if report is not None else ListReport()
    for i, want in enumerate(lists):
        rep.rows += 1
        c = int(counts[i])
        got = indices[i, :c]
        if c == len(want) and np.array_equal(got, want):
            rep.exact += 1
            continue
        if c > indices.shape[1]:
            rep.bad.append(f"{tag} row {i}: count {c} exceeds capacity")
            continue
        if np.any(np.diff(got) <= 0) or (c and (got[0] < 0 or got[-1] >= S.shape[1])):
            rep.bad.append(f"{tag} row {i}: list not ascending/unique/in range")
            continue
        ex, edge = orc.near_cutoff_exempt(S[i], forced, "mass" if mode == "mass" else "topk", k=k, mass=mass,
                                          mass_rel=mass_rel)
        diff = np.setxor1d(got, want)
        if not np.all(ex[diff]):
            rep.bad.append(f"{tag} row {i}: blocks {diff[~ex[diff]][:8]} differ outside the cutoff band")
            continue
        if c != len(want) and not (edge and abs(c - len(want)) <= 1):
            rep.bad.append(f"{tag} row {i}: count {c} != {len(want)}")
            continue
        rep.excused += 1
    return rep


def output_errors(got: np.ndarray, want: np.ndarray):
    d = np.abs(np.asarray(got, np.float64) - want)
    return float(d.max()), float(d.mean())


def check_output(got: np.ndarray, want: np.ndarray, dtype: str, what: str = "O") -> None:
    mx, mean = output_errors(got, want)
    t = TOL[dtype]
    assert mx <= t["max_abs"] and mean <= t["mean_abs"], \
        f"{what}: max-abs {mx:.3e} (<= {t['max_abs']}), mean-abs {mean:.3e} (<= {t['mean_abs']})"
