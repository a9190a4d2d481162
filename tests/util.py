"""Helpers shared by the parity tests: run the CUDA library and the CPU oracle on the same
instance and compare everything the search outputs, bit for bit."""
from __future__ import annotations

from typing import Dict, Optional, Tuple

import oracle
from xp_instances import Sketch


def windows_for(sk: Sketch, hole: int, windows: Optional[Dict[int, Tuple[int, int]]]):
    """Oracle-style {size: (begin, end)} and library-style [(hole, size, begin, end)]."""
    if windows is None:
        return None, None
    return dict(windows), [(hole, s, b, e) for s, (b, e) in windows.items()]


def assert_same(got, want, where=""):
    assert got.cand_count == want.cand_count, where
    assert got.match_count == want.match_count, where
    assert got.solved == want.solved, where
    if want.solved:
        assert (got.least_size, got.least_rank, got.least_text) == (want.least_size, want.least_rank, want.least_text), where


def check_sketch(xp, sk: Sketch, windows: Optional[Dict[int, Tuple[int, int]]] = None, first_points=None, **kw):
    """Full comparison of every hole of one sketch; returns the library's results."""
    gr = xp.xp_grammar_create(sk.grammar)
    ls = xp.xp_sketch_load(gr, sk)
    lib_rr = []
    for h in range(len(sk.holes)):
        _, rr = windows_for(sk, h, windows)
        lib_rr += rr or []
    res = xp.xp_repair(ls, rank_ranges=lib_rr or None, **kw)
    for h in range(len(sk.holes)):
        want = oracle.repair_hole(sk, h, rank_ranges=windows, first_points=first_points)
        assert_same(res[h], want, f"{sk.name} hole {h}")
    return res
