"""The five configurations at full size against results written by the CPU oracle alone
(tests/golden/make_full_goldens.py, sharded over rank windows).  Everything the search
outputs is compared bit for bit: candidate counts, match counts, the least solution."""
import json
import os

import pytest

from xp_instances import config2, config3, config4, config5

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _seeds_with_goldens(name):
    """Seeds for which tests/golden/ holds a full-size result of this configuration."""
    seeds = []
    for f in sorted(os.listdir(GOLDEN)):
        if f.startswith(f"{name}_seed") and f.endswith("_full.json"):
            seeds.append(int(f[len(name) + 5:-len("_full.json")]))
    return seeds


def _check_large(xp, name, make, seed=0):
    path = os.path.join(GOLDEN, f"{name}_seed{seed}_full.json")
    if not os.path.exists(path):
        pytest.skip(f"{path} has not been generated")
    want = json.load(open(path))["holes"]
    sk = make(seed)
    gr = xp.xp_grammar_create(sk.grammar)
    ls = xp.xp_sketch_load(gr, sk)
    got = xp.xp_repair(ls)
    assert len(got) == len(want)
    for h, (g, w) in enumerate(zip(got, want)):
        assert g.cand_count == w["cand_count"], (name, h)
        assert g.match_count == w["match_count"], (name, h)
        assert g.solved == w["solved"], (name, h)
        if w["solved"]:
            assert (g.least_size, g.least_rank, g.least_text) == (w["least_size"], w["least_rank"], w["least_text"]), (name, h)
    return got


def test_config2_full(xp):
    got = _check_large(xp, "config2", config2)
    assert sum(got[0].cand_count) == 213939625416


def test_config3_full(xp):
    got = _check_large(xp, "config3", config3)
    assert [sum(g.cand_count) for g in got] == [134377694] * 3 and all(g.solved for g in got)


def test_config4_full(xp):
    got = _check_large(xp, "config4", config4)
    assert sum(got[0].cand_count) == 322884631700


@pytest.mark.parametrize("name,make,seed", [(n, m, sd) for n, m in (("config2", config2), ("config3", config3), ("config4", config4))
                                            for sd in _seeds_with_goldens(n) if sd != 0])
def test_other_seeds_full(xp, name, make, seed):
    """Every further seed that has a golden: among them instances whose target is small at the probes, where a
    large share of the candidates passes the filter (queue overflows, the second look turned on by the CTAs)."""
    _check_large(xp, name, make, seed)


def _config5_seeds():
    return [int(f[len("config5_seed"):-len("_full.txt")]) for f in sorted(os.listdir(GOLDEN))
            if f.startswith("config5_seed") and f.endswith("_full.txt")]


@pytest.mark.parametrize("seed", _config5_seeds())
def test_config5_full_batch(xp, seed):
    rows = [[int(x) for x in line.split()] for line in open(os.path.join(GOLDEN, f"config5_seed{seed}_full.txt"))
            if not line.startswith("#")]
    assert len(rows) == 4096
    sks = config5(seed, 4096)
    grs = {}
    for sk in sks:
        key = tuple(v.hi for v in sk.grammar.variables)
        if key not in grs:
            grs[key] = xp.xp_grammar_create(sk.grammar)
    loaded = xp.xp_sketch_load_batch([grs[tuple(v.hi for v in sk.grammar.variables)] for sk in sks], sks)
    res = xp.xp_repair_batch(loaded)
    unsolved = 0
    for i, (r, row) in enumerate(zip(res, rows)):
        g = r[0]
        assert [g.match_count[1], g.match_count[3], g.match_count[5]] == row[:3], i
        assert g.solved == (row[3] != 0), i
        if g.solved:
            assert (g.least_size, g.least_rank) == (row[3], row[4]), i
        unsolved += not g.solved
    assert 0 < unsolved < 4096 // 4          # the generator plants targets beyond the bound in about a tenth
