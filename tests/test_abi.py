"""CPU-side checks of the C-ABI library: it loads, exports what include/xp.h declares, and its
host logic (counts, unranking, argument checking) agrees with the oracle.  No GPU work."""
import ctypes as C
import os
import random
import re

import pytest

import oracle
import paper_2505_02146_b200 as xp
from paper_2505_02146_b200 import binding as B
from xp_instances import (Variable, config1, config2_grammar, config3, config4, config5_instance, free_grammar,
                          quasi_affine_grammar)

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    lib = xp.load()
    header = open(os.path.join(ROOT, "include", "xp.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(xp_[a-z0-9_]+)\s*\(", header))
    assert {"xp_grammar_create", "xp_sketch_load", "xp_repair", "xp_repair_batch", "xp_result_get"} <= declared
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(B.EXPORTS)


def test_counts_agree_with_oracle():
    for g, K in [(config1(0).grammar, 5), (config2_grammar(), 7), (config3(0).grammar, 6),
                 (config4(0, 4096).grammar, 9), (config5_instance(0, 0).grammar, 6)]:
        gr = xp.xp_grammar_create(g)
        for nt in range(g.n_nonterminals):
            assert xp.xp_grammar_count(gr, nt, K) == oracle.counts(g, nt, K)


def test_unranking_agrees_with_oracle_listing():
    rnd = random.Random(1)
    vs = [Variable("p", 0, 2), Variable("q", 0, 3), Variable("r", 1, 3)]
    cases = [(free_grammar(vs[:2], [-2, 0, 1, 3]), 7), (quasi_affine_grammar(vs, [-2, 0, 3], [1, 2]), 7),
             (config1(0).grammar, 5)]
    for g, K in cases:
        gr = xp.xp_grammar_create(g)
        for nt in range(g.n_nonterminals):
            cnt = oracle.counts(g, nt, K)
            for size in range(1, K + 1):
                if cnt[size] == 0:
                    continue
                if cnt[size] <= 3000:
                    want = oracle.listing(g, nt, size)
                    got = [xp.xp_grammar_unrank(gr, nt, size, r)[0] for r in range(cnt[size])]
                    assert got == want
                else:
                    for r in [0, cnt[size] - 1] + [rnd.randrange(cnt[size]) for _ in range(60)]:
                        assert xp.xp_grammar_unrank(gr, nt, size, r)[0] == oracle.listing(g, nt, size, r, r + 1)[0]
    # large ranks of the big configs
    for g, size in [(config2_grammar(), 7), (config4(0, 4096).grammar, 9)]:
        gr = xp.xp_grammar_create(g)
        n = oracle.counts(g, 0, size)[size]
        for r in [0, n - 1] + [rnd.randrange(n) for _ in range(40)]:
            assert xp.xp_grammar_unrank(gr, 0, size, r)[0] == oracle.listing(g, 0, size, r, r + 1)[0]


def test_argument_checking_and_error_strings():
    lib = xp.load()
    out = C.c_void_p()
    assert lib.xp_grammar_create(None, C.byref(out)) == 1
    assert b"null" in lib.xp_last_error()
    g = config1(0).grammar
    gr = xp.xp_grammar_create(g)
    with pytest.raises(xp.XpError) as e:
        xp.xp_grammar_unrank(gr, 0, 5, 342950)
    assert e.value.status == 1
    with pytest.raises(xp.XpError) as e:
        xp.xp_grammar_count(gr, 3, 5)
    assert e.value.status == 1
    big = free_grammar([Variable("x", 0, 4)], list(range(2000)))
    gb = xp.xp_grammar_create(big)
    assert xp.xp_grammar_count(gb, 0, 5)[5] == 2 * 25 * 2001 ** 3
    with pytest.raises(xp.XpError) as e:
        xp.xp_grammar_count(gb, 0, 13)
    assert e.value.status == 4
    bad = config1(0).grammar
    bad.productions[-1] = type(bad.productions[-1])(lhs=0, kind=2, op=7, left=0, right=0)     # '<' is not a grammar operator
    with pytest.raises(xp.XpError) as e:
        xp.xp_grammar_create(bad)
    assert e.value.status == 2


def test_no_cpu_fallback_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    gr = xp.xp_grammar_create(config1(0).grammar)
    with pytest.raises(xp.XpError) as e:
        xp.xp_sketch_load(gr, config1(0))
    assert e.value.status == 6
    with pytest.raises(xp.XpError) as e:
        xp.xp_sketch_load_batch([gr, gr], [config1(0), config1(1)])
    assert e.value.status == 6 and "sketch 0" in str(e.value)


def test_batch_load_checks_its_arguments_before_touching_a_device():
    lib = xp.load()
    outs = (C.c_void_p * 2)()
    assert lib.xp_sketch_load_batch(None, None, 2, outs) == 1
    assert b"null" in lib.xp_last_error()
    gr = xp.xp_grammar_create(config1(0).grammar)
    sk = config1(0)
    sk.holes[0].max_size = 99                       # beyond XP_MAX_SIZE: refused by the host-side checks
    with pytest.raises(xp.XpError) as e:
        xp.xp_sketch_load_batch([gr], [sk])
    assert e.value.status == 3 and "sketch 0" in str(e.value)
