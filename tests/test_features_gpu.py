"""GPU tests of what surrounds the search proper: large families of operand tiles, the honest work
counters, refinement of the probe points from whole-domain failures, cancellation and time limit,
packed batch results, and one search cut into rank windows and merged."""
import ctypes as C
import os
import subprocess
import sys
import threading
import time

import numpy as np
import pytest

import oracle
from tests.util import assert_same, check_sketch
from xp_instances import (Hole, Sketch, Variable, config1, config2, config5, config5_instance, constant_set,
                          free_grammar, parse_expr)
from xp_instances.model import OP_CODE, P_BIN, P_CONST, P_VAR, Grammar, Production

pytestmark = pytest.mark.gpu

PATHS = [0, 1, 2]


def test_more_tile_segments_than_one_family_holds(xp):
    """Segments that share their register-side operands form families of at most 8; a grammar
    with more of them (here 4 nonterminals x 7 operators, then 9 copies of one production) must
    still have every candidate searched."""
    vs = [Variable("a", -3, 4), Variable("b", 0, 3)]
    ops = ["+", "-", "*", "/", "%", "min", "max"]
    prods = [Production(lhs=0, kind=P_VAR, var=0), Production(lhs=0, kind=P_VAR, var=1),
             Production(lhs=0, kind=P_CONST, value=2)]
    for nt, consts in [(1, [1, 3]), (2, [-2, 5]), (3, [0, 4, 7])]:
        prods += [Production(lhs=nt, kind=P_CONST, value=c) for c in consts]
    for right in (0, 1, 2, 3):
        prods += [Production(lhs=0, kind=P_BIN, op=OP_CODE[o], left=0, right=right) for o in ops]
    g = Grammar(vs, 4, prods)
    for spec in ["(a*3)-b", "min(a,5)+b", "(a%3)+4"]:
        sk = Sketch(g, [Hole(0, 5, spec_expr=parse_expr(spec, vs))], name=f"four operand kinds: {spec}")
        for flags in PATHS:
            check_sketch(xp, sk, flags=flags)
    g9 = free_grammar([Variable("x", 0, 5)], [1, 2, 3], ops=[])
    for _ in range(9):
        g9.productions.append(Production(lhs=0, kind=P_BIN, op=OP_CODE["+"], left=0, right=0))
    sk9 = Sketch(g9, [Hole(0, 5, spec_expr=parse_expr("(x+2)+1", g9.variables))], name="nine plus productions")
    for flags in PATHS:
        res = check_sketch(xp, sk9, flags=flags)
        assert res[0].cand_count == [0, 4, 0, 9 * 16, 0, 2 * 81 * 64]


def test_work_counters_add_up(xp):
    """Every candidate of a tile is either tested at the first probe or counted as skipped; the
    evaluations reported are the tests that ran plus the exact checks, never more than one filter
    test per candidate."""
    sk = config1(0)
    ls = xp.xp_sketch_load(xp.xp_grammar_create(sk.grammar), sk)
    r = xp.xp_repair(ls, flags=xp.XP_FLAG_ALWAYS_FILTER)[0]
    in_tiles = r.cand_count[3] + r.cand_count[5]
    assert r.filter_tests + r.candidates_skipped == in_tiles
    assert 0 < r.filter_tests <= in_tiles
    assert r.evals_executed >= r.filter_tests + r.cand_count[1]          # size 1 is checked rank by rank
    assert r.h2d_bytes > 0 and r.d2h_bytes > 0
    # a remainder-free grammar on a spec with no zero divisors: nothing is skipped
    vs = [Variable("i", 1, 9), Variable("j", 1, 9)]
    g = free_grammar(vs, [1, 2, 3], ops=["+", "-", "*"])
    ls2 = xp.xp_sketch_load(xp.xp_grammar_create(g), Sketch(g, [Hole(0, 5, spec_expr=parse_expr("(i*3)+j", vs))]))
    r2 = xp.xp_repair(ls2, flags=xp.XP_FLAG_ALWAYS_FILTER)[0]
    assert r2.candidates_skipped == 0 and r2.filter_tests == r2.cand_count[3] + r2.cand_count[5]
    info = xp.xp_sketch_info_get(ls2)
    assert info.n_holes == 1 and info.n_points == 64 and info.load_h2d_bytes > 0 and info.load_d2h_bytes > 0


def _one_odd_point_sketch():
    """i + j everywhere except at one interior point: every candidate equal to i + j on the
    static probes passes them and then fails the whole-domain check at that point."""
    vs = [Variable("i", 0, 48), Variable("j", 0, 48)]
    g = free_grammar(vs, constant_set(-2, 2))
    ids = np.arange(48 * 48, dtype=np.int64)
    coords = np.stack([ids // 48, ids % 48], axis=1).astype(np.int32)
    spec = (coords[:, 0].astype(np.int64) + coords[:, 1])
    odd = 17 * 48 + 29
    spec[odd] += 1
    return Sketch(g, [Hole(0, 5, spec_table=spec)], coords, name="i+j but for one point"), odd


def test_refinement_promotes_the_points_that_ended_whole_domain_checks(xp):
    sk, odd = _one_odd_point_sketch()
    want = oracle.repair_hole(sk)
    assert not want.solved
    ls = xp.xp_sketch_load(xp.xp_grammar_create(sk.grammar), sk)
    before = xp.xp_repair(ls)[0]
    assert_same(before, want)
    assert before.probe_survivors > 20                      # i+j, j+i, (i+j)+0, ... all reach the whole-domain check
    n = xp.xp_sketch_refine(ls)
    assert n >= 1 and xp.xp_sketch_info_get(ls).n_refined == n
    after = xp.xp_repair(ls)[0]
    assert_same(after, want)
    assert after.probe_survivors < before.probe_survivors and after.probe_survivors == 0
    assert xp.xp_sketch_refine(ls) == 0                     # nothing new was noted by the second search
    assert_same(xp.xp_repair(ls, flags=xp.XP_FLAG_NO_FILTER)[0], want)
    # on instances the static probes already decide, refinement changes nothing
    sk1 = config1(2)
    l1 = xp.xp_sketch_load(xp.xp_grammar_create(sk1.grammar), sk1)
    w1 = oracle.repair_hole(sk1)
    assert_same(xp.xp_repair(l1)[0], w1)
    xp.xp_sketch_refine(l1)
    assert_same(xp.xp_repair(l1)[0], w1)


def test_refinement_on_a_guard_that_fails_at_one_interior_point(xp):
    """A loop-bound hole (context ``j < HOLE``) whose spec differs from ``j < 40`` at a single
    interior point: constants >= 40 and many other candidates survive the probes."""
    vs = [Variable("i", 0, 40), Variable("j", 0, 40)]
    g = free_grammar(vs, constant_set(38, 44) + [0, 1])
    ids = np.arange(1600, dtype=np.int64)
    coords = np.stack([ids // 40, ids % 40], axis=1).astype(np.int32)
    spec = np.ones(1600, dtype=np.int64)
    spec[23 * 40 + 31] = 0
    sk = Sketch(g, [Hole(0, 3, ctx=parse_expr("j<HOLE", vs), spec_table=spec)], coords, name="guard with one odd point")
    want = oracle.repair_hole(sk)
    ls = xp.xp_sketch_load(xp.xp_grammar_create(g), sk)
    before = xp.xp_repair(ls)[0]
    assert_same(before, want)
    if before.probe_survivors > want.match_count[1] + want.match_count[3]:
        assert xp.xp_sketch_refine(ls) >= 1
        after = xp.xp_repair(ls)[0]
        assert_same(after, want)
        assert after.probe_survivors < before.probe_survivors


def test_cancel_word_and_time_limit(xp):
    sk = config2(0)
    ls = xp.xp_sketch_load(xp.xp_grammar_create(sk.grammar), sk)
    slow = dict(rank_ranges=[(0, 7, 0, 3_000_000_000)], flags=xp.XP_FLAG_NO_FILTER)      # rank by rank: hundreds of ms
    word = C.c_int32(1)
    with pytest.raises(xp.XpError) as e:
        xp.xp_repair(ls, cancel=word)
    assert e.value.status == 8 and "before launch" in str(e.value)
    word = C.c_int32(0)
    threading.Timer(0.03, lambda: setattr(word, "value", 1)).start()
    t0 = time.perf_counter()
    with pytest.raises(xp.XpError) as e:
        xp.xp_repair(ls, cancel=word, **slow)
    assert e.value.status == 8 and "between launches" in str(e.value)
    cancelled_after = time.perf_counter() - t0
    with pytest.raises(xp.XpError) as e:
        xp.xp_repair(ls, timeout_ms=5, **slow)
    assert e.value.status == 7
    # the library is usable afterwards, and a search that polls gives the same answer as one that does not
    word = C.c_int32(0)
    small = [(0, 7, 10 ** 9, 10 ** 9 + 50_000_000)]
    a = xp.xp_repair(ls, rank_ranges=small, cancel=word, timeout_ms=60_000)[0]
    b = xp.xp_repair(ls, rank_ranges=small)[0]
    assert a.match_count == b.match_count and a.least_rank == b.least_rank and a.n_launches > b.n_launches
    assert cancelled_after < 5.0


def test_packed_batch_results(xp):
    sks = config5(0, 24)
    grs = {}
    for sk in sks:
        key = tuple(v.hi for v in sk.grammar.variables)
        grs.setdefault(key, xp.xp_grammar_create(sk.grammar))
    keys = [tuple(v.hi for v in sk.grammar.variables) for sk in sks]
    loaded = xp.xp_sketch_load_batch([grs[k] for k in keys], sks, xp.marshal_sketches(sks))
    plain = xp.xp_repair_batch(loaded)
    packed, view = xp.xp_repair_batch(loaded, packed=True)
    arr = xp.summaries_as_numpy(packed)
    assert len(packed) == 24 and view.n_launches >= 2
    for i, sk in enumerate(sks):
        r = plain[i][0]
        assert_same(r, oracle.repair_hole(sk))
        assert list(arr["match_count"][i][:r.cand_count.__len__()]) == r.match_count
        assert bool(arr["solved"][i]) == r.solved and int(arr["least_rank"][i]) == r.least_rank
        assert (arr["least_text"][i].decode() if r.solved else "") == r.least_text
        assert int(arr["evals_executed"][i]) > 0
    lib = xp.load()
    out = (xp.binding.xp_hole_summary * 2)()
    assert lib.xp_result_pack(None, 1, out, 2, None) == 1


@pytest.mark.parametrize("world", [1, 2, 3, 7])
def test_one_search_cut_into_rank_windows_and_merged(xp, world):
    """The multi-GPU partition of one search, run here rank after rank on one GPU: disjoint rank
    windows per size through the library, merged by sum (counts) and minimum (least rank)."""
    from paper_2505_02146_b200.sharding import shard_rank_windows
    for sk, flags in [(config1(1), 0), (config1(4), xp.XP_FLAG_ALWAYS_FILTER), (config5_instance(0, 3), 0)]:
        want = oracle.repair_hole(sk)
        gr = xp.xp_grammar_create(sk.grammar)
        ls = xp.xp_sketch_load(gr, sk)
        counts = xp.xp_grammar_count(gr, 0, sk.holes[0].max_size)
        total = [0] * (sk.holes[0].max_size + 1)
        found = []
        for rank in range(world):
            r = xp.xp_repair(ls, rank_ranges=shard_rank_windows(counts, world, rank, hole=0), flags=flags)[0]
            total = [a + b for a, b in zip(total, r.match_count)]
            if r.solved:
                found.append((r.least_size, r.least_rank))
        assert total == want.match_count
        assert bool(found) == want.solved
        if found:
            assert min(found) == (want.least_size, want.least_rank)


def test_small_parity_cases_under_the_checked_build():
    """The library compiled with -DXP_CHECKS carries index checks (ranks against counts, table and
    queue slots, stack depths, point ids, segment numbers) that record a code instead of faulting;
    the small parity cases must run through it with nothing recorded (a recorded code makes every
    search return an error)."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, XP_CHECKED_BUILD="1")
    cases = "config1 or contexts or repeated or min_max or edge or windows or table_domain"
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
                        "tests/test_parity_gpu.py", "tests/test_features_gpu.py", "-k",
                        f"({cases} or family or refinement or rank_windows or one_point) and not checked_build"],
                       cwd=root, env=env, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-1000:]
    assert " passed" in r.stdout


def test_shifts_as_grammar_operators(xp):
    """<< and >> in productions, contexts and specs: no 32-bit filter loop exists for them, their
    operand tiles are evaluated exactly; a count outside 0..63 fails the candidate at that point."""
    vs = [Variable("i", 0, 6), Variable("j", -2, 5)]
    g = free_grammar(vs, [1, 2, 3, 64], ops=["+", "*", "<<", ">>"])
    for spec, ctx in [("(i<<2)+j", ""), ("(i+j)>>1", ""), ("i<<j", ""), ("j>>64", ""), ("(i<<3)+(j<<1)", "HOLE<<1"),
                      ("((i*3)>>1)<4", "(HOLE>>1)<4")]:
        sk = Sketch(g, [Hole(0, 5, ctx=parse_expr(ctx, vs) if ctx else [], spec_expr=parse_expr(spec, vs))], name=f"shifts: {spec}")
        for flags in PATHS:
            check_sketch(xp, sk, flags=flags)
    wide = [Variable("x", 2 ** 33, 2 ** 33 + 4), Variable("s", 0, 66)]
    gw = free_grammar(wide, [1, 31], ops=["-", "<<", ">>"])
    skw = Sketch(gw, [Hole(0, 5, spec_expr=parse_expr("(x>>s)-(1<<31)", wide))], name="wide shifts")
    for flags in PATHS:
        check_sketch(xp, skw, flags=flags)


def test_constant_only_holes(xp):
    """Instruction-parameter and buffer-size holes: the hole is filled from constants alone (a
    nonterminal with constant productions only, size bound 1).  The vector length of an
    instruction that must cover exactly the elements the source touches (2309 was written where
    1024 is right), and the row pitch of a staging buffer."""
    vs = [Variable("e", 0, 4096)]
    lengths = [16, 64, 256, 1000, 1024, 2048, 2309, 4096]
    prods = [Production(lhs=0, kind=P_CONST, value=c) for c in lengths]
    g = Grammar(vs, 1, prods)
    sk = Sketch(g, [Hole(0, 1, ctx=parse_expr("e<HOLE", vs), spec_expr=parse_expr("e<1024", vs))], name="vector length")
    res = check_sketch(xp, sk)
    assert res[0].least_text == "1024" and res[0].match_count == [0, 1] and res[0].cand_count == [0, 8]
    vs2 = [Variable("r", 0, 32), Variable("c", 0, 48)]
    prods2 = [Production(lhs=0, kind=P_VAR, var=0), Production(lhs=0, kind=P_VAR, var=1)]
    prods2 += [Production(lhs=1, kind=P_CONST, value=c) for c in (32, 40, 48, 64, 96)]
    g2 = Grammar(vs2, 2, prods2)
    sk2 = Sketch(g2, [Hole(1, 1, ctx=parse_expr("(r*HOLE)+c", vs2), spec_expr=parse_expr("(r*48)+c", vs2))], name="row pitch")
    res2 = check_sketch(xp, sk2)
    assert res2[0].least_text == "48" and res2[0].solved
    sk3 = Sketch(g2, [Hole(1, 1, ctx=parse_expr("(r*HOLE)+c", vs2), spec_expr=parse_expr("(r*50)+c", vs2))], name="no such pitch")
    assert not check_sketch(xp, sk3)[0].solved


def test_one_point_domain_where_a_large_share_of_the_candidates_match(xp):
    """A typed grammar of the large search's shape (leaves, E+E, E-E, E*K, E/P, E%P) on a domain of one
    point: there is one probe, so no second look, and every candidate whose value at that point is
    the target is a match.  Hits are frequent in every member of a family, the small ones included,
    the warps' hit queues run over, and the global survivor queue fills up; counts and least
    solutions must still be exact."""
    vs = [Variable("a", 3, 4), Variable("b", 5, 6), Variable("c", 2, 3), Variable("d", 7, 8)]
    prods = [Production(lhs=0, kind=P_VAR, var=i) for i in range(4)]
    prods += [Production(lhs=1, kind=P_CONST, value=k) for k in (-2, -1, 2, 3, 4, 6)]
    prods += [Production(lhs=2, kind=P_CONST, value=p) for p in (2, 3, 4, 5)]
    prods += [Production(lhs=0, kind=P_BIN, op=OP_CODE["+"], left=0, right=0),
              Production(lhs=0, kind=P_BIN, op=OP_CODE["-"], left=0, right=0),
              Production(lhs=0, kind=P_BIN, op=OP_CODE["*"], left=0, right=1),
              Production(lhs=0, kind=P_BIN, op=OP_CODE["/"], left=0, right=2),
              Production(lhs=0, kind=P_BIN, op=OP_CODE["%"], left=0, right=2)]
    g = Grammar(vs, 3, prods)
    for spec in ["a+b", "c-c", "(d*3)-1"]:
        sk = Sketch(g, [Hole(0, 9, spec_expr=parse_expr(spec, vs))], name=f"one point, target {spec}")
        res = check_sketch(xp, sk)
        assert res[0].cand_count[1:10:2] == [4, 88, 2640, 94688, 3769920]
        assert sum(res[0].match_count) > 1000


def test_negation_as_zero_minus_operand(xp):
    """Negation enters a grammar as  E -> Z - E  with  Z -> 0  (the reading taken for a unary minus): a typed
    production like the others, through the filter and both exact paths."""
    vs = [Variable("i", 0, 6), Variable("j", -2, 5)]
    prods = [Production(lhs=0, kind=P_VAR, var=0), Production(lhs=0, kind=P_VAR, var=1)]
    prods += [Production(lhs=0, kind=P_CONST, value=c) for c in (1, 2, 3)]
    prods += [Production(lhs=1, kind=P_CONST, value=0)]
    prods += [Production(lhs=0, kind=P_BIN, op=OP_CODE["+"], left=0, right=0),
              Production(lhs=0, kind=P_BIN, op=OP_CODE["*"], left=0, right=0),
              Production(lhs=0, kind=P_BIN, op=OP_CODE["-"], left=1, right=0)]
    g = Grammar(vs, 2, prods)
    for spec, ctx, least in [("0-(i+j)", "", "(0-(i+j))"), ("(0-i)*3", "", None), ("(0-(i*j))+7", "HOLE+7", "(i*(0-j))")]:
        sk = Sketch(g, [Hole(0, 7 if not ctx else 5, ctx=parse_expr(ctx, vs) if ctx else [], spec_expr=parse_expr(spec, vs))],
                    name=f"negation: {spec}")
        for flags in PATHS:
            res = check_sketch(xp, sk, flags=flags)
        if least:
            assert res[0].least_text == least
