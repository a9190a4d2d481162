"""Pins for the CPU oracle: closed forms, hand-derived sets, a separate pure-Python
brute force over materialised trees, invariants and C division identities.  None of
these re-use the oracle's own code to produce the expected values."""
import itertools
import math
import os
import random

import numpy as np
import pytest

import oracle
from tests import pybrute
from xp_instances import (Hole, JointHole, Sketch, Variable, config1, config2_grammar, config3, config4,
                          config5_instance, constant_set, free_grammar, parse_expr,
                          quasi_affine_grammar)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def catalan(n):
    return math.comb(2 * n, n) // (n + 1)


def free_closed_form(L, B, size):
    """Free binary grammar with L leaves and B operators: Catalan(n) * B^n * L^(n+1) at size 2n+1."""
    if size % 2 == 0:
        return 0
    n = (size - 1) // 2
    return catalan(n) * B ** n * L ** (n + 1)


# ---------------------------------------------------------------- closed-form counts

@pytest.mark.parametrize("name,L,K,expected", [
    ("c1", 19, 5, [19, 1805, 342950]),
    ("c2", 136, 7, [136, 92480, 125772800, 213813760000]),
    ("c3", 139, 6, [139, 96605, 134280950]),
])
def test_counts_free_grammar_closed_form(name, L, K, expected):
    if name == "c1":
        g = config1(0).grammar
    elif name == "c2":
        g = config2_grammar()
    else:
        g = config3(0).grammar
    assert g.leaf_count() == L
    got = oracle.counts(g, 0, K)
    assert [got[s] for s in range(1, K + 1, 2)] == expected
    assert all(got[s] == 0 for s in range(0, K + 1, 2))
    assert [got[s] for s in range(K + 1)] == [free_closed_form(L, 5, s) if s else 0 for s in range(K + 1)]


def test_counts_config5_closed_form():
    for idx in range(6):
        g = config5_instance(0, idx).grammar
        L = len(g.variables) + 33
        assert oracle.counts(g, 0, 6) == [0, L, 0, 5 * L * L, 0, 2 * 25 * L ** 3, 0]


def test_counts_typed_grammar_recurrence():
    """E ::= v | E+E | E-E | E*K | E/P | E%P with |K| = 257, |P| = 128, 4 variables:
    b_1 = 4, b_s = 2*sum_a b_a*b_(s-1-a) + (257 + 128 + 128)*b_(s-2)."""
    g = config4(0, n_points=4096).grammar
    b = {1: 4}
    for s in range(3, 10, 2):
        b[s] = 2 * sum(b[a] * b[s - 1 - a] for a in range(1, s - 1, 2)) + 513 * b[s - 2]
    assert [b[s] for s in (1, 3, 5, 7, 9)] == [4, 2084, 1102436, 591874756, 322291652420]
    got = oracle.counts(g, 0, 9)
    assert got == [0, 4, 0, 2084, 0, 1102436, 0, 591874756, 0, 322291652420]
    assert oracle.counts(g, 1, 3) == [0, 257, 0, 0]
    assert oracle.counts(g, 2, 3) == [0, 128, 0, 0]


def test_constant_set_is_a_set():
    cs = constant_set(-64, 64, [2 ** e for e in range(11)])
    assert len(cs) == 133 and len(set(cs)) == 133
    assert cs[:129] == list(range(-64, 65)) and cs[129:] == [128, 256, 512, 1024]


def test_count_overflow_is_reported():
    vs = [Variable("x", 0, 4)]
    g = free_grammar(vs, list(range(2000)))
    with pytest.raises(OverflowError):
        oracle.counts(g, 0, 13)


# ---------------------------------------------------------------- hand-derived sets (golden file)

def _golden_rows():
    rows, sets, ranks = [], [], []
    for line in open(os.path.join(GOLDEN, "config1_hand_derived.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        parts = [p.strip() for p in line.split("|")]
        if parts[0].startswith("set"):
            size, spec = parts[0].split(None, 1)
            sets.append((int(size[3:]), spec, parts[1].split()))
        elif parts[0].startswith("rank"):
            size, text = parts[0].split(None, 1)
            ranks.append((int(size[4:]), text, int(parts[1])))
        else:
            rows.append((parts[0], [int(x) for x in parts[1].split()], int(parts[2]), int(parts[3]), parts[4]))
    return rows, sets, ranks


def _c1(spec):
    vs = [Variable("i", 0, 16), Variable("j", 0, 16)]
    g = free_grammar(vs, constant_set(-8, 8))
    return Sketch(g, [Hole(0, 5, spec_expr=parse_expr(spec, vs))])


def test_hand_derived_match_counts_and_least():
    rows, sets, ranks = _golden_rows()
    assert len(rows) == 4 and len(sets) == 3 and len(ranks) == 5
    for spec, m135, lsize, lrank, ltext in rows:
        r = oracle.repair_hole(_c1(spec))
        assert [r.match_count[1], r.match_count[3], r.match_count[5]] == m135, spec
        assert (r.solved, r.least_size, r.least_rank, r.least_text) == (True, lsize, lrank, ltext), spec
    g = _c1("i").grammar
    for size, text, rank in ranks:
        assert oracle.listing(g, 0, size, rank, rank + 1) == [text]


def test_hand_derived_match_sets_are_complete():
    rows, sets, ranks = _golden_rows()
    for size, spec, members in sets:
        sk = _c1(spec)
        texts = oracle.listing(sk.grammar, 0, size)
        found = []
        for rank, t in enumerate(texts):
            if t in members:
                r = oracle.repair_hole(sk, rank_ranges={1: (0, 0), 3: (0, 0), 5: (0, 0), size: (rank, rank + 1)})
                assert r.match_count[size] == 1, (spec, t)
                found.append(t)
        assert sorted(found) == sorted(members)
        full = oracle.repair_hole(sk)
        assert full.match_count[size] == len(members)


# ---------------------------------------------------------------- brute force on tiny inputs

def _tiny_cases():
    rnd = random.Random(7)
    cases = []
    vs2 = [Variable("a", 0, 3), Variable("b", -1, 2)]
    cases.append((free_grammar(vs2, [-2, 0, 1, 3]), vs2))
    vs1 = [Variable("x", -2, 3)]
    cases.append((free_grammar(vs1, [0, 1, 2, -1, 4]), vs1))
    cases.append((free_grammar(vs2, [2, -3], ops=["-", "/", "%"]), vs2))
    vs3 = [Variable("p", 0, 2), Variable("q", 0, 3), Variable("r", 1, 3)]
    cases.append((quasi_affine_grammar(vs3, [-2, 0, 3], [1, 2]), vs3))
    return cases, rnd


def test_listing_equals_materialised_enumeration():
    cases, _ = _tiny_cases()
    for g, vs in cases:
        T = pybrute.all_trees(g, 5)
        for nt in range(g.n_nonterminals):
            for size in range(1, 6):
                want = [pybrute.tree_text(t, g) for t in T[(nt, size)]]
                assert oracle.counts(g, nt, size)[size] == len(want)
                assert oracle.listing(g, nt, size) == want
                if len(want) > 10:           # windows are slices of the full listing
                    for lo, hi in [(0, 1), (3, 9), (len(want) // 2, len(want) // 2 + 7), (len(want) - 2, len(want))]:
                        assert oracle.listing(g, nt, size, lo, hi) == want[lo:hi]


def test_repair_equals_brute_force():
    cases, rnd = _tiny_cases()
    n_checked = 0
    for g, vs in cases:
        T = pybrute.all_trees(g, 5)
        names = [v.name for v in vs]
        specs = []
        for size in (1, 3, 5, 5, 5):                 # specs drawn from the grammar itself ...
            specs.append(pybrute.tree_text(rnd.choice(T[(0, size)]), g))
        specs += [f"({names[0]}*2)-1", "0", f"{names[-1]}<1"]       # ... and a few outside it
        ctxs = ["", f"HOLE*2+{names[0]}", f"{names[0]}<HOLE", "min(HOLE,1)", f"HOLE/{names[-1]}"]
        for spec in specs:
            for ctx in ctxs[:2] if spec != specs[0] else ctxs:
                sk = Sketch(g, [Hole(0, 5, ctx=parse_expr(ctx, vs) if ctx else [], spec_expr=parse_expr(spec, vs))])
                cand, match, least, matches = pybrute.repair(sk)
                r = oracle.repair_hole(sk)
                assert r.cand_count == cand and r.match_count == match, (spec, ctx)
                if least is None:
                    assert not r.solved
                else:
                    assert (r.solved, r.least_size, r.least_rank, r.least_text) == (True,) + least
                # every single rank decided alike (match set, not only its size), on a sample of ranks
                for s in (3, 5):
                    for rank in rnd.sample(range(cand[s]), 5) + [m[1] for m in matches if m[0] == s][:5]:
                        one = oracle.repair_hole(sk, rank_ranges={1: (0, 0), 3: (0, 0), 5: (0, 0), s: (rank, rank + 1)})
                        assert one.match_count[s] == int((s, rank) in matches)
                n_checked += 1
    assert n_checked >= 40


def test_table_domain_and_table_spec_equal_brute_force():
    rnd = random.Random(3)
    vs = [Variable("u", 0, 5), Variable("w", 0, 4)]
    g = free_grammar(vs, [1, 2, 3])
    coords = np.array([[4, 3], [0, 0], [2, 1], [3, 3], [1, 2], [4, 0]], dtype=np.int32)
    for text in ["(u*2)+w", "(u%3)", "((u+w)/2)"]:
        spec = np.array([pybrute.code_value(parse_expr(text, vs), tuple(int(x) for x in row)) for row in coords], dtype=np.int64)
        sk = Sketch(g, [Hole(0, 5, spec_table=spec)], coords)
        cand, match, least, _ = pybrute.repair(sk)
        r = oracle.repair_hole(sk)
        assert r.cand_count == cand and r.match_count == match
        assert (r.least_size, r.least_rank, r.least_text) == least


# ---------------------------------------------------------------- invariants

def _points(sk):
    return pybrute.points_of(sk)


def test_returned_solution_matches_everywhere_independent_evaluator():
    for seed in range(5):
        sk = config1(seed)
        r = oracle.repair_hole(sk)
        assert r.solved
        h = sk.holes[0]
        for pt in _points(sk):
            assert pybrute.text_value(r.least_text, sk.grammar, pt) == pybrute.code_value(h.spec_expr, pt)


def test_planted_target_is_recovered_or_beaten():
    for seed in range(5):
        sk = config1(seed)
        planted = sk.holes[0].note
        r = oracle.repair_hole(sk)
        texts5 = oracle.listing(sk.grammar, 0, 5)
        planted_rank = texts5.index(planted)
        assert r.solved and (r.least_size, r.least_rank) <= (5, planted_rank)
        assert r.match_count[5] >= 1


def test_point_order_does_not_change_results():
    sk = _c1("(i*8)+j")
    base = oracle.repair_hole(sk)
    perm = list(range(256)); random.Random(5).shuffle(perm)
    other = oracle.repair_hole(sk, first_points=perm)
    assert (base.match_count, base.least_rank, base.least_text) == (other.match_count, other.least_rank, other.least_text)
    assert other.evals != base.evals      # only the work changes


def test_domain_subset_is_monotone():
    vs = [Variable("i", 0, 16), Variable("j", 0, 16)]
    g = free_grammar(vs, constant_set(-8, 8))
    full = np.array(list(itertools.product(range(16), range(16))), dtype=np.int32)
    spec = parse_expr("(i/4)+j", vs)
    sub = full[[0, 1, 17]]
    r_full = oracle.repair_hole(Sketch(g, [Hole(0, 5, spec_expr=spec)], full))
    r_box = oracle.repair_hole(Sketch(g, [Hole(0, 5, spec_expr=spec)], None))
    r_sub = oracle.repair_hole(Sketch(g, [Hole(0, 5, spec_expr=spec)], sub))
    assert r_full.match_count == r_box.match_count and r_full.least_rank == r_box.least_rank
    assert all(a <= b for a, b in zip(r_full.match_count, r_sub.match_count))
    assert r_sub.match_count[5] > r_full.match_count[5]


def test_commutative_pairs_match_together():
    sk = _c1("(i*8)+j")
    texts = oracle.listing(sk.grammar, 0, 5)
    where = {t: k for k, t in enumerate(texts)}
    for a, b in [("(j+(i*8))", "((i*8)+j)"), ("(j+(8*i))", "((8*i)+j)")]:
        for t in (a, b):
            one = oracle.repair_hole(sk, rank_ranges={1: (0, 0), 3: (0, 0), 5: (where[t], where[t] + 1)})
            assert one.match_count[5] == 1


def test_constant_spec_at_size_one():
    for c, present in [(7, True), (-8, True), (9, False), (0, True)]:
        r = oracle.repair_hole(_c1(str(c)))
        assert r.match_count[1] == int(present)


def test_zero_divisor_candidates_are_counted_but_never_match():
    vs = [Variable("x", 0, 3)]
    g = free_grammar(vs, [0], ops=["/", "%"])
    # size 3: x/x, x/0, 0/x, 0/0, x%x, x%0, 0%x, 0%0 -- every one divides by zero somewhere on x in {0,1,2}
    sk = Sketch(g, [Hole(0, 3, spec_expr=parse_expr("0", vs))])
    r = oracle.repair_hole(sk)
    assert r.cand_count == [0, 2, 0, 8] and r.match_count == [0, 1, 0, 0]
    # on x in {1,2} only: 0/x, 0%x and x%x are 0 everywhere
    sk2 = Sketch(free_grammar([Variable("x", 1, 3)], [0], ops=["/", "%"]),
                 [Hole(0, 3, spec_expr=parse_expr("0", [Variable("x", 1, 3)]))])
    assert oracle.repair_hole(sk2).match_count == [0, 1, 0, 3]
    # an invalid subtree poisons the tree even under *0
    g3 = free_grammar(vs, [0], ops=["*", "/"])
    sk3 = Sketch(g3, [Hole(0, 5, spec_expr=parse_expr("0", vs))])
    texts = oracle.listing(g3, 0, 5)
    rank = texts.index("(0*(x/0))")
    one = oracle.repair_hole(sk3, rank_ranges={1: (0, 0), 3: (0, 0), 5: (rank, rank + 1)})
    assert one.match_count[5] == 0


def test_rank_windows_partition_the_search():
    sk = _c1("i%4")
    full = oracle.repair_hole(sk)
    total = 0
    cuts = [0, 1, 68590, 100000, 342949, 342950]
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        part = oracle.repair_hole(sk, rank_ranges={1: (0, 0), 3: (0, 0), 5: (lo, hi)})
        assert part.cand_count == full.cand_count          # counts stay syntactic
        total += part.match_count[5]
    assert total == full.match_count[5]


# ---------------------------------------------------------------- C arithmetic

def test_c_division_identities():
    vs = [Variable("a", 0, 1), Variable("b", 0, 1)]
    div, mod = parse_expr("a/b", vs), parse_expr("a%b", vs)
    for a, b, q, r in [(-7, 2, -3, -1), (7, -2, -3, 1), (-7, -2, 3, -1), (7, 2, 3, 1), (0, 5, 0, 0), (-1, 5, 0, -1)]:
        assert oracle.eval_code(div, [a, b]) == q and oracle.eval_code(mod, [a, b]) == r
    rnd = random.Random(11)
    for _ in range(2000):
        a = rnd.randrange(-2 ** 63, 2 ** 63) >> rnd.randrange(0, 60)
        b = rnd.randrange(-2 ** 63, 2 ** 63) >> rnd.randrange(0, 62)
        if b == 0:
            assert oracle.eval_code(div, [a, b]) is None and oracle.eval_code(mod, [a, b]) is None
            continue
        q, r = oracle.eval_code(div, [a, b]), oracle.eval_code(mod, [a, b])
        if (a, b) != (-2 ** 63, -1):
            assert q * b + r == a and abs(r) < abs(b) and (r == 0 or (r < 0) == (a < 0))
    lo = -2 ** 63
    assert oracle.eval_code(div, [lo, -1]) == lo and oracle.eval_code(mod, [lo, -1]) == 0
    assert oracle.eval_code(parse_expr("a*b", vs), [2 ** 62, 4]) == 0                 # wraps
    assert oracle.eval_code(parse_expr("a+b", vs), [2 ** 63 - 1, 1]) == -2 ** 63
    assert oracle.eval_code(parse_expr("a-b", vs), [-2 ** 63, 1]) == 2 ** 63 - 1


def test_context_operators():
    vs = [Variable("a", 0, 1), Variable("b", 0, 1)]
    for text, pt, want in [("a<b", [1, 2], 1), ("a<b", [2, 2], 0), ("a<=b", [2, 2], 1), ("a==b", [3, 3], 1),
                           ("a!=b", [3, 3], 0), ("min(a,b)", [-4, 9], -4), ("max(a,b)", [-4, 9], 9),
                           ("a&&b", [5, 0], 0), ("a&&b", [5, -1], 1), ("a||b", [0, 0], 0), ("a||b", [0, 7], 1),
                           ("(a/b)||1", [1, 0], None), ("HOLE*56+a", [3, 0], 563)]:
        assert oracle.eval_code(parse_expr(text, vs), pt, hole=10) == want, text


def test_min_max_as_grammar_operators():
    """min and max in the grammar: counts follow the closed form with 7 operators, listing and
    search agree with the materialised brute force, and the trip count of a remainder tile
    (8, 8, 8, 6 for io = 0..3 of a 30-long loop split by 8) is found as min(8,(30-(io*8)))."""
    vs = [Variable("io", 0, 4)]
    g = free_grammar(vs, [8, 30], ops=["-", "*", "min"])
    assert oracle.counts(g, 0, 7) == [0, 3, 0, 27, 0, 486, 0, 10935]
    T = pybrute.all_trees(g, 5)
    for size in (1, 3, 5):
        assert oracle.listing(g, 0, size) == [pybrute.tree_text(t, g) for t in T[(0, size)]]
    coords = np.array([[0], [1], [2], [3]], dtype=np.int32)
    sk = Sketch(g, [Hole(0, 7, spec_table=np.array([8, 8, 8, 6], dtype=np.int64))], coords)
    r = oracle.repair_hole(sk)
    cand, match, least, _ = pybrute.repair(sk)
    assert r.cand_count == cand and r.match_count == match == [0, 0, 0, 0, 0, 0, 0, 4]
    assert (r.least_size, r.least_rank, r.least_text) == least == (7, 7840, "min(8,(30-(io*8)))")
    for io in range(4):
        assert pybrute.text_value(r.least_text, g, (io,)) == min(8, 30 - io * 8)
    full = free_grammar([Variable("a", -3, 4), Variable("b", 0, 3)], [0, 2], ops=["+", "-", "*", "/", "%", "min", "max"])
    assert oracle.counts(full, 0, 5) == [0, 4, 0, 7 * 16, 0, 2 * 49 * 64]
    for spec in ["max(a,0)", "min(a,b)*2", "max(a,b)-min(a,b)"]:
        sk = Sketch(full, [Hole(0, 5, spec_expr=parse_expr(spec, full.variables))])
        cand, match, least, _ = pybrute.repair(sk)
        r = oracle.repair_hole(sk)
        assert r.match_count == match and r.solved == (least is not None)
        if least is not None:
            assert (r.least_size, r.least_rank, r.least_text) == least


def test_loop_bound_hole_reading():
    """Loop-bound holes are checked through the guard predicate on the enclosing box:
    ``kh < HOLE`` against ``(oh+kh-1) < 6`` is solved by ``7-oh`` (small version of the 56-wide case)."""
    vs = [Variable("oh", 0, 6), Variable("kh", 0, 3)]
    g = free_grammar(vs, [-1, 0, 1, 6, 7])
    sk = Sketch(g, [Hole(0, 3, ctx=parse_expr("kh<HOLE", vs), spec_expr=parse_expr("((oh+kh)-1)<6", vs))])
    r = oracle.repair_hole(sk)
    cand, match, least, matches = pybrute.repair(sk)
    assert r.match_count == match and (r.least_size, r.least_rank, r.least_text) == least
    texts = oracle.listing(g, 0, 3)
    assert (3, texts.index("(7-oh)")) in matches


# ---------------------------------------------------------------------------------------------
# shifts as operators; two holes inside one constraint
# ---------------------------------------------------------------------------------------------

def test_shift_semantics():
    """<< is a multiplication by 2^b with wrap-around, >> the floor division by 2^b (sign kept);
    a count outside 0..63 is undefined.  Checked against Python's unbounded integers."""
    rnd = random.Random(7)
    vs = [Variable("a", 0, 1), Variable("b", 0, 1)]
    shl, shr = parse_expr("a<<b", vs), parse_expr("a>>b", vs)
    cases = [(1, 0), (1, 63), (-1, 63), (-2 ** 63, 63), (-2 ** 63, 1), (2 ** 62, 1), (5, 64), (5, -1), (-7, 1), (7, 1)]
    cases += [(rnd.randrange(-2 ** 63, 2 ** 63), rnd.randrange(-3, 67)) for _ in range(2000)]
    for a, b in cases:
        l, r = oracle.eval_code(shl, [a, b]), oracle.eval_code(shr, [a, b])
        if b < 0 or b > 63:
            assert l is None and r is None
            continue
        want = (a * 2 ** b) & (2 ** 64 - 1)
        assert l == (want - 2 ** 64 if want >= 2 ** 63 else want)
        assert r == a // 2 ** b
    assert oracle.eval_code(parse_expr("(a<<1)<b+1", vs), [3, 6]) == 1        # precedence: + above << above <


def test_shifts_as_grammar_operators_equal_brute_force():
    vs = [Variable("i", 0, 5), Variable("j", -2, 3)]
    g = free_grammar(vs, [1, 2, 64], ops=["+", "<<", ">>"])
    for spec in ["(i<<2)+j", "i>>1", "(i+j)<<1", "j>>64"]:
        sk = Sketch(g, [Hole(0, 5, spec_expr=parse_expr(spec, vs))])
        got = oracle.repair_hole(sk)
        cand, match, least, _ = pybrute.repair(sk)
        assert got.cand_count == cand and got.match_count == match
        assert (got.solved, got.least_size, got.least_rank, got.least_text) == \
            ((True,) + least if least else (False, 0, 0, ""))
    sk = Sketch(g, [Hole(0, 5, spec_expr=parse_expr("(i<<2)+j", vs))])
    assert oracle.repair_hole(sk).least_text == "(j+(i<<2))"


def test_joint_counts_are_products_of_closed_forms():
    vs = [Variable("i", 0, 3)]
    g = free_grammar(vs, [0, 1, 2, 3], ops=["+", "-", "*"])                 # L = 5, B = 3
    cnt = {1: 5, 3: 3 * 25, 5: 2 * 9 * 125}
    J = JointHole((0, 0), (5, 3), parse_expr("HOLE0+HOLE1", vs), spec_expr=parse_expr("i", vs))
    r = oracle.repair_joint(Sketch(g, [Hole(0, 1, spec_expr=parse_expr("i", vs))]), J)
    want = [0] * 9
    for s0 in (1, 3, 5):
        for s1 in (1, 3):
            want[s0 + s1] += cnt[s0] * cnt[s1]
    assert r.cand_count == want


def test_joint_hand_derived():
    """ctx HOLE0*4 + HOLE1 against i*4 + j over i in [0,4), j in [0,4), leaves i j 0 1 4: part 1
    must be j up to multiples of 4 moved into part 0; at total size 2 the only pair is (i, j); it is
    the least.  At total size 4 the pairs are (size 1, size 3) and (size 3, size 1): with part 0 = i
    the size-3 trees equal to j on the whole domain are j+0, 0+j, j-0, j*1, 1*j, j/1 and j%4 (j < 4):
    seven; with part 1 = j the size-3 trees equal to i are the same seven forms of i: 14 in all."""
    vs = [Variable("i", 0, 4), Variable("j", 0, 4)]
    g = free_grammar(vs, [0, 1, 4])
    base = Sketch(g, [Hole(0, 1, spec_expr=parse_expr("i", vs))])
    J = JointHole((0, 0), (3, 3), parse_expr("(HOLE0*4)+HOLE1", vs), spec_expr=parse_expr("(i*4)+j", vs))
    r = oracle.repair_joint(base, J)
    assert r.cand_count[2] == 25 and r.match_count[2] == 1
    assert (r.solved, r.least_total, r.least_size0, r.least_rank0, r.least_rank1, r.least_text0, r.least_text1) == \
        (True, 2, 1, 0, 1, "i", "j")
    assert r.match_count[4] == 14


def test_joint_equals_brute_force():
    rnd = random.Random(11)
    vs = [Variable("p", 0, 3), Variable("q", -1, 2)]
    cases = [(free_grammar(vs, [0, 2], ops=["+", "*"]), "(HOLE0*3)+HOLE1", "(p*3)+(q+2)", (3, 3)),
             (free_grammar(vs, [1, -1], ops=["-", "/"]), "HOLE0-HOLE1", "p-(q/1)", (3, 3)),
             (free_grammar(vs, [1, 2], ops=["+", "%"]), "HOLE1<HOLE0", "q<(p+1)", (3, 1)),
             (quasi_affine_grammar(vs, [-1, 2], [1, 2]), "(HOLE0+HOLE1)*HOLE1", "(p+q)*q", (3, 3))]
    for g, ctx, spec, K in cases:
        sk = Sketch(g, [Hole(0, 1, spec_expr=parse_expr("p", vs))])
        J = JointHole((0, 0), K, parse_expr(ctx, vs), spec_expr=parse_expr(spec, vs))
        r = oracle.repair_joint(sk, J)
        pts = pybrute.points_of(sk)
        want = [pybrute.code_value(J.spec_expr, p) for p in pts]
        cand, match, least = pybrute.repair_joint(g, J.start_nt, J.max_size, J.ctx, pts, want)
        assert r.cand_count == cand and r.match_count == match
        if least is None:
            assert not r.solved
        else:
            assert (r.least_total, r.least_size0, r.least_rank0, r.least_rank1, r.least_text0, r.least_text1) == least
    assert rnd is not None


def test_joint_reduces_to_the_single_hole_search_when_one_part_is_cancelled():
    """With a context that multiplies part 1 by zero and a grammar without division (every tree
    defined everywhere), a pair matches iff part 0 matches on its own: the joint match count at
    total size s is the sum over s0 + s1 = s of match_single[s0] * cnt[s1]."""
    vs = [Variable("i", 0, 4), Variable("j", 0, 3)]
    g = free_grammar(vs, [0, 1, 2], ops=["+", "-", "*"])
    single = oracle.repair_hole(Sketch(g, [Hole(0, 5, spec_expr=parse_expr("(i*2)+j", vs))]))
    cnt = oracle.counts(g, 0, 3)
    J = JointHole((0, 0), (5, 3), parse_expr("HOLE0+(HOLE1*0)", vs), spec_expr=parse_expr("(i*2)+j", vs))
    r = oracle.repair_joint(Sketch(g, [Hole(0, 1, spec_expr=parse_expr("i", vs))]), J)
    for s in range(2, 9):
        assert r.match_count[s] == sum(single.match_count[s0] * cnt[s - s0] for s0 in range(1, 6) if 1 <= s - s0 <= 3)
    assert r.solved and r.least_size0 == single.least_size and r.least_rank0 == single.least_rank and r.least_rank1 == 0


# ---------------------------------------------------------------------------------------------
# behaviour mode: bottom-up enumeration with observational-equivalence pruning
# ---------------------------------------------------------------------------------------------

def _behaviours_by_brute_force(g, nt, K, pts):
    """Value vectors on ``pts`` of ALL syntactic trees, by the smallest size at which each occurs
    (trees undefined at some point are left out): what pruning must not change."""
    T = pybrute.all_trees(g, K)
    seen, per_size = set(), [0] * (K + 1)
    for s in range(1, K + 1):
        new = set()
        for t in T[(nt, s)]:
            sig = tuple(pybrute.tree_value(t, p) for p in pts)
            if None in sig or sig in seen:
                continue
            new.add(sig)
        per_size[s] = len(new)
        seen |= new
    return per_size


def test_behaviour_counts_equal_brute_force_over_all_trees():
    """A behaviour first realised by a syntactic tree of size s is first realised in the pruned
    space at size s too (subtrees can be swapped for their class representatives, which are no
    larger), so the per-size counts of new behaviours must equal a brute force over every tree."""
    vs = [Variable("p", 0, 3), Variable("q", -1, 2)]
    cases = [(free_grammar(vs, [0, 1, 2], ops=["+", "*"]), 5), (free_grammar(vs, [1, -2], ops=["-", "/", "%"]), 5),
             (quasi_affine_grammar(vs, [-1, 2], [1, 2]), 7), (free_grammar(vs[:1], [1, 3], ops=["+", "<<", "min"]), 7)]
    for g, K in cases:
        sk = Sketch(g, [Hole(0, K, spec_expr=parse_expr("p", vs))])
        pts = pybrute.points_of(sk)
        for sig in (list(range(len(pts))), [0, len(pts) - 1, 2]):
            r = oracle.behaviours(sk, sig)
            assert r.distinct == _behaviours_by_brute_force(g, 0, K, [pts[i] for i in sig])
            assert r.enumerated[1] == g.leaf_count(0)


def test_behaviour_mode_with_every_point_as_signature_agrees_with_the_exhaustive_search():
    """With the whole domain as signature the first matching representative has the size of the
    exhaustive search's least solution, is verified, and evaluates to the spec everywhere."""
    vs = [Variable("i", 0, 6), Variable("j", 0, 5)]
    g = free_grammar(vs, constant_set(-2, 3))
    for spec in ["(i*3)+j", "i%3", "j", "(i+j)/2", "(i*i)*(j+7)"]:
        sk = Sketch(g, [Hole(0, 5, spec_expr=parse_expr(spec, vs))])
        full = oracle.repair_hole(sk)
        r = oracle.behaviours(sk, list(range(sk.n_points)))
        assert r.solved == full.solved and r.hit == full.solved
        if full.solved:
            assert r.solution_size == full.least_size and r.hit_verified and r.sig_matches == 1
            for p in pybrute.points_of(sk):
                assert pybrute.text_value(r.solution_text, g, p) == pybrute.code_value(sk.holes[0].spec_expr, p)


def test_behaviour_mode_on_a_partial_signature_reports_an_unverified_hit():
    vs = [Variable("i", 0, 8), Variable("j", 0, 8)]
    g = free_grammar(vs, [0, 1, 2])
    sk = Sketch(g, [Hole(0, 3, spec_expr=parse_expr("i*j", vs))])
    diag = [k * 8 + k for k in range(8)]                      # on the diagonal i*j and i*i look the same
    r = oracle.behaviours(sk, diag)
    assert r.hit and r.hit_text == "(i*i)" and not r.hit_verified and not r.solved and r.sig_matches == 1
    r2 = oracle.behaviours(sk, diag + [19])                   # (2, 3): 6 against 4
    assert r2.solved and r2.solution_text == "(i*j)"
    # through a context that is not injective several representatives satisfy the signature
    sk3 = Sketch(g, [Hole(0, 3, ctx=parse_expr("HOLE/4", vs), spec_expr=parse_expr("(i*j)/4", vs))])
    r3 = oracle.behaviours(sk3, list(range(64)))
    assert r3.sig_matches >= 1 and r3.solved and r3.hit_verified


def _negation_grammar(vs):
    """Negation as the production  E -> Z - E  with the one-constant nonterminal  Z -> 0  (the reading
    taken for a unary minus: it costs two nodes more than its operand, not one)."""
    from xp_instances.model import OP_CODE, P_BIN, P_CONST, P_VAR, Grammar, Production
    prods = [Production(lhs=0, kind=P_VAR, var=i) for i in range(len(vs))]
    prods += [Production(lhs=0, kind=P_CONST, value=c) for c in (1, 2, 3)]
    prods += [Production(lhs=1, kind=P_CONST, value=0)]
    prods += [Production(lhs=0, kind=P_BIN, op=OP_CODE["+"], left=0, right=0),
              Production(lhs=0, kind=P_BIN, op=OP_CODE["*"], left=0, right=0),
              Production(lhs=0, kind=P_BIN, op=OP_CODE["-"], left=1, right=0)]
    return Grammar(vs, 2, prods)


def test_negation_as_zero_minus_operand():
    """Counts by the closed form (with L leaves: n1 = L, n3 = 2 L^2 + L, n5 = 2 (2 n1 n3) + n3), results
    equal to brute force, and the least solution of a negated target is the `0 - e` form."""
    vs = [Variable("i", 0, 5), Variable("j", -2, 3)]
    g = _negation_grammar(vs)
    L = 5
    n3 = 2 * L * L + L
    assert oracle.counts(g, 0, 5) == [0, L, 0, n3, 0, 4 * L * n3 + n3]
    for spec, least in [("0-(i+j)", "(0-(i+j))"), ("(0-i)*3", None), ("0-i", "(0-i)")]:
        sk = Sketch(g, [Hole(0, 5, spec_expr=parse_expr(spec, vs))])
        got = oracle.repair_hole(sk)
        cand, match, want, _ = pybrute.repair(sk)
        assert got.cand_count == cand and got.match_count == match
        assert (got.solved, got.least_size, got.least_rank, got.least_text) == ((True,) + want if want else (False, 0, 0, ""))
        if least:
            assert got.least_text == least
