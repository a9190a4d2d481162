"""Parity of the CUDA library against the CPU oracle, through the C ABI, bit for bit:
per-size candidate counts, per-size match counts and the least solution."""
import random

import numpy as np
import pytest

import oracle
from tests import pybrute
from tests.util import assert_same, check_sketch
from xp_instances import (Hole, Sketch, Variable, config1, config2, config3, config4, config5, constant_set,
                          free_grammar, parse_expr, quasi_affine_grammar)

pytestmark = pytest.mark.gpu

# 0: the library's own choice of path per rank window; 1: every candidate unranked on its own;
# 2: the probe filter over operand tiles wherever it is legal, however small the window.
PATHS = [0, 1, 2]


def _c1(spec, ctx=""):
    vs = [Variable("i", 0, 16), Variable("j", 0, 16)]
    g = free_grammar(vs, constant_set(-8, 8))
    return Sketch(g, [Hole(0, 5, ctx=parse_expr(ctx, vs) if ctx else [], spec_expr=parse_expr(spec, vs))], name=f"c1:{spec}")


@pytest.mark.parametrize("seed", range(5))
def test_config1_full(xp, seed):
    res = check_sketch(xp, config1(seed))
    assert res[0].solved and res[0].cand_count == [0, 19, 0, 1805, 0, 342950]


@pytest.mark.parametrize("flags", PATHS)
@pytest.mark.parametrize("spec", ["i", "(i*8)+j", "i%4", "7", "(i/3)-j", "100", "(i*j)%5", "0", "j-j"])
def test_config1_grammar_specs(xp, spec, flags):
    check_sketch(xp, _c1(spec), flags=flags)


@pytest.mark.parametrize("ctx", ["HOLE*2+i", "i<HOLE", "min(HOLE,3)", "HOLE/j", "(HOLE%3)==(i%3)", "HOLE-HOLE"])
@pytest.mark.parametrize("flags", PATHS)
def test_contexts(xp, ctx, flags):
    check_sketch(xp, _c1("(i+j)<9" if "<" in ctx or "==" in ctx else "i+j", ctx), flags=flags)


@pytest.mark.parametrize("ctx,spec", [("HOLE<=i", "(j*2)<=i"), ("(i+3)<HOLE", "(i+3)<(j+5)"), ("(7-HOLE)<=j", "(7-(i/2))<=j"),
                                       ("i<(HOLE-2)", "i<((i*j)-2)"), ("j<=(3-HOLE)", "j<=(3-(i%3))"), ("i<HOLE", "i+j"),
                                       ("(HOLE+HOLE)<i", "(j+j)<i"), ("(HOLE<i)+1", "(j<i)+1")])
def test_comparison_contexts_through_the_filter(xp, ctx, spec):
    """Guard predicates (loop bounds): the filter works on the interval of hole values that
    satisfies the comparison at a probe; other shapes fall back to rank-by-rank search."""
    for flags in PATHS:
        check_sketch(xp, _c1(spec, ctx), flags=flags)


def test_comparison_context_with_wide_values(xp):
    vs = [Variable("x", 2 ** 40, 2 ** 40 + 3), Variable("y", -2, 2)]
    g = free_grammar(vs, [1, 2 ** 31, -2 ** 62], ops=["+", "-", "*"])
    for ctx, spec in [("y<HOLE", "y<(x*y)"), ("HOLE<=(x*2)", "((x+x)+y)<=(x*2)")]:
        sk = Sketch(g, [Hole(0, 5, ctx=parse_expr(ctx, vs), spec_expr=parse_expr(spec, vs))], name=f"wide cmp:{ctx}")
        for flags in PATHS:
            check_sketch(xp, sk, flags=flags)


@pytest.mark.parametrize("ctx,spec", [("(HOLE*3)+(i*16)", "((i+j)*3)+(i*16)"), ("j-(HOLE*-5)", "j+(i*40)"),
                                       ("(2*HOLE)-(HOLE*3)", "0-(i%5)"), ("HOLE*0", "0"), ("(i*j)+7", "(i*j)+7")])
def test_affine_contexts_through_the_filter(xp, ctx, spec):
    for flags in PATHS:
        check_sketch(xp, _c1(spec, ctx), flags=flags)


def test_path_flags_change_work_not_results(xp):
    sk = _c1("(i*8)+j")
    a = check_sketch(xp, sk)
    b = check_sketch(xp, sk, flags=xp.XP_FLAG_NO_FILTER)
    c = check_sketch(xp, sk, flags=xp.XP_FLAG_ALWAYS_FILTER)
    assert a[0].match_count == b[0].match_count == c[0].match_count and a[0].least_rank == b[0].least_rank == c[0].least_rank
    assert b[0].filter_survivors == b[0].probe_survivors          # no filter stage: nothing is dropped before the probes
    assert c[0].filter_survivors < sum(c[0].cand_count)           # the filter drops candidates at probe 0


def test_tiny_grammars_against_oracle_and_brute_force(xp):
    rnd = random.Random(9)
    vs2 = [Variable("a", 0, 3), Variable("b", -1, 2)]
    vs3 = [Variable("p", 0, 2), Variable("q", 0, 3), Variable("r", 1, 3)]
    cases = [(free_grammar(vs2, [-2, 0, 1, 3]), vs2), (free_grammar(vs2, [2, -3], ops=["-", "/", "%"]), vs2),
             (quasi_affine_grammar(vs3, [-2, 0, 3], [1, 2]), vs3)]
    for g, vs in cases:
        T = pybrute.all_trees(g, 5)
        for size in (1, 3, 5, 5):
            spec = pybrute.tree_text(rnd.choice(T[(0, size)]), g)
            for ctx in ["", f"HOLE*2+{vs[0].name}"]:
                sk = Sketch(g, [Hole(0, 5, ctx=parse_expr(ctx, vs) if ctx else [], spec_expr=parse_expr(spec, vs))])
                res = check_sketch(xp, sk)
                for flags in (1, 2):
                    other = check_sketch(xp, sk, flags=flags)
                    assert other[0].match_count == res[0].match_count
                cand, match, least, _ = pybrute.repair(sk)
                assert res[0].cand_count == cand and res[0].match_count == match
                if least:
                    assert (res[0].least_size, res[0].least_rank, res[0].least_text) == least


def test_larger_sizes_small_grammar(xp):
    vs = [Variable("x", 0, 5), Variable("y", -2, 3)]
    g = free_grammar(vs, [1, 2])
    for K, spec in [(7, "((x*2)+y)-(x%2)"), (9, "((x+y)*(x-y))+1")]:
        for flags in (0, 2):
            check_sketch(xp, Sketch(g, [Hole(0, K, spec_expr=parse_expr(spec, vs))], name=f"K{K}"), flags=flags)
    gq = quasi_affine_grammar(vs, [-1, 2, 3], [1, 2, 4])
    for flags in (0, 2):
        check_sketch(xp, Sketch(gq, [Hole(0, 9, spec_expr=parse_expr("((x/2)*3)+(y%4)", vs))], name="typed K9"), flags=flags)


def test_repeated_productions_and_the_largest_size(xp):
    """Two productions with the same operator are distinct candidates (they cannot share a
    filter segment); size 15 is the library's limit (8 leaves, operand stack of 8)."""
    from xp_instances.model import OP_CODE, P_BIN, Production
    g2 = free_grammar([Variable("x", 0, 4)], [1, 2], ops=["+", "*"])
    g2.productions.append(Production(lhs=0, kind=P_BIN, op=OP_CODE["+"], left=0, right=0))
    sk = Sketch(g2, [Hole(0, 7, spec_expr=parse_expr("(x*2)+1", g2.variables))], name="two plus productions")
    for flags in PATHS:
        res = check_sketch(xp, sk, flags=flags)
        assert res[0].cand_count == [0, 3, 0, 27, 0, 486, 0, 10935]
    g3 = free_grammar([Variable("x", 0, 3)], [1], ops=["+"])
    sk3 = Sketch(g3, [Hole(0, 15, spec_expr=parse_expr("((x+x)+(x+1))+((1+1)+(x+1))", g3.variables))], name="size 15")
    for flags in PATHS:
        res = check_sketch(xp, sk3, flags=flags)
        assert res[0].cand_count[15] == 109824 and res[0].match_count[15] == 30030


def test_min_max_as_grammar_operators(xp):
    coords = np.array([[0], [1], [2], [3]], dtype=np.int32)
    g = free_grammar([Variable("io", 0, 4)], [8, 30], ops=["-", "*", "min"])
    sk = Sketch(g, [Hole(0, 7, spec_table=np.array([8, 8, 8, 6], dtype=np.int64))], coords, name="remainder tile")
    for flags in PATHS:
        res = check_sketch(xp, sk, flags=flags)
        assert res[0].least_text == "min(8,(30-(io*8)))"
    vs = [Variable("a", -3, 4), Variable("b", 0, 3)]
    full = free_grammar(vs, [0, 2, -5, 7], ops=["+", "-", "*", "/", "%", "min", "max"])
    for spec, ctx in [("max(a,0)", ""), ("min(a,b)*2", ""), ("max(a,b)-min(a,b)", ""), ("(max(a,2)*3)+b", "(HOLE*3)+b"),
                      ("min(a,b)<1", "HOLE<1")]:
        sk = Sketch(full, [Hole(0, 5, ctx=parse_expr(ctx, vs) if ctx else [], spec_expr=parse_expr(spec, vs))], name=f"minmax:{spec}")
        for flags in PATHS:
            check_sketch(xp, sk, flags=flags)
    # a larger space so that whole tiles of every operator group run (7 operators: two segments per split)
    big = free_grammar([Variable("i", 0, 16), Variable("j", 0, 16)], constant_set(-8, 8), ops=["+", "-", "*", "/", "%", "min", "max"])
    for spec in ["min(i,j)+3", "max((i*2),j)"]:
        check_sketch(xp, Sketch(big, [Hole(0, 5, spec_expr=parse_expr(spec, big.variables))], name=f"minmax big:{spec}"))


def test_zero_divisors_and_wraparound(xp):
    vs = [Variable("x", 0, 3)]
    for flags in PATHS:
        check_sketch(xp, Sketch(free_grammar(vs, [0], ops=["/", "%", "*"]), [Hole(0, 5, spec_expr=parse_expr("0", vs))]), flags=flags)
    big = [Variable("x", 2 ** 62 - 1, 2 ** 62 + 2)]
    g = free_grammar(big, [2, 4, -1, -2 ** 63], ops=["+", "*", "/", "%", "-"])
    for spec in ["x*4", "(x+x)+(x+x)", "(x*2)/-1"]:
        for flags in PATHS:
            check_sketch(xp, Sketch(g, [Hole(0, 5, spec_expr=parse_expr(spec, big))], name=f"wrap:{spec}"), flags=flags)
    table = np.array([-2 ** 63, 0], dtype=np.int64)                 # INT64_MIN / -1 and % -1
    gm = free_grammar([Variable("x", 0, 2)], [-1, -2 ** 63, 0], ops=["/", "%", "*"])
    coords = np.array([[0], [1]], dtype=np.int32)
    for flags in PATHS:
        check_sketch(xp, Sketch(gm, [Hole(0, 5, spec_table=table)], coords, name="int64min"), flags=flags)
    # operands around the int32 boundary: tiles mix 32-bit and 64-bit operand values
    edge = [Variable("x", 2 ** 31 - 3, 2 ** 31 + 2)]
    ge = free_grammar(edge, [1, 2, -1, 2 ** 31, -2 ** 31], ops=["+", "-", "*", "/", "%"])
    for spec in ["x-2147483648", "(x*2)/2", "x%-2147483648"]:
        for flags in (0, 2):
            check_sketch(xp, Sketch(ge, [Hole(0, 5, spec_expr=parse_expr(spec, edge))], name=f"edge32:{spec}"), flags=flags)


def test_table_domain_host_and_device_tensors(xp):
    import torch
    vs = [Variable("u", 0, 50), Variable("w", 0, 40)]
    g = free_grammar(vs, [1, 2, 3, 7])
    rnd = np.random.default_rng(0)
    coords = np.stack([rnd.integers(0, 50, 3000), rnd.integers(0, 40, 3000)], axis=1).astype(np.int32)
    spec = (coords[:, 0].astype(np.int64) * 7 + coords[:, 1] // 3)
    sk = Sketch(g, [Hole(0, 5, spec_table=spec)], coords, name="table")
    res = check_sketch(xp, sk)
    gr = xp.xp_grammar_create(g)
    ls = xp.xp_sketch_load(gr, sk, coords=torch.from_numpy(coords).cuda(), spec_tables={0: torch.from_numpy(spec).cuda()})
    ws = torch.empty(xp.xp_workspace_bytes([ls]), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    dev = xp.xp_repair(ls, workspace=ws, stream=stream.cuda_stream)
    assert dev[0].match_count == res[0].match_count and dev[0].least_text == res[0].least_text


def test_box_check_on_the_mentioned_variables_only(xp):
    """On a box the whole-domain check leaves out variables that neither the candidate nor the
    context nor the spec mention.  17 920 points (five chunks of the check); the sub-boxes have
    between 1 and 17 920 points depending on the candidate."""
    vs = [Variable("i", 0, 64), Variable("j", 0, 40), Variable("k", 0, 7)]
    g = free_grammar(vs, [0, 1, 2, 7])
    cases = [("i*2", ""), ("k", ""), ("(i*2)+k", ""), ("7", ""), ("i<3", "HOLE<3"), ("(j*5)+i", "(HOLE*5)+i"),
             ("k<2", "k<HOLE"), ("(i+j)+k", ""), ("(j/7)*0", "")]
    for spec, ctx in cases:
        sk = Sketch(g, [Hole(0, 5, ctx=parse_expr(ctx, vs) if ctx else [], spec_expr=parse_expr(spec, vs))], name=f"subbox:{spec}")
        for flags in PATHS:
            check_sketch(xp, sk, flags=flags)
    # a spec TABLE on the same kind of points may depend on any variable: nothing is left out
    pts = np.stack(np.meshgrid(np.arange(12), np.arange(9), np.arange(50), indexing="ij"), axis=-1).reshape(-1, 3).astype(np.int32)
    vt = [Variable("i", 0, 12), Variable("j", 0, 9), Variable("k", 0, 50)]
    table = pts[:, 0].astype(np.int64) * 2
    table[-1] += 1                                  # only the last point tells i*2 from the spec
    r = check_sketch(xp, Sketch(free_grammar(vt, [0, 1, 2]), [Hole(0, 3, spec_table=table)], pts, name="table: last point differs"))
    assert not r[0].solved


def test_whole_domain_check_in_64_bit(xp):
    """Coordinates of a table domain, not the declared ranges, bound the values: rows far outside
    the ranges make products that need 64 bits; small rows let the check run in 32 bits."""
    vs = [Variable("x", 0, 4), Variable("y", 0, 4)]
    g = free_grammar(vs, [1, 3, 70000])
    rnd = np.random.default_rng(5)
    for xmax, ymax in [(200000, 100000), (300, 200), (2 ** 31 - 1, 3)]:
        coords = np.stack([rnd.integers(0, xmax, 6000), rnd.integers(0, ymax, 6000)], axis=1).astype(np.int32)
        coords[0] = (xmax - 1, ymax - 1)
        spec = coords[:, 0].astype(np.int64) * coords[:, 1] + 3
        sk = Sketch(g, [Hole(0, 5, spec_table=spec)], coords, name=f"bounds:{xmax}x{ymax}")
        res = check_sketch(xp, sk)
        assert res[0].solved and res[0].least_text in ("((x*y)+3)", "(3+(x*y))")
    coords = np.stack([rnd.integers(-2 ** 31, -2 ** 31 + 5, 5000), rnd.integers(0, 3, 5000)], axis=1).astype(np.int32)
    spec = coords[:, 0].astype(np.int64) - coords[:, 1]            # INT32_MIN itself among the coordinates
    check_sketch(xp, Sketch(g, [Hole(0, 3, spec_table=spec)], coords, name="bounds:int32 min"))


def test_edge_domains(xp):
    vs = [Variable("u", 0, 4)]
    g = free_grammar(vs, [0, 1])
    empty = Sketch(g, [Hole(0, 3, spec_table=np.zeros(0, dtype=np.int64))], np.zeros((0, 1), dtype=np.int32), name="empty")
    r = check_sketch(xp, empty)                    # no constraint: every candidate matches
    assert r[0].match_count == r[0].cand_count and (r[0].least_size, r[0].least_rank) == (1, 0)
    one = Sketch(g, [Hole(0, 3, spec_table=np.array([3], dtype=np.int64))], np.array([[3]], dtype=np.int32), name="one")
    check_sketch(xp, one)
    check_sketch(xp, Sketch(g, [Hole(0, 1, spec_expr=parse_expr("u", vs))], name="K1"))
    check_sketch(xp, Sketch(g, [Hole(0, 3, spec_expr=parse_expr("u/0", vs))], name="spec undefined"))
    check_sketch(xp, _c1("(i*8)+j"), windows={1: (0, 0), 3: (5, 5), 5: (2545, 2546)})
    check_sketch(xp, _c1("(i*8)+j"), windows={5: (2546, 342950)})


def test_ragged_rank_windows_partition(xp):
    sk = _c1("i%4")
    full = check_sketch(xp, sk)
    cuts = [0, 1, 1023, 1025, 68590, 100001, 342949, 342950]
    total = 0
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        total += check_sketch(xp, sk, windows={1: (0, 0), 3: (0, 0), 5: (lo, hi)})[0].match_count[5]
    assert total == full[0].match_count[5]


def test_config5_batch_slice(xp):
    sks = config5(0, 24)
    grs = {}
    loaded = []
    for sk in sks:
        key = len(sk.grammar.variables), tuple(v.hi for v in sk.grammar.variables)
        if key not in grs:
            grs[key] = xp.xp_grammar_create(sk.grammar)
        loaded.append(xp.xp_sketch_load(grs[key], sk))
    res = xp.xp_repair_batch(loaded)
    n_unsolved = 0
    for sk, r in zip(sks, res):
        want = oracle.repair_hole(sk)
        assert_same(r[0], want, sk.name)
        n_unsolved += not want.solved
    single = xp.xp_repair(loaded[3])
    assert single[0].match_count == res[3][0].match_count and single[0].least_rank == res[3][0].least_rank


def test_batch_load_equals_single_loads(xp):
    """xp_sketch_load_batch leaves every sketch as xp_sketch_load would: table and box domains,
    several holes, different grammars in one batch; a bad description fails the whole batch."""
    sks = config5(1, 12) + [config1(2), _c1("i<3", "HOLE<3"), _c1("(i*8)+j")]
    vs = [Variable("i", 0, 64), Variable("j", 0, 40), Variable("k", 0, 7)]
    g3 = free_grammar(vs, [0, 1, 2, 7])
    sks.append(Sketch(g3, [Hole(0, 5, spec_expr=parse_expr("(i*2)+k", vs)), Hole(0, 3, ctx=parse_expr("k<HOLE", vs), spec_expr=parse_expr("k<2", vs)),
                           Hole(0, 3, spec_expr=parse_expr("j/0", vs))], name="three holes"))
    grs = [xp.xp_grammar_create(sk.grammar) for sk in sks]
    batch = xp.xp_sketch_load_batch(grs, sks)
    together = xp.xp_repair_batch(batch)
    for sk, gr, ls, res in zip(sks, grs, batch, together):
        alone = xp.xp_repair(xp.xp_sketch_load(gr, sk))
        one_by_one = xp.xp_repair(ls)
        for h in range(len(sk.holes)):
            want = oracle.repair_hole(sk, h)
            assert_same(res[h], want, f"{sk.name} hole {h} (batch load, batch search)")
            assert_same(one_by_one[h], want, f"{sk.name} hole {h} (batch load)")
            assert_same(alone[h], want, f"{sk.name} hole {h} (single load)")
            assert (res[h].filter_survivors, res[h].probe_survivors) == (alone[h].filter_survivors, alone[h].probe_survivors)
    bad = Sketch(g3, [Hole(7, 5, spec_expr=parse_expr("i", vs))], name="bad start symbol")
    with pytest.raises(xp.XpError, match="sketch 1"):
        xp.xp_sketch_load_batch([grs[0], xp.xp_grammar_create(g3)], [sks[0], bad])
    assert xp.xp_repair(xp.xp_sketch_load(grs[0], sks[0]))[0].match_count == together[0][0].match_count      # still usable


def test_config2_rank_slices(xp):
    sk = config2(0)
    n7 = 213813760000
    rnd = random.Random(2)
    win = {1: (0, 136), 3: (0, 92480), 5: (1000000, 1400000)}
    for lo in [0, n7 - 300000, rnd.randrange(n7 - 10 ** 6), rnd.randrange(n7 - 10 ** 6)]:
        w = dict(win)
        w[7] = (lo, lo + 300000)
        check_sketch(xp, sk, windows=w)


def test_config3_rank_slices_three_holes(xp):
    sk = config3(0)
    corners_first = [0, 1806335, 27726, 55 * 56 * 9 + 2 * 3]
    rnd = random.Random(4)
    lo = rnd.randrange(134280950 - 10 ** 6)
    check_sketch(xp, sk, windows={1: (0, 139), 3: (0, 20000), 5: (lo, lo + 200000)}, first_points=corners_first)


def test_config4_rank_slices(xp):
    sk = config4(0, n_points=1 << 14)
    n9 = 322291652420
    rnd = random.Random(6)
    lo = rnd.randrange(n9 - 10 ** 6)
    check_sketch(xp, sk, windows={1: (0, 4), 3: (0, 2084), 5: (0, 200000), 7: (10 ** 8, 10 ** 8 + 200000), 9: (lo, lo + 200000)})


def test_planted_targets_are_found_in_their_windows(xp):
    """The planted target's own rank (looked up with the oracle's listing) must match."""
    for sk, size in [(config2(1), 7), (config4(1, n_points=1 << 14), 9)]:
        target = sk.holes[0].note
        rank = _structural_rank(sk.grammar, target)
        assert oracle.listing(sk.grammar, 0, size, rank, rank + 1) == [target]
        res = check_sketch(xp, sk, windows={s: (0, 0) if s != size else (rank, rank + 1) for s in range(1, size + 1)})
        assert res[0].match_count[size] == 1 and res[0].least_text == target


def _structural_rank(g, text):
    """Rank of a fully parenthesised expression, computed from the oracle's counts by the
    definition of the canonical order (test-side code, independent of the library)."""
    from xp_instances.model import OPS, P_BIN, P_CONST, P_VAR
    cnt = {nt: oracle.counts(g, nt, 9) for nt in range(g.n_nonterminals)}

    def parse(s):
        if s[0] != "(":
            return ("leaf", s)
        j = 1                                   # split at the top-level operator
        if s[j] == "(":
            depth = 0
            while True:
                depth += s[j] == "("
                depth -= s[j] == ")"
                j += 1
                if depth == 0:
                    break
        else:
            j += 1
            while s[j].isalnum():
                j += 1
        left, op, right = s[1:j], s[j], s[j + 1:-1]
        return (op, parse(left), parse(right))

    def size(t):
        return 1 if t[0] == "leaf" else 1 + size(t[1]) + size(t[2])

    def rank(t, nt):
        if t[0] == "leaf":
            leaves = [p for p in g.productions if p.lhs == nt and p.kind != P_BIN]
            for r, p in enumerate(leaves):
                if (p.kind == P_VAR and g.variables[p.var].name == t[1]) or (p.kind == P_CONST and str(p.value) == t[1]):
                    return r
            raise KeyError(t)
        s = size(t)
        a = size(t[1])
        base = 0
        for p in g.productions:
            if p.lhs != nt or p.kind != P_BIN:
                continue
            if OPS[p.op] == t[0]:
                for aa in range(1, a):
                    base += cnt[p.left][aa] * cnt[p.right][s - 1 - aa]
                return base + rank(t[1], p.left) * cnt[p.right][s - 1 - a] + rank(t[2], p.right)
            for aa in range(1, s - 1):
                base += cnt[p.left][aa] * cnt[p.right][s - 1 - aa]
        raise KeyError(t)

    return rank(parse(text), 0)


def test_integer_peak_microbenchmark_is_plausible(xp):
    """The roofline denominator: independent 32-bit add chains reach about SMs x 128 lanes x clock,
    multiply-add chains about half of that (they issue on one pipe of 64 lanes per SM)."""
    import torch
    add, mad = xp.xp_int32_peak()
    props = torch.cuda.get_device_properties(0)
    lanes = props.multi_processor_count * 128
    assert 0.3e9 * lanes < add < 2.3e9 * lanes          # between 0.3 and 2.3 GHz worth of one add per lane and clock
    assert 0.35 * add < mad < 0.75 * add


def test_division_cost_microbenchmark_is_plausible(xp):
    """A general int64 division costs tens to a few hundred 32-bit operations, a division by a
    constant through its reciprocal a handful."""
    add, _ = xp.xp_int32_peak()
    general, reciprocal = xp.xp_int_div_rate()
    assert 20 < add / general < 2000
    assert 2 < add / reciprocal < 40
    assert reciprocal > 4 * general
