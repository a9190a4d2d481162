"""Two holes inside one constraint (xp_repair_joint) against the CPU oracle, bit for bit: pair
counts and match counts per total size, and the least pair (total size, size of part 0, ranks, texts)."""
import numpy as np
import pytest

import oracle
from xp_instances import Hole, JointHole, Sketch, Variable, constant_set, free_grammar, parse_expr, quasi_affine_grammar

pytestmark = pytest.mark.gpu


def _check(xp, sk, J):
    want = oracle.repair_joint(sk, J)
    ls = xp.xp_sketch_load(xp.xp_grammar_create(sk.grammar), sk)
    got = xp.xp_repair_joint(ls, J)
    assert got.cand_count == want.cand_count and got.match_count == want.match_count, sk.name
    assert got.solved == want.solved, sk.name
    if want.solved:
        assert (got.least_total, got.least_size0, got.least_rank0, got.least_rank1, got.least_text0, got.least_text1) == \
            (want.least_total, want.least_size0, want.least_rank0, want.least_rank1, want.least_text0, want.least_text1), sk.name
    return got


def _base(g, vs):
    return Sketch(g, [Hole(0, 1, spec_expr=parse_expr(vs[0].name, vs))], name="joint")


@pytest.mark.parametrize("ctx,spec,K", [
    ("(HOLE0*16)+HOLE1", "(i*16)+j", (3, 3)),                 # stride and offset wrong at once
    ("(HOLE0*16)+HOLE1", "((i+j)*16)+(j*2)", (3, 3)),
    ("HOLE0-HOLE1", "(i/2)-(j%3)", (3, 3)),
    ("HOLE1<HOLE0", "j<(i+2)", (3, 1)),                       # a guard with both sides missing
    ("(HOLE0+HOLE1)*HOLE1", "(i+j)*j", (3, 3)),
    ("HOLE0/HOLE1", "(i*4)/(j-2)", (3, 3)),                   # zero divisors at some points for some pairs
    ("HOLE0+HOLE1", "12345", (3, 3)),                          # no solution
    ("HOLE0+(HOLE1*0)", "i+j", (5, 1)),
])
def test_joint_small_products(xp, ctx, spec, K):
    vs = [Variable("i", 0, 8), Variable("j", 0, 6)]
    g = free_grammar(vs, constant_set(-1, 4))
    J = JointHole((0, 0), K, parse_expr(ctx, vs), spec_expr=parse_expr(spec, vs))
    got = _check(xp, _base(g, vs), J)
    assert (got.evals_executed > 0 or not got.solved) and got.n_launches >= 3


def test_joint_typed_grammar_table_domain_and_table_spec(xp):
    vs = [Variable("r", 0, 12), Variable("c", 0, 10), Variable("k", 0, 3)]
    g = quasi_affine_grammar(vs, [-2, -1, 2, 3, 10], [1, 2, 3])
    rng = np.random.default_rng(5)
    ids = rng.permutation(12 * 10 * 3)[:200]
    coords = np.stack([ids // 30, (ids // 3) % 10, ids % 3], axis=1).astype(np.int32)
    spec = (coords[:, 0].astype(np.int64) * 10 + coords[:, 1]) * 3 + coords[:, 2]
    sk = Sketch(g, [Hole(0, 1, spec_table=spec)], coords, name="typed joint")
    J = JointHole((0, 0), (5, 1), parse_expr("(HOLE0*3)+HOLE1", vs), spec_table=spec)
    got = _check(xp, sk, J)
    assert got.solved and (got.least_text0, got.least_text1) == ("(c+(r*10))", "k")
    import torch
    J2 = JointHole((0, 0), (5, 1), parse_expr("(HOLE0*3)+HOLE1", vs), spec_table=torch.from_numpy(spec).cuda())
    ls = xp.xp_sketch_load(xp.xp_grammar_create(g), sk)
    again = xp.xp_repair_joint(ls, J2)
    assert again.match_count == got.match_count and again.least_rank0 == got.least_rank0
    # different bounds per part, parts from different nonterminals (a multiplier constant and an expression)
    J3 = JointHole((1, 0), (1, 5), parse_expr("HOLE0*HOLE1", vs), spec_expr=parse_expr("((r*10)+c)*3", vs))
    _check(xp, sk, J3)


def test_joint_edges(xp):
    vs = [Variable("x", 0, 3)]
    g = free_grammar(vs, [0, 1], ops=["+", "/"])
    empty = Sketch(g, [Hole(0, 1, spec_table=np.zeros(0, dtype=np.int64))], np.zeros((0, 1), dtype=np.int32), name="no points")
    J = JointHole((0, 0), (3, 3), parse_expr("HOLE0+HOLE1", vs), spec_table=np.zeros(0, dtype=np.int64))
    got = _check(xp, empty, J)
    assert got.match_count == got.cand_count                   # no constraint at all
    one = Sketch(g, [Hole(0, 1, spec_expr=parse_expr("x", vs))], np.array([[2]], dtype=np.int32), name="one point")
    _check(xp, one, JointHole((0, 0), (3, 3), parse_expr("HOLE0+HOLE1", vs), spec_expr=parse_expr("x/0", vs)))     # spec undefined
    _check(xp, one, JointHole((0, 0), (3, 3), parse_expr("HOLE0+HOLE1", vs), spec_expr=parse_expr("x+1", vs)))
    ls = xp.xp_sketch_load(xp.xp_grammar_create(g), one)
    with pytest.raises(xp.XpError) as e:
        xp.xp_repair_joint(ls, JointHole((0, 0), (3, 3), parse_expr("HOLE0+1", vs), spec_expr=parse_expr("x", vs)))
    assert e.value.status == 3 and "both parts" in str(e.value)
    big = free_grammar(vs, list(range(300)))
    lb = xp.xp_sketch_load(xp.xp_grammar_create(big), Sketch(big, [Hole(0, 1, spec_expr=parse_expr("x", vs))]))
    with pytest.raises(xp.XpError) as e:
        xp.xp_repair_joint(lb, JointHole((0, 0), (5, 1), parse_expr("HOLE0+HOLE1", vs), spec_expr=parse_expr("x", vs)))
    assert e.value.status == 4
