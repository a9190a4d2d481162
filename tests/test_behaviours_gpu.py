"""The behaviour mode (xp_behaviours: bottom-up enumeration with observational-equivalence pruning
on signature points) against the CPU oracle, value for value: candidates enumerated and new
behaviours per size, representatives that satisfy the signature, the first hit and the first
solution verified on the whole domain."""
import numpy as np
import pytest

import oracle
from xp_instances import (Hole, Sketch, Variable, config1, config5_instance, constant_set, free_grammar, parse_expr,
                          quasi_affine_grammar)

pytestmark = pytest.mark.gpu


def _check(xp, sk, sig, hole=0, **kw):
    want = oracle.behaviours(sk, sig, hole)
    ls = xp.xp_sketch_load(xp.xp_grammar_create(sk.grammar), sk)
    got = xp.xp_behaviours(ls, sig, hole=hole, **kw)
    K = sk.holes[hole].max_size
    assert [int(got.enumerated[k]) for k in range(K + 1)] == want.enumerated, sk.name
    assert [int(got.distinct[k]) for k in range(K + 1)] == want.distinct, sk.name
    assert int(got.sig_matches) == want.sig_matches
    assert bool(got.hit) == want.hit and bool(got.solved) == want.solved
    if want.hit:
        assert (got.hit_size, int(got.hit_index), bool(got.hit_verified), got.hit_text.decode()) == \
            (want.hit_size, want.hit_index, want.hit_verified, want.hit_text)
    if want.solved:
        assert (got.solution_size, int(got.solution_index), got.solution_text.decode()) == \
            (want.solution_size, want.solution_index, want.solution_text)
    return got


def test_behaviours_small_grammars(xp):
    vs = [Variable("p", 0, 5), Variable("q", -2, 3)]
    pts = 5 * 5
    cases = [(free_grammar(vs, [0, 1, 2], ops=["+", "*"]), 7, "(p*2)+q", ""),
             (free_grammar(vs, [1, -2], ops=["-", "/", "%"]), 5, "(p%2)-q", ""),
             (quasi_affine_grammar(vs, [-1, 2, 3], [1, 2]), 7, "((p/2)*3)+(q%2)", ""),
             (free_grammar(vs, [1, 3], ops=["+", "<<", "min"]), 7, "min(p,3)<<1", ""),
             (free_grammar(vs, [0, 1, 2], ops=["+", "*"]), 5, "((p*q)+1)/3", "HOLE/3"),
             (free_grammar(vs, [0, 1], ops=["+", "/"]), 5, "p/0", "")]
    for g, K, spec, ctx in cases:
        sk = Sketch(g, [Hole(0, K, ctx=parse_expr(ctx, vs) if ctx else [], spec_expr=parse_expr(spec, vs))], name=f"behaviours: {spec}")
        for sig in (list(range(pts)), [0, pts - 1, 7, 13], [3]):
            _check(xp, sk, sig[:16])


def test_behaviours_beyond_the_exhaustive_bound(xp):
    """The two-index grammar at size 9: 2.2e10 syntactic trees, a few million behaviours on eight
    signature points.  The planted size-7 form is found although the exhaustive search stops at 5."""
    vs = [Variable("i", 0, 16), Variable("j", 0, 16)]
    g = free_grammar(vs, constant_set(-8, 8))
    sk = Sketch(g, [Hole(0, 7, spec_expr=parse_expr("((i*8)+j)%5", vs))], name="two-index size 7")
    sig = [0, 255, 15, 240, 100, 37, 201, 77, 18, 129, 66, 250]
    got = _check(xp, sk, sig)
    assert got.solved and got.solution_size == 7 and got.representatives > 100000
    assert got.bytes_moved > 0 and got.kernel_ms > 0
    with pytest.raises(xp.XpError) as e:
        xp.xp_behaviours(xp.xp_sketch_load(xp.xp_grammar_create(g), sk), sig, max_representatives=1000)
    assert e.value.status == 4 and "representatives" in str(e.value)


def test_behaviours_table_domain_and_seeded_instances(xp):
    for inst in (config5_instance(0, 0), config5_instance(0, 5)):
        n = inst.n_points
        _check(xp, inst, [0, 1, 2, 3, n // 2, n - 1, n // 3, n // 5, 17, 91])
    sk = config1(1)
    _check(xp, sk, list(range(0, 256, 17)))
    ls = xp.xp_sketch_load(xp.xp_grammar_create(sk.grammar), sk)
    for bad in ([], list(range(17)), [256]):
        with pytest.raises(xp.XpError) as e:
            xp.xp_behaviours(ls, bad)
        assert e.value.status == 1
