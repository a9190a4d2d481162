"""Algorithm 3 from end to end for one expression (xp_repair_pair): sketches from a (source,
erroneous) pair, constraints per concrete index, batched search, stitching.  The expected result is
restated here with plain loops over the CPU oracle: one single-hole problem per node of the
erroneous expression, the choice among the solvable ones, the substitution."""
import pytest

import oracle
from tests import pybrute
from xp_instances import Hole, Sketch, Variable, constant_set, free_grammar, parse_expr, postfix_to_text
from xp_instances.model import K_HOLE, K_OP, K_VAR

pytestmark = pytest.mark.gpu


def _subtree_first(code):
    st, first = [], []
    for i, (kind, _, _) in enumerate(code):
        if kind == K_OP:
            st.pop()
            first.append(st[-1])
        else:
            first.append(i)
            st.append(i)
    return first


def _expected(g, source_over_target, erroneous, max_size):
    """Plain restatement: every node's sketch searched by the oracle; smallest solution, then the
    smallest subtree taken out, then the leftmost."""
    first = _subtree_first(erroneous)
    best = None
    for i in range(len(erroneous)):
        ctx = erroneous[:first[i]] + [(K_HOLE, 0, 0)] + erroneous[i + 1:]
        sk = Sketch(g, [Hole(0, max_size, ctx=[] if len(ctx) == 1 else ctx, spec_expr=source_over_target)])
        r = oracle.repair_hole(sk)
        if not r.solved:
            continue
        key = (r.least_size, i - first[i] + 1, first[i])
        if best is None or key < best[0]:
            best = (key, i, first[i], r, ctx)
    return best


@pytest.mark.parametrize("source,erroneous", [
    ("(i*16)+j", "(i*8)+j"),                 # a wrong stride: the constant is replaced
    ("(i*16)+j", "(i*16)+i"),                # a wrong variable
    ("((i*4)+j)%7", "((i+4)+j)%7"),          # a wrong operator deep inside: the smallest fix replaces (i+4)
    ("(i*16)+j", "(i*16)+j"),                # nothing wrong: some leaf is "replaced" by itself
    ("(i*j)*(i*j)", "(i+1)<j"),              # no single-subtree fix within the bound
])
def test_pair_repair_equals_the_plain_restatement(xp, source, erroneous):
    vs = [Variable("i", 0, 8), Variable("j", 0, 16)]
    g = free_grammar(vs, constant_set(-2, 4) + [8, 16])
    S, E = parse_expr(source, vs), parse_expr(erroneous, vs)
    want = _expected(g, S, E, 3)
    got = xp.xp_repair_pair(xp.xp_grammar_create(g), S, E, 0, 3)
    assert got.n_sketches == len(E)
    if want is None:
        assert not got.solved
        return
    _, node, first, r, ctx = want
    assert got.solved and (got.node_first, got.node_last) == (first, node)
    assert (got.least_size, got.least_rank, got.hole_text) == (r.least_size, r.least_rank, r.least_text)
    assert got.sketch_text == postfix_to_text(ctx, vs)
    assert got.stitched_text == got.sketch_text.replace("HOLE", r.least_text)
    # the stitched expression agrees with the source at every point (independent evaluator)
    for i in range(8):
        for j in range(16):
            assert pybrute.text_value(got.stitched_text, g, (i, j)) == pybrute.code_value(S, (i, j))
    assert postfix_to_text(got.stitched_code, vs) == got.stitched_text


def test_pair_repair_across_a_split_loop(xp):
    """The source iterates over i in [0,32); the transformed program over io in [0,4), ii in [0,8)
    with i = io*8 + ii (a loop split).  Its index expression uses a wrong stride."""
    tv = [Variable("io", 0, 4), Variable("ii", 0, 8), Variable("k", 0, 3)]
    sv = [Variable("i", 0, 32), Variable("k", 0, 3)]
    g = free_grammar(tv, [1, 2, 3, 4, 8, 96])
    S = parse_expr("(i*3)+k", sv)
    E = parse_expr("((io*16)+(ii*3))+k", tv)
    var_map = [parse_expr("(io*8)+ii", tv), parse_expr("k", tv)]
    S_t = parse_expr("(((io*8)+ii)*3)+k", tv)
    want = _expected(g, S_t, E, 3)
    got = xp.xp_repair_pair(xp.xp_grammar_create(g), S, E, 0, 3, var_map=var_map)
    assert want is not None and got.solved
    _, node, first, r, ctx = want
    assert (got.node_first, got.node_last, got.least_size, got.least_rank, got.hole_text) == \
        (first, node, r.least_size, r.least_rank, r.least_text)
    assert got.stitched_text == postfix_to_text(ctx, tv).replace("HOLE", r.least_text)
    assert got.stitched_text == "(((io*(3*8))+(ii*3))+k)"
    assert got.candidates > 0 and got.evals_executed > 0


def test_pair_repair_rejects_malformed_input(xp):
    vs = [Variable("i", 0, 4)]
    g = free_grammar(vs, [1])
    gr = xp.xp_grammar_create(g)
    with pytest.raises(xp.XpError) as e:
        xp.xp_repair_pair(gr, parse_expr("i", vs), [(K_OP, 0, 0)], 0, 3)
    assert e.value.status == 3 and "malformed" in str(e.value)
    with pytest.raises(xp.XpError) as e:
        xp.xp_repair_pair(gr, parse_expr("i", vs), parse_expr("HOLE+1", vs), 0, 3)
    assert e.value.status == 3
    with pytest.raises(xp.XpError) as e:
        xp.xp_repair_pair(gr, [(K_VAR, 3, 0)], parse_expr("i", vs), 0, 3, var_map=[parse_expr("i", vs)])
    assert e.value.status == 3
