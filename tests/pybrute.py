"""A third, deliberately different statement of the search, in pure Python, for
tiny inputs only: every tree of every size is materialised bottom-up as a nested
tuple, evaluated with Python's unbounded integers (reduced to int64 by hand) on
every point with no early exit.  Used to pin the C++ oracle; shares nothing with
it or with the CUDA library."""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

from xp_instances.model import (K_CONST, K_HOLE, K_OP, K_VAR, OPS, P_BIN, P_CONST, P_VAR,
                                Grammar, Sketch)

M64 = 1 << 64


def wrap(x: int) -> int:
    x &= M64 - 1
    return x - M64 if x >= (1 << 63) else x


def c_op(op: str, a: int, b: int) -> Optional[int]:
    """int64 C semantics; None when the divisor is zero."""
    if op == "+": return wrap(a + b)
    if op == "-": return wrap(a - b)
    if op == "*": return wrap(a * b)
    if op in ("/", "%"):
        if b == 0:
            return None
        q = abs(a) // abs(b)
        if (a < 0) != (b < 0):
            q = -q
        return wrap(q) if op == "/" else wrap(a - q * b)
    if op == "<": return int(a < b)
    if op == "<=": return int(a <= b)
    if op == "==": return int(a == b)
    if op == "!=": return int(a != b)
    if op == "min": return min(a, b)
    if op == "max": return max(a, b)
    if op == "&&": return int(a != 0 and b != 0)
    if op == "||": return int(a != 0 or b != 0)
    if op in ("<<", ">>"):                    # a shift count outside 0..63 is undefined, like a zero divisor
        if b < 0 or b > 63:
            return None
        return wrap(a * (1 << b)) if op == "<<" else a // (1 << b)      # >> keeps the sign (floor division)
    raise ValueError(op)


def all_trees(g: Grammar, max_size: int) -> Dict[Tuple[int, int], List[tuple]]:
    """trees[(nt, size)] in canonical order; a tree is ('v', i), ('c', value) or (op, l, r)."""
    T: Dict[Tuple[int, int], List[tuple]] = {}
    for s in range(1, max_size + 1):
        for nt in range(g.n_nonterminals):
            out: List[tuple] = []
            for p in g.productions:
                if p.lhs != nt:
                    continue
                if p.kind == P_VAR:
                    if s == 1: out.append(("v", p.var))
                elif p.kind == P_CONST:
                    if s == 1: out.append(("c", p.value))
                else:
                    for a in range(1, s - 1):
                        for l in T.get((p.left, a), []):
                            for r in T.get((p.right, s - 1 - a), []):
                                out.append((OPS[p.op], l, r))
            T[(nt, s)] = out
    return T


def tree_value(t: tuple, pt: Sequence[int]) -> Optional[int]:
    if t[0] == "v": return pt[t[1]]
    if t[0] == "c": return t[1]
    a = tree_value(t[1], pt)
    b = tree_value(t[2], pt)
    if a is None or b is None:
        return None
    return c_op(t[0], a, b)


def tree_text(t: tuple, g: Grammar) -> str:
    if t[0] == "v": return g.variables[t[1]].name
    if t[0] == "c": return str(t[1])
    if t[0] in ("min", "max"):
        return f"{t[0]}({tree_text(t[1], g)},{tree_text(t[2], g)})"
    return f"({tree_text(t[1], g)}{t[0]}{tree_text(t[2], g)})"


def code_value(code, pt: Sequence[int], hole=0) -> Optional[int]:
    """``hole``: the hole's value, or a sequence of values for the parts of a joint sketch."""
    st: List[Optional[int]] = []
    bad = False
    for kind, arg, value in code:
        if kind == K_VAR: st.append(pt[arg])
        elif kind == K_CONST: st.append(value)
        elif kind == K_HOLE: st.append(hole[arg] if isinstance(hole, (list, tuple)) else hole)
        else:
            b = st.pop(); a = st.pop()
            r = c_op(OPS[arg], a, b)
            if r is None:
                bad = True; r = 0
            st.append(r)
    return None if bad else st[0]


def points_of(sk: Sketch) -> List[Tuple[int, ...]]:
    if sk.coords is not None:
        return [tuple(int(x) for x in row) for row in sk.coords]
    pts = [()]
    for v in sk.grammar.variables:           # first variable slowest
        pts = [p + (x,) for p in pts for x in range(v.lo, v.hi)]
    return pts


def repair(sk: Sketch, hole_index: int = 0):
    """(cand_count, match_count, least(size, rank, text) or None, matching (size, rank) set)."""
    h = sk.holes[hole_index]
    pts = points_of(sk)
    if h.spec_table is not None:
        spec = [int(x) for x in h.spec_table]
    else:
        spec = [code_value(h.spec_expr, p) for p in pts]
    T = all_trees(sk.grammar, h.max_size)
    cand = [0] * (h.max_size + 1)
    match = [0] * (h.max_size + 1)
    least = None
    matches = set()
    for s in range(1, h.max_size + 1):
        trees = T[(h.start_nt, s)]
        cand[s] = len(trees)
        for rank, t in enumerate(trees):
            good = True
            for p, want in zip(pts, spec):           # no early exit on purpose
                v = tree_value(t, p)
                if v is not None and h.ctx:
                    v = code_value(h.ctx, p, v)
                if v is None or want is None or v != want:
                    good = False
            if good:
                match[s] += 1
                matches.add((s, rank))
                if least is None:
                    least = (s, rank, tree_text(t, sk.grammar))
    return cand, match, least, matches


def repair_joint(g: Grammar, starts, max_sizes, ctx, pts, spec):
    """Two holes in one context, brute force: (cand_count, match_count, least) by TOTAL size, where
    least = (total size, size of part 0, rank of part 0, rank of part 1, text 0, text 1) in the order
    total size, size of part 0, rank of part 0, rank of part 1."""
    T = all_trees(g, max(max_sizes))
    K = max_sizes[0] + max_sizes[1]
    cand = [0] * (K + 1)
    match = [0] * (K + 1)
    least = None
    for s in range(2, K + 1):
        for s0 in range(1, s):
            s1 = s - s0
            if s0 > max_sizes[0] or s1 > max_sizes[1]:
                continue
            A, B = T[(starts[0], s0)], T[(starts[1], s1)]
            cand[s] += len(A) * len(B)
            for r0, t0 in enumerate(A):
                for r1, t1 in enumerate(B):
                    good = True
                    for p, want in zip(pts, spec):
                        v0, v1 = tree_value(t0, p), tree_value(t1, p)
                        v = None if v0 is None or v1 is None else code_value(ctx, p, (v0, v1))
                        if v is None or want is None or v != want:
                            good = False
                    if good:
                        match[s] += 1
                        if least is None:
                            least = (s, s0, r0, r1, tree_text(t0, g), tree_text(t1, g))
    return cand, match, least


def text_value(text: str, g: Grammar, pt: Sequence[int]) -> Optional[int]:
    """Re-evaluates a solution text ``(L op R)`` / leaf independently of any postfix code."""
    names = {v.name: i for i, v in enumerate(g.variables)}
    pos = 0

    def node() -> Optional[int]:
        nonlocal pos
        if text.startswith(("min(", "max("), pos):
            op = text[pos:pos + 3]; pos += 4
            a = node()
            assert text[pos] == ","; pos += 1
            b = node()
            assert text[pos] == ")"; pos += 1
            if a is None or b is None:
                return None
            return c_op(op, a, b)
        if text[pos] == "(":
            pos += 1
            a = node()
            op = text[pos]; pos += 1
            if op in "<>" and text[pos] == op:  # a shift
                op += op; pos += 1
            b = node()
            assert text[pos] == ")"; pos += 1
            if a is None or b is None:
                return None
            return c_op(op, a, b)
        j = pos
        while j < len(text) and (text[j].isalnum() or text[j] in "_." or (j == pos and text[j] == "-")):
            j += 1
        tok = text[pos:j]; pos = j
        return pt[names[tok]] if tok in names else int(tok)

    v = node()
    assert pos == len(text), text
    return v
