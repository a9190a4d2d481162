"""Plain data model of a repair instance, shared by every consumer of the
seeded generators (the CPU oracle wrapper and the CUDA binding each marshal
these objects into their own C structures).

A repair instance follows the statement of the repair problem in Section 4.4
(Algorithm 3): a code sketch whose missing expressions ("holes") must be
filled from a bounded expression grammar so that the snippet agrees with the
source program on every concrete index of the iteration domain.

This module holds descriptions only: no candidate counting, enumeration or
expression evaluation lives here.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple, Union

import numpy as np

# Operator codes.  The first five, min, max and the two shifts may appear in grammar
# productions; all of them in context and spec expressions.
OPS = ["+", "-", "*", "/", "%", "<", "<=", "==", "!=", "min", "max", "&&", "||", "<<", ">>"]
OP_CODE = {s: i for i, s in enumerate(OPS)}
GRAMMAR_OPS = OPS[:5]

# Instruction kinds of the postfix code used for contexts and specs.
K_VAR, K_CONST, K_HOLE, K_OP = 0, 1, 2, 3

# Production kinds.
P_VAR, P_CONST, P_BIN = 0, 1, 2


@dataclass(frozen=True)
class Variable:
    name: str
    lo: int  # inclusive
    hi: int  # exclusive


@dataclass(frozen=True)
class Production:
    """One grammar production ``lhs -> var | const | left op right``."""
    lhs: int
    kind: int                 # P_VAR / P_CONST / P_BIN
    var: int = 0              # P_VAR: variable index
    value: int = 0            # P_CONST: the constant
    op: int = 0               # P_BIN: operator code (one of the first five)
    left: int = 0             # P_BIN: nonterminal of the left operand
    right: int = 0            # P_BIN: nonterminal of the right operand


@dataclass
class Grammar:
    variables: List[Variable]
    n_nonterminals: int
    productions: List[Production]   # canonical order = list order

    def leaf_count(self, nt: int = 0) -> int:
        return sum(1 for p in self.productions if p.lhs == nt and p.kind != P_BIN)


# A postfix instruction: (kind, arg, value)
Instr = Tuple[int, int, int]


@dataclass
class Hole:
    start_nt: int
    max_size: int
    ctx: List[Instr] = field(default_factory=list)      # empty = identity
    spec_expr: Optional[List[Instr]] = None              # spec as expression ...
    spec_table: Optional[np.ndarray] = None              # ... or int64[n_points]
    note: str = ""                                       # e.g. text of the planted target


@dataclass
class JointHole:
    """Two holes inside ONE constraint: ``ctx`` mentions ``HOLE0`` and ``HOLE1``; the candidates
    are pairs of expressions (part 0 from ``start_nt[0]`` up to ``max_size[0]`` nodes, part 1
    likewise) and the constraint is stated once for the pair."""
    start_nt: Tuple[int, int]
    max_size: Tuple[int, int]
    ctx: List[Instr]
    spec_expr: Optional[List[Instr]] = None
    spec_table: Optional[np.ndarray] = None
    note: str = ""


@dataclass
class Sketch:
    grammar: Grammar
    holes: List[Hole]
    coords: Optional[np.ndarray] = None   # None = full box; else int32[n_points, n_vars]
    name: str = ""

    @property
    def n_points(self) -> int:
        if self.coords is not None:
            return int(self.coords.shape[0])
        n = 1
        for v in self.grammar.variables:
            n *= (v.hi - v.lo)
        return n


# --------------------------------------------------------------------------
# Grammar builders
# --------------------------------------------------------------------------

def free_grammar(variables: Sequence[Variable], constants: Sequence[int],
                 ops: Sequence[str] = GRAMMAR_OPS) -> Grammar:
    """One nonterminal; leaves first (variables in declaration order, then the
    constants in the order given), then one binary production per operator."""
    prods: List[Production] = []
    for i, _ in enumerate(variables):
        prods.append(Production(lhs=0, kind=P_VAR, var=i))
    for c in constants:
        prods.append(Production(lhs=0, kind=P_CONST, value=int(c)))
    for o in ops:
        prods.append(Production(lhs=0, kind=P_BIN, op=OP_CODE[o], left=0, right=0))
    return Grammar(list(variables), 1, prods)


def quasi_affine_grammar(variables: Sequence[Variable], mul_constants: Sequence[int],
                         div_constants: Sequence[int]) -> Grammar:
    """Typed grammar ``E ::= v | E+E | E-E | E*K | E/P | E%P`` with constant-only
    nonterminals K (multipliers) and P (positive divisors)."""
    E, K, P = 0, 1, 2
    prods: List[Production] = []
    for i, _ in enumerate(variables):
        prods.append(Production(lhs=E, kind=P_VAR, var=i))
    prods.append(Production(lhs=E, kind=P_BIN, op=OP_CODE["+"], left=E, right=E))
    prods.append(Production(lhs=E, kind=P_BIN, op=OP_CODE["-"], left=E, right=E))
    prods.append(Production(lhs=E, kind=P_BIN, op=OP_CODE["*"], left=E, right=K))
    prods.append(Production(lhs=E, kind=P_BIN, op=OP_CODE["/"], left=E, right=P))
    prods.append(Production(lhs=E, kind=P_BIN, op=OP_CODE["%"], left=E, right=P))
    for c in mul_constants:
        prods.append(Production(lhs=K, kind=P_CONST, value=int(c)))
    for c in div_constants:
        prods.append(Production(lhs=P, kind=P_CONST, value=int(c)))
    return Grammar(list(variables), 3, prods)


def constant_set(lo: int, hi: int, extra: Sequence[int] = ()) -> List[int]:
    """The inclusive range ascending, then the extra values not already present,
    ascending (a set: no value appears twice)."""
    base = list(range(lo, hi + 1))
    seen = set(base)
    for e in sorted(extra):
        if e not in seen:
            base.append(e)
            seen.add(e)
    return base


# --------------------------------------------------------------------------
# Text <-> postfix for context / spec expressions (syntax only)
# --------------------------------------------------------------------------

_BINARY_LEVELS = [["||"], ["&&"], ["==", "!="], ["<", "<="], ["<<", ">>"], ["+", "-"], ["*", "/", "%"]]


def _tokenize(text: str) -> List[str]:
    toks: List[str] = []
    i, n = 0, len(text)
    while i < n:
        ch = text[i]
        if ch.isspace():
            i += 1
        elif ch.isalpha() or ch == "_":
            j = i
            while j < n and (text[j].isalnum() or text[j] in "_."):
                j += 1
            toks.append(text[i:j]); i = j
        elif ch.isdigit():
            j = i
            while j < n and text[j].isdigit():
                j += 1
            toks.append(text[i:j]); i = j
        elif text[i:i + 2] in ("<<", ">>", "<=", "==", "!=", "&&", "||"):
            toks.append(text[i:i + 2]); i += 2
        elif ch in "+-*/%<(),":
            toks.append(ch); i += 1
        else:
            raise ValueError(f"bad character {ch!r} in expression {text!r}")
    return toks


def parse_expr(text: str, variables: Sequence[Variable]) -> List[Instr]:
    """Infix text -> postfix instruction list.  ``HOLE`` names the hole (``HOLE0``, ``HOLE1`` the
    parts of a joint sketch); ``<<`` and ``>>`` bind tighter than comparisons and looser than ``+``; ``min(a,b)``
    and ``max(a,b)`` are calls; a minus sign directly before a number literal in
    operand position is part of the literal (there is no unary minus operator)."""
    names = {v.name: i for i, v in enumerate(variables)}
    toks = _tokenize(text)
    pos = 0
    out: List[Instr] = []

    def peek() -> Optional[str]:
        return toks[pos] if pos < len(toks) else None

    def take(expected: Optional[str] = None) -> str:
        nonlocal pos
        if pos >= len(toks):
            raise ValueError(f"unexpected end of expression {text!r}")
        t = toks[pos]
        if expected is not None and t != expected:
            raise ValueError(f"expected {expected!r}, got {t!r} in {text!r}")
        pos += 1
        return t

    def primary() -> None:
        t = take()
        if t == "(":
            level(0); take(")")
        elif t == "-" and peek() is not None and peek().isdigit():
            out.append((K_CONST, 0, -int(take())))
        elif t.isdigit():
            out.append((K_CONST, 0, int(t)))
        elif t in ("min", "max"):
            take("("); level(0); take(","); level(0); take(")")
            out.append((K_OP, OP_CODE[t], 0))
        elif t == "HOLE" or (t.startswith("HOLE") and t[4:].isdigit()):
            out.append((K_HOLE, int(t[4:] or 0), 0))      # HOLE = HOLE0; HOLE1, ... name the other parts of a joint sketch
        elif t in names:
            out.append((K_VAR, names[t], 0))
        else:
            raise ValueError(f"unknown name {t!r} in {text!r}")

    def level(k: int) -> None:
        if k == len(_BINARY_LEVELS):
            primary(); return
        level(k + 1)
        while peek() in _BINARY_LEVELS[k]:
            op = take()
            level(k + 1)
            out.append((K_OP, OP_CODE[op], 0))

    level(0)
    if pos != len(toks):
        raise ValueError(f"trailing tokens in {text!r}")
    return out


def postfix_to_text(code: Sequence[Instr], variables: Sequence[Variable]) -> str:
    """Fully parenthesised infix without spaces: a leaf prints bare, an operator
    node as ``(L op R)``; ``min``/``max`` as calls."""
    st: List[str] = []
    for kind, arg, value in code:
        if kind == K_VAR:
            st.append(variables[arg].name)
        elif kind == K_CONST:
            st.append(str(int(value)))
        elif kind == K_HOLE:
            st.append("HOLE" if arg == 0 else f"HOLE{arg}")
        else:
            r = st.pop(); l = st.pop()
            s = OPS[arg]
            st.append(f"{s}({l},{r})" if s in ("min", "max") else f"({l}{s}{r})")
    assert len(st) == 1
    return st[0]
