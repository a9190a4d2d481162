"""Seeded synthetic repair instances.

The paper's own evaluation programs (21 operators x 8 shapes, Table 5) are not
available; these generators stand in for them and take their shapes: a small
two-index nest, a 256x256 matmul tile nest, a ResNet-style 56x56 3x3 im2col
convolution, a large quasi-affine index map and a batch of small elementwise
nests.  Every instance is a function of (config, seed, instance index) only.

The "source program" side of an instance is the planted target.  Where a
config hands the solvers a value table instead of an expression, the table is
produced here with plain numpy integer arithmetic on templates whose ``/`` and
``%`` operands are non-negative with positive divisors, so no rounding or sign
convention is involved.  Nothing here counts, enumerates or ranks candidates.
"""
from __future__ import annotations

from typing import Callable, List, Sequence, Tuple

import numpy as np

from .model import (Grammar, Hole, Sketch, Variable, constant_set, free_grammar,
                    parse_expr, quasi_affine_grammar)


def _rng(config: int, seed: int, instance: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([0x5850, config, seed, instance])))


# --------------------------------------------------------------------------
# Point sets
# --------------------------------------------------------------------------

def box_coords(extents: Sequence[int], ids: np.ndarray) -> np.ndarray:
    """Coordinates of box point ids; mixed radix with the first variable slowest."""
    ids = np.asarray(ids, dtype=np.int64)
    out = np.empty((ids.shape[0], len(extents)), dtype=np.int32)
    rem = ids.copy()
    for d in range(len(extents) - 1, -1, -1):
        out[:, d] = rem % extents[d]
        rem //= extents[d]
    return out


def boundary_ids(extents: Sequence[int]) -> np.ndarray:
    """Corners and 1-D edges of the box (every variable but at most one at an
    extreme), as point ids, each once, in a fixed order (corners first)."""
    n = len(extents)
    strides = [1] * n
    for d in range(n - 2, -1, -1):
        strides[d] = strides[d + 1] * extents[d + 1]
    seen, order = set(), []

    def add(coord):
        pid = sum(c * s for c, s in zip(coord, strides))
        if pid not in seen:
            seen.add(pid); order.append(pid)

    for mask in range(1 << n):
        add([(extents[d] - 1) if (mask >> d) & 1 else 0 for d in range(n)])
    for free in range(n):
        others = [d for d in range(n) if d != free]
        for mask in range(1 << (n - 1)):
            base = [0] * n
            for b, d in enumerate(others):
                base[d] = (extents[d] - 1) if (mask >> b) & 1 else 0
            for x in range(extents[free]):
                base[free] = x
                add(base)
    return np.asarray(order, dtype=np.int64)


def sampled_point_ids(extents: Sequence[int], n_points: int, rng: np.random.Generator) -> np.ndarray:
    """Boundary ids first, then seeded uniform sampling without replacement up to
    exactly ``n_points`` ids (the whole box, in id order, if it has that many)."""
    total = int(np.prod([int(e) for e in extents], dtype=object))
    if total == n_points:
        return np.arange(total, dtype=np.int64)
    assert total > n_points
    first = boundary_ids(extents)[:n_points]
    ids = first
    while ids.shape[0] < n_points:
        need = n_points - ids.shape[0]
        draw = rng.integers(0, total, size=max(1024, 2 * need), dtype=np.int64)
        _, where = np.unique(draw, return_index=True)      # first occurrence of each id,
        draw = draw[np.sort(where)]                        # kept in draw order
        draw = draw[~np.isin(draw, ids)]
        ids = np.concatenate([ids, draw[:need]])
    assert ids.shape[0] == n_points and np.unique(ids).shape[0] == n_points
    return ids


# --------------------------------------------------------------------------
# Config 1: single-hole index repair, i,j in [0,16)
# --------------------------------------------------------------------------

def config1(seed: int) -> Sketch:
    r = _rng(1, seed)
    vs = [Variable("i", 0, 16), Variable("j", 0, 16)]
    g = free_grammar(vs, constant_set(-8, 8))
    a, b = (("i", "j"), ("j", "i"))[int(r.integers(2))]
    C = int(r.integers(2, 9))
    forms = [f"(({a}*{C})+{b})", f"({b}+({a}*{C}))", f"(({a}*{C})-{b})",
             f"(({a}+{b})%{C})", f"(({a}/{C})+{b})", f"(({C}*{a})+{b})"]
    target = forms[int(r.integers(len(forms)))]
    hole = Hole(start_nt=0, max_size=5, spec_expr=parse_expr(target, vs), note=target)
    return Sketch(g, [hole], None, name=f"config1/seed{seed}")


# --------------------------------------------------------------------------
# Config 2: thread-binding repair for a 256x256 matmul tile nest
# --------------------------------------------------------------------------

def config2_grammar() -> Grammar:
    vs = [Variable("bx", 0, 64), Variable("tx", 0, 256), Variable("k", 0, 8)]
    return free_grammar(vs, constant_set(-64, 64, [2 ** e for e in range(11)]))


def config2(seed: int) -> Sketch:
    r = _rng(2, seed)
    g = config2_grammar()
    vs = g.variables
    pow2 = [2, 4, 8, 16, 32, 64, 128, 256, 512, 1024]
    C1 = pow2[int(r.integers(3, len(pow2)))]
    C2 = pow2[int(r.integers(0, 6))]
    forms = [f"((bx*{C1})+(tx*{C2}))", f"(((bx*{C1})+tx)+k)", f"(((bx*{C1})+tx)/{C2})",
             f"((bx*{C1})+(tx%{C2}))", f"(((tx/{C2})*{C1})+k)", f"((tx*{C2})+(bx*{C1}))"]
    target = forms[int(r.integers(len(forms)))]
    hole = Hole(start_nt=0, max_size=7, spec_expr=parse_expr(target, vs), note=target)
    return Sketch(g, [hole], None, name=f"config2/seed{seed}")


# --------------------------------------------------------------------------
# Config 3: three holes of a conv2d NCHW im2col lowering
# --------------------------------------------------------------------------

def config3(seed: int) -> Sketch:
    r = _rng(3, seed)
    vs = [Variable("c", 0, 64), Variable("oh", 0, 56), Variable("ow", 0, 56),
          Variable("kh", 0, 3), Variable("kw", 0, 3)]
    g = free_grammar(vs, constant_set(-64, 64, [128, 256, 512, 1024, 3136]))
    wvar = bool(r.integers(2))        # repair the column (w) or the row (h) expressions
    flip = bool(r.integers(2))        # operand order inside the fixed context
    o, k = ("ow", "kw") if wvar else ("oh", "kh")
    row, col = "((oh+kh)-1)", "((ow+kw)-1)"
    if wvar:
        ctx1 = f"((c*3136)+({row}*56))+HOLE" if not flip else f"HOLE+((c*3136)+({row}*56))"
    else:
        ctx1 = f"((c*3136)+(HOLE*56))+{col}" if not flip else f"{col}+((HOLE*56)+(c*3136))"
    spec1 = f"((c*3136)+({row}*56))+{col}"
    t1 = col if wvar else row
    ctx2 = "((((c*9)+HOLE)*3136)+(oh*56))+ow" if not flip else "ow+((oh*56)+(3136*(HOLE+(c*9))))"
    spec2 = "((((c*9)+((kh*3)+kw))*3136)+(oh*56))+ow"
    t2 = "((kh*3)+kw)"
    ctx3 = f"{k}<HOLE"
    spec3 = f"(({o}+{k})-1)<56"
    t3 = f"(57-{o})"
    holes = [
        Hole(0, 6, ctx=parse_expr(ctx1, vs), spec_expr=parse_expr(spec1, vs), note=t1),
        Hole(0, 6, ctx=parse_expr(ctx2, vs), spec_expr=parse_expr(spec2, vs), note=t2),
        Hole(0, 6, ctx=parse_expr(ctx3, vs), spec_expr=parse_expr(spec3, vs), note=t3),
    ]
    return Sketch(g, holes, None, name=f"config3/seed{seed}")


# --------------------------------------------------------------------------
# Config 4: large typed search over a sampled 2^20-point table
# --------------------------------------------------------------------------

def config4(seed: int, n_points: int = 1 << 20) -> Sketch:
    r = _rng(4, seed)
    while True:
        ext = [int(x) for x in r.integers(1, 257, size=4)]
        if int(np.prod(ext, dtype=object)) >= (1 << 22):
            break
    vs = [Variable(f"v{d}", 0, ext[d]) for d in range(4)]
    g = quasi_affine_grammar(vs, constant_set(-128, 128), list(range(1, 129)))
    ids = sampled_point_ids(ext, n_points, r)
    coords = box_coords(ext, ids)
    big = [d for d in range(4) if ext[d] >= 8]
    a, b = [int(x) for x in r.choice(big, size=2, replace=False)]
    P1 = int(r.integers(2, min(128, ext[a]) + 1))
    P2 = int(r.integers(2, min(128, ext[b]) + 1))
    K1 = int(r.integers(2, 129)) * (1 if r.integers(2) else -1)
    target = f"(((v{a}/{P1})*{K1})+(v{b}%{P2}))"
    va = coords[:, a].astype(np.int64)
    vb = coords[:, b].astype(np.int64)
    spec = (va // P1) * K1 + (vb % P2)          # va, vb >= 0 and P1, P2 > 0
    hole = Hole(start_nt=0, max_size=9, spec_table=spec.astype(np.int64), note=target)
    return Sketch(g, [hole], coords, name=f"config4/seed{seed}")


# --------------------------------------------------------------------------
# Config 5: batch of small single-hole instances with explicit tables
# --------------------------------------------------------------------------

def _small_target(r: np.random.Generator, names: Sequence[str], cols: Sequence[np.ndarray],
                  unsolvable: bool) -> Tuple[str, np.ndarray]:
    nv = len(names)
    ia, ib = [int(x) for x in r.choice(nv, size=2, replace=False)]
    a, b, xa, xb = names[ia], names[ib], cols[ia], cols[ib]
    C = int(r.integers(2, 17))
    D = int(r.integers(2, 17))
    if unsolvable:      # planted size-7 target (4 leaves), beyond the size bound
        forms: List[Tuple[str, Callable[[], np.ndarray]]] = [
            (f"(({a}*{C})+({b}*{D}))", lambda: xa * C + xb * D),
            (f"((({a}/{C})*{D})+{b})", lambda: (xa // C) * D + xb),
            (f"(({a}%{C})+({b}*{D}))", lambda: (xa % C) + xb * D),
        ]
    else:               # planted target of size <= 5
        forms = [
            (f"(({a}*{C})+{b})", lambda: xa * C + xb),
            (f"(({a}/{C})+{b})", lambda: xa // C + xb),
            (f"(({a}+{b})%{C})", lambda: (xa + xb) % C),
            (f"(({a}*{C})-{b})", lambda: xa * C - xb),
            (f"({a}+({b}*{D}))", lambda: xa + xb * D),
            (f"({a}%{C})", lambda: xa % C),
            (f"({a}*{C})", lambda: xa * C),
        ]
    text, fn = forms[int(r.integers(len(forms)))]
    return text, fn().astype(np.int64)


def config5_instance(seed: int, index: int, n_points: int = 4096) -> Sketch:
    r = _rng(5, seed, index)
    nv = int(r.integers(2, 4))
    while True:          # re-draw the extents until the box has enough points
        cand = r.integers(1, 65, size=(4096, nv))
        ok = np.flatnonzero(np.prod(cand, axis=1) >= n_points)
        if ok.size:
            ext = [int(x) for x in cand[ok[0]]]
            break
    names = ["x", "y", "z"][:nv]
    vs = [Variable(names[d], 0, ext[d]) for d in range(nv)]
    g = free_grammar(vs, constant_set(-16, 16))
    ids = sampled_point_ids(ext, n_points, r)
    coords = box_coords(ext, ids)
    cols = [coords[:, d].astype(np.int64) for d in range(nv)]
    unsolvable = bool(r.random() < 0.10)
    text, spec = _small_target(r, names, cols, unsolvable)
    hole = Hole(start_nt=0, max_size=6, spec_table=spec, note=text)
    return Sketch(g, [hole], coords, name=f"config5/seed{seed}/inst{index}")


def config5(seed: int, n_instances: int = 4096, n_points: int = 4096) -> List[Sketch]:
    return [config5_instance(seed, i, n_points) for i in range(n_instances)]
