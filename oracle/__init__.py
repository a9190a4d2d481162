"""CPU oracle wrapper -- TEST INFRASTRUCTURE ONLY.

Marshals :mod:`xp_instances` objects into the plain C++ oracle
(``xp_oracle.cpp``) through ctypes.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this package; the CUDA library and its
binding never do, and nothing here touches them.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

from xp_instances.model import Grammar, Hole, Sketch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "xp_oracle.cpp")
_LIB = os.path.join(_HERE, "libxp_oracle.so")
XO_MAX_SIZE = 15


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (plain -O2, no tuning flags)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


class _Prod(C.Structure):
    _fields_ = [("lhs", C.c_int32), ("kind", C.c_int32), ("var", C.c_int32), ("op", C.c_int32),
                ("left", C.c_int32), ("right", C.c_int32), ("value", C.c_int64)]


class _Instr(C.Structure):
    _fields_ = [("kind", C.c_int32), ("arg", C.c_int32), ("value", C.c_int64)]


class _Grammar(C.Structure):
    _fields_ = [("n_vars", C.c_int32), ("lo", C.POINTER(C.c_int64)), ("hi", C.POINTER(C.c_int64)),
                ("var_names", C.POINTER(C.c_char_p)), ("n_nt", C.c_int32), ("n_prods", C.c_int32),
                ("prods", C.POINTER(_Prod))]


class _Problem(C.Structure):
    _fields_ = [("g", _Grammar), ("n_points", C.c_int64), ("coords", C.POINTER(C.c_int32)),
                ("n_first", C.c_int64), ("first_points", C.POINTER(C.c_int64)),
                ("start_nt", C.c_int32), ("max_size", C.c_int32),
                ("ctx_len", C.c_int32), ("ctx", C.POINTER(_Instr)),
                ("spec_len", C.c_int32), ("spec_expr", C.POINTER(_Instr)),
                ("spec_table", C.POINTER(C.c_int64)),
                ("rank_begin", C.POINTER(C.c_uint64)), ("rank_end", C.POINTER(C.c_uint64))]


class _Result(C.Structure):
    _fields_ = [("cand_count", C.c_uint64 * (XO_MAX_SIZE + 1)), ("match_count", C.c_uint64 * (XO_MAX_SIZE + 1)),
                ("solved", C.c_int32), ("least_size", C.c_int32), ("least_rank", C.c_uint64),
                ("evals", C.c_uint64), ("least_text", C.c_char * 1024)]


class _JointProblem(C.Structure):
    _fields_ = [("g", _Grammar), ("n_points", C.c_int64), ("coords", C.POINTER(C.c_int32)),
                ("start_nt", C.c_int32 * 2), ("max_size", C.c_int32 * 2),
                ("ctx_len", C.c_int32), ("ctx", C.POINTER(_Instr)),
                ("spec_len", C.c_int32), ("spec_expr", C.POINTER(_Instr)),
                ("spec_table", C.POINTER(C.c_int64))]


class _JointResult(C.Structure):
    _fields_ = [("cand_count", C.c_uint64 * (2 * XO_MAX_SIZE + 1)), ("match_count", C.c_uint64 * (2 * XO_MAX_SIZE + 1)),
                ("solved", C.c_int32), ("least_total", C.c_int32), ("least_size0", C.c_int32), ("pad", C.c_int32),
                ("least_rank0", C.c_uint64), ("least_rank1", C.c_uint64), ("evals", C.c_uint64),
                ("least_text0", C.c_char * 512), ("least_text1", C.c_char * 512)]


class _BehaviourProblem(C.Structure):
    _fields_ = [("base", _Problem), ("n_sig", C.c_int64), ("sig_points", C.POINTER(C.c_int64))]


class _BehaviourResult(C.Structure):
    _fields_ = [("enumerated", C.c_uint64 * (XO_MAX_SIZE + 1)), ("distinct", C.c_uint64 * (XO_MAX_SIZE + 1)),
                ("sig_matches", C.c_uint64), ("hit", C.c_int32), ("hit_size", C.c_int32), ("hit_index", C.c_uint64),
                ("hit_verified", C.c_int32), ("solved", C.c_int32), ("solution_size", C.c_int32),
                ("solution_index", C.c_uint64), ("hit_text", C.c_char * 1024), ("solution_text", C.c_char * 1024)]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        lib.xo_counts.restype = C.c_int
        lib.xo_counts.argtypes = [C.POINTER(_Grammar), C.c_int, C.c_int, C.POINTER(C.c_uint64)]
        lib.xo_list.restype = C.c_int64
        lib.xo_list.argtypes = [C.POINTER(_Grammar), C.c_int, C.c_int, C.c_uint64, C.c_uint64, C.c_char_p, C.c_int64]
        lib.xo_eval_code.restype = C.c_int
        lib.xo_eval_code.argtypes = [C.POINTER(_Instr), C.c_int, C.POINTER(C.c_int64), C.c_int64, C.POINTER(C.c_int64)]
        lib.xo_repair.restype = C.c_int
        lib.xo_repair.argtypes = [C.POINTER(_Problem), C.POINTER(_Result)]
        lib.xo_behaviours.restype = C.c_int
        lib.xo_behaviours.argtypes = [C.POINTER(_BehaviourProblem), C.POINTER(_BehaviourResult)]
        lib.xo_repair_joint.restype = C.c_int
        lib.xo_repair_joint.argtypes = [C.POINTER(_JointProblem), C.POINTER(_JointResult)]
        _lib = lib
    return _lib


def _code(instrs) -> "C.Array":
    arr = (_Instr * max(1, len(instrs)))()
    for i, (k, a, v) in enumerate(instrs):
        arr[i].kind, arr[i].arg, arr[i].value = k, a, v
    return arr


class _GrammarC:
    """Keeps the ctypes buffers of one grammar alive."""

    def __init__(self, g: Grammar):
        nv = len(g.variables)
        self.lo = (C.c_int64 * max(1, nv))(*[v.lo for v in g.variables])
        self.hi = (C.c_int64 * max(1, nv))(*[v.hi for v in g.variables])
        self.names = (C.c_char_p * max(1, nv))(*[v.name.encode() for v in g.variables])
        self.prods = (_Prod * len(g.productions))()
        for i, p in enumerate(g.productions):
            q = self.prods[i]
            q.lhs, q.kind, q.var, q.op, q.left, q.right, q.value = p.lhs, p.kind, p.var, p.op, p.left, p.right, p.value
        self.c = _Grammar(nv, self.lo, self.hi, self.names, g.n_nonterminals, len(g.productions), self.prods)


@dataclass
class OracleResult:
    cand_count: List[int]
    match_count: List[int]
    solved: bool
    least_size: int
    least_rank: int
    least_text: str
    evals: int


def counts(g: Grammar, nt: int, max_size: int) -> List[int]:
    """Number of derivation trees of nonterminal ``nt`` for sizes 0..max_size."""
    gc = _GrammarC(g)
    out = (C.c_uint64 * (max_size + 1))()
    rc = _load().xo_counts(C.byref(gc.c), nt, max_size, out)
    if rc:
        raise OverflowError("a candidate count reaches 2^63")
    return [int(x) for x in out]


def listing(g: Grammar, nt: int, size: int, begin: int = 0, end: Optional[int] = None) -> List[str]:
    """Texts of the trees of (nt, size) with ranks in [begin, end), canonical order."""
    gc = _GrammarC(g)
    if end is None:
        end = counts(g, nt, size)[size]
    need = _load().xo_list(C.byref(gc.c), nt, size, begin, end, None, 0)
    buf = C.create_string_buffer(int(need))
    _load().xo_list(C.byref(gc.c), nt, size, begin, end, buf, need)
    text = buf.value.decode()
    return text.split("\n")[:-1] if text else []


def eval_code(instrs, point: Sequence[int], hole: int = 0):
    """Value of a postfix expression at one point, or None if a divisor is zero."""
    pt = (C.c_int64 * max(1, len(point)))(*point)
    out = C.c_int64(0)
    ok = _load().xo_eval_code(_code(instrs), len(instrs), pt, hole, C.byref(out))
    return int(out.value) if ok else None


def repair_hole(sk: Sketch, hole_index: int = 0, rank_ranges: Optional[dict] = None,
                first_points: Optional[Sequence[int]] = None) -> OracleResult:
    """The repair search for one hole of a sketch.

    ``rank_ranges`` maps size -> (begin, end) and restricts the match search at
    that size to those ranks (sizes not named are searched in full).
    ``first_points`` are point indices tried before the rest; the result does not
    depend on them."""
    P, keep = _problem(sk, hole_index, rank_ranges, first_points)
    h: Hole = sk.holes[hole_index]
    R = _Result()
    rc = _load().xo_repair(C.byref(P), C.byref(R))
    if rc:
        raise ValueError("oracle rejected the problem")
    K = h.max_size
    return OracleResult([int(x) for x in R.cand_count[:K + 1]], [int(x) for x in R.match_count[:K + 1]],
                        bool(R.solved), int(R.least_size), int(R.least_rank), R.least_text.decode(), int(R.evals))


def _problem(sk: Sketch, hole_index: int, rank_ranges=None, first_points=None):
    """The C description of one hole's problem and the buffers it points into."""
    h: Hole = sk.holes[hole_index]
    gc = _GrammarC(sk.grammar)
    P = _Problem()
    P.g = gc.c
    P.n_points = sk.n_points
    keep = [gc]
    if sk.coords is not None:
        co = np.ascontiguousarray(sk.coords, dtype=np.int32)
        keep.append(co)
        P.coords = co.ctypes.data_as(C.POINTER(C.c_int32))
    if first_points is not None and len(first_points):
        fp = np.ascontiguousarray(first_points, dtype=np.int64)
        keep.append(fp)
        P.n_first = fp.shape[0]
        P.first_points = fp.ctypes.data_as(C.POINTER(C.c_int64))
    P.start_nt, P.max_size = h.start_nt, h.max_size
    ctx = _code(h.ctx); keep.append(ctx)
    P.ctx_len, P.ctx = len(h.ctx), ctx
    if h.spec_table is not None:
        st = np.ascontiguousarray(h.spec_table, dtype=np.int64)
        assert st.shape[0] == sk.n_points
        keep.append(st)
        P.spec_table = st.ctypes.data_as(C.POINTER(C.c_int64))
    else:
        se = _code(h.spec_expr); keep.append(se)
        P.spec_len, P.spec_expr = len(h.spec_expr), se
    if rank_ranges is not None:
        rb = (C.c_uint64 * (h.max_size + 1))(*([0] * (h.max_size + 1)))
        re = (C.c_uint64 * (h.max_size + 1))(*([2 ** 64 - 1] * (h.max_size + 1)))
        for s, (b, e) in rank_ranges.items():
            rb[s], re[s] = b, e
        keep += [rb, re]
        P.rank_begin, P.rank_end = rb, re
    return P, keep


@dataclass
class JointResult:
    cand_count: List[int]          # index = total size of the pair
    match_count: List[int]
    solved: bool
    least_total: int
    least_size0: int
    least_rank0: int
    least_rank1: int
    least_text0: str
    least_text1: str
    evals: int


def repair_joint(sk: Sketch, joint) -> JointResult:
    """The repair search for two holes inside one constraint (``joint``: a ``JointHole``) over the
    domain and grammar of ``sk``: every pair of trees, by total size, then size of part 0, then
    rank of part 0, then rank of part 1."""
    gc = _GrammarC(sk.grammar)
    P = _JointProblem()
    P.g = gc.c
    P.n_points = sk.n_points
    keep = []
    if sk.coords is not None:
        co = np.ascontiguousarray(sk.coords, dtype=np.int32)
        keep.append(co)
        P.coords = co.ctypes.data_as(C.POINTER(C.c_int32))
    P.start_nt[0], P.start_nt[1] = joint.start_nt
    P.max_size[0], P.max_size[1] = joint.max_size
    ctx = _code(joint.ctx); keep.append(ctx)
    P.ctx_len, P.ctx = len(joint.ctx), ctx
    if joint.spec_table is not None:
        st = np.ascontiguousarray(joint.spec_table, dtype=np.int64)
        assert st.shape[0] == sk.n_points
        keep.append(st)
        P.spec_table = st.ctypes.data_as(C.POINTER(C.c_int64))
    else:
        se = _code(joint.spec_expr); keep.append(se)
        P.spec_len, P.spec_expr = len(joint.spec_expr), se
    R = _JointResult()
    if _load().xo_repair_joint(C.byref(P), C.byref(R)):
        raise ValueError("oracle rejected the joint problem")
    K = joint.max_size[0] + joint.max_size[1]
    return JointResult([int(x) for x in R.cand_count[:K + 1]], [int(x) for x in R.match_count[:K + 1]], bool(R.solved),
                       int(R.least_total), int(R.least_size0), int(R.least_rank0), int(R.least_rank1),
                       R.least_text0.decode(), R.least_text1.decode(), int(R.evals))


@dataclass
class BehaviourResult:
    enumerated: List[int]          # candidates generated for the start nonterminal, per size
    distinct: List[int]            # new behaviours among them
    sig_matches: int
    hit: bool
    hit_size: int
    hit_index: int
    hit_verified: bool
    hit_text: str
    solved: bool
    solution_size: int
    solution_index: int
    solution_text: str


def behaviours(sk: Sketch, sig_points: Sequence[int], hole_index: int = 0) -> BehaviourResult:
    """Bottom-up enumeration with observational-equivalence pruning on the given signature points
    (indices into the sketch's domain, in the given order)."""
    P, keep = _problem(sk, hole_index)
    B = _BehaviourProblem()
    B.base = P
    sp = np.ascontiguousarray(sig_points, dtype=np.int64)
    B.n_sig = sp.shape[0]
    B.sig_points = sp.ctypes.data_as(C.POINTER(C.c_int64))
    R = _BehaviourResult()
    if _load().xo_behaviours(C.byref(B), C.byref(R)):
        raise ValueError("oracle rejected the problem")
    K = sk.holes[hole_index].max_size
    return BehaviourResult([int(x) for x in R.enumerated[:K + 1]], [int(x) for x in R.distinct[:K + 1]], int(R.sig_matches),
                           bool(R.hit), int(R.hit_size), int(R.hit_index), bool(R.hit_verified), R.hit_text.decode(),
                           bool(R.solved), int(R.solution_size), int(R.solution_index), R.solution_text.decode())
