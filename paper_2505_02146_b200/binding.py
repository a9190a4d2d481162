"""ctypes binding of libxpiler_repair.so: argument marshalling only.

Every step of the repair search runs inside the CUDA library; nothing here
evaluates, counts or ranks candidates, and there is no CPU fallback: a missing
or unloadable library raises.  The functions carry the names of the C ABI
(``include/xp.h``); ``Grammar`` / ``LoadedSketch`` are thin handle owners.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from . import build as _build

XP_MAX_SIZE = 15
XP_FLAG_NO_FILTER = 1
XP_FLAG_ALWAYS_FILTER = 2
_STATUS = {0: "XP_OK", 1: "XP_ERR_INVALID_ARG", 2: "XP_ERR_GRAMMAR", 3: "XP_ERR_SKETCH", 4: "XP_ERR_TOO_LARGE",
           5: "XP_ERR_NOMEM", 6: "XP_ERR_CUDA", 7: "XP_ERR_TIMEOUT", 8: "XP_ERR_CANCELLED"}

EXPORTS = ["xp_grammar_create", "xp_grammar_destroy", "xp_grammar_count", "xp_grammar_unrank",
           "xp_sketch_load", "xp_sketch_load_batch", "xp_sketch_destroy", "xp_workspace_bytes", "xp_repair", "xp_repair_batch",
           "xp_result_get", "xp_result_free", "xp_last_error", "xp_int32_peak", "xp_repair_static",
           "xp_sketch_info_get", "xp_sketch_refine", "xp_result_pack",
           "xp_repair_pair", "xp_pair_result_get", "xp_pair_result_free",
           "xp_repair_joint", "xp_joint_result_get", "xp_joint_result_free", "xp_behaviours", "xp_int_div_rate"]


class XpError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{_STATUS.get(status, status)}: {message}")
        self.status = status


class xp_variable(C.Structure):
    _fields_ = [("name", C.c_char_p), ("lo", C.c_int64), ("hi", C.c_int64)]


class xp_production(C.Structure):
    _fields_ = [("lhs", C.c_int32), ("kind", C.c_int32), ("var", C.c_int32), ("op", C.c_int32),
                ("left", C.c_int32), ("right", C.c_int32), ("value", C.c_int64)]


class xp_grammar_desc(C.Structure):
    _fields_ = [("n_vars", C.c_int32), ("vars", C.POINTER(xp_variable)), ("n_nonterminals", C.c_int32),
                ("n_productions", C.c_int32), ("productions", C.POINTER(xp_production))]


class xp_instr(C.Structure):
    _fields_ = [("kind", C.c_int32), ("arg", C.c_int32), ("value", C.c_int64)]


class xp_hole_desc(C.Structure):
    _fields_ = [("start_nt", C.c_int32), ("max_size", C.c_int32), ("ctx_len", C.c_int32), ("ctx", C.POINTER(xp_instr)),
                ("spec_kind", C.c_int32), ("spec_len", C.c_int32), ("spec_expr", C.POINTER(xp_instr)),
                ("spec_table", C.c_void_p), ("spec_table_on_device", C.c_int32)]


class xp_sketch_desc(C.Structure):
    _fields_ = [("domain_kind", C.c_int32), ("n_points", C.c_int64), ("coords", C.c_void_p),
                ("coords_on_device", C.c_int32), ("n_holes", C.c_int32), ("holes", C.POINTER(xp_hole_desc))]


class xp_rank_range(C.Structure):
    _fields_ = [("hole", C.c_int32), ("size", C.c_int32), ("begin", C.c_uint64), ("end", C.c_uint64)]


class xp_repair_opts(C.Structure):
    _fields_ = [("size_min", C.c_int32), ("size_max", C.c_int32), ("n_rank_ranges", C.c_int32),
                ("rank_ranges", C.POINTER(xp_rank_range)), ("stream", C.c_void_p), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_size_t), ("flags", C.c_uint32), ("cancel", C.POINTER(C.c_int32)),
                ("timeout_ms", C.c_int64)]


class xp_result_view(C.Structure):
    _fields_ = [("solved", C.c_int32), ("max_size", C.c_int32), ("cand_count", C.POINTER(C.c_uint64)),
                ("match_count", C.POINTER(C.c_uint64)), ("least_size", C.c_int32), ("least_rank", C.c_uint64),
                ("least_code", C.POINTER(xp_instr)), ("least_len", C.c_int32), ("least_text", C.c_char_p),
                ("evals_executed", C.c_uint64), ("filter_survivors", C.c_uint64), ("probe_survivors", C.c_uint64),
                ("nominal_ops", C.c_uint64), ("kernel_ms", C.c_double), ("total_ms", C.c_double), ("n_launches", C.c_int32),
                ("filter_tests", C.c_uint64), ("candidates_skipped", C.c_uint64), ("h2d_bytes", C.c_uint64),
                ("d2h_bytes", C.c_uint64)]


class xp_sketch_info(C.Structure):
    _fields_ = [("n_holes", C.c_int32), ("device", C.c_int32), ("n_points", C.c_int64), ("device_bytes", C.c_uint64),
                ("load_h2d_bytes", C.c_uint64), ("load_d2h_bytes", C.c_uint64), ("n_probes", C.c_int32 * 8),
                ("n_refined", C.c_int32)]


class xp_hole_summary(C.Structure):
    _fields_ = [("solved", C.c_int32), ("max_size", C.c_int32), ("least_size", C.c_int32), ("pad", C.c_int32),
                ("least_rank", C.c_uint64), ("cand_count", C.c_uint64 * (XP_MAX_SIZE + 1)),
                ("match_count", C.c_uint64 * (XP_MAX_SIZE + 1)), ("evals_executed", C.c_uint64),
                ("least_text", C.c_char * 256)]


class xp_pair_desc(C.Structure):
    _fields_ = [("source", C.POINTER(xp_instr)), ("source_len", C.c_int32), ("erroneous", C.POINTER(xp_instr)),
                ("erroneous_len", C.c_int32), ("n_source_vars", C.c_int32), ("var_map", C.POINTER(C.POINTER(xp_instr))),
                ("var_map_len", C.POINTER(C.c_int32)), ("start_nt", C.c_int32), ("max_size", C.c_int32)]


class xp_pair_view(C.Structure):
    _fields_ = [("solved", C.c_int32), ("n_sketches", C.c_int32), ("node_first", C.c_int32), ("node_last", C.c_int32),
                ("least_size", C.c_int32), ("least_rank", C.c_uint64), ("hole_text", C.c_char_p),
                ("sketch_text", C.c_char_p), ("stitched_text", C.c_char_p), ("stitched_code", C.POINTER(xp_instr)),
                ("stitched_len", C.c_int32), ("candidates", C.c_uint64), ("evals_executed", C.c_uint64),
                ("load_ms", C.c_double), ("search_ms", C.c_double)]


class xp_behaviour_desc(C.Structure):
    _fields_ = [("hole", C.c_int32), ("n_sig", C.c_int32), ("sig_points", C.POINTER(C.c_int64)),
                ("max_representatives", C.c_uint64)]


class xp_behaviour_summary(C.Structure):
    _fields_ = [("max_size", C.c_int32), ("pad", C.c_int32), ("enumerated", C.c_uint64 * (XP_MAX_SIZE + 1)),
                ("distinct", C.c_uint64 * (XP_MAX_SIZE + 1)), ("sig_matches", C.c_uint64), ("hit", C.c_int32),
                ("hit_size", C.c_int32), ("hit_index", C.c_uint64), ("hit_verified", C.c_int32), ("solved", C.c_int32),
                ("solution_size", C.c_int32), ("pad2", C.c_int32), ("solution_index", C.c_uint64),
                ("hit_text", C.c_char * 256), ("solution_text", C.c_char * 256), ("representatives", C.c_uint64),
                ("bytes_moved", C.c_uint64), ("kernel_ms", C.c_double), ("total_ms", C.c_double),
                ("n_launches", C.c_int32), ("pad3", C.c_int32)]


class xp_joint_desc(C.Structure):
    _fields_ = [("start_nt", C.c_int32 * 2), ("max_size", C.c_int32 * 2), ("ctx_len", C.c_int32), ("ctx", C.POINTER(xp_instr)),
                ("spec_kind", C.c_int32), ("spec_len", C.c_int32), ("spec_expr", C.POINTER(xp_instr)),
                ("spec_table", C.c_void_p), ("spec_table_on_device", C.c_int32)]


class xp_joint_view(C.Structure):
    _fields_ = [("solved", C.c_int32), ("max_total", C.c_int32), ("cand_count", C.POINTER(C.c_uint64)),
                ("match_count", C.POINTER(C.c_uint64)), ("least_total", C.c_int32), ("least_size", C.c_int32 * 2),
                ("least_rank", C.c_uint64 * 2), ("least_text", C.c_char_p * 2), ("evals_executed", C.c_uint64),
                ("probe_survivors", C.c_uint64), ("kernel_ms", C.c_double), ("total_ms", C.c_double), ("n_launches", C.c_int32)]


_lib = None


def load(path: Optional[str] = None):
    """Loads (building first if the sources are newer) the shared library; raises if that fails."""
    global _lib
    if _lib is not None:
        return _lib
    # XP_CHECKED_BUILD=1 in the environment selects the variant with index checks compiled in
    lib = C.CDLL(path or _build.build(checked=os.environ.get("XP_CHECKED_BUILD", "") == "1"))
    vp = C.c_void_p
    lib.xp_grammar_create.argtypes = [C.POINTER(xp_grammar_desc), C.POINTER(vp)]
    lib.xp_grammar_destroy.argtypes = [vp]
    lib.xp_grammar_destroy.restype = None
    lib.xp_grammar_count.argtypes = [vp, C.c_int32, C.c_int32, C.POINTER(C.c_uint64)]
    lib.xp_grammar_unrank.argtypes = [vp, C.c_int32, C.c_int32, C.c_uint64, C.POINTER(xp_instr), C.c_int32,
                                      C.c_char_p, C.c_size_t]
    lib.xp_sketch_load.argtypes = [vp, C.POINTER(xp_sketch_desc), C.POINTER(vp)]
    lib.xp_sketch_load_batch.argtypes = [C.POINTER(vp), C.POINTER(xp_sketch_desc), C.c_size_t, C.POINTER(vp)]
    lib.xp_sketch_destroy.argtypes = [vp]
    lib.xp_sketch_destroy.restype = None
    lib.xp_workspace_bytes.argtypes = [C.POINTER(vp), C.c_size_t, C.POINTER(xp_repair_opts)]
    lib.xp_workspace_bytes.restype = C.c_size_t
    lib.xp_repair.argtypes = [vp, C.POINTER(xp_repair_opts), C.POINTER(vp)]
    lib.xp_repair_batch.argtypes = [C.POINTER(vp), C.c_size_t, C.POINTER(xp_repair_opts), C.POINTER(vp)]
    lib.xp_result_get.argtypes = [vp, C.c_int32, C.POINTER(xp_result_view)]
    lib.xp_result_free.argtypes = [vp]
    lib.xp_result_free.restype = None
    lib.xp_last_error.restype = C.c_char_p
    lib.xp_int32_peak.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_double)]
    lib.xp_int_div_rate.argtypes = [C.POINTER(C.c_double)]
    lib.xp_repair_static.argtypes = [vp, C.POINTER(xp_repair_opts), C.POINTER(xp_hole_summary), C.c_int32]
    lib.xp_sketch_info_get.argtypes = [vp, C.POINTER(xp_sketch_info)]
    lib.xp_sketch_refine.argtypes = [vp, C.c_int32, C.POINTER(C.c_int32)]
    lib.xp_result_pack.argtypes = [C.POINTER(vp), C.c_size_t, C.POINTER(xp_hole_summary), C.c_size_t, C.POINTER(C.c_size_t)]
    lib.xp_behaviours.argtypes = [vp, C.POINTER(xp_behaviour_desc), C.POINTER(xp_repair_opts), C.POINTER(xp_behaviour_summary)]
    lib.xp_repair_joint.argtypes = [vp, C.POINTER(xp_joint_desc), C.POINTER(xp_repair_opts), C.POINTER(vp)]
    lib.xp_joint_result_get.argtypes = [vp, C.POINTER(xp_joint_view)]
    lib.xp_joint_result_free.argtypes = [vp]
    lib.xp_joint_result_free.restype = None
    lib.xp_repair_pair.argtypes = [vp, C.POINTER(xp_pair_desc), C.POINTER(vp)]
    lib.xp_pair_result_get.argtypes = [vp, C.POINTER(xp_pair_view)]
    lib.xp_pair_result_free.argtypes = [vp]
    lib.xp_pair_result_free.restype = None
    for name in EXPORTS:
        getattr(lib, name)
    _lib = lib
    return lib


def _check(status: int) -> None:
    if status != 0:
        raise XpError(status, load().xp_last_error().decode())


def _code(instrs) -> "C.Array":
    arr = (xp_instr * max(1, len(instrs)))()
    for i, (k, a, v) in enumerate(instrs):
        arr[i].kind, arr[i].arg, arr[i].value = k, a, v
    return arr


# ------------------------------------------------------------------------------------------
# the C ABI, one Python function per entry point
# ------------------------------------------------------------------------------------------

class Grammar:
    """Owns an ``xp_grammar*``."""

    def __init__(self, handle: int, model):
        self.handle, self.model = handle, model

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.xp_grammar_destroy(self.handle)
            self.handle = None


class GrammarDesc:
    """A grammar's C descriptor in host memory (``marshal_grammar``), with what it points to kept alive."""

    def __init__(self, desc, model, keep):
        self.desc, self.model, self._keep = desc, model, keep


def marshal_grammar(g) -> GrammarDesc:
    """Encodes an ``xp_instances.Grammar`` as the C descriptor ``xp_grammar_create`` takes; a caller that
    creates the same grammar again and again does this once."""
    nv = len(g.variables)
    names = [v.name.encode() for v in g.variables]
    vs = (xp_variable * max(1, nv))()
    for i, v in enumerate(g.variables):
        vs[i].name, vs[i].lo, vs[i].hi = names[i], v.lo, v.hi
    ps = (xp_production * len(g.productions))()
    for i, p in enumerate(g.productions):
        q = ps[i]
        q.lhs, q.kind, q.var, q.op, q.left, q.right, q.value = p.lhs, p.kind, p.var, p.op, p.left, p.right, p.value
    return GrammarDesc(xp_grammar_desc(nv, vs, g.n_nonterminals, len(g.productions), ps), g, (names, vs, ps))


def xp_grammar_create(g) -> Grammar:
    """``g``: an ``xp_instances.Grammar`` (variables with ranges, productions in canonical order), or the
    descriptor ``marshal_grammar`` made of one."""
    lib = load()
    d = g if isinstance(g, GrammarDesc) else marshal_grammar(g)
    out = C.c_void_p()
    _check(lib.xp_grammar_create(C.byref(d.desc), C.byref(out)))
    return Grammar(out.value, d.model)


def xp_grammar_count(gr: Grammar, nt: int, max_size: int) -> List[int]:
    out = (C.c_uint64 * (max_size + 1))()
    _check(load().xp_grammar_count(gr.handle, nt, max_size, out))
    return [int(x) for x in out]


def xp_grammar_unrank(gr: Grammar, nt: int, size: int, rank: int) -> Tuple[str, List[Tuple[int, int, int]]]:
    code = (xp_instr * XP_MAX_SIZE)()
    text = C.create_string_buffer(1024)
    _check(load().xp_grammar_unrank(gr.handle, nt, size, rank, code, XP_MAX_SIZE, text, 1024))
    return text.value.decode(), [(code[i].kind, code[i].arg, code[i].value) for i in range(size)]


class LoadedSketch:
    """Owns an ``xp_sketch*`` and keeps the grammar and any device tensors it refers to alive."""

    def __init__(self, handle: int, grammar: Grammar, n_holes: int, keep):
        self.handle, self.grammar, self.n_holes, self._keep = handle, grammar, n_holes, keep

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.xp_sketch_destroy(self.handle)
            self.handle = None


def _ptr_of(x) -> Tuple[int, int, object]:
    """(address, on_device, keep-alive) of a numpy array (host) or a torch CUDA tensor (device)."""
    if isinstance(x, np.ndarray):
        return x.ctypes.data, 0, x
    return int(x.data_ptr()), int(x.is_cuda), x      # torch tensor: device memory only, no torch compute


def _fill_sketch_desc(desc, sk, coords, spec_tables, keep) -> int:
    """Marshals one ``xp_instances.Sketch`` into ``desc``; everything that must outlive the call goes to ``keep``."""
    nh = len(sk.holes)
    holes = (xp_hole_desc * nh)()
    keep.append(holes)
    for i, h in enumerate(sk.holes):
        d = holes[i]
        d.start_nt, d.max_size = h.start_nt, h.max_size
        ctx = _code(h.ctx); keep.append(ctx)
        d.ctx_len, d.ctx = len(h.ctx), ctx
        table = (spec_tables or {}).get(i, h.spec_table)
        if table is not None:
            if isinstance(table, np.ndarray):
                table = np.ascontiguousarray(table, dtype=np.int64)
            d.spec_kind = 1
            d.spec_table, d.spec_table_on_device, k = _ptr_of(table)
            keep.append(k)
        else:
            se = _code(h.spec_expr); keep.append(se)
            d.spec_kind, d.spec_len, d.spec_expr = 0, len(h.spec_expr), se
    co = coords if coords is not None else sk.coords
    if co is not None:
        if isinstance(co, np.ndarray):
            co = np.ascontiguousarray(co, dtype=np.int32)
        desc.domain_kind = 1
        desc.n_points = int(co.shape[0])
        desc.coords, desc.coords_on_device, k = _ptr_of(co)
        keep.append(k)
    desc.n_holes, desc.holes = nh, holes
    return nh


def xp_sketch_load(gr: Grammar, sk, coords=None, spec_tables: Optional[Dict[int, object]] = None) -> LoadedSketch:
    """``sk``: an ``xp_instances.Sketch``.  ``coords`` / ``spec_tables[hole]`` may override the
    sketch's host tables with contiguous torch CUDA tensors (int32 [n, n_vars] / int64 [n]),
    which the library then uses in place."""
    lib = load()
    keep = []
    desc = xp_sketch_desc()
    nh = _fill_sketch_desc(desc, sk, coords, spec_tables, keep)
    out = C.c_void_p()
    _check(lib.xp_sketch_load(gr.handle, C.byref(desc), C.byref(out)))
    return LoadedSketch(out.value, gr, nh, [k for k in keep if not isinstance(k, C.Array)])


def marshal_sketches(sks: Sequence):
    """The C descriptors (``xp_sketch_desc`` array and what it points to, all in host memory) of a
    list of sketches, for callers that load the same descriptions more than once."""
    n = len(sks)
    descs = (xp_sketch_desc * n)()
    keeps, nhs = [], []
    for i, sk in enumerate(sks):
        keep = []
        nhs.append(_fill_sketch_desc(descs[i], sk, None, None, keep))
        keeps.append(keep)
    return descs, nhs, keeps


def xp_sketch_load_batch(grs: Sequence[Grammar], sks: Sequence, marshalled=None) -> List[LoadedSketch]:
    """Loads ``sks[i]`` against ``grs[i]`` in one call (one wait for the device for the whole batch).
    ``marshalled``: the result of ``marshal_sketches(sks)``, to skip building the descriptors again."""
    lib = load()
    n = len(sks)
    assert len(grs) == n and n > 0
    descs, nhs, keeps = marshalled if marshalled is not None else marshal_sketches(sks)
    handles = (C.c_void_p * n)(*[g.handle for g in grs])
    outs = (C.c_void_p * n)()
    _check(lib.xp_sketch_load_batch(handles, descs, n, outs))
    return [LoadedSketch(outs[i], grs[i], nhs[i], [k for k in keeps[i] if not isinstance(k, C.Array)]) for i in range(n)]


@dataclass
class HoleResult:
    solved: bool
    cand_count: List[int]
    match_count: List[int]
    least_size: int
    least_rank: int
    least_text: str
    least_code: List[Tuple[int, int, int]]
    evals_executed: int
    filter_survivors: int
    probe_survivors: int
    nominal_ops: int
    kernel_ms: float
    total_ms: float
    n_launches: int
    filter_tests: int = 0
    candidates_skipped: int = 0
    h2d_bytes: int = 0
    d2h_bytes: int = 0


def xp_result_get(result_handle: int, hole: int) -> HoleResult:
    v = xp_result_view()
    _check(load().xp_result_get(result_handle, hole, C.byref(v)))
    K = v.max_size
    return HoleResult(bool(v.solved), [int(v.cand_count[k]) for k in range(K + 1)],
                      [int(v.match_count[k]) for k in range(K + 1)], int(v.least_size), int(v.least_rank),
                      v.least_text.decode() if v.solved else "",
                      [(v.least_code[i].kind, v.least_code[i].arg, v.least_code[i].value) for i in range(v.least_len)],
                      int(v.evals_executed), int(v.filter_survivors), int(v.probe_survivors),
                      int(v.nominal_ops), float(v.kernel_ms), float(v.total_ms), int(v.n_launches),
                      int(v.filter_tests), int(v.candidates_skipped), int(v.h2d_bytes), int(v.d2h_bytes))


def _opts(size_min=0, size_max=0, rank_ranges=None, stream=None, workspace=None, flags=0, cancel=None, timeout_ms=0):
    o = xp_repair_opts()
    o.size_min, o.size_max, o.flags, o.timeout_ms = size_min, size_max, flags, int(timeout_ms)
    keep = []
    if cancel is not None:             # a ctypes.c_int32 that another thread may set
        o.cancel = C.pointer(cancel)
        keep.append(cancel)
    if rank_ranges:
        rr = (xp_rank_range * len(rank_ranges))()
        for i, (hole, size, b, e) in enumerate(rank_ranges):
            rr[i].hole, rr[i].size, rr[i].begin, rr[i].end = hole, size, b, e
        o.n_rank_ranges, o.rank_ranges = len(rank_ranges), rr
        keep.append(rr)
    if stream is not None:
        o.stream = int(stream)
    if workspace is not None:          # a torch CUDA tensor (uint8) used as scratch
        o.workspace, o.workspace_bytes = int(workspace.data_ptr()), int(workspace.numel() * workspace.element_size())
        keep.append(workspace)
    return o, keep


def xp_workspace_bytes(sketches: Sequence[LoadedSketch], **kw) -> int:
    o, _keep = _opts(**kw)
    arr = (C.c_void_p * len(sketches))(*[s.handle for s in sketches])
    return int(load().xp_workspace_bytes(arr, len(sketches), C.byref(o)))


def xp_repair(sketch: LoadedSketch, **kw) -> List[HoleResult]:
    """Keyword options: size_min, size_max, rank_ranges=[(hole, size, begin, end)], stream (raw
    cudaStream_t), workspace (torch CUDA uint8 tensor), flags, cancel (a ``ctypes.c_int32`` polled
    between launches), timeout_ms.  Returns one result per hole."""
    o, _keep = _opts(**kw)
    out = C.c_void_p()
    _check(load().xp_repair(sketch.handle, C.byref(o), C.byref(out)))
    try:
        return [xp_result_get(out.value, h) for h in range(sketch.n_holes)]
    finally:
        load().xp_result_free(out.value)


def xp_repair_batch(sketches: Sequence[LoadedSketch], packed: bool = False, **kw):
    """``packed=False``: one list of ``HoleResult`` per sketch.  ``packed=True``: ``(summaries, view)``
    where ``summaries`` is ONE ctypes array of ``xp_hole_summary`` (the holes of sketch 0, then of sketch 1,
    ...) filled by a single ``xp_result_pack`` call, and ``view`` is the full ``HoleResult`` of the first
    hole (timings, counters and byte counts of the whole call)."""
    o, _keep = _opts(**kw)
    lib = load()
    n = len(sketches)
    arr = (C.c_void_p * n)(*[s.handle for s in sketches])
    outs = (C.c_void_p * n)()
    _check(lib.xp_repair_batch(arr, n, C.byref(o), outs))
    try:
        if packed:
            total = sum(s.n_holes for s in sketches)
            out = (xp_hole_summary * total)()
            got = C.c_size_t()
            _check(lib.xp_result_pack(outs, n, out, total, C.byref(got)))
            return out, xp_result_get(outs[0], 0)
        return [[xp_result_get(outs[i], h) for h in range(sketches[i].n_holes)] for i in range(n)]
    finally:
        for i in range(n):
            lib.xp_result_free(outs[i])


def xp_sketch_info_get(sketch: LoadedSketch) -> xp_sketch_info:
    out = xp_sketch_info()
    _check(load().xp_sketch_info_get(sketch.handle, C.byref(out)))
    return out


def xp_sketch_refine(sketch: LoadedSketch, max_promote: int = 0) -> int:
    """Promotes the domain points that ended whole-domain checks in earlier searches to probe
    points; returns how many were promoted."""
    n = C.c_int32()
    _check(load().xp_sketch_refine(sketch.handle, max_promote, C.byref(n)))
    return int(n.value)


def xp_repair_static(sketch: LoadedSketch, **kw) -> List[xp_hole_summary]:
    """The search of one sketch with the scratch in the library's fixed device array: for
    callers that may not allocate device memory at call time.  The summaries are ctypes
    structures owned by the caller (cand_count, match_count, solved, least_size, least_rank,
    least_text).  Keyword options as for ``xp_repair`` (``workspace`` is ignored)."""
    o, _keep = _opts(**kw)
    out = (xp_hole_summary * sketch.n_holes)()
    _check(load().xp_repair_static(sketch.handle, C.byref(o), out, sketch.n_holes))
    return list(out)


SUMMARY_DTYPE = np.dtype([("solved", "<i4"), ("max_size", "<i4"), ("least_size", "<i4"), ("pad", "<i4"),
                          ("least_rank", "<u8"), ("cand_count", "<u8", (XP_MAX_SIZE + 1,)),
                          ("match_count", "<u8", (XP_MAX_SIZE + 1,)), ("evals_executed", "<u8"), ("least_text", "S256")])


def summaries_as_numpy(packed) -> np.ndarray:
    """A structured numpy view (no copy) of an array of ``xp_hole_summary``."""
    assert C.sizeof(xp_hole_summary) == SUMMARY_DTYPE.itemsize
    return np.frombuffer(packed, dtype=SUMMARY_DTYPE)


def xp_behaviours(sketch: LoadedSketch, sig_points: Sequence[int], hole: int = 0, max_representatives: int = 0,
                  stream=None) -> xp_behaviour_summary:
    """The behaviour mode: bottom-up enumeration with observational-equivalence pruning on the given
    signature points (domain point ids).  Returns the C summary (per-size ``enumerated`` / ``distinct``,
    ``sig_matches``, the first hit and the first verified solution)."""
    d = xp_behaviour_desc()
    pts = (C.c_int64 * len(sig_points))(*[int(p) for p in sig_points])
    d.hole, d.n_sig, d.sig_points, d.max_representatives = hole, len(sig_points), pts, max_representatives
    o, _keep = _opts(stream=stream)
    out = xp_behaviour_summary()
    _check(load().xp_behaviours(sketch.handle, C.byref(d), C.byref(o), C.byref(out)))
    return out


@dataclass
class JointResult:
    solved: bool
    cand_count: List[int]          # index = total size of the pair
    match_count: List[int]
    least_total: int
    least_size0: int
    least_rank0: int
    least_rank1: int
    least_text0: str
    least_text1: str
    evals_executed: int
    probe_survivors: int
    kernel_ms: float
    total_ms: float
    n_launches: int


def xp_repair_joint(sketch: LoadedSketch, joint, stream=None) -> JointResult:
    """``joint``: an ``xp_instances.JointHole`` (two parts inside one constraint) searched over the
    domain and grammar of ``sketch``."""
    lib = load()
    d = xp_joint_desc()
    d.start_nt[0], d.start_nt[1] = joint.start_nt
    d.max_size[0], d.max_size[1] = joint.max_size
    ctx = _code(joint.ctx)
    d.ctx_len, d.ctx = len(joint.ctx), ctx
    keep = [ctx]
    if joint.spec_table is not None:
        table = joint.spec_table
        if isinstance(table, np.ndarray):
            table = np.ascontiguousarray(table, dtype=np.int64)
        d.spec_kind = 1
        d.spec_table, d.spec_table_on_device, k = _ptr_of(table)
        keep.append(k)
    else:
        se = _code(joint.spec_expr); keep.append(se)
        d.spec_kind, d.spec_len, d.spec_expr = 0, len(joint.spec_expr), se
    o, _keep = _opts(stream=stream)
    out = C.c_void_p()
    _check(lib.xp_repair_joint(sketch.handle, C.byref(d), C.byref(o), C.byref(out)))
    try:
        v = xp_joint_view()
        _check(lib.xp_joint_result_get(out.value, C.byref(v)))
        K = v.max_total
        return JointResult(bool(v.solved), [int(v.cand_count[k]) for k in range(K + 1)], [int(v.match_count[k]) for k in range(K + 1)],
                           int(v.least_total), int(v.least_size[0]), int(v.least_rank[0]), int(v.least_rank[1]),
                           (v.least_text[0] or b"").decode(), (v.least_text[1] or b"").decode(), int(v.evals_executed),
                           int(v.probe_survivors), float(v.kernel_ms), float(v.total_ms), int(v.n_launches))
    finally:
        lib.xp_joint_result_free(out.value)


@dataclass
class PairResult:
    solved: bool
    n_sketches: int
    node_first: int
    node_last: int
    least_size: int
    least_rank: int
    hole_text: str
    sketch_text: str
    stitched_text: str
    stitched_code: List[Tuple[int, int, int]]
    candidates: int
    evals_executed: int
    load_ms: float
    search_ms: float


def xp_repair_pair(gr: Grammar, source, erroneous, start_nt: int, max_size: int, var_map=None, n_source_vars=None) -> PairResult:
    """``source`` / ``erroneous``: postfix instruction lists; ``var_map``: per source variable its value
    as a postfix list over the grammar's variables (None: the snippets share their variables)."""
    lib = load()
    d = xp_pair_desc()
    src, err = _code(source), _code(erroneous)
    d.source, d.source_len, d.erroneous, d.erroneous_len = src, len(source), err, len(erroneous)
    d.start_nt, d.max_size = start_nt, max_size
    keep = []
    if var_map is not None:
        arrs = [_code(m) for m in var_map]
        keep.append(arrs)
        ptrs = (C.POINTER(xp_instr) * len(var_map))(*[C.cast(a, C.POINTER(xp_instr)) for a in arrs])
        lens = (C.c_int32 * len(var_map))(*[len(m) for m in var_map])
        d.var_map, d.var_map_len, d.n_source_vars = ptrs, lens, len(var_map)
        keep += [ptrs, lens]
    else:
        d.n_source_vars = n_source_vars if n_source_vars is not None else len(gr.model.variables)
    out = C.c_void_p()
    _check(lib.xp_repair_pair(gr.handle, C.byref(d), C.byref(out)))
    try:
        v = xp_pair_view()
        _check(lib.xp_pair_result_get(out.value, C.byref(v)))
        return PairResult(bool(v.solved), int(v.n_sketches), int(v.node_first), int(v.node_last), int(v.least_size),
                          int(v.least_rank), (v.hole_text or b"").decode(), (v.sketch_text or b"").decode(),
                          (v.stitched_text or b"").decode(),
                          [(v.stitched_code[i].kind, v.stitched_code[i].arg, v.stitched_code[i].value) for i in range(v.stitched_len)],
                          int(v.candidates), int(v.evals_executed), float(v.load_ms), float(v.search_ms))
    finally:
        lib.xp_pair_result_free(out.value)


def xp_int32_peak() -> Tuple[float, float]:
    out = (C.c_double * 2)()
    _check(load().xp_int32_peak(out, None))
    return float(out[0]), float(out[1])


def xp_int_div_rate() -> Tuple[float, float]:
    """(int64 general divisions per second, int32 reciprocal divisions by a constant per second)."""
    out = (C.c_double * 2)()
    _check(load().xp_int_div_rate(out))
    return float(out[0]), float(out[1])
