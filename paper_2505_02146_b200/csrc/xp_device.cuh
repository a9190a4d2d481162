// Device-side building blocks: int64 C-semantics arithmetic, combinatorial unranking of a
// candidate into postfix code, and the postfix interpreters.
#pragma once

#include "xp_dev.h"

namespace xp {

// Index checks of the checked build (-DXP_CHECKS; the stand-in for a memory checker on tiny
// cases): XP_CHECKED(cond, code) is `true` and costs nothing in the normal build; in the checked
// build a false condition is recorded (the first code wins) and the caller takes a safe value
// instead of the bad index.  Nothing traps, spins or faults: the search finishes, and the host
// turns a recorded code into an error status.
#ifdef XP_CHECKS
static __device__ unsigned int g_check_word;      // (one per source file; the search kernels' copy is the one the host reads)
__device__ __forceinline__ bool xp_checked(bool cond, unsigned int code) {
    if (!cond) atomicCAS(&g_check_word, 0u, code);
    return cond;
}
#define XP_CHECKED(cond, code) xp_checked((cond), (code))
#else
#define XP_CHECKED(cond, code) true
#endif
enum { kChkRank = 1, kChkTable = 2, kChkQueue = 3, kChkStack = 4, kChkPoint = 5, kChkSlot = 6, kChkSegment = 7 };

// One binary operation in int64 C semantics with wrap-around.  Returns false when the
// divisor is zero (the candidate is then invalid at this point).  INT64_MIN / -1 wraps to
// INT64_MIN and INT64_MIN % -1 is 0; the trapping machine division is never issued.
__device__ __forceinline__ bool apply_op(int op, i64 a, i64 b, i64& r) {
    switch (op) {
        case XP_OP_ADD: r = (i64)((u64)a + (u64)b); return true;
        case XP_OP_SUB: r = (i64)((u64)a - (u64)b); return true;
        case XP_OP_MUL: r = (i64)((u64)a * (u64)b); return true;
        case XP_OP_DIV:
        case XP_OP_MOD: {
            if (b == 0) return false;
            i64 q;
            if (b == -1) q = (i64)(0ull - (u64)a);
            else if (a == (i64)(i32)a && b == (i64)(i32)b) q = (i64)((i32)a / (i32)b);   // both fit 32 bits, b != -1
            else q = a / b;
            r = (op == XP_OP_DIV) ? q : (i64)((u64)a - (u64)q * (u64)b);
            return true;
        }
        case XP_OP_LT: r = a < b; return true;
        case XP_OP_LE: r = a <= b; return true;
        case XP_OP_EQ: r = a == b; return true;
        case XP_OP_NE: r = a != b; return true;
        case XP_OP_MIN: r = a < b ? a : b; return true;
        case XP_OP_MAX: r = a > b ? a : b; return true;
        case XP_OP_AND: r = (a != 0) & (b != 0); return true;
        case XP_OP_OR: r = (a != 0) | (b != 0); return true;
        case XP_OP_SHL: r = (i64)((u64)a << (b & 63)); return b >= 0 && b <= 63;
        case XP_OP_SHR: r = a >> (b & 63); return b >= 0 && b <= 63;      // (device >> on a signed value keeps the sign)
    }
    return false;
}

__device__ __forceinline__ void divmod_u64(u64 n, u64 d, u64& q, u64& r) {
    if (((n | d) >> 32) == 0) { u32 qq = (u32)n / (u32)d; q = qq; r = (u32)n - qq * (u32)d; }
    else { q = n / d; r = n - q * d; }
}

// rank -> postfix code of the tree of (nt, size) with that rank in canonical order.
// code[i] is a leaf index into GrammarDev::leaves, or kOpBit | operator.  Returns the length
// (== size).  Walks the tree with an explicit stack: a frame is a subtree still to be
// expanded, or (size 0) an operator to be emitted after its operands.
static __device__ __noinline__ int unrank(const GrammarDev* __restrict__ g, int nt, int size, u64 rank, u32* code) {
    struct Frame { u64 rank; i32 nt; i32 size; };
    Frame st[kMaxSize + 1];
    int sp = 0, n = 0;
    if (!XP_CHECKED(size >= 1 && size <= kMaxSize && rank < g->cnt[nt][size], kChkRank)) { rank = 0; size = 1; }
    st[sp++] = Frame{rank, nt, size};
    while (sp > 0) {
        const Frame f = st[--sp];
        if (f.size == 0) { code[n++] = kOpBit | (u32)f.nt; continue; }
        if (f.size == 1) { code[n++] = (u32)(g->leaf_begin[f.nt] + (i32)f.rank); continue; }
        int p = g->bin_begin[f.nt];
        const int pe = g->bin_begin[f.nt + 1];
        while (p + 1 < pe && g->bins[p + 1].off[f.size] <= f.rank) ++p;
        const BinDev* bp = &g->bins[p];
        u64 rem = f.rank - bp->off[f.size];
        const int lnt = bp->lnt, rnt = bp->rnt;
        int a = 1;
        u64 cr;
        for (;; ++a) {                                   // left size: blocks of cnt[L][a] * cnt[R][size-1-a]
            cr = g->cnt[rnt][f.size - 1 - a];
            const u64 block = g->cnt[lnt][a] * cr;
            if (rem < block || a == f.size - 2) break;
            rem -= block;
        }
        u64 l, r;
        divmod_u64(rem, cr, l, r);
        st[sp++] = Frame{0, bp->op, 0};
        st[sp++] = Frame{r, rnt, f.size - 1 - a};
        st[sp++] = Frame{l, lnt, a};
    }
    return n;
}

// One level of unranking: the root production and the operand subtrees (sizes and ranks) of
// the tree of (nt, size >= 3) with the given rank.
__device__ __forceinline__ void unrank_root(const GrammarDev* __restrict__ g, int nt, int size, u64 rank,
                                            int& op, int& lnt, int& rnt, int& a, u64& l, u64& r) {
    if (!XP_CHECKED(size >= 3 && rank < g->cnt[nt][size], kChkRank)) rank = 0;
    int p = g->bin_begin[nt];
    const int pe = g->bin_begin[nt + 1];
    while (p + 1 < pe && g->bins[p + 1].off[size] <= rank) ++p;
    const BinDev* bp = &g->bins[p];
    u64 rem = rank - bp->off[size];
    op = bp->op; lnt = bp->lnt; rnt = bp->rnt;
    u64 cr;
    for (a = 1;; ++a) {
        cr = g->cnt[rnt][size - 1 - a];
        const u64 block = g->cnt[lnt][a] * cr;
        if (rem < block || a == size - 2) break;
        rem -= block;
    }
    divmod_u64(rem, cr, l, r);
}

// Value of a candidate (postfix code over the grammar's leaves) at one point.
__device__ __forceinline__ bool eval_cand(const u32* code, int n, const LeafDev* __restrict__ leaves,
                                          const i64* pt, i64& out) {
    i64 st[kCandStack];
    int sp = 0;
    for (int i = 0; i < n; ++i) {
        const u32 w = code[i];
        if (w & kOpBit) {
            const i64 b = st[--sp];
            const i64 a = st[sp - 1];
            i64 r;
            if (!apply_op((int)(w & 0xff), a, b, r)) return false;
            st[sp - 1] = r;
        } else {
            const LeafDev lf = leaves[w];
            if (!XP_CHECKED(sp < kCandStack, kChkStack)) return false;
            st[sp++] = lf.var >= 0 ? pt[lf.var] : lf.value;
        }
    }
    out = st[0];
    return true;
}

// Value of a context or spec expression at one point; `hole` is the value of the hole.
__device__ __forceinline__ bool eval_code(const xp_instr* code, int n, const i64* pt, i64 hole, i64& out) {
    i64 st[kMaxStack];
    int sp = 0;
    for (int i = 0; i < n; ++i) {
        const xp_instr c = code[i];
        if (c.kind == XP_I_OP) {
            const i64 b = st[--sp];
            const i64 a = st[sp - 1];
            i64 r;
            if (!apply_op(c.arg, a, b, r)) return false;
            st[sp - 1] = r;
        } else {
            if (!XP_CHECKED(sp < kMaxStack, kChkStack)) return false;
            st[sp++] = c.kind == XP_I_VAR ? pt[c.arg] : (c.kind == XP_I_CONST ? c.value : hole);
        }
    }
    out = st[0];
    return true;
}

// Coordinates of domain point `pid`: a table row, or the mixed-radix digits of the id over
// the box (first variable slowest).
__device__ __forceinline__ void point_coords(const SketchDev* __restrict__ s, i64 pid, i64* pt) {
    const int nv = s->n_vars;
    if (!XP_CHECKED(pid >= 0 && pid < s->n_points, kChkPoint)) pid = 0;
    if (s->coords != nullptr) {
        const i32* row = s->coords + pid * nv;
        for (int d = 0; d < nv; ++d) pt[d] = row[d];
    } else {
        u64 rem = (u64)pid;
        for (int d = nv - 1; d >= 0; --d) {
            u64 q, r;
            divmod_u64(rem, (u64)s->ext[d], q, r);
            pt[d] = s->lo[d] + (i64)r;
            rem = q;
        }
    }
}

// Does candidate value h satisfy hole's constraint at point pt whose spec value is `want`?
__device__ __forceinline__ bool ctx_matches(const HoleDev* __restrict__ hole, const i64* pt, i64 h, i64 want) {
    i64 v = h;
    if (hole->ctx_len > 0 && !eval_code(hole->ctx, hole->ctx_len, pt, h, v)) return false;
    return v == want;
}

}  // namespace xp
