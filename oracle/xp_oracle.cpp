// CPU ORACLE -- TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, single-threaded statement of what the repair search computes.
// Only the tests, the smoke check and the CPU-baseline leg of the benchmark may
// build or call this file; the product path never does, and it shares no code
// with the CUDA library.
//
// What it computes (Section 4.4, Algorithm 3: the CreateSMTQuery / SynthesisCode
// steps).  The paper enumerates one constraint per concrete index of the snippet
// and asks a solver to fill the sketch's missing expressions so that all of them
// hold.  Here that question is answered by its definition over a bounded grammar:
//
//   for every size k = 1..K and every derivation tree e of the start symbol with
//   exactly k nodes, taken in canonical order,
//       match(e)  <=>  for every domain point p:
//                      e(p) is defined, ctx(e(p), p) is defined and equals spec(p)
//   cand_count[k]  = number of trees of size k
//   match_count[k] = number of matching trees of size k
//   least          = the matching tree with the smallest (size, rank)
//
// Readings the paper leaves open (it prints no grammar, order or arithmetic):
//   * size = number of tree nodes (each leaf 1, each operator 1);
//   * canonical order within (nonterminal, size): by production in the order the
//     grammar lists them; for a binary production by left size ascending, then
//     left subtree rank, then right subtree rank (fastest); a size-1 tree's rank
//     is the position of its leaf production among the nonterminal's leaves;
//   * values are int64 with wrap-around; '/' truncates toward zero, '%' takes the
//     dividend's sign; INT64_MIN / -1 = INT64_MIN and INT64_MIN % -1 = 0;
//   * a zero divisor anywhere in a tree (or in the context, or in the spec) at a
//     point makes the candidate fail at that point, with no short-circuiting;
//   * comparison and logic operators (context / spec only) yield 0 or 1 and
//     evaluate both operands;
//   * a grammar may also use min and max as binary operators (printed min(a,b)):
//     the remainder-tile bounds of a split loop need them;
//   * and the shifts << and >> (strength-reduced index arithmetic): the count must lie in
//     0..63, anything else makes the candidate fail at that point like a zero divisor;
//     << wraps, >> keeps the sign;
//   * a joint sketch has two holes inside ONE constraint (xo_repair_joint): the candidates
//     are the pairs of trees, ordered by total size, then the size of the first tree, then
//     its rank, then the second tree's rank; counts are per total size;
//   * the behaviour mode (xo_behaviours) enumerates bottom-up with observational-equivalence
//     pruning on a given list of signature points: a tree's signature is its value at every
//     signature point; per nonterminal and size, the candidates are the leaves (size 1) and, for
//     each binary production in order, each left size ascending, the pairs (left representative,
//     right representative) in the order the representatives were found, right fastest; a
//     candidate undefined at a signature point is dropped; one whose signature a representative
//     of the same nonterminal already has (smaller size, or earlier at this size) is dropped;
//     the others become the representatives of this size, in that order.
//
// Parity against the paper itself is unpinned: it prints no instance, query or
// solution for this step (its constraint figure is not available).  The functions
// below are pinned by the tests against closed-form counts, hand-derived match
// sets, a separate brute force over materialised trees, and invariants.

#include <cstdint>
#include <cstdio>
#include <cstring>
#include <functional>
#include <map>
#include <memory>
#include <string>
#include <vector>

typedef uint64_t u64;
typedef int64_t i64;

enum { XO_MAX_SIZE = 15 };
enum { OP_ADD = 0, OP_SUB, OP_MUL, OP_DIV, OP_MOD, OP_LT, OP_LE, OP_EQ, OP_NE, OP_MIN, OP_MAX, OP_AND, OP_OR, OP_SHL, OP_SHR, OP_COUNT };
enum { K_VAR = 0, K_CONST = 1, K_HOLE = 2, K_OP = 3 };
enum { P_VAR = 0, P_CONST = 1, P_BIN = 2 };

extern "C" {

struct xo_prod { int32_t lhs, kind, var, op, left, right; i64 value; };
struct xo_instr { int32_t kind, arg; i64 value; };

struct xo_grammar {
    int32_t n_vars;
    const i64* lo;                 // inclusive lower bounds
    const i64* hi;                 // exclusive upper bounds
    const char* const* var_names;
    int32_t n_nt;
    int32_t n_prods;
    const xo_prod* prods;
};

struct xo_problem {
    xo_grammar g;
    i64 n_points;
    const int32_t* coords;         // null: the full box of the variable ranges, first variable slowest
    i64 n_first;                   // optional: point indices checked before the rest (any order is allowed:
    const i64* first_points;       //   mismatch and invalidity are not told apart, so the order is free)
    int32_t start_nt, max_size;
    int32_t ctx_len;  const xo_instr* ctx;         // 0 = identity
    int32_t spec_len; const xo_instr* spec_expr;   // used when spec_table is null
    const i64* spec_table;                          // n_points values
    const u64* rank_begin;         // optional windows per size [max_size+1]; null = everything
    const u64* rank_end;
};

struct xo_result {
    u64 cand_count[XO_MAX_SIZE + 1];
    u64 match_count[XO_MAX_SIZE + 1];
    int32_t solved, least_size;
    u64 least_rank;
    u64 evals;                     // candidate-point evaluations carried out
    char least_text[1024];
};

// Two holes in one constraint.  HOLE instructions of ctx carry the part (0 or 1) in arg.
struct xo_joint_problem {
    xo_grammar g;
    i64 n_points;
    const int32_t* coords;
    int32_t start_nt[2], max_size[2];
    int32_t ctx_len;  const xo_instr* ctx;         // must mention both parts
    int32_t spec_len; const xo_instr* spec_expr;
    const i64* spec_table;
};

struct xo_joint_result {
    u64 cand_count[2 * XO_MAX_SIZE + 1];           // index = total size
    u64 match_count[2 * XO_MAX_SIZE + 1];
    int32_t solved, least_total, least_size0, pad;
    u64 least_rank0, least_rank1;
    u64 evals;
    char least_text0[512], least_text1[512];
};

// Bottom-up enumeration with observational-equivalence pruning on signature points.
struct xo_behaviour_problem {
    xo_problem base;               // grammar, domain, hole (start_nt, max_size, ctx, spec); rank windows unused
    i64 n_sig;                     // signature points: indices into the domain, in this order
    const i64* sig_points;
};

struct xo_behaviour_result {
    u64 enumerated[XO_MAX_SIZE + 1];   // candidates generated for the start nonterminal, per size
    u64 distinct[XO_MAX_SIZE + 1];     // of them, new behaviours (representatives)
    u64 sig_matches;                   // representatives (all sizes) that satisfy the constraint at every signature point
    int32_t hit, hit_size;             // the first of them in (size, order found) ...
    u64 hit_index;                     // ... its position among the representatives of its size
    int32_t hit_verified;              // ... and whether it satisfies the constraint on the whole domain
    int32_t solved, solution_size;     // the first of them that does
    u64 solution_index;
    char hit_text[1024], solution_text[1024];
};

}  // extern "C"

namespace {

// ---- arithmetic (C semantics on int64, zero divisors reported) ---------------

bool apply_op(int op, i64 a, i64 b, i64& out) {
    switch (op) {
        case OP_ADD: out = (i64)((u64)a + (u64)b); return true;
        case OP_SUB: out = (i64)((u64)a - (u64)b); return true;
        case OP_MUL: out = (i64)((u64)a * (u64)b); return true;
        case OP_DIV:
            if (b == 0) return false;
            out = (b == -1) ? (i64)(0 - (u64)a) : a / b;
            return true;
        case OP_MOD:
            if (b == 0) return false;
            out = (b == -1) ? 0 : a % b;
            return true;
        case OP_LT: out = a < b; return true;
        case OP_LE: out = a <= b; return true;
        case OP_EQ: out = a == b; return true;
        case OP_NE: out = a != b; return true;
        case OP_MIN: out = a < b ? a : b; return true;
        case OP_MAX: out = a > b ? a : b; return true;
        case OP_AND: out = (a != 0) && (b != 0); return true;
        case OP_OR: out = (a != 0) || (b != 0); return true;
        case OP_SHL:
            if (b < 0 || b > 63) return false;
            out = (i64)((u64)a << b);
            return true;
        case OP_SHR:
            if (b < 0 || b > 63) return false;
            out = a < 0 ? ~(~a >> b) : a >> b;           // sign-propagating, written without relying on the compiler's choice
            return true;
    }
    return false;
}

const char* const OP_TEXT[OP_COUNT] = {"+", "-", "*", "/", "%", "<", "<=", "==", "!=", "min", "max", "&&", "||", "<<", ">>"};

// Postfix evaluation of a context or spec expression at one point.  `holes`: the value of the
// hole (a joint sketch: of its parts; a HOLE instruction's arg says which).
bool eval_code(const xo_instr* code, int n, const i64* pt, const i64* holes, i64& out) {
    i64 st[64];
    int sp = 0;
    for (int i = 0; i < n; ++i) {
        const xo_instr& c = code[i];
        if (c.kind == K_VAR) st[sp++] = pt[c.arg];
        else if (c.kind == K_CONST) st[sp++] = c.value;
        else if (c.kind == K_HOLE) st[sp++] = holes[c.arg];
        else {
            i64 b = st[--sp], a = st[--sp], r;
            if (!apply_op(c.arg, a, b, r)) return false;
            st[sp++] = r;
        }
        if (sp >= 63) return false;
    }
    if (sp != 1) return false;
    out = st[0];
    return true;
}

// ---- grammar, counts -------------------------------------------------------------

struct Node { const xo_prod* p; Node* l; Node* r; };

struct Gram {
    const xo_grammar* g;
    std::vector<std::vector<const xo_prod*>> of;          // productions per nonterminal, in order
    std::vector<std::vector<u64>> cnt;                     // cnt[nt][size]
    bool overflow = false;

    Gram(const xo_grammar* g_, int max_size) : g(g_) {
        of.resize(g->n_nt);
        for (int i = 0; i < g->n_prods; ++i) of[g->prods[i].lhs].push_back(&g->prods[i]);
        cnt.assign(g->n_nt, std::vector<u64>(max_size + 1, 0));
        for (int s = 1; s <= max_size; ++s)
            for (int nt = 0; nt < g->n_nt; ++nt) {
                unsigned __int128 c = 0;
                for (const xo_prod* p : of[nt]) {
                    if (p->kind != P_BIN) { if (s == 1) c += 1; }
                    else for (int a = 1; a <= s - 2; ++a)
                        c += (unsigned __int128)cnt[p->left][a] * cnt[p->right][s - 1 - a];
                    if (c >> 63) { overflow = true; c = 0; }
                }
                cnt[nt][s] = (u64)c;
            }
    }
};

typedef std::function<void()> Fn;

// Calls k() once for every tree of (nt, size) whose rank lies in [lo, hi), in
// canonical order, with `out` pointing at the tree.
void gen(const Gram& G, int nt, int size, u64 lo, u64 hi, Node*& out, const Fn& k) {
    u64 base = 0;
    for (const xo_prod* p : G.of[nt]) {
        if (p->kind != P_BIN) {
            if (size == 1) {
                if (base >= lo && base < hi) { Node n{p, nullptr, nullptr}; out = &n; k(); }
                ++base;
            }
            continue;
        }
        for (int a = 1; a <= size - 2; ++a) {
            const int b = size - 1 - a;
            const u64 cl = G.cnt[p->left][a], cr = G.cnt[p->right][b];
            const u64 block = cl * cr;
            if (block == 0) continue;
            if (base + block <= lo || base >= hi) { base += block; continue; }
            const u64 wlo = lo > base ? lo - base : 0;                     // window inside this block
            const u64 whi = (hi - base < block) ? hi - base : block;
            Node n{p, nullptr, nullptr};
            out = &n;
            u64 l = wlo / cr;                                              // rank of the current left subtree
            gen(G, p->left, a, wlo / cr, (whi + cr - 1) / cr, n.l, [&]() {
                const u64 row = l * cr;
                const u64 rlo = wlo > row ? wlo - row : 0;
                const u64 rhi = (whi - row < cr) ? whi - row : cr;
                gen(G, p->right, b, rlo, rhi, n.r, [&]() { out = &n; k(); });
                ++l;
            });
            base += block;
        }
    }
}

bool eval_tree(const Node* n, const i64* pt, i64& out) {
    if (n->p->kind == P_VAR) { out = pt[n->p->var]; return true; }
    if (n->p->kind == P_CONST) { out = n->p->value; return true; }
    i64 a, b;
    const bool va = eval_tree(n->l, pt, a);
    const bool vb = eval_tree(n->r, pt, b);
    if (!va || !vb) return false;
    return apply_op(n->p->op, a, b, out);
}

void tree_text(const xo_grammar* g, const Node* n, std::string& s) {
    if (n->p->kind == P_VAR) { s += g->var_names ? g->var_names[n->p->var] : ("v" + std::to_string(n->p->var)); return; }
    if (n->p->kind == P_CONST) { s += std::to_string((long long)n->p->value); return; }
    if (n->p->op == OP_MIN || n->p->op == OP_MAX) {
        s += OP_TEXT[n->p->op]; s += "("; tree_text(g, n->l, s); s += ","; tree_text(g, n->r, s); s += ")";
        return;
    }
    s += "("; tree_text(g, n->l, s); s += OP_TEXT[n->p->op]; tree_text(g, n->r, s); s += ")";
}

}  // namespace

extern "C" {

// Number of derivation trees per size for nonterminal nt; returns 1 if a count reaches 2^63.
int xo_counts(const xo_grammar* g, int nt, int max_size, u64* out) {
    Gram G(g, max_size);
    for (int s = 0; s <= max_size; ++s) out[s] = G.cnt[nt][s];
    return G.overflow ? 1 : 0;
}

// Texts of the trees of (nt, size) with rank in [begin, end), one per line.
// Returns the number of bytes needed (including the final NUL).
i64 xo_list(const xo_grammar* g, int nt, int size, u64 begin, u64 end, char* buf, i64 buflen) {
    Gram G(g, size);
    std::string all;
    Node* root = nullptr;
    if (end > G.cnt[nt][size]) end = G.cnt[nt][size];
    gen(G, nt, size, begin, end, root, [&]() { tree_text(g, root, all); all += "\n"; });
    if ((i64)all.size() + 1 <= buflen) memcpy(buf, all.c_str(), all.size() + 1);
    return (i64)all.size() + 1;
}

// Value of a postfix expression at one point (returns 0 when a divisor is zero).
int xo_eval_code(const xo_instr* code, int n, const i64* pt, i64 hole, i64* out) {
    return eval_code(code, n, pt, &hole, *out) ? 1 : 0;
}

// The repair search for one hole.  Returns 0, or 1 on a malformed problem.
int xo_repair(const xo_problem* P, xo_result* R) {
    memset(R, 0, sizeof(*R));
    const xo_grammar* g = &P->g;
    const int K = P->max_size;
    if (K < 1 || K > XO_MAX_SIZE || g->n_vars > 16) return 1;
    Gram G(g, K);
    if (G.overflow) return 1;
    const int nv = g->n_vars;
    const i64 np = P->n_points;

    // Every domain point and the spec's value there.
    std::vector<i64> pts((size_t)np * (nv ? nv : 1));
    for (i64 p = 0; p < np; ++p) {
        if (P->coords) for (int d = 0; d < nv; ++d) pts[p * nv + d] = P->coords[p * nv + d];
        else {
            i64 rem = p;
            for (int d = nv - 1; d >= 0; --d) {
                const i64 ext = g->hi[d] - g->lo[d];
                pts[p * nv + d] = g->lo[d] + rem % ext;
                rem /= ext;
            }
        }
    }
    std::vector<i64> spec(np);
    std::vector<char> spec_ok(np, 1);
    for (i64 p = 0; p < np; ++p) {
        if (P->spec_table) spec[p] = P->spec_table[p];
        else { const i64 none = 0; spec_ok[p] = eval_code(P->spec_expr, P->spec_len, &pts[p * nv], &none, spec[p]); }
    }
    // Order in which points are tried: the caller's "first" points, then all of them.
    std::vector<i64> order;
    for (i64 i = 0; i < P->n_first; ++i) order.push_back(P->first_points[i]);
    for (i64 p = 0; p < np; ++p) order.push_back(p);

    for (int k = 1; k <= K; ++k) {
        R->cand_count[k] = G.cnt[P->start_nt][k];
        u64 lo = 0, hi = R->cand_count[k];
        if (P->rank_begin) {
            lo = P->rank_begin[k];
            if (P->rank_end[k] < hi) hi = P->rank_end[k];
        }
        if (lo >= hi) continue;
        Node* root = nullptr;
        u64 rank = lo;
        gen(G, P->start_nt, k, lo, hi, root, [&]() {
            bool ok = true;
            for (i64 p : order) {
                ++R->evals;
                const i64* pt = &pts[p * nv];
                i64 h, v;
                ok = spec_ok[p] && eval_tree(root, pt, h);
                if (ok) {
                    if (P->ctx_len == 0) v = h;
                    else ok = eval_code(P->ctx, P->ctx_len, pt, &h, v);
                }
                ok = ok && v == spec[p];
                if (!ok) break;
            }
            if (ok) {
                ++R->match_count[k];
                if (!R->solved) {
                    R->solved = 1; R->least_size = k; R->least_rank = rank;
                    std::string s; tree_text(g, root, s);
                    snprintf(R->least_text, sizeof(R->least_text), "%s", s.c_str());
                }
            }
            ++rank;
        });
    }
    return 0;
}

// The repair search for a joint sketch: every pair (tree of part 0, tree of part 1), by total
// size, then size of part 0, then rank of part 0, then rank of part 1.  Returns 0, or 1 on a
// malformed problem.
int xo_repair_joint(const xo_joint_problem* P, xo_joint_result* R) {
    memset(R, 0, sizeof(*R));
    const xo_grammar* g = &P->g;
    const int K0 = P->max_size[0], K1 = P->max_size[1];
    if (K0 < 1 || K0 > XO_MAX_SIZE || K1 < 1 || K1 > XO_MAX_SIZE || g->n_vars > 16 || P->ctx_len < 1) return 1;
    Gram G(g, K0 > K1 ? K0 : K1);
    if (G.overflow) return 1;
    const int nv = g->n_vars;
    const i64 np = P->n_points;
    std::vector<i64> pts((size_t)np * (nv ? nv : 1));
    for (i64 p = 0; p < np; ++p) {
        if (P->coords) for (int d = 0; d < nv; ++d) pts[p * nv + d] = P->coords[p * nv + d];
        else {
            i64 rem = p;
            for (int d = nv - 1; d >= 0; --d) {
                const i64 ext = g->hi[d] - g->lo[d];
                pts[p * nv + d] = g->lo[d] + rem % ext;
                rem /= ext;
            }
        }
    }
    std::vector<i64> spec(np);
    std::vector<char> spec_ok(np, 1);
    const i64 none[2] = {0, 0};
    for (i64 p = 0; p < np; ++p) {
        if (P->spec_table) spec[p] = P->spec_table[p];
        else spec_ok[p] = eval_code(P->spec_expr, P->spec_len, &pts[p * nv], none, spec[p]);
    }
    for (int s = 2; s <= K0 + K1; ++s) {
        for (int s0 = 1; s0 < s; ++s0) {
            const int s1 = s - s0;
            if (s0 > K0 || s1 > K1) continue;
            const u64 c0 = G.cnt[P->start_nt[0]][s0], c1 = G.cnt[P->start_nt[1]][s1];
            const unsigned __int128 prod = (unsigned __int128)c0 * c1;
            if ((prod >> 63) || R->cand_count[s] + (u64)prod < R->cand_count[s]) return 1;
            R->cand_count[s] += (u64)prod;
            Node* t0 = nullptr;
            u64 r0 = 0;
            gen(G, P->start_nt[0], s0, 0, c0, t0, [&]() {
                Node* t1 = nullptr;
                u64 r1 = 0;
                gen(G, P->start_nt[1], s1, 0, c1, t1, [&]() {
                    bool ok = true;
                    for (i64 p = 0; p < np && ok; ++p) {
                        ++R->evals;
                        const i64* pt = &pts[p * nv];
                        i64 h[2], v;
                        const bool d0 = eval_tree(t0, pt, h[0]);
                        const bool d1 = eval_tree(t1, pt, h[1]);
                        ok = spec_ok[p] && d0 && d1 && eval_code(P->ctx, P->ctx_len, pt, h, v) && v == spec[p];
                    }
                    if (ok) {
                        ++R->match_count[s];
                        if (!R->solved) {
                            R->solved = 1; R->least_total = s; R->least_size0 = s0; R->least_rank0 = r0; R->least_rank1 = r1;
                            std::string a, b; tree_text(g, t0, a); tree_text(g, t1, b);
                            snprintf(R->least_text0, sizeof(R->least_text0), "%s", a.c_str());
                            snprintf(R->least_text1, sizeof(R->least_text1), "%s", b.c_str());
                        }
                    }
                    ++r1;
                });
                ++r0;
            });
        }
    }
    return 0;
}

// The behaviour mode.  Returns 0, or 1 on a malformed problem.
int xo_behaviours(const xo_behaviour_problem* B, xo_behaviour_result* R) {
    memset(R, 0, sizeof(*R));
    const xo_problem* P = &B->base;
    const xo_grammar* g = &P->g;
    const int K = P->max_size, nv = g->n_vars;
    const i64 np = P->n_points, ns = B->n_sig;
    if (K < 1 || K > XO_MAX_SIZE || nv > 16 || ns < 0) return 1;
    auto coords_of = [&](i64 p, i64* pt) {
        if (P->coords) { for (int d = 0; d < nv; ++d) pt[d] = P->coords[p * nv + d]; return; }
        i64 rem = p;
        for (int d = nv - 1; d >= 0; --d) { const i64 ext = g->hi[d] - g->lo[d]; pt[d] = g->lo[d] + rem % ext; rem /= ext; }
    };
    auto spec_at = [&](i64 p, const i64* pt, i64& v) {
        if (P->spec_table) { v = P->spec_table[p]; return true; }
        const i64 none = 0;
        return eval_code(P->spec_expr, P->spec_len, pt, &none, v);
    };
    std::vector<i64> sig_pt((size_t)ns * (nv ? nv : 1)), sig_spec(ns);
    std::vector<char> sig_ok(ns, 1);
    for (i64 j = 0; j < ns; ++j) {
        if (B->sig_points[j] < 0 || B->sig_points[j] >= np) return 1;
        coords_of(B->sig_points[j], &sig_pt[j * nv]);
        sig_ok[j] = spec_at(B->sig_points[j], &sig_pt[j * nv], sig_spec[j]);
    }
    std::vector<std::vector<const xo_prod*>> of(g->n_nt);
    for (int i = 0; i < g->n_prods; ++i) of[g->prods[i].lhs].push_back(&g->prods[i]);
    struct Rep { std::vector<i64> sig; const xo_prod* p; int a; u64 l, r; };
    std::vector<std::vector<std::vector<Rep>>> reps(g->n_nt, std::vector<std::vector<Rep>>(K + 1));
    std::vector<std::map<std::vector<i64>, int>> seen(g->n_nt);
    std::function<void(int, int, u64, std::string&)> text = [&](int nt, int size, u64 idx, std::string& out) {
        const Rep& t = reps[nt][size][idx];
        if (t.p->kind == P_VAR) { out += g->var_names ? g->var_names[t.p->var] : ("v" + std::to_string(t.p->var)); return; }
        if (t.p->kind == P_CONST) { out += std::to_string((long long)t.p->value); return; }
        const bool call = t.p->op == OP_MIN || t.p->op == OP_MAX;
        out += call ? std::string(OP_TEXT[t.p->op]) + "(" : std::string("(");
        text(t.p->left, t.a, t.l, out);
        out += call ? "," : OP_TEXT[t.p->op];
        text(t.p->right, size - 1 - t.a, t.r, out);
        out += ")";
    };
    std::function<bool(int, int, u64, const i64*, i64&)> value = [&](int nt, int size, u64 idx, const i64* pt, i64& out) {
        const Rep& t = reps[nt][size][idx];
        if (t.p->kind == P_VAR) { out = pt[t.p->var]; return true; }
        if (t.p->kind == P_CONST) { out = t.p->value; return true; }
        i64 a, b;
        const bool va = value(t.p->left, t.a, t.l, pt, a), vb = value(t.p->right, size - 1 - t.a, t.r, pt, b);
        return va && vb && apply_op(t.p->op, a, b, out);
    };
    for (int s = 1; s <= K; ++s)
        for (int nt = 0; nt < g->n_nt; ++nt) {
            u64 enumerated = 0;
            auto offer = [&](Rep&& c, bool defined) {
                ++enumerated;
                if (!defined) return;
                if (seen[nt].count(c.sig)) return;
                seen[nt][c.sig] = 1;
                reps[nt][s].push_back(std::move(c));
            };
            for (const xo_prod* p : of[nt]) {
                if (p->kind != P_BIN) {
                    if (s != 1) continue;
                    Rep c{std::vector<i64>(ns), p, 0, 0, 0};
                    for (i64 j = 0; j < ns; ++j) c.sig[j] = p->kind == P_VAR ? sig_pt[j * nv + p->var] : p->value;
                    offer(std::move(c), true);
                    continue;
                }
                for (int a = 1; a <= s - 2; ++a) {
                    const auto& L = reps[p->left][a];
                    const auto& Rr = reps[p->right][s - 1 - a];
                    for (u64 l = 0; l < L.size(); ++l)
                        for (u64 r = 0; r < Rr.size(); ++r) {
                            Rep c{std::vector<i64>(ns), p, a, l, r};
                            bool defined = true;
                            for (i64 j = 0; j < ns && defined; ++j) defined = apply_op(p->op, L[l].sig[j], Rr[r].sig[j], c.sig[j]);
                            offer(std::move(c), defined);
                        }
                }
            }
            if (nt == P->start_nt) { R->enumerated[s] = enumerated; R->distinct[s] = reps[nt][s].size(); }
        }
    // representatives of the start nonterminal against the constraint
    for (int s = 1; s <= K; ++s)
        for (u64 i = 0; i < reps[P->start_nt][s].size(); ++i) {
            const Rep& t = reps[P->start_nt][s][i];
            bool ok = true;
            for (i64 j = 0; j < ns && ok; ++j) {
                i64 v = t.sig[j];
                ok = sig_ok[j] && (P->ctx_len == 0 || eval_code(P->ctx, P->ctx_len, &sig_pt[j * nv], &t.sig[j], v)) && v == sig_spec[j];
            }
            if (!ok) continue;
            ++R->sig_matches;
            if (R->solved) continue;
            bool all = true;
            for (i64 p = 0; p < np && all; ++p) {
                i64 pt[16], want, h, v;
                coords_of(p, pt);
                all = spec_at(p, pt, want) && value(P->start_nt, s, i, pt, h);
                if (all) { v = h; all = (P->ctx_len == 0 || eval_code(P->ctx, P->ctx_len, pt, &h, v)) && v == want; }
            }
            std::string txt;
            text(P->start_nt, s, i, txt);
            if (!R->hit) {
                R->hit = 1; R->hit_size = s; R->hit_index = i; R->hit_verified = all ? 1 : 0;
                snprintf(R->hit_text, sizeof(R->hit_text), "%s", txt.c_str());
            }
            if (all) {
                R->solved = 1; R->solution_size = s; R->solution_index = i;
                snprintf(R->solution_text, sizeof(R->solution_text), "%s", txt.c_str());
            }
        }
    return 0;
}

}  // extern "C"
