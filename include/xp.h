/* xp.h -- C ABI of libxpiler_repair: bounded-grammar repair of sketch holes on one GPU.
 *
 * The operation is the query-creation and synthesis step of the paper's symbolic code
 * repair (Section 4.4, Algorithm 3: CreateSMTQuery + SynthesisCode): a code sketch has
 * missing expressions ("holes": a buffer index, a thread binding, a loop bound); one
 * constraint is stated per concrete index of the snippet's iteration domain; the holes are
 * filled so that every constraint holds.  The paper hands the constraints to an SMT solver.
 * This library decides the same question by exhaustive enumeration of a bounded expression
 * grammar on the GPU:
 *
 *   for each hole, each size k = 1..max_size and each derivation tree e of the hole's start
 *   nonterminal with exactly k nodes (leaf = 1 node, operator = 1 node), in canonical order:
 *       e matches  <=>  at every domain point p:  e(p) is defined, ctx(e(p), p) is defined,
 *                       and ctx(e(p), p) == spec(p)
 *   cand_count[k]  = number of trees of size k          (syntactic, closed by recurrence)
 *   match_count[k] = number of matching trees of size k (restricted to the rank window, if any)
 *   least          = the matching tree with the smallest (size, rank)
 *
 * Arithmetic: int64 with wrap-around; '/' truncates toward zero; '%' takes the dividend's
 * sign; INT64_MIN / -1 = INT64_MIN and INT64_MIN % -1 = 0; a zero divisor anywhere in the
 * candidate, the context or the spec at a point makes the candidate fail there (no
 * short-circuit, also under a multiplication by zero).  Comparison / logic operators (context
 * and spec only) give 0 or 1 and evaluate both operands.
 *
 * Canonical order inside (nonterminal, size): by production, in the order the grammar lists
 * them; inside a binary production by left-subtree size ascending, then left-subtree rank,
 * then right-subtree rank (fastest).  A size-1 tree's rank is the position of its leaf
 * production among the nonterminal's leaf productions.
 *
 * General rules.  All functions return an xp_status (0 = XP_OK) and never throw or abort;
 * xp_last_error() gives a message for the calling thread's last failure.  Descriptor
 * structures and everything they point to are borrowed for the duration of the call and
 * deep-copied (exception: device-resident tables, see xp_sketch_desc).  Handles are immutable
 * after creation and owned by the caller until the matching destroy/free.  Every pointer is
 * a HOST pointer unless its comment says "device".  "No solution within the bound" is not an
 * error.  Every entry point that touches the GPU fails with XP_ERR_CUDA when no CUDA device
 * is usable: there is no CPU fallback.
 */
#ifndef XP_H_
#define XP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t xp_status;
enum {
    XP_OK = 0,
    XP_ERR_INVALID_ARG = 1,   /* null pointer, index out of range, malformed bytecode */
    XP_ERR_GRAMMAR = 2,       /* malformed grammar description */
    XP_ERR_SKETCH = 3,        /* malformed sketch description */
    XP_ERR_TOO_LARGE = 4,     /* a candidate count reaches 2^63, or a size limit of the library is exceeded */
    XP_ERR_NOMEM = 5,         /* host or device allocation failed, or the caller's workspace is too small */
    XP_ERR_CUDA = 6,          /* a CUDA call failed (message in xp_last_error) */
    XP_ERR_TIMEOUT = 7,       /* the call's time limit (xp_repair_opts.timeout_ms) ran out between launches */
    XP_ERR_CANCELLED = 8      /* the caller's cancel word became non-zero before or between launches */
};

/* Library limits. */
enum {
    XP_MAX_SIZE = 15,         /* largest candidate size (nodes) */
    XP_MAX_VARS = 8,
    XP_MAX_NONTERMINALS = 8,
    XP_MAX_CODE = 64          /* instructions in one context or spec expression */
};

/* Operators.  The first five, MIN, MAX and the shifts may appear in grammar productions (min and max
 * let a hole express the bound of a remainder tile, e.g. min(T, N - io*T); shifts are what strength-
 * reduced index arithmetic uses); all of them in context and spec expressions.  A shift count outside
 * 0..63 makes the candidate fail at the point, like a zero divisor; << wraps around, >> keeps the sign. */
enum {
    XP_OP_ADD = 0, XP_OP_SUB = 1, XP_OP_MUL = 2, XP_OP_DIV = 3, XP_OP_MOD = 4,
    XP_OP_LT = 5, XP_OP_LE = 6, XP_OP_EQ = 7, XP_OP_NE = 8, XP_OP_MIN = 9, XP_OP_MAX = 10,
    XP_OP_AND = 11, XP_OP_OR = 12, XP_OP_SHL = 13, XP_OP_SHR = 14
};

/* Variables of the snippet: name (copied) and range lo <= v < hi. */
typedef struct { const char* name; int64_t lo, hi; } xp_variable;

/* Grammar production  lhs -> variable | constant | left op right. */
enum { XP_PROD_VAR = 0, XP_PROD_CONST = 1, XP_PROD_BIN = 2 };
typedef struct {
    int32_t lhs;        /* nonterminal index, 0 <= lhs < n_nonterminals */
    int32_t kind;       /* XP_PROD_* */
    int32_t var;        /* XP_PROD_VAR: variable index */
    int32_t op;         /* XP_PROD_BIN: XP_OP_ADD .. XP_OP_MOD, XP_OP_MIN, XP_OP_MAX, XP_OP_SHL, XP_OP_SHR */
    int32_t left;       /* XP_PROD_BIN: nonterminal of the left operand */
    int32_t right;      /* XP_PROD_BIN: nonterminal of the right operand */
    int64_t value;      /* XP_PROD_CONST: the constant */
} xp_production;

typedef struct {
    int32_t n_vars;                     /* <= XP_MAX_VARS */
    const xp_variable* vars;
    int32_t n_nonterminals;             /* <= XP_MAX_NONTERMINALS */
    int32_t n_productions;
    const xp_production* productions;   /* canonical order = array order */
} xp_grammar_desc;

/* Postfix instruction of a context, spec or solution expression. */
enum { XP_I_VAR = 0, XP_I_CONST = 1, XP_I_HOLE = 2, XP_I_OP = 3 };
typedef struct {
    int32_t kind;       /* XP_I_* */
    int32_t arg;        /* XP_I_VAR: variable index; XP_I_OP: XP_OP_* */
    int64_t value;      /* XP_I_CONST: the constant */
} xp_instr;

/* One hole of the sketch: the missing expression, the fixed expression around it and what
 * the source program computes at the same iteration. */
enum { XP_SPEC_EXPR = 0, XP_SPEC_TABLE = 1 };
typedef struct {
    int32_t start_nt;           /* nonterminal the hole is filled from */
    int32_t max_size;           /* size bound K, 1 <= K <= XP_MAX_SIZE */
    int32_t ctx_len;            /* 0: identity context (the hole is the whole expression) */
    const xp_instr* ctx;        /* postfix over variables, constants and XP_I_HOLE (<= XP_MAX_CODE) */
    int32_t spec_kind;          /* XP_SPEC_EXPR or XP_SPEC_TABLE */
    int32_t spec_len;           /* XP_SPEC_EXPR: postfix over variables and constants */
    const xp_instr* spec_expr;
    const int64_t* spec_table;  /* XP_SPEC_TABLE: n_points values, point order of the domain */
    int32_t spec_table_on_device; /* non-zero: spec_table is a DEVICE pointer; it is not copied
                                     and must stay valid and unchanged until xp_sketch_destroy */
} xp_hole_desc;

/* The sketch: an iteration domain and its holes.  A loop-bound hole is stated through its
 * guard predicate on the enclosing box (context "loopvar < HOLE", spec = the source's
 * executes-here predicate, 0 or 1).  Each hole has its own spec and is searched on its own. */
enum { XP_DOMAIN_BOX = 0, XP_DOMAIN_TABLE = 1 };
typedef struct {
    int32_t domain_kind;        /* XP_DOMAIN_BOX: every point of the variable ranges, point id ->
                                   coordinates by mixed radix with the first variable slowest;
                                   XP_DOMAIN_TABLE: explicit points */
    int64_t n_points;           /* XP_DOMAIN_TABLE: number of rows (may be 0) */
    const int32_t* coords;      /* XP_DOMAIN_TABLE: int32 [n_points][n_vars], row-major */
    int32_t coords_on_device;   /* non-zero: coords is a DEVICE pointer, kept by reference (as above) */
    int32_t n_holes;
    const xp_hole_desc* holes;
} xp_sketch_desc;

/* Restricts the match search of one (hole, size) to ranks begin <= rank < end.  Counts of
 * candidates stay syntactic; match counts and the least solution refer to the window. */
typedef struct { int32_t hole; /* -1: every hole */ int32_t size; uint64_t begin, end; } xp_rank_range;

typedef struct {
    int32_t size_min, size_max;         /* 0, 0: every size 1..max_size of each hole */
    int32_t n_rank_ranges;
    const xp_rank_range* rank_ranges;
    void* stream;                       /* cudaStream_t to launch on; NULL: the default stream */
    void* workspace;                    /* DEVICE memory for the call's scratch (256-byte aligned), */
    size_t workspace_bytes;             /*   at least xp_workspace_bytes(); NULL: the library uses a block of its
                                             own that it keeps from call to call (cudaMalloc when it must grow) */
    uint32_t flags;                     /* XP_FLAG_* */
    const volatile int32_t* cancel;     /* optional host word.  When it is given (or timeout_ms is), the search runs
                                           as a series of bounded launches (at most XP_CANCEL_TICKETS work tickets,
                                           a few milliseconds, each); the host waits for each, then reads the word:
                                           non-zero ends the call with XP_ERR_CANCELLED and no result.  Nothing on
                                           the device waits for the word, and no kernel is in flight on return. */
    int64_t timeout_ms;                 /* > 0: the same series of launches, and the call ends with XP_ERR_TIMEOUT
                                           once this much wall time has passed when a launch has finished */
} xp_repair_opts;
enum { XP_CANCEL_TICKETS = 8192 };

enum {
    XP_FLAG_NO_FILTER = 1u,             /* skip the probe-point filter stage (every candidate is unranked
                                           and checked on its own); same results, for testing */
    XP_FLAG_ALWAYS_FILTER = 2u          /* use the filter stage also for rank windows too small to gain
                                           from it; same results, for testing */
};

typedef struct xp_grammar xp_grammar;
typedef struct xp_sketch xp_sketch;
typedef struct xp_result xp_result;

/* Result of one hole.  Pointers live until xp_result_free. */
typedef struct {
    int32_t solved;                 /* 1 if some candidate inside the bound (and window) matches */
    int32_t max_size;
    const uint64_t* cand_count;     /* [max_size + 1], index = size */
    const uint64_t* match_count;    /* [max_size + 1] */
    int32_t least_size;             /* valid when solved */
    uint64_t least_rank;
    const xp_instr* least_code;     /* postfix of the least solution */
    int32_t least_len;
    const char* least_text;         /* fully parenthesised infix, e.g. "(j+(i*8))", "(i<<2)"; min and max as calls, "min(a,b)" */
    uint64_t evals_executed;        /* candidate-point evaluations that ran for this hole: filter_tests plus the exact
                                       evaluations of stage 2 (a hit at a probe point) and stage 3 (a survivor at a
                                       domain point).  Candidates decided without a test are not in here. */
    uint64_t filter_survivors;      /* candidates that passed the first probe point */
    uint64_t probe_survivors;       /* candidates that passed every probe point */
    uint64_t nominal_ops;           /* 32-bit integer operations the filter stage's candidate-point evaluations
                                       that were carried out amount to under the library's cost model: one operation and one
                                       comparison per evaluation, with + - * min max = 1, a reciprocal division = 7
                                       (/ and % of one operand pair share it), a remainder's multiply-subtract = 1 */
    double kernel_ms;               /* device time of the whole call's kernels (CUDA events) */
    double total_ms;                /* host wall time of the whole call */
    int32_t n_launches;             /* kernels the call launched */
    uint64_t filter_tests;          /* filter-stage tests at the first probe point that ran: pairs of operand subtrees
                                       both defined there, times the operators whose test loop was entered */
    uint64_t candidates_skipped;    /* candidates of the operand tiles visited that were decided without a test: an
                                       operand undefined at the probe (a zero divisor inside it), a remainder whose
                                       divisor cannot exceed the target's magnitude, a quotient or remainder of 32-bit
                                       operands against a target outside 32 bits.  With a rank window the tiles also
                                       cover some ranks outside it; those count here or in filter_tests as well. */
    uint64_t h2d_bytes, d2h_bytes;  /* bytes the call copied to and from the device (the whole call, every hole) */
} xp_result_view;

/* Grammar (Section 4.4: the expressions the synthesis step may put into a hole).  Builds the
 * per-(nonterminal, size) candidate counts and rank offsets on the host; no GPU is touched.
 * Errors: XP_ERR_GRAMMAR (bad indices, operator outside + - * / % min max << >>), XP_ERR_TOO_LARGE. */
xp_status xp_grammar_create(const xp_grammar_desc* desc, xp_grammar** out);
void xp_grammar_destroy(xp_grammar* g);

/* Host-side views of the grammar's enumeration (no GPU): counts per size of a nonterminal,
 * out[0..max_size] (XP_ERR_TOO_LARGE if one reaches 2^63), and the text / postfix of the tree
 * with a given rank.  text may be NULL; returns XP_ERR_INVALID_ARG if rank >= count or a
 * buffer is too small (code needs `size` instructions). */
xp_status xp_grammar_count(const xp_grammar* g, int32_t nt, int32_t max_size, uint64_t* out);
xp_status xp_grammar_unrank(const xp_grammar* g, int32_t nt, int32_t size, uint64_t rank,
                            xp_instr* code, int32_t code_cap, char* text, size_t text_cap);

/* Sketch (Algorithm 3: GenerateCodeSketch gives the holes, CreateSMTQuery the per-index
 * constraints = domain + spec).  Encodes contexts and specs, copies host tables to the GPU
 * and chooses the probe points.  The grammar must outlive the sketch.
 * Errors: XP_ERR_SKETCH, XP_ERR_INVALID_ARG, XP_ERR_NOMEM, XP_ERR_CUDA. */
xp_status xp_sketch_load(const xp_grammar* g, const xp_sketch_desc* desc, xp_sketch** out);
void xp_sketch_destroy(xp_sketch* s);

/* The same for n sketches at once (Algorithm 3 runs once per failing snippet, and a pass can leave
 * many of them): descs[i] is loaded against grammars[i] (the same grammar may appear many times)
 * and outs[i] receives its handle.  The sketches come out exactly as n calls of xp_sketch_load
 * would leave them; the difference is cost: the copies and the load's kernels of the whole batch
 * are queued together (one launch covers every sketch) and the host waits for the device once,
 * where n single loads wait n times.  On error nothing is loaded and every outs[i] is NULL; the
 * message names the first offending sketch.
 * Errors: as xp_sketch_load. */
xp_status xp_sketch_load_batch(const xp_grammar* const* grammars, const xp_sketch_desc* descs, size_t n,
                               xp_sketch** outs);

/* What a loaded sketch holds and what its load moved (no GPU is touched). */
typedef struct {
    int32_t n_holes, device;        /* device: the CUDA device the sketch was loaded on; calls on it must be made
                                       with that device current (XP_ERR_INVALID_ARG otherwise) */
    int64_t n_points;
    uint64_t device_bytes;          /* device memory of the sketch (tables included, the caller's own tables not) */
    uint64_t load_h2d_bytes, load_d2h_bytes;   /* bytes the load copied to and from the device (grammar tables
                                                  included when this load was the grammar's first) */
    int32_t n_probes[8];            /* probe points of the first 8 holes */
    int32_t n_refined;              /* points promoted to probes by xp_sketch_refine so far */
} xp_sketch_info;
xp_status xp_sketch_info_get(const xp_sketch* s, xp_sketch_info* out);

/* Counterexample-guided refinement of the probe points (the enumerative counterpart of the solver
 * loop inside Algorithm 3's SynthesisCode: a candidate that satisfies every constraint looked at so
 * far and then fails one gives that constraint to the next round).  Every search notes, per hole,
 * the domain points at which candidates that had passed all probe points failed their whole-domain
 * check.  This call promotes the most frequent of them (at most max_promote per hole, 0: the
 * default of 4) to probe points, directly behind the first one, rebuilds the probe tables and
 * clears the notes; n_promoted (may be NULL) receives how many points were promoted over all holes.
 * Results of later searches are unchanged (a probe point is a domain point, and a match must hold
 * at every domain point); only the work changes: candidates that used to reach the whole-domain
 * check now end at a probe.  The sketch must not be in use by a search during the call.
 * Errors: XP_ERR_INVALID_ARG, XP_ERR_CUDA. */
xp_status xp_sketch_refine(xp_sketch* s, int32_t max_promote, int32_t* n_promoted);

/* Device scratch a call over these sketches needs (0 on invalid arguments). */
size_t xp_workspace_bytes(const xp_sketch* const* sketches, size_t n, const xp_repair_opts* opts);

/* The search (Algorithm 3: SynthesisCode), all sizes of all holes, synchronous on return.
 * opts may be NULL.  Distinct calls may run concurrently on distinct streams and workspaces.
 * xp_repair_batch searches n independent sketches in one pass over the GPU and writes n
 * results (outs[i] belongs to sketches[i]); on error no result is returned.
 * Errors: XP_ERR_INVALID_ARG, XP_ERR_NOMEM, XP_ERR_CUDA, XP_ERR_CANCELLED. */
xp_status xp_repair(const xp_sketch* sketch, const xp_repair_opts* opts, xp_result** out);
xp_status xp_repair_batch(const xp_sketch* const* sketches, size_t n, const xp_repair_opts* opts,
                          xp_result** outs);

/* Algorithm 3 hands the filled snippet back (SynthesisCode -> StitchBack): the per-hole answer. */
xp_status xp_result_get(const xp_result* r, int32_t hole, xp_result_view* out);
void xp_result_free(xp_result* r);

/* The same search as xp_repair for ONE sketch, for callers that must not allocate device
 * memory while they run.  (The paper has no counterpart for this entry point: it exists for
 * how the library is embedded, not for the method.)  Such callers are, for example, a
 * framework whose caching allocator owns all device memory after start-up, a serving loop in
 * which the implicit device-wide synchronisation of cudaMalloc / cudaFree is not acceptable,
 * or a process that runs under a hard device-memory budget fixed before the first request.
 * xp_repair either takes a caller-allocated workspace or calls cudaMalloc itself, and it
 * creates CUDA events; this entry point does neither.  Its scratch (counters, segment table,
 * accumulators, survivor queue) lives in a fixed array of XP_STATIC_SCRATCH_BYTES inside the library,
 * which every GPU that loads the library holds until the process exits.
 *
 *  - Inputs and outputs stay the caller's: the sketch (loaded earlier with xp_sketch_load,
 *    which does allocate) and `out`, an array of at least n_holes summaries, filled in place.
 *  - opts->workspace is ignored; size / rank windows, flags and stream work as in xp_repair;
 *    cancel is read once, before the launch; timeout_ms is ignored.  The call copies from
 *    pageable host memory and returns after the stream has been synchronised.
 *  - A call whose plan needs more than the fixed array, or a sketch with more than 64 holes,
 *    fails with XP_ERR_TOO_LARGE and a message giving the limit; nothing is launched.
 *  - The first call on a device looks up the array's device address (cudaGetSymbolAddress) and
 *    keeps it per device; make that first call before any stream capture begins elsewhere in
 *    the process.  Two threads making their first calls on one device at the same moment both
 *    look the address up and store the same value: harmless, and not locked.
 *  - All calls share the one array per device.  Each call overwrites the whole part it uses
 *    (counter and accumulators are staged in their start state), so earlier contents never
 *    leak into a result; but two calls that overlap in time on the same device race on it.
 *    Serialise them (same stream, or wait for the previous call to return).
 *  - No cudaMalloc, cudaFree, event or stream creation happens inside; kernel_ms is therefore
 *    not measured here.
 * Errors: XP_ERR_INVALID_ARG, XP_ERR_TOO_LARGE, XP_ERR_CUDA, XP_ERR_CANCELLED. */
enum { XP_STATIC_SCRATCH_BYTES = 1 << 20 };
typedef struct {
    int32_t solved, max_size, least_size, pad;
    uint64_t least_rank;
    uint64_t cand_count[XP_MAX_SIZE + 1];
    uint64_t match_count[XP_MAX_SIZE + 1];
    uint64_t evals_executed;
    char least_text[256];
} xp_hole_summary;
xp_status xp_repair_static(const xp_sketch* sketch, const xp_repair_opts* opts, xp_hole_summary* out,
                           int32_t out_cap);

/* The answers of n results (as xp_repair_batch returns them) in one array: the summaries of result 0's
 * holes, then result 1's, and so on (Algorithm 3's hand-back step for a batch of snippets).  out_cap is
 * the number of entries `out` holds; *n_out (may be NULL) receives the number written.
 * Errors: XP_ERR_INVALID_ARG (null result, out too short). */
xp_status xp_result_pack(const xp_result* const* results, size_t n, xp_hole_summary* out, size_t out_cap, size_t* n_out);

/* Two holes inside ONE constraint (a product search, for small products): `ctx` mentions both parts
 * (XP_I_HOLE with arg = 0 or 1) and the constraint "ctx(e0(p), e1(p), p) == spec(p) at every point p" is
 * stated for the PAIR (e0, e1), e_k a tree of start_nt[k] with at most max_size[k] nodes.  Where a snippet's
 * missing expressions cannot be given a spec of their own each (a wrong stride AND a wrong offset inside
 * one index), this is the form SynthesisCode's query takes.  The pairs are ordered by total size s0 + s1,
 * then s0, then the rank of e0, then the rank of e1; counts are per total size.  Domain, variables and
 * grammar are those of `sketch` (its own holes play no role).  Every candidate of either part up to its
 * bound is tabulated at up to 16 probe points (so each count per size must stay below 2^22), every pair
 * is tested on the probes from the tables, and a pair that passes them is checked on the whole domain.
 * Errors: XP_ERR_INVALID_ARG, XP_ERR_SKETCH (malformed ctx / spec, ctx without both parts),
 * XP_ERR_TOO_LARGE (a count of 2^22 or more, or more than 2^40 pairs), XP_ERR_NOMEM, XP_ERR_CUDA. */
typedef struct {
    int32_t start_nt[2], max_size[2];
    int32_t ctx_len; const xp_instr* ctx;
    int32_t spec_kind;              /* XP_SPEC_EXPR or XP_SPEC_TABLE */
    int32_t spec_len; const xp_instr* spec_expr;
    const int64_t* spec_table;      /* n_points values, point order of the domain */
    int32_t spec_table_on_device;
} xp_joint_desc;
typedef struct xp_joint_result xp_joint_result;
typedef struct {
    int32_t solved, max_total;      /* max_total = max_size[0] + max_size[1] */
    const uint64_t* cand_count;     /* [max_total + 1], index = total size of the pair */
    const uint64_t* match_count;
    int32_t least_total, least_size[2];
    uint64_t least_rank[2];
    const char* least_text[2];
    uint64_t evals_executed;        /* (pair, point) evaluations that ran: probe tests and whole-domain points */
    uint64_t probe_survivors;       /* pairs that passed every probe point */
    double kernel_ms, total_ms;
    int32_t n_launches;
} xp_joint_view;
xp_status xp_repair_joint(const xp_sketch* sketch, const xp_joint_desc* joint, const xp_repair_opts* opts, xp_joint_result** out);
xp_status xp_joint_result_get(const xp_joint_result* r, xp_joint_view* out);
void xp_joint_result_free(xp_joint_result* r);

/* The behaviour mode: bottom-up enumeration with observational-equivalence pruning (the paper keeps
 * its symbolic synthesis "limited scale" because the space of expressions explodes; pruning by behaviour
 * is the enumerative way to push the bound).  A different contract from xp_repair: what is counted is
 * BEHAVIOURS on a caller-given list of signature points, not syntactic candidates.
 *   A tree's signature is the vector of its values at the signature points.  Per nonterminal and size
 *   (ascending), the candidates are the leaf productions (size 1) and, for each binary production in the
 *   grammar's order, each left size ascending, every pair (left representative, right representative) in
 *   the order the representatives were found, right fastest.  A candidate that is undefined at a signature
 *   point (zero divisor, bad shift count) is dropped; one whose signature a representative of the same
 *   nonterminal already has (a smaller size, or earlier at this size) is dropped; the others become
 *   the representatives of this size, in that order.  A behaviour first realised by some tree of size s is
 *   found at size s (subtrees can be swapped for their representatives, which are no larger).
 * For hole `hole` of the sketch (start nonterminal, size bound, context, spec) the call reports, per size,
 * the candidates enumerated and the new behaviours found for the start nonterminal; how many
 * representatives satisfy the constraint at every signature point; the first of them (size, then order
 * found) and whether it satisfies the constraint on the whole domain; and the first that does.
 * Signatures live in device memory (8 bytes x n_sig per representative) beside a hash table of
 * fingerprints; an equal fingerprint is always confirmed by comparing the signatures themselves, so the
 * result does not depend on the hash.  The work is bound by memory traffic, not by the integer units.
 * Errors: XP_ERR_INVALID_ARG (bad hole, n_sig outside 1..XP_MAX_SIG, a point id outside the domain),
 * XP_ERR_TOO_LARGE (more representatives than max_representatives), XP_ERR_NOMEM, XP_ERR_CUDA. */
enum { XP_MAX_SIG = 16 };
typedef struct {
    int32_t hole;
    int32_t n_sig;
    const int64_t* sig_points;          /* domain point ids (box: mixed radix, first variable slowest), in signature order */
    uint64_t max_representatives;       /* of all nonterminals and sizes together; 0: 2^22 */
} xp_behaviour_desc;
typedef struct {
    int32_t max_size, pad;
    uint64_t enumerated[XP_MAX_SIZE + 1];
    uint64_t distinct[XP_MAX_SIZE + 1];
    uint64_t sig_matches;
    int32_t hit, hit_size;              /* first representative that satisfies the signature points */
    uint64_t hit_index;                 /* its position among the representatives of its size */
    int32_t hit_verified;               /* it satisfies the constraint on the whole domain */
    int32_t solved, solution_size, pad2;  /* first representative that does */
    uint64_t solution_index;
    char hit_text[256], solution_text[256];
    uint64_t representatives;           /* of all nonterminals and sizes */
    uint64_t bytes_moved;               /* algorithmic bytes of the signature passes (see DESIGN notes in the source) */
    double kernel_ms, total_ms;
    int32_t n_launches, pad3;
} xp_behaviour_summary;
xp_status xp_behaviours(const xp_sketch* sketch, const xp_behaviour_desc* desc, const xp_repair_opts* opts,
                        xp_behaviour_summary* out);

/* Algorithm 3 from end to end for one expression: the source snippet's expression S_s and the
 * erroneous expression S_e that the transformed program computes in its place go in, the repaired
 * expression comes out.
 *   GenerateCodeSketch: every subtree of S_e in turn is taken out and replaced by a hole, giving one
 *     single-hole sketch per node of S_e (context = the rest of S_e);
 *   CreateSMTQuery: the constraint per concrete index is "sketch == S_s at this point" over the box of
 *     the grammar's variables; where the two snippets iterate over different variables (a loop that the
 *     pass split, fused or bound to threads), var_map gives the value of each source variable as an
 *     expression over the grammar's (= the transformed program's) variables, and S_s is rewritten with it;
 *   SynthesisCode: all sketches are searched in one batch (xp_sketch_load_batch + xp_repair_batch);
 *   StitchBack: among the sketches that have a solution the one with the smallest solution is taken
 *     (ties: the smallest subtree taken out, then the leftmost) and its solution is put in place of
 *     the subtree.
 * S_s is postfix over source variables (XP_I_VAR arg < n_source_vars) and constants; S_e postfix over the
 * grammar's variables and constants; both may use every operator.  var_map may be NULL when the snippets
 * share their variables (n_source_vars must then equal the grammar's n_vars).
 * Errors: XP_ERR_INVALID_ARG, XP_ERR_SKETCH (malformed expression, rewritten spec longer than XP_MAX_CODE),
 * and those of the load and the search. */
typedef struct {
    const xp_instr* source;    int32_t source_len;       /* S_s */
    const xp_instr* erroneous; int32_t erroneous_len;    /* S_e */
    int32_t n_source_vars;
    const xp_instr* const* var_map;                      /* [n_source_vars] postfix expressions, or NULL */
    const int32_t* var_map_len;
    int32_t start_nt, max_size;                          /* what a hole is filled from */
} xp_pair_desc;
typedef struct xp_pair_result xp_pair_result;
typedef struct {
    int32_t solved;                 /* some single-subtree replacement makes S_e agree with S_s everywhere */
    int32_t n_sketches;             /* sketches generated (= nodes of S_e) and searched */
    int32_t node_first, node_last;  /* the subtree taken out: instructions [node_first, node_last] of S_e */
    int32_t least_size;             /* the solution that replaced it */
    uint64_t least_rank;
    const char* hole_text;          /* ... as text */
    const char* sketch_text;        /* S_e with HOLE in place of the subtree */
    const char* stitched_text;      /* the repaired expression */
    const xp_instr* stitched_code;  /* ... and as postfix */
    int32_t stitched_len;
    uint64_t candidates;            /* candidates of all sketches together */
    uint64_t evals_executed;
    double load_ms, search_ms;
} xp_pair_view;
xp_status xp_repair_pair(const xp_grammar* g, const xp_pair_desc* desc, xp_pair_result** out);
xp_status xp_pair_result_get(const xp_pair_result* r, xp_pair_view* out);
void xp_pair_result_free(xp_pair_result* r);

/* Message of the calling thread's last failed call ("" if none). */
const char* xp_last_error(void);

/* Measures the integer-ALU peak this library's roofline is quoted against: independent
 * 32-bit add chains (out[0]) and multiply-add chains (out[1]) in thread-operations per
 * second, on the current device and stream NULL.  Errors: XP_ERR_CUDA. */
xp_status xp_int32_peak(double* out_ops_per_s /* [2] */, double* out_ms /* [2], may be NULL */);

/* Measures what a division costs on the current device: out[0] = int64 truncating divisions per second
 * with divisors not known in advance (the general form of the exact evaluators), out[1] = int32 divisions
 * per second by a constant through a precomputed reciprocal (multiply-high, multiply-subtract, one
 * correction: the form the whole-domain check folds constant divisors into).  Dividing xp_int32_peak's
 * add figure by these gives the cost of one division in 32-bit operations.  Errors: XP_ERR_CUDA. */
xp_status xp_int_div_rate(double* out_divs_per_s /* [2] */);

#ifdef __cplusplus
}
#endif
#endif  /* XP_H_ */
