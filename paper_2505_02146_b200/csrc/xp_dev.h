// Structures shared by the host encoder and the device kernels of libxpiler_repair.
// Everything here is plain data laid out by the host and read by the kernels.
#pragma once

#include <stdint.h>

#include "xp.h"

namespace xp {

typedef unsigned long long u64;
typedef long long i64;
typedef unsigned int u32;
typedef int i32;

constexpr int kMaxSize = XP_MAX_SIZE;
constexpr int kMaxVars = XP_MAX_VARS;
constexpr int kMaxNt = XP_MAX_NONTERMINALS;
constexpr int kMaxCode = XP_MAX_CODE;
constexpr int kMaxStack = 16;        // deepest operand stack of a context / spec expression
constexpr int kCandStack = 8;        // deepest operand stack of a candidate (size <= 15 => <= 8 leaves)
constexpr int kMaxProbe = 16;        // probe points per sketch
constexpr int kProbeSamples = 64;    // sample points the probes are chosen from
constexpr int kThreads = 256;        // threads per CTA of the evaluation kernel
constexpr int kLinearChunk = kThreads * 4;   // ranks per linear ticket
constexpr int kNA = 8;                // tile tickets: register-side operands per thread
constexpr int kRegTile = kThreads * kNA;     // register-side operands per tile
constexpr int kBcTile = 512;          // broadcast-side operands per tile
constexpr int kBcTileSlow = 8;        // ... of a hole whose context compares (interval test in 64 bits per candidate)
constexpr u64 kStageMaxPoints = 1ull << 26;  // largest box whose points and spec values are staged in HBM at load
constexpr int kProgMax = 64;          // candidate substituted into its context: longest staged program
constexpr u64 kTabBudgetBytes = 64ull << 20;   // subtree-value tables of one hole, all probes together
constexpr u64 kTabMaxEntries = 1ull << 22;   // largest (nonterminal, size) subtree-value table per hole
constexpr u64 kBigMaxEntries = 1ull << 30;   // ... of the one further size that is tabulated at the first probe only
constexpr u64 kBigBudgetBytes = 12ull << 30; // ... and its bytes (9 per entry), per hole
constexpr u32 kOpBit = 0x80000000u;  // candidate code word: operator (low bits = XP_OP_*) or leaf index
constexpr int kMaxFamily = 8;         // tile segments that may share one fill of the register-side operands (a hit's
                                      // queue entry names its member in 3 bits)

// A leaf production: a variable (var >= 0) or a constant.
struct LeafDev { i32 var; i32 pad; i64 value; };

// A binary production and, per candidate size s, the number of trees of its nonterminal that
// precede its first tree (off[s]), i.e. the rank offset of the production at that size.
struct BinDev { i32 op, lnt, rnt, pad; u64 off[kMaxSize + 2]; };

struct GrammarDev {
    i32 n_vars, n_nt, n_leaves, n_bins;
    i32 leaf_begin[kMaxNt + 1];      // leaves of nonterminal nt: leaves[leaf_begin[nt] .. leaf_begin[nt+1])
    i32 bin_begin[kMaxNt + 1];       // binary productions of nt: bins[bin_begin[nt] .. bin_begin[nt+1])
    u64 cnt[kMaxNt][kMaxSize + 1];   // trees of nt with exactly s nodes
    const LeafDev* leaves;           // device
    const BinDev* bins;              // device
};

struct HoleDev {
    i32 start_nt, max_size, ctx_len, spec_len;   // spec_len == 0: the spec is a table
    const i64* spec_table;                        // device, n_points values: the caller's table, or the spec
                                                  // expression evaluated once per point at load (null: evaluate)
    xp_instr ctx[kMaxCode];
    xp_instr spec[kMaxCode];
    // Probe points of this hole, most discriminating first (written by the prepare kernel).
    i32 n_probe;
    u32 probe_spec_ok;                            // bit j: the spec is defined at probe j
    i64 probe_id[kMaxProbe];
    i64 probe_pt[kMaxProbe][kMaxVars];
    i64 probe_spec[kMaxProbe];                    // spec at the probe points
    // Context at probe 0 as an affine map of the hole value, ctx(h) = aff_A * h + aff_B in
    // wrap-around arithmetic (possible when the hole only passes through + - * with
    // hole-free operands); aff_ok == 0: not of that form, the probe filter is not used.
    i32 aff_ok;
    u32 aff_okmask;                               // bit j: the context is affine in the hole at probe j too,
    u64 aff_A, aff_B;                             //        ctx(h) = aff_Aj[j] * h + aff_Bj[j]
    u64 aff_Aj[kMaxProbe], aff_Bj[kMaxProbe];
    // Contexts that compare: when the context is  X < c,  X <= c,  c < X  or  c <= X  with X = +-h + B
    // (h the hole value, B and c hole-free), the hole values that satisfy the constraint at probe j
    // form the interval [rng_lo[j], rng_hi[j]] (LLONG_MIN / LLONG_MAX for an open end; lo > hi: none).
    // Such a hole (a loop bound stated through its guard predicate) is filtered on that interval
    // where an affine context is filtered on equality.  Bit j of rng_okmask: probe j has the form.
    u32 rng_okmask, pad3;
    i64 rng_lo[kMaxProbe], rng_hi[kMaxProbe];
    // Values at probe 0 of every subtree of the small sizes 1..tab_max_size, by (nonterminal,
    // size, rank): tab_val[tab_off[nt][size] + rank], with tab_ok telling whether the subtree
    // is defined there (no zero divisor).  Built bottom-up once per sketch; operands of the
    // filter stage are looked up here instead of being unranked again in every tile.
    // The tables exist for the probes 0 .. tab_probes-1, one copy after the other (stride tab_total).
    // Hits of the filter are checked exactly there (two lookups and one operation per probe); only
    // probes without tables need the candidate unranked in full.
    // second: filter hits are also checked exactly at probe 1 before they are queued (needs tables, a
    // defined spec and an affine context at probe 1); sample_pass0: how many of the sample_n small
    // candidates sampled at load satisfied probe 0, sample_big: how many of the kPrepBigSamples random
    // candidates of the largest size did (a high rate of either makes the second look worth its cost).
    i32 second, sample_pass0, sample_n, sample_big;
    i32 second_ok;                                // the second look is possible (tables, spec and context at probe 1): a
                                                  // CTA that sees many filter hits for this hole turns it on for itself
    // Set by the host before the load's kernels run: the largest subtree size and the number of
    // probes that the tables may cover (their memory is laid out for that many), and whether the
    // search is small (then the second look is always taken).  prepare_kernel derives
    // tab_max_size, tab_probes, second and filter_ok from them and from the probes it chose.
    i32 tab_size_cap, tab_probes_cap, small_search;
    i32 filter_ok;                                // the probe filter applies: probe 0 exists, its context is affine or compares
    i32 tab_max_size, tab_probes;
    // One size further (big_size = the next size above tab_size_cap that has trees, when operands of that size occur and its trees fit
    // kBigMaxEntries / kBigBudgetBytes) the values are tabulated at probe 0 ONLY: these are the register-side
    // operands of the largest candidates (config 4: 5.9e8 subtrees of size 7, 5.3 GB), which every search
    // would otherwise rebuild from the smaller tables tile by tile -- a third of such a search's time.
    // The memory of a B200 has room for them; they stay resident with the sketch.  big_on is set by the
    // load's kernels once the smaller tables exist at probe 0.
    i32 big_size, big_on;
    u64 big_off[kMaxNt];                          // first entry of each nonterminal
    u64 big_total;
    i64* big_val;                                 // device
    unsigned char* big_ok;                        // device
    u64 tab_total;
    u64 tab_off[kMaxNt][kMaxSize + 1];
    i64* tab_val;                                 // device
    unsigned char* tab_ok;                        // device
    unsigned char* tab_vars;                      // device, one copy: bit v set if variable v occurs in the subtree
    // Variables that the context or the spec expression mention (all of them when the spec is the
    // caller's table).  On a box domain a candidate is checked on the sub-box of these and its
    // own variables only: no other variable can change either side of the constraint.
    u32 fixed_vars, pad2;
    // Points that ended a survivor's whole-domain check (a candidate that passed every probe and then
    // failed somewhere): a small open-addressed table of point ids (-1: free) with the number of
    // survivors each has ended.  Written by verify_kernel, read and cleared by xp_sketch_refine, which
    // promotes the most frequent ones to probes.  (Counters only: nothing in a search reads them.)
    i64* kill_pid;                                // device, kKillSlots entries
    u32* kill_cnt;                                // device, kKillSlots entries
};
constexpr int kKillSlots = 64;

struct SketchDev {
    const GrammarDev* g;                          // device
    i32 n_vars, n_holes, domain_kind, n_samples;
    i32 prep_cands, project;                      // project: box domain with staged points (see HoleDev::fixed_vars)                         // sampled candidates the probe choice is based on (<= 1024)
    i64 n_points;
    const i32* coords;                            // device: the points of a table domain, or the staged
                                                  // points of a box (null: derive them from the point id)
    i64 lo[kMaxVars], ext[kMaxVars];              // box: range start and extent per variable
    i64 vmin[kMaxVars], vmax[kMaxVars];           // smallest and largest coordinate of each variable over the domain
                                                  // (box: from the ranges; table: reduced over the rows at load)
    HoleDev* holes;                               // device
    i64 sample_id[kProbeSamples];                 // point ids the probes are chosen from (host-chosen)
};

// One hole of one sketch, for the kernels that run at load over a whole batch of sketches.
struct LoadJob { SketchDev* s; i32 hole, pad; };

// Per (sketch, hole) accumulators, zeroed (min_rank to all-ones) by the host before the launch.
struct AccDev {
    u64 match_count[kMaxSize + 1];
    u64 min_rank[kMaxSize + 1];
    u64 evals;                       // exact candidate-point evaluations that ran: stage 2 (probes) and stage 3 (domain points)
    u64 filter_survivors, probe_survivors, pad;
    u64 ops_skipped;                 // cost-model operations that the filter did not have to carry out (remainders
                                     // of a tile none of whose divisors exceeds the target's magnitude)
    u64 filter_tests;                // filter-stage tests at probe 0 that ran: (register operand defined there) x
                                     // (broadcast operand defined there) x (operators whose loop was entered)
    u64 tile_cands;                  // candidates of the tiles visited, tested or not
};

// One contiguous piece of work.  kind 0 (linear): ranks [rank_begin, rank_end) of `size`,
// every candidate unranked on its own.  kind 1 (tile): the product of left subtrees
// [a_begin, a_begin+a_count) x right subtrees of one (production group, left size).
enum { kSegLinear = 0, kSegTile = 1 };
struct SegDev {
    u64 first_ticket;                // tickets before this segment
    u64 rank_begin, rank_end;        // window of ranks searched at this size
    i32 sketch, hole, size, kind;
    i32 acc;                         // accumulator slot
    // tile segments
    i32 reg_nt, reg_size;            // register-side operand: nonterminal, size
    i32 bc_nt, bc_size;              // broadcast-side operand
    i32 swap;                        // 1: the register side is the RIGHT operand
    i32 n_ops;                       // productions sharing (left nt, right nt) at this split
    i32 op[5];
    u64 op_base[5];                  // rank of (left 0, right 0) for each of them
    u64 reg_begin, reg_count;        // register-side subtree ranks covered by the window
    u64 bc_begin, bc_count;          // broadcast-side subtree ranks covered
    u64 right_count;                 // trees of the right operand (rank = base + l * right_count + r)
    u32 reg_tiles, bc_tiles;         // tickets = reg_tiles * bc_tiles
    i32 has_div;                     // some production of the group is / or %
    i32 generic;                     // some production of the group has no 32-bit filter loop (the shifts): the group's
                                     // candidates are evaluated exactly, in 64 bits, at the probe
    i32 bc_base, bc_keep;            // slots [bc_base, bc_base + bc_count) of the CTA's broadcast tile belong to this
                                     // segment; bc_keep (first of a family): all members' broadcast operands fit the
                                     // tile side by side and do not depend on the ticket, so a CTA fills them once
    i32 bc_tile;                     // broadcast operands per ticket (<= kBcTile; smaller where a candidate costs
                                     // more than a comparison, so that the search still spreads over all SMs)
    i32 family;                      // tile segments that share the register-side operands sit next to each
                                     // other: the first holds the tickets and the count of them (>= 1), the
                                     // others (family == 0) are visited by its tickets, one fill for all
};

// A candidate that passed every probe point and waits for the whole-domain check.  The check
// is cut into chunks of kVerifyChunk points that any CTA may take; state counts the chunks
// that passed, its top bit says that some point failed.
constexpr int kVerifyChunk = 4096;
constexpr u32 kSurvFailed = 0x80000000u;
struct SurvDev { u64 rank; i32 sketch, hole, size, acc; u32 state, vars; };   // vars: variables the candidate mentions

struct PlanDev {
    u64 ticket_base;                 // tickets [ticket_base, n_tickets) belong to this launch (a search that polls a
                                     // cancel word is cut into several launches); the counter starts at zero each time
    u64 n_tickets;
    i32 n_segs, n_sketches;
    const SegDev* segs;              // device
    const SketchDev* const* sketches;  // device table of device pointers
    AccDev* acc;                     // device
    u64* ticket;                     // device counter, zero at launch
    SurvDev* surv;                   // device queue of survivors
    u32* surv_n;                     // device counter of pushes (may run past surv_cap), zero at launch
    u64* verify_ticket;              // device counter, zero at launch
    u32 surv_cap;
    u32 max_chunks;                  // chunks of the largest domain among the sketches
    u32* err;                        // device word for the checked build's index checks (0: none failed)
    // Survivors in hole order (null when the call has one hole): queued survivors per accumulator slot
    // (counted by eval_kernel), the slots' offsets (a scan of the counts) and, per slot side by side, the
    // queue indices of its survivors (a scatter).  The verification kernel walks surv_sorted.
    i32 n_acc;
    u32* surv_hist;                  // device, n_acc, zero at launch
    u32* surv_off;                   // device, n_acc + 1
    u32* surv_sorted;                // device, surv_cap
    // Survivors whose check spans more than one chunk of points (queue indices, in no particular order),
    // listed after the search so that the later chunks are walked for them alone.
    u32* surv_long;                  // device, surv_cap
    u32* surv_long_n;                // device counter, zero at launch
};

}  // namespace xp
