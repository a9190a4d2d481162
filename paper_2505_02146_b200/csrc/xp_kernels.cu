// Device kernels of libxpiler_repair (sm_100a).
//
//   prepare_kernel  -- per sketch, once at load: coordinates and spec values of the sample
//                      points, choice and order of each hole's probe points.
//   subvalue_kernel, stage_points_kernel, stage_spec_kernel, coord_bounds_kernel -- per sketch,
//                      once at load: values (and variable sets) of all small subtrees at the probes;
//                      points and spec values of a box; coordinate bounds of a table.
//   eval_kernel     -- the search.  Persistent CTAs take tickets (pieces of the rank space)
//                      from an atomic counter; no CTA ever waits for another.
//                        stage 1 (tile segments): probe-point filter over a product of operand tiles,
//                                 with a second, exact look at probe 1 for what the filter lets through;
//                        stage 2: exact int64 check of a hit on the probe points (lane = candidate).
//                      Survivors of stage 2 go to a global queue.
//   verify_kernel   -- stage 3: check on the whole domain (lane = 2 or 4 points, warp-wide early
//                      exit), cut into (survivor, chunk of points) items that any warp takes; on a
//                      box only the sub-box of the variables that occur is visited.
//   count_kernel    -- survivors that passed every chunk become matches: per-size counts (sum)
//                      and least rank (min) by atomics.
//   finish_kernel   -- reduction of the per-size results to the least solution per hole.
//   int32_peak_*    -- integer-ALU peak microbenchmarks.
#include <cuda_runtime.h>

#include <climits>

#include "xp_device.cuh"
#include "xp_launch.h"

namespace xp {

// ------------------------------------------------------------------------------------------
// prepare
// ------------------------------------------------------------------------------------------

// Context of a hole at one point as an affine map of the hole value (wrap-around ring
// arithmetic): walks the postfix code with entries "A*h + B".  Fails when the hole meets an
// operator other than + - *, or itself under *, or when a hole-free operand divides by zero.
__device__ bool ctx_affine(const HoleDev* hole, const i64* pt, u64& A, u64& B) {
    if (hole->ctx_len == 0) { A = 1; B = 0; return true; }
    u64 sa[kMaxStack], sb[kMaxStack];
    int sp = 0;
    u32 has = 0;                                        // bit i: stack entry i contains the hole
    for (int i = 0; i < hole->ctx_len; ++i) {
        const xp_instr c = hole->ctx[i];
        if (c.kind != XP_I_OP) {
            sa[sp] = c.kind == XP_I_HOLE ? 1ull : 0ull;
            sb[sp] = c.kind == XP_I_VAR ? (u64)pt[c.arg] : (c.kind == XP_I_CONST ? (u64)c.value : 0ull);
            has = (has & ~(1u << sp)) | ((c.kind == XP_I_HOLE ? 1u : 0u) << sp);
            ++sp;
            continue;
        }
        --sp;
        const bool hy = (has >> sp) & 1, hx = (has >> (sp - 1)) & 1;
        const u64 xa = sa[sp - 1], xb = sb[sp - 1], ya = sa[sp], yb = sb[sp];
        if (!hx && !hy) {
            i64 r;
            if (!apply_op(c.arg, (i64)xb, (i64)yb, r)) return false;
            sb[sp - 1] = (u64)r;
            continue;
        }
        if (c.arg == XP_OP_ADD) { sa[sp - 1] = xa + ya; sb[sp - 1] = xb + yb; }
        else if (c.arg == XP_OP_SUB) { sa[sp - 1] = xa - ya; sb[sp - 1] = xb - yb; }
        else if (c.arg == XP_OP_MUL && !(hx && hy)) {
            if (hx) { sa[sp - 1] = xa * yb; sb[sp - 1] = xb * yb; }
            else { sa[sp - 1] = ya * xb; sb[sp - 1] = yb * xb; }
        } else return false;
        has |= 1u << (sp - 1);
    }
    A = sa[0]; B = sb[0];
    return true;
}

// Context of a hole at one point as a comparison of +-h + B with a hole-free value (see
// HoleDev::rng_lo): walks the postfix code with entries that are a constant, the form a*h + b
// with a = +-1, or (last instruction only) the predicate.  On success gives the interval of
// hole values h for which the context's value equals `spec`.  All magnitudes are kept below
// 2^61, so that the interval is exact for every h below 2^62 in magnitude.
__device__ bool ctx_interval(const HoleDev* hole, const i64* pt, i64 spec, i64& lo, i64& hi) {
    constexpr i64 kBig = 1ll << 61;
    i64 sa[kMaxStack], sb[kMaxStack];                   // entry = sa * h + sb; sa == 0: a constant
    int sp = 0;
    const int n = hole->ctx_len;
    if (n < 3) return false;
    for (int i = 0; i < n; ++i) {
        const xp_instr c = hole->ctx[i];
        if (c.kind != XP_I_OP) {
            sa[sp] = c.kind == XP_I_HOLE ? 1 : 0;
            sb[sp] = c.kind == XP_I_VAR ? pt[c.arg] : (c.kind == XP_I_CONST ? c.value : 0);
            ++sp;
            continue;
        }
        --sp;
        const i64 xa = sa[sp - 1], xb = sb[sp - 1], ya = sa[sp], yb = sb[sp];
        if (xb <= -kBig || xb >= kBig || yb <= -kBig || yb >= kBig) return false;
        if (xa == 0 && ya == 0) {
            i64 r;
            if (!apply_op(c.arg, xb, yb, r)) return false;
            sb[sp - 1] = r;
            continue;
        }
        if (i == n - 1 && (c.arg == XP_OP_LT || c.arg == XP_OP_LE) && (xa == 0) != (ya == 0)) {
            // value = [ a*h + b < T ] xor neg
            i64 a, b, T;
            bool neg;
            if (ya == 0) { a = xa; b = xb; T = c.arg == XP_OP_LT ? yb : yb + 1; neg = false; }      // X < c, X <= c
            else { a = ya; b = yb; T = c.arg == XP_OP_LT ? xb + 1 : xb; neg = true; }              // c < X, c <= X
            if (spec != 0 && spec != 1) { lo = 1; hi = 0; return true; }
            const bool want = (spec == 1) != neg;                  // a*h + b < T must be `want`
            if (a == 1) {                                          // h < T - b
                if (want) { lo = LLONG_MIN; hi = T - b - 1; } else { lo = T - b; hi = LLONG_MAX; }
            } else {                                               // -h + b < T  <=>  h > b - T
                if (want) { lo = b - T + 1; hi = LLONG_MAX; } else { lo = LLONG_MIN; hi = b - T; }
            }
            return true;
        }
        if (c.arg == XP_OP_ADD && (xa == 0 || ya == 0)) { sa[sp - 1] = xa + ya; sb[sp - 1] = xb + yb; }
        else if (c.arg == XP_OP_SUB && (xa == 0 || ya == 0)) { sa[sp - 1] = xa - ya; sb[sp - 1] = xb - yb; }
        else return false;
    }
    return false;
}

constexpr int kPrepBigSamples = 8192;                    // random candidates of the largest size, held against the first probe

// The context at every probe (affine in the hole, or a comparison; one thread per probe), and what
// the rest of the load and the searches go by.  Called by every thread of the CTA once the n
// probes (ids, coordinates, spec values) are in place; ncand / pass0: how many sampled candidates
// the probe choice looked at and how many of them satisfied the first probe; big_hits: how many of
// the kPrepBigSamples candidates of the largest size did.
__device__ __forceinline__ void probe_contexts(HoleDev* hole, int n, int ncand, int pass0, int big_hits) {
    const int t = threadIdx.x;
    if (t < kMaxProbe) {
        u64 A = 0, B = 0;
        const bool aff = t < n && ctx_affine(hole, hole->probe_pt[t], A, B);
        i64 lo = 1, hi = 0;
        const bool rng = t < n && !aff && ((hole->probe_spec_ok >> t) & 1u) &&
                         ctx_interval(hole, hole->probe_pt[t], hole->probe_spec[t], lo, hi);
        hole->aff_Aj[t] = aff ? A : 0;
        hole->aff_Bj[t] = aff ? B : 0;
        hole->rng_lo[t] = lo;
        hole->rng_hi[t] = hi;
        const u32 amask = __ballot_sync(0x0000ffffu, aff), rmask = __ballot_sync(0x0000ffffu, rng);
        if (t == 0) {
            hole->aff_ok = aff ? 1 : 0;
            hole->aff_A = aff ? A : 0;
            hole->aff_B = aff ? B : 0;
            hole->aff_okmask = amask;
            hole->rng_okmask = rmask;
            // what the rest of the load and the searches go by
            const u32 spec_ok = hole->probe_spec_ok;
            const bool filter_ok = n > 0 && (aff || (rmask & spec_ok & 1u));
            hole->filter_ok = filter_ok ? 1 : 0;
            int probes = 0;
            if (filter_ok && hole->tab_size_cap > 0 && hole->tab_total > 0) probes = n < hole->tab_probes_cap ? n : hole->tab_probes_cap;
            hole->tab_probes = probes;
            hole->tab_max_size = probes > 0 ? hole->tab_size_cap : 0;
            hole->big_on = 0;                             // (the kernel that fills the big table turns it on)
            // Second look at probe 1 inside the filter: for small searches (its cost is in the operand
            // fills, which large tiles amortise anyway) and wherever the sampled candidates say that
            // probe 0 alone lets many through.
            const bool possible = n >= 2 && probes >= 2 && ((spec_ok & (amask | rmask)) >> 1 & 1u);
            // (one in 256 of the small sample, or one in 4096 of the large candidates: the dense form of the
            // loops wins from about there, see kAdaptRate)
            const bool frequent = (ncand > 0 && (u64)pass0 * 256 >= (u64)ncand) || (u64)big_hits * 4096 >= (u64)kPrepBigSamples;
            hole->second = possible && (hole->small_search || frequent) ? 1 : 0;
            hole->second_ok = possible ? 1 : 0;
        }
    }
}

// Choice of each hole's probe points, once per sketch (one CTA per hole).  Threads evaluate the sample
// points; then a sample of small candidates (sizes 1, 3, 5, ranks spread evenly) is run on
// every sample point, giving each a bit set of the samples where it satisfies the constraint.
// The probes are picked greedily: each next probe is the sample that the fewest of the
// sampled candidates still alive (satisfying all probes picked so far) also satisfy; ties go
// to the larger |spec| + sum |coordinate| (large, distinct operand values make coincidences
// rare).  Only the amount of work downstream depends on this choice, never a result.
constexpr int kPrepThreads = 1024;
constexpr int kPrepCands = 1024;
constexpr int kPrepParts = 4;                           // a sampled candidate's sample points are split over this many threads
__global__ void __launch_bounds__(kPrepThreads) prepare_kernel(const LoadJob* jobs) {
    SketchDev* s = jobs[blockIdx.x].s;
    __shared__ i64 s_pt[kProbeSamples][kMaxVars];
    __shared__ i64 s_spec[kProbeSamples];
    __shared__ int s_ok[kProbeSamples];
    __shared__ u64 s_score[kProbeSamples];
    __shared__ u64 s_sig[kPrepCands];                   // per sampled candidate: bit j = it satisfies sample j
    __shared__ u32 s_mask[kProbeSamples][kPrepCands / 32];    // the same bits, per sample over the candidates
    __shared__ u32 s_alive[kPrepCands / 32];            // candidates that satisfy every probe chosen so far
    __shared__ u32 s_count[kProbeSamples];
    __shared__ u64 s_chosen;
    __shared__ int s_best;
    __shared__ int s_big_hits;
    const int t = threadIdx.x;
    const int ns = s->n_samples;
    const int nv = s->n_vars;
    const GrammarDev* g = s->g;
    HoleDev* hole = &s->holes[jobs[blockIdx.x].hole];    // one CTA per hole
    if (t < ns) {
        i64 pt[kMaxVars];
        u64 coord_mag = 0;
        point_coords(s, s->sample_id[t], pt);
        for (int d = 0; d < nv; ++d) {
            s_pt[t][d] = pt[d];
            coord_mag += (u64)(pt[d] < 0 ? -pt[d] : pt[d]);
        }
        i64 v = 0;
        bool ok = true;
        if (hole->spec_table != nullptr) v = hole->spec_table[s->sample_id[t]];
        else ok = eval_code(hole->spec, hole->spec_len, pt, 0, v);
        s_spec[t] = v;
        s_ok[t] = ok;
        const u64 mag = (u64)(v < 0 ? -v : v);
        s_score[t] = ok ? (mag > (1ull << 62) ? (1ull << 62) : mag) + coord_mag : 0;
    }
    // behaviour of sampled small candidates on the sample points
    int sizes[3], nsz = 0;
    for (int k = 1; k <= 5 && k <= hole->max_size; k += 2)
        if (g->cnt[hole->start_nt][k] > 0) sizes[nsz++] = k;
    const int ncand = nsz > 0 ? (s->prep_cands < kPrepCands ? s->prep_cands : kPrepCands) : 0;
    for (int c = t; c < kPrepCands; c += kPrepThreads) s_sig[c] = 0;
    if (t == 0) s_chosen = 0;
    __syncthreads();
    for (int item = t; item < ncand * kPrepParts; item += kPrepThreads) {
        const int c = item / kPrepParts, part = item % kPrepParts;
        const int size = sizes[c % nsz];
        const u64 cnt = g->cnt[hole->start_nt][size];
        const u64 per = (u64)(ncand / nsz) + 1;
        const u64 slot = (u64)(c / nsz);
        if (slot < cnt || cnt >= per) {                       // small sizes: every rank once, the rest unused
            const u64 rank = cnt >= per ? slot * (cnt / per) : slot;
            u32 code[kMaxSize];
            const int n = unrank(g, hole->start_nt, size, rank, code);
            u64 sig = 0;
            for (int j = part; j < ns; j += kPrepParts) {
                i64 v;
                if (s_ok[j] && eval_cand(code, n, g->leaves, s_pt[j], v) && ctx_matches(hole, s_pt[j], v, s_spec[j]))
                    sig |= 1ull << j;
            }
            if (sig) atomicOr(&s_sig[c], sig);
        }
    }
    __syncthreads();
    const int nw = (ncand + 31) / 32;
    for (int i = t; i < ns * nw; i += kPrepThreads) {         // transpose the bits: per sample, a set of candidates
        const int j = i / nw, w = i % nw;
        u32 word = 0;
        for (int b = 0; b < 32 && w * 32 + b < ncand; ++b) word |= (u32)((s_sig[w * 32 + b] >> j) & 1ull) << b;
        s_mask[j][w] = word;
    }
    if (t < nw) s_alive[t] = (t + 1) * 32 <= ncand ? 0xffffffffu : (1u << (ncand - t * 32)) - 1u;
    __syncthreads();
    int n = 0;
    int pass0 = 0;
    for (; n < kMaxProbe && n < ns; ++n) {
        const u64 chosen = s_chosen;
        if (t < ns) {
            u32 count = 0xffffffffu;
            if (!((chosen >> t) & 1ull)) {
                count = 0;
                for (int w = 0; w < nw; ++w) count += (u32)__popc(s_alive[w] & s_mask[t][w]);
            }
            s_count[t] = count;
        }
        __syncthreads();
        if (t == 0) {
            int best = -1;
            for (int i = 0; i < ns; ++i) {
                if ((chosen >> i) & 1ull) continue;
                if (best < 0 || s_count[i] < s_count[best] || (s_count[i] == s_count[best] && s_score[i] > s_score[best])) best = i;
            }
            hole->probe_id[n] = s->sample_id[best];
            for (int d = 0; d < nv; ++d) hole->probe_pt[n][d] = s_pt[best][d];
            hole->probe_spec[n] = s_spec[best];
            if (n == 0) { hole->probe_spec_ok = 0; pass0 = (int)s_count[best]; }
            if (s_ok[best]) hole->probe_spec_ok |= 1u << n;
            s_chosen = chosen | (1ull << best);
            s_best = best;
        }
        __syncthreads();
        if (t < nw) s_alive[t] &= s_mask[s_best][t];
        __syncthreads();
    }
    if (t == 0) {
        hole->n_probe = n;
        if (n == 0) hole->probe_spec_ok = 0;
        s_big_hits = 0;
    }
    __syncthreads();
    // How often the first probe lets a candidate through is estimated once more on random candidates
    // of the largest size, where nearly all of a search's work is: the behaviour of expressions of one
    // to five nodes says little about those of nine.
    int big_size = hole->max_size;
    while (big_size > 1 && g->cnt[hole->start_nt][big_size] == 0) --big_size;
    const bool sample_big = n > 0 && big_size >= 3 && (hole->probe_spec_ok & 1u) && !hole->small_search;      // (a small search takes the second look anyway)
    if (sample_big) {
        const u64 cnt = g->cnt[hole->start_nt][big_size];
        i64 pt0[kMaxVars];
        for (int d = 0; d < nv; ++d) pt0[d] = hole->probe_pt[0][d];
        const i64 spec0 = hole->probe_spec[0];
        for (int c = t; c < kPrepBigSamples; c += kPrepThreads) {
            u64 x = (u64)(c + 1) * 0x9E3779B97F4A7C15ull;     // (a fixed scramble of the sample's number)
            x ^= x >> 29; x *= 0xBF58476D1CE4E5B9ull; x ^= x >> 32;
            u32 code[kMaxSize];
            const int len = unrank(g, hole->start_nt, big_size, __umul64hi(x, cnt), code);
            i64 v;
            if (eval_cand(code, len, g->leaves, pt0, v) && ctx_matches(hole, pt0, v, spec0)) atomicAdd(&s_big_hits, 1);
        }
    }
    __syncthreads();
    const int big_hits = sample_big ? s_big_hits : 0;
    if (t == 0) {
        hole->sample_pass0 = pass0;                       // sampled candidates that satisfy the first probe chosen
        hole->sample_n = ncand;
        hole->sample_big = big_hits;
    }
    __syncthreads();
    probe_contexts(hole, n, ncand, pass0, big_hits);
}

// The probes of a hole replaced by the host (xp_sketch_refine: points that ended whole-domain
// checks are promoted): hole->probe_id[0 .. n_probe) is given; coordinates, spec values and the
// context forms are derived again, as prepare_kernel does for the probes it picks.  One warp per hole.
__global__ void __launch_bounds__(32) reprobe_kernel(const LoadJob* jobs) {
    SketchDev* s = jobs[blockIdx.x].s;
    HoleDev* hole = &s->holes[jobs[blockIdx.x].hole];
    const int t = threadIdx.x, n = hole->n_probe;
    bool ok = false;
    if (t < n) {
        i64 pt[kMaxVars];
        point_coords(s, hole->probe_id[t], pt);
        for (int d = 0; d < s->n_vars; ++d) hole->probe_pt[t][d] = pt[d];
        i64 v = 0;
        ok = true;
        if (hole->spec_table != nullptr) v = hole->spec_table[hole->probe_id[t]];
        else ok = eval_code(hole->spec, hole->spec_len, pt, 0, v);
        hole->probe_spec[t] = v;
    }
    const u32 okmask = __ballot_sync(0xffffffffu, ok);
    if (t == 0) hole->probe_spec_ok = okmask;
    __syncthreads();
    probe_contexts(hole, n, hole->sample_n, hole->sample_pass0, hole->sample_big);
}

// ------------------------------------------------------------------------------------------
// eval
// ------------------------------------------------------------------------------------------

constexpr int kLinearPerThread = kLinearChunk / kThreads; // ranks per thread per linear ticket
constexpr u64 kAdaptRate = 4096;                          // filter hits per evaluation above 1 / kAdaptRate are "many"
constexpr int kWarps = kThreads / 32;
constexpr int kQueueCap = 3072;                           // filter hits waiting for the exact probe check (all warps)
constexpr int kWarpQueue = kQueueCap / kWarps;            // ... per warp: every warp keeps and empties its own queue
 constexpr int kQueueTags = 8;                             // tiles whose hits may wait in a warp's queue at a time
constexpr u32 kDrainMin = 32;                             // hits a warp lets gather before it checks them (resident families)
constexpr int kChunkB = 512;                              // broadcast operands between block-wide queue checks
static_assert(kRegTile <= 2048 && kBcTile <= 1024, "queue entries pack the tile indices in 11 + 10 bits");
static_assert(32 * 5 <= kWarpQueue / 2, "one replay step of a warp must fit the free half of its queue");

// A broadcast-side operand of a tile, as three 16-byte records so that each loop fetches what
// it needs with one shared-memory load.  All per-operand arithmetic that does not depend on
// the register operand is done once, when the tile is filled:
//   BcRing: t_add = the value a register operand (times A) must have for +; t_pm = the
//           sign-free form that covers + and - in one comparison (see ring_pass); and for *
//           the operand itself and the negated target:  (A*a) * b - tp == 0 (mod 2^32)  (one
//           multiply-add, which issues on a pipe that the comparisons do not use);
//   BcDiv:  magnitudes for / and %, see div_pass;
//   BcMeta: the value itself, meta = index inside the tile | ctz(|value|) << 16 | bit 31: pad holds
//           the operand's exact value at probe 1 (second look).
struct __align__(16) BcRing { u32 t_add, t_pm, mul_b, mul_nt; };
struct __align__(16) BcDiv { u32 low, ub, inv, cmax; };
struct __align__(16) BcMeta { u32 lo, hi, meta, pad; };

// The candidate under whole-domain check as one postfix program shared by the CTA: the
// hole's context with the candidate's code substituted for every HOLE leaf, leaves resolved.
// depth = deepest operand stack; depth == 0 marks a program too long to stage (the slow
// interpreters are used instead).
struct CandShared {
    i32 len, depth;
    i32 cand_len;
    // Sub-box the check runs on (see proj_points): its variables from the fastest down, with the
    // extent of each and its stride in point ids of the full box; n_proj_vars == 0: every point.
    i32 n_proj_vars;
    u32 proj_ext[kMaxVars], proj_stride[kMaxVars];
    i32 narrow;                  // every value the program can produce over the domain fits int32 (proved from
                                 // the variables' coordinate bounds): the check may run in 32-bit arithmetic
    i32 var[kProgMax];           // >= 0: variable; -1: constant; -2 - op: operator
    i64 val[kProgMax];
    i32 cvar[kMaxSize];          // the candidate alone (for the slow path)
    i64 cval[kMaxSize];
};

struct MemberState {
    u64 bc_first; i32 lo, hi; u32 n, nspecial; i32 wide;
    u32 mask, opip;              // the member's operators: bit per operator slot, and (3 bits per slot) each one's index
                                 // in the segment's list
    i32 mod_possible;            // some operand of the member, as a divisor, exceeds the target's magnitude: only
                                 // then can a remainder equal the target (|n % d| < |d|)
};

struct EvalShared {
    u64 ticket;
    i32 seg_index;
    SegDev seg;
    CandShared wcand[kWarps];    // per warp: the candidate of a whole-domain check the warp does itself
    // results of the (sketch, hole) the CTA is working on
    i32 cur_acc;
    u64 match_count[kMaxSize + 1];
    u64 min_rank[kMaxSize + 1];
    u64 filter_survivors, probe_survivors, ops_skipped;
    u64 filter_tests, tile_cands;
    u64 warp_evals[kThreads / 32];
    // tile tickets: the broadcast-side operands at probe 0 (entries invalid there are dropped) with
    // what the loops need of each, and the warps' queues of filter hits
    i32 chunk_hint[kWarps];      // broadcast slots per look at the hit queue (adapts to the hit rate)
    // The members of the family at hand (a single segment is a family of one): their segments and,
    // per member, the broadcast slots [lo, hi) it owns in the tile; general operands fill them from lo
    // up (n of them), those of magnitude <= 1 from hi down (nspecial).  When all members' slots lie
    // side by side (bc_keep) they stay valid from ticket to ticket: kept_head names the family
    // resident in the tile (-1: none), and the next ticket of that family does not fill again.
    SegDev mseg[kMaxFamily];
    MemberState mb[kMaxFamily];
    i32 kept_head;
    i32 reg_wide;                // some register-side operand of the ticket does not fit int32
    u32 wmember[kWarps];         // member the warp is working on, and (<< 3) the tag of its tile: both go into its queue entries
    u32 wq_n[kWarps], wq_over[kWarps];
    // second look (HoleDev::second): context factor, offset and spec value at probe 1 of the hole at hand
    i32 adapt_second;            // this CTA has seen more than one filter hit per kAdaptRate evaluations for the
                                 // hole it works on: it takes the second look from now on (until it changes hole)
    // what the loops need of the hole at the first probe (read from the hole once per ticket)
    u64 h_A, h_tq;               // context factor; spec value minus the context's offset
    i64 h_rng_lo, h_rng_hi;      // interval of values that satisfy a comparing context
    i32 h_aff_ok;
    i32 p1_on, p1_rng;           // p1_rng: the context compares at probe 1; the value must lie in [p1_lo, p1_hi]
    u64 p1_A, p1_B, p1_spec;
    i64 p1_lo, p1_hi;
    BcRing bc_ring[kBcTile];
    BcDiv bc_div[kBcTile];
    BcMeta bc_meta[kBcTile];
    u32 queue[kWarps][kWarpQueue];   // reg index | broadcast slot << 11 | op index << 21 | member << 24 | tile tag << 27
    // Hits may wait in a warp's queue over several tickets of one resident family, until there are
    // enough of them to give every lane of the exact check one (a tile of a sparse search leaves a
    // handful per warp).  An entry names its tile by a tag: wq_first holds the first register-side rank
    // of the warp's last kQueueTags tiles, wq_tiles counts the warp's tiles, wq_age the tiles since the
    // queue was last emptied (it is emptied before a tag comes round again).  q_sketch and q_hole name
    // the hole the waiting hits belong to.
    u64 wq_first[kWarps][kQueueTags];
    u32 wq_tiles[kWarps], wq_age[kWarps];
    i32 q_sketch, q_hole;
    i32 q_waiting;               // some warp has let hits wait
};

// Moves the CTA's private results of one (sketch, hole) into the global accumulators.
// Counts are sums and ranks are minima, so the order of flushes cannot change the result.
__device__ __noinline__ void flush_acc(EvalShared& sh, const PlanDev& plan, u64& my_evals) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    u64 e = my_evals;
    for (int o = 16; o > 0; o >>= 1) e += __shfl_down_sync(0xffffffffu, e, o);
    if (lane == 0) sh.warp_evals[warp] = e;
    __syncthreads();
    if (sh.cur_acc >= 0) {
        AccDev* acc = &plan.acc[sh.cur_acc];
        const int t = threadIdx.x;
        if (t <= kMaxSize) {
            if (sh.match_count[t]) atomicAdd(&acc->match_count[t], sh.match_count[t]);
            if (sh.min_rank[t] != ~0ull) atomicMin(&acc->min_rank[t], sh.min_rank[t]);
        }
        if (t == 32) {
            u64 tot = 0;
            for (int w = 0; w < kThreads / 32; ++w) tot += sh.warp_evals[w];
            if (tot) atomicAdd(&acc->evals, tot);
            if (sh.filter_survivors) atomicAdd(&acc->filter_survivors, sh.filter_survivors);
            if (sh.probe_survivors) atomicAdd(&acc->probe_survivors, sh.probe_survivors);
            if (sh.ops_skipped) atomicAdd(&acc->ops_skipped, sh.ops_skipped);
            if (sh.filter_tests) atomicAdd(&acc->filter_tests, sh.filter_tests);
            if (sh.tile_cands) atomicAdd(&acc->tile_cands, sh.tile_cands);
        }
    }
    __syncthreads();
    if (threadIdx.x <= kMaxSize) { sh.match_count[threadIdx.x] = 0; sh.min_rank[threadIdx.x] = ~0ull; }
    if (threadIdx.x == 0) { sh.filter_survivors = 0; sh.probe_survivors = 0; sh.ops_skipped = 0; sh.adapt_second = 0; sh.filter_tests = 0; sh.tile_cands = 0; }
    my_evals = 0;
    __syncthreads();
}

// Stage 2: exact check of one candidate on the hole's probe points, first failure ends it.
__device__ __noinline__ bool probe_check(const GrammarDev* g, const HoleDev* hole, const u32* code, int n,
                                            u64& my_evals) {
    const int np = hole->n_probe;
    for (int j = 0; j < np; ++j) {
        ++my_evals;
        if (!((hole->probe_spec_ok >> j) & 1)) return false;
        i64 h;
        if (!eval_cand(code, n, g->leaves, hole->probe_pt[j], h)) return false;
        if (!ctx_matches(hole, hole->probe_pt[j], h, hole->probe_spec[j])) return false;
    }
    return true;
}

__device__ __noinline__ void stage_candidate(CandShared& c, const SketchDev* sk, const HoleDev* hole, int size, u64 rank) {
    const GrammarDev* g = sk->g;
    u32 code[kMaxSize];
    const int n = unrank(g, hole->start_nt, size, rank, code);
    c.cand_len = n;
    for (int k = 0; k < n; ++k) {
        if (code[k] & kOpBit) { c.cvar[k] = -2 - (i32)(code[k] & 0xff); c.cval[k] = 0; }
        else { const LeafDev lf = g->leaves[code[k]]; c.cvar[k] = lf.var >= 0 ? lf.var : -1; c.cval[k] = lf.value; }
    }
    // the context with the candidate in place of each HOLE; alongside, an upper bound of the
    // magnitude of every value on the operand stack (saturating at 2^62), from the coordinate
    // bounds of the variables: if no bound reaches 2^31 the program is exact in int32
    int len = 0, sp = 0, depth = 0;
    bool fits = true, narrow = true;
    constexpr u64 kSat = 1ull << 62;
    u64 mag[kMaxStack + kCandStack + 1];
    auto mag_of = [](i64 v) { return v < 0 ? 0ull - (u64)v : (u64)v; };
    auto emit = [&](i32 var, i64 val) {
        if (len >= kProgMax || sp > kMaxStack + kCandStack - 1) { fits = false; return; }
        c.var[len] = var; c.val[len] = val; ++len;
        u64 m;
        if (var >= -1) {
            if (var >= 0) { const u64 a = mag_of(sk->vmin[var]), b = mag_of(sk->vmax[var]); m = a > b ? a : b; }
            else m = mag_of(val);
            mag[sp] = m < kSat ? m : kSat;
            if (++sp > depth) depth = sp;
        } else {
            --sp;
            const u64 a = mag[sp - 1], b = mag[sp];
            switch (-2 - var) {
                case XP_OP_ADD: case XP_OP_SUB: m = a + b; break;
                case XP_OP_MUL: m = (a >> 31 || b >> 31) ? kSat : a * b; break;
                case XP_OP_DIV: m = a; break;
                case XP_OP_MOD: m = a < b ? a : b; break;
                case XP_OP_MIN: case XP_OP_MAX: m = a > b ? a : b; break;
                case XP_OP_SHL: m = kSat; break;
                case XP_OP_SHR: m = a; break;
                default: m = 1; break;
            }
            mag[sp - 1] = m < kSat ? m : kSat;
        }
        narrow = narrow && (m >> 31) == 0;
    };
    if (hole->ctx_len == 0) {
        for (int k = 0; k < n; ++k) emit(c.cvar[k], c.cval[k]);
    } else {
        for (int i = 0; i < hole->ctx_len && fits; ++i) {
            const xp_instr in = hole->ctx[i];
            if (in.kind == XP_I_HOLE) for (int k = 0; k < n; ++k) emit(c.cvar[k], c.cval[k]);
            else if (in.kind == XP_I_OP) emit(-2 - in.arg, 0);
            else emit(in.kind == XP_I_VAR ? in.arg : -1, in.value);
        }
    }
    bool has_hole = hole->ctx_len == 0;
    for (int i = 0; i < hole->ctx_len; ++i) has_hole = has_hole || hole->ctx[i].kind == XP_I_HOLE;
    c.len = len;
    c.n_proj_vars = 0;                            // every point, unless the caller sets a sub-box (proj_points)
    c.depth = (fits && has_hole) ? depth : 0;     // a context that ignores the hole still needs the candidate to be defined
    c.narrow = narrow ? 1 : 0;
}

// Operators that exist only inside a staged int32 program: division and remainder by a constant
// that is not zero.  "push c; x / y" becomes one instruction on the top of the stack whose val
// holds the constant (low half) and floor(2^32 / |c|) (high half), so that a point costs a
// multiply-high and a correction instead of a 32-bit division.
constexpr int kOpDivC = 32, kOpModC = 33;

// Rewrites the constant divisions of a staged program that runs in int32 (only the vectorised
// whole-domain check understands the result).  One lane.
__device__ void fold_constant_divisors(CandShared& c) {
    int w = 0;
    for (int k = 0; k < c.len; ++k) {
        const i32 cv = c.var[k];
        const bool divmod = cv == -2 - XP_OP_DIV || cv == -2 - XP_OP_MOD;
        if (divmod && w > 0 && c.var[w - 1] == -1 && c.val[w - 1] != 0 && c.val[w - 1] > -(1ll << 31) && c.val[w - 1] < (1ll << 31)) {
            const i32 d = (i32)c.val[w - 1];
            const u32 ad = d < 0 ? 0u - (u32)d : (u32)d;
            const u32 M = ad == 1u ? 0xffffffffu : (u32)((1ull << 32) / ad);
            c.var[w - 1] = -2 - (cv == -2 - XP_OP_DIV ? kOpDivC : kOpModC);
            c.val[w - 1] = (i64)(((u64)M << 32) | (u32)d);
            continue;                                     // (the operator took the place of the push)
        }
        c.var[w] = cv; c.val[w] = c.val[k]; ++w;
    }
    c.len = w;
}

// The staged program at one point with an operand stack of D registers (D >= its depth): a
// push shifts the registers up, an operator combines the two lowest and shifts down.  The
// program is the same for every thread, so all branches are uniform.
template <int D>
__device__ __forceinline__ bool run_program(const CandShared& c, const i32* __restrict__ row, i64& out) {
    i64 st[D];
#pragma unroll
    for (int i = 0; i < D; ++i) st[i] = 0;
    const int n = c.len;
    for (int k = 0; k < n; ++k) {
        const i32 cv = c.var[k];
        if (cv >= -1) {
            const i64 v = cv >= 0 ? (i64)row[cv] : c.val[k];
#pragma unroll
            for (int i = D - 1; i > 0; --i) st[i] = st[i - 1];
            st[0] = v;
        } else {
            i64 r;
            if (!apply_op(-2 - cv, st[1], st[0], r)) return false;
            st[0] = r;
#pragma unroll
            for (int i = 1; i < D - 1; ++i) st[i] = st[i + 1];
        }
    }
    out = st[0];
    return true;
}

// Points that the whole-domain check of a survivor has to visit.  On a box whose points are
// staged, variables that neither the candidate nor the context nor the spec mention cannot
// change either side of the constraint, so the sub-box of the mentioned variables (the others
// at their first value) decides for the whole box.  Returns the number of points of that
// sub-box (the whole domain when nothing can be left out, or when the sub-box does not fit 31
// bits) and, if `c` is given, writes its digits there.
__device__ __forceinline__ i64 proj_points(const SketchDev* sk, const HoleDev* hole, u32 cand_vars, CandShared* c) {
    if (c) c->n_proj_vars = 0;
    const int nv = sk->n_vars;
    const u32 all = nv >= 32 ? 0xffffffffu : (1u << nv) - 1u;
    const u32 used = (cand_vars | hole->fixed_vars) & all;
    if (!sk->project || used == all) return sk->n_points;
    u64 n = 1, stride = 1;
    int k = 0;
    for (int v = nv - 1; v >= 0; --v) {                 // last variable fastest
        const u64 ext = (u64)sk->ext[v];
        if ((used >> v) & 1u) {
            if (stride >> 31 || ext >> 31) return sk->n_points;
            if (c) { c->proj_ext[k] = (u32)ext; c->proj_stride[k] = (u32)stride; }
            ++k;
            n *= ext;
            if (n >> 31) return sk->n_points;
        }
        stride *= ext;
    }
    if (c) c->n_proj_vars = k;
    return (i64)n;
}

// Point id in the full box of point q of the sub-box.
__device__ __forceinline__ i64 proj_pid(const CandShared& c, i64 q) {
    u32 rem = (u32)q, pid = 0;
    for (int k = 0; k < c.n_proj_vars; ++k) {
        const u32 e = c.proj_ext[k], d = rem / e;
        pid += (rem - d * e) * c.proj_stride[k];
        rem = d;
    }
    return (i64)pid;
}

// Stage 3 core: one WARP checks the staged candidate on the points [first, last), 32 points
// per step; a failing point anywhere ends the scan at the next warp vote.  Returns true if
// every point passed; adds the points tried by this lane to evals.
// Fast form: points and spec values come from tables in HBM (the caller's, or staged at load)
// and the program runs on a register stack.  Otherwise coordinates are derived from the point
// id and the interpreters with a stack in local memory are used.
// On failure *fail_pid is the domain point id of one point that failed (the same for all lanes).
template <int D>
__device__ __forceinline__ bool check_points_fast(const CandShared& c, const SketchDev* sk, const HoleDev* hole,
                                                  i64 first, i64 last, u64& evals, i64* fail_pid) {
    const int nv = sk->n_vars;
    const int lane = threadIdx.x & 31;
    for (i64 base = first; base < last; base += 32) {
        bool bad = false;
        if (base + lane < last) {
            i64 pid = c.n_proj_vars ? proj_pid(c, base + lane) : base + lane;
            if (!XP_CHECKED(pid >= 0 && pid < sk->n_points, kChkPoint)) pid = 0;
            ++evals;
            i64 v;
            bad = !run_program<D>(c, sk->coords + pid * nv, v) || v != hole->spec_table[pid];
        }
        const u32 bm = __ballot_sync(0xffffffffu, bad);
        if (bm) {
            const i64 q = base + (__ffs((int)bm) - 1);
            *fail_pid = c.n_proj_vars ? proj_pid(c, q) : q;
            return false;
        }
    }
    return true;
}

// Stage 3, the form the verification kernel uses: every lane runs the staged program on P
// points at once (points base + i*32 + lane, so that the table reads of a step are coalesced),
// 32*P points per step and warp vote.  The top of the operand stack is kept in registers; the
// entries below it live in shared memory, one 16-byte slot per lane and level (read and
// written as one vector access).  T = i32 with P = 4 when the program is proved exact in
// int32 (CandShared::narrow), else T = i64 with P = 2.  The program is the same for all
// lanes, so the dispatch branches are uniform.  Points and spec values come from the tables.
constexpr int kVecDepth = 8;                              // deepest operand stack this form takes
template <typename T, int P> union VecSlot { uint4 q; T v[P]; };

// One operator of a staged program on P points at once.  Binary: t = a op t.  The folded constant
// divisions (int32 programs only; kval = the constant and floor(2^32 / |constant|)) work on t alone.
// `bad` collects zero divisors.
template <typename T, int P>
__device__ __forceinline__ void vec_op(int op, i64 kval, const VecSlot<T, P>& a, VecSlot<T, P>& t, bool& bad) {
    if (sizeof(T) == 4 && op >= kOpDivC) {                // x / c or x % c, c != 0 a constant
        const i32 d = (i32)(u32)(u64)kval;
        const u32 M = (u32)((u64)kval >> 32), ad = d < 0 ? 0u - (u32)d : (u32)d;
#pragma unroll
        for (int i = 0; i < P; ++i) {
            const i32 x = (i32)t.v[i];
            const u32 ux = x < 0 ? 0u - (u32)x : (u32)x;      // |x| < 2^31: the estimate is the quotient or one less
            u32 q = __umulhi(ux, M), r = ux - q * ad;
            if (r >= ad) { ++q; r -= ad; }
            t.v[i] = (T)(op == kOpDivC ? (((x < 0) != (d < 0)) ? (i32)(0u - q) : (i32)q) : (x < 0 ? (i32)(0u - r) : (i32)r));
        }
        return;
    }
    if (sizeof(T) == 8) {
#pragma unroll
        for (int i = 0; i < P; ++i) {
            i64 r = 0;
            bad |= !apply_op(op, (i64)a.v[i], (i64)t.v[i], r);
            t.v[i] = (T)r;
        }
        return;
    }
    switch (op) {                                         // int32: no result can overflow (proved at staging)
#define XP_EACH(expr) _Pragma("unroll") for (int i = 0; i < P; ++i) { const i32 x = (i32)a.v[i], y = (i32)t.v[i]; t.v[i] = (T)(expr); } break;
        case XP_OP_ADD: XP_EACH(x + y)
        case XP_OP_SUB: XP_EACH(x - y)
        case XP_OP_MUL: XP_EACH(x * y)
        case XP_OP_DIV:
        case XP_OP_MOD:
#pragma unroll
            for (int i = 0; i < P; ++i) {
                const i32 x = (i32)a.v[i], y = (i32)t.v[i];
                bad |= y == 0;
                const i32 d = y == 0 ? 1 : y;             // |x| < 2^31, so x / -1 does not overflow
                const i32 q = x / d;
                t.v[i] = (T)(op == XP_OP_DIV ? q : x - q * d);
            }
            break;
        case XP_OP_LT: XP_EACH(x < y)
        case XP_OP_LE: XP_EACH(x <= y)
        case XP_OP_EQ: XP_EACH(x == y)
        case XP_OP_NE: XP_EACH(x != y)
        case XP_OP_MIN: XP_EACH(x < y ? x : y)
        case XP_OP_MAX: XP_EACH(x > y ? x : y)
        case XP_OP_AND: XP_EACH((x != 0) & (y != 0))
        case XP_OP_OR: XP_EACH((x != 0) | (y != 0))
        case XP_OP_SHR:                                   // (a left shift never stays in an int32 program: its bound saturates)
#pragma unroll
            for (int i = 0; i < P; ++i) {
                const i32 x = (i32)a.v[i], y = (i32)t.v[i];
                bad |= y < 0 || y > 63;
                t.v[i] = (T)(x >> (y > 31 ? 31 : (y < 0 ? 0 : y)));
            }
            break;
#undef XP_EACH
        default: bad = true; break;
    }
}

template <typename T, int P>
__device__ __forceinline__ bool check_points_vec(const CandShared& c, uint4* __restrict__ stack, const SketchDev* sk,
                                                 const HoleDev* hole, i64 first, i64 last, i64* fail_pid) {
    static_assert(sizeof(T) * P == sizeof(uint4), "one stack level of a lane is one 16-byte slot");
    const int nv = sk->n_vars;
    const int lane = threadIdx.x & 31;
    const int n = c.len;
    const i32* __restrict__ coords = sk->coords;
    const i64* __restrict__ spec = hole->spec_table;
    typedef VecSlot<T, P> Slot;
    for (i64 base = first; base < last; base += 32 * P) {
        const i32* row[P];
        i64 want[P];
        bool in[P];
#pragma unroll
        for (int i = 0; i < P; ++i) {
            const i64 pid = base + i * 32 + lane;
            in[i] = pid < last;
            i64 at = in[i] ? pid : first;                 // lanes past the end repeat a valid point
            if (c.n_proj_vars) at = proj_pid(c, at);      // (uniform branch)
            if (!XP_CHECKED(at >= 0 && at < sk->n_points, kChkPoint)) at = 0;
            row[i] = coords + at * nv;
            want[i] = spec[at];
        }
        Slot t;
#pragma unroll
        for (int i = 0; i < P; ++i) t.v[i] = 0;
        bool bad = false;
        int below = 0;                                    // entries under the top of the stack
        for (int k = 0; k < n; ++k) {
            const i32 cv = c.var[k];
            if (cv >= -1) {
                stack[below * 32 + lane] = t.q;           // (the very first push stores an unused slot)
                ++below;
                if (cv >= 0) {
#pragma unroll
                    for (int i = 0; i < P; ++i) t.v[i] = (T)row[i][cv];
                } else {
                    const T v = (T)c.val[k];
#pragma unroll
                    for (int i = 0; i < P; ++i) t.v[i] = v;
                }
                continue;
            }
            const int op = -2 - cv;
            Slot a;
            a.q = t.q;
            if (!(sizeof(T) == 4 && op >= kOpDivC)) { --below; a.q = stack[below * 32 + lane]; }
            vec_op<T, P>(op, c.val[k], a, t, bad);
        }
        // a zero divisor at a repeated point is a zero divisor at a real point of this candidate
        // too (the repeated point is `first`, which lane 0 holds in range), so `bad` needs no mask
        u32 which = bad ? 1u : 0u;                        // bit i: this lane's point i failed (a zero divisor: point 0)
#pragma unroll
        for (int i = 0; i < P; ++i) which |= (u32)(in[i] && (i64)t.v[i] != want[i]) << i;
        const u32 bm = __ballot_sync(0xffffffffu, which != 0u);
        if (bm) {
            const int src = __ffs((int)bm) - 1;
            const u32 w = __shfl_sync(0xffffffffu, which, src);
            const i64 q = base + (i64)(__ffs((int)w) - 1) * 32 + src;
            const i64 qq = q < last ? q : first;
            *fail_pid = c.n_proj_vars ? proj_pid(c, qq) : qq;
            return false;
        }
    }
    return true;
}

__device__ __noinline__ bool check_points(const CandShared& c, const SketchDev* sk, const HoleDev* hole, i64 first,
                                          i64 last, u64& evals, i64* fail_pid) {
    if (sk->coords != nullptr && hole->spec_table != nullptr && c.depth >= 1) {
        if (c.depth <= 4) return check_points_fast<4>(c, sk, hole, first, last, evals, fail_pid);
        if (c.depth <= 8) return check_points_fast<8>(c, sk, hole, first, last, evals, fail_pid);
    }
    const int n = c.cand_len;
    const int lane = threadIdx.x & 31;
    for (i64 base = first; base < last; base += 32) {
        bool bad = false;
        if (base + lane < last) {
            const i64 pid = c.n_proj_vars ? proj_pid(c, base + lane) : base + lane;
            ++evals;
            i64 pt[kMaxVars];
            point_coords(sk, pid, pt);
            i64 want = 0;
            bool ok = true;
            if (hole->spec_table != nullptr) want = hole->spec_table[pid];
            else ok = eval_code(hole->spec, hole->spec_len, pt, 0, want);
            i64 st[kCandStack];
            int sp = 0;
            for (int k = 0; k < n && ok; ++k) {
                const i32 cv = c.cvar[k];
                if (cv >= -1) st[sp++] = cv >= 0 ? pt[cv] : c.cval[k];
                else {
                    const i64 b = st[--sp];
                    i64 r;
                    ok = apply_op(-2 - cv, st[sp - 1], b, r);
                    st[sp - 1] = r;
                }
            }
            bad = !ok || !ctx_matches(hole, pt, st[0], want);
        }
        const u32 bm = __ballot_sync(0xffffffffu, bad);
        if (bm) {
            const i64 q = base + (__ffs((int)bm) - 1);
            *fail_pid = c.n_proj_vars ? proj_pid(c, q) : q;
            return false;
        }
    }
    return true;
}

// A candidate that passed the probes goes into the global queue for the verification kernel.
// Returns false if the queue is full: the caller's warp then checks the candidate itself.
__device__ __forceinline__ bool push_survivor(const PlanDev& plan, const SegDev& seg, u64 rank, u32 vars) {
    // (the counter saturates: once the queue is full nothing is added, so it cannot wrap around
    // and hand out a slot twice however many survivors a search has)
    if (*(volatile const u32*)plan.surv_n >= plan.surv_cap) return false;
    const u32 at = atomicAdd(plan.surv_n, 1u);
    if (at >= plan.surv_cap) return false;
    SurvDev r;
    r.rank = rank; r.sketch = seg.sketch; r.hole = seg.hole; r.size = seg.size; r.acc = seg.acc;
    r.state = 0; r.vars = vars;
    plan.surv[at] = r;
    if (plan.surv_hist) atomicAdd(&plan.surv_hist[r.acc], 1u);       // (for the hole order the verification walks)
    return true;
}

// The warp checks one candidate on the whole domain itself and records a match in the CTA's
// private results.  Called by all 32 lanes together.
__device__ __noinline__ void warp_verify(EvalShared& sh, const SketchDev* sk, const HoleDev* hole, int size, u64 rank,
                                         u64& my_evals) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) stage_candidate(sh.wcand[warp], sk, hole, size, rank);
    __syncwarp();
    i64 fail_pid = 0;
    const bool ok = check_points(sh.wcand[warp], sk, hole, 0, sk->n_points, my_evals, &fail_pid);
    if (ok && lane == 0) {
        atomicAdd(&sh.match_count[size], 1ull);
        atomicMin(&sh.min_rank[size], rank);
    }
    __syncwarp();
}

// Lanes holding a survivor that the global queue did not take hand it to their warp, one
// after the other.  Called by all 32 lanes together.
__device__ __forceinline__ void warp_verify_pending(EvalShared& sh, const SketchDev* sk, const HoleDev* hole, int size,
                                                    bool pending, u64 rank, u64& my_evals) {
    u32 m = __ballot_sync(0xffffffffu, pending);
    while (m) {
        const int src = __ffs((int)m) - 1;
        m &= m - 1;
        const u64 r = __shfl_sync(0xffffffffu, rank, src);
        warp_verify(sh, sk, hole, size, r, my_evals);
    }
}

// Adds a per-lane count over the warp into a counter of the CTA's private results.
__device__ __forceinline__ void warp_tally(u64* counter, u32 mine) {
    for (int o = 16; o > 0; o >>= 1) mine += __shfl_down_sync(0xffffffffu, mine, o);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(counter, (u64)mine);
}

// A linear ticket: kLinearChunk consecutive ranks, each unranked and checked on its own.
__device__ __noinline__ void linear_ticket(EvalShared& sh, const PlanDev& plan, const SketchDev* sk, const HoleDev* hole,
                                          u64 local, u64& my_evals) {
    const SegDev& seg = sh.seg;
    const GrammarDev* g = sk->g;
    const u64 first = seg.rank_begin + local * (u64)kLinearChunk;
    u32 passes = 0;
    for (int i = 0; i < kLinearPerThread; ++i) {
        const u64 rank = first + (u64)i * kThreads + threadIdx.x;
        bool pending = false;
        if (rank < seg.rank_end) {
            u32 code[kMaxSize];
            const int n = unrank(g, hole->start_nt, seg.size, rank, code);
            if (probe_check(g, hole, code, n, my_evals)) {
                ++passes;
                u32 vars = 0;
                for (int k = 0; k < n; ++k)
                    if (!(code[k] & kOpBit)) { const i32 var = g->leaves[code[k]].var; if (var >= 0) vars |= 1u << var; }
                pending = !push_survivor(plan, seg, rank, vars);
            }
        }
        warp_verify_pending(sh, sk, hole, seg.size, pending, rank, my_evals);
    }
    warp_tally(&sh.filter_survivors, passes);
    warp_tally(&sh.probe_survivors, passes);
}


// ------------------------------------------------------------------------------------------
// stage 1: probe-point filter over a product of operand tiles
// ------------------------------------------------------------------------------------------
//
// A tile ticket covers candidates  L op R  for one group of productions and one left size:
// kRegTile subtrees of one operand (kNA per thread, in registers) times up to kBcTile subtrees
// of the other (in shared memory, read as warp-wide broadcasts).  Each operand subtree is
// unranked and evaluated ONCE at probe 0; a candidate then costs one operation and one
// comparison.  Everything the filter lets through is re-checked exactly (stage 2), so the
// filter only has to be a necessary condition:
//   * operands that fit int32 are combined in 32-bit arithmetic and compared with the low
//     32 bits of the target (+ - * commute with reduction mod 2^32; / and % of int32 operands
//     are exact);
//   * an affine context  A*h + B  is folded into the operands (ring operators) or applied to
//     the quotient / remainder;
//   * everything that depends on one operand only is computed when the tile is filled, so a
//     candidate costs one comparison for + and -, a multiply-add and a minimum for *, and for / and %
//     a range test and a divisibility test on magnitudes (see ring_pass and div_pass).

__device__ __forceinline__ u32 abs_u32(i32 x) { return x < 0 ? 0u - (u32)x : (u32)x; }

__device__ __forceinline__ void push_hit(EvalShared& sh, u32 reg_idx, u32 slot, u32 opi) {
    const int warp = threadIdx.x >> 5;
    const u32 at = atomicAdd(&sh.wq_n[warp], 1u);
    if (at < (u32)kWarpQueue) sh.queue[warp][at] = reg_idx | (slot << 11) | (opi << 21) | (sh.wmember[warp] << 24);
    else sh.wq_over[warp] = 1u;
}

// Value of the subtree (nt, size, rank) at the hole's probe `pr` (one the hole has tables
// for); false when a divisor is zero.  Small sizes come from the hole's subtree-value
// tables; a larger subtree whose operands are both in the tables costs one level of unranking;
// anything else is unranked in full.
__device__ __noinline__ bool operand_value(const GrammarDev* g, const HoleDev* hole, int pr, int nt, int size, u64 rank, i64& v) {
    const int tmax = hole->tab_max_size;
    const u64 pbase = (u64)pr * hole->tab_total;
    if (pr == 0 && size == hole->big_size && hole->big_on) {
        const u64 at = hole->big_off[nt] + rank;
        v = hole->big_val[at];
        return hole->big_ok[at] != 0;
    }
    if (size <= tmax) {
        u64 at = pbase + hole->tab_off[nt][size] + rank;
        if (!XP_CHECKED(pr < hole->tab_probes && hole->tab_off[nt][size] + rank < hole->tab_total && rank < g->cnt[nt][size], kChkTable)) at = 0;
        v = hole->tab_val[at];
        return hole->tab_ok[at] != 0;
    }
    if (size == 1) {
        const LeafDev lf = g->leaves[g->leaf_begin[nt] + (i32)rank];
        v = lf.var >= 0 ? hole->probe_pt[pr][lf.var] : lf.value;
        return true;
    }
    if (tmax >= 1) {
        int op, lnt, rnt, a;
        u64 l, r;
        unrank_root(g, nt, size, rank, op, lnt, rnt, a, l, r);
        if (a <= tmax && size - 1 - a <= tmax) {
            const u64 la = pbase + hole->tab_off[lnt][a] + l, ra = pbase + hole->tab_off[rnt][size - 1 - a] + r;
            if (!hole->tab_ok[la] || !hole->tab_ok[ra]) return false;
            return apply_op(op, hole->tab_val[la], hole->tab_val[ra], v);
        }
    }
    u32 code[kMaxSize];
    const int n = unrank(g, nt, size, rank, code);
    return eval_cand(code, n, g->leaves, hole->probe_pt[pr], v);
}

// Variables that the subtree (nt, size, rank) mentions, from the tables where they reach (one
// level of unranking above them); all variables otherwise, which is always a safe answer.
__device__ __noinline__ u32 operand_vars(const GrammarDev* g, const HoleDev* hole, int nt, int size, u64 rank) {
    const int tmax = hole->tab_max_size;
    if (size <= tmax) return hole->tab_vars[hole->tab_off[nt][size] + rank];
    if (tmax >= 1 && size >= 3) {
        int op, lnt, rnt, a;
        u64 l, r;
        unrank_root(g, nt, size, rank, op, lnt, rnt, a, l, r);
        if (a <= tmax && size - 1 - a <= tmax)
            return (u32)hole->tab_vars[hole->tab_off[lnt][a] + l] | (u32)hole->tab_vars[hole->tab_off[rnt][size - 1 - a] + r];
    }
    return 0xffu;
}

// Values at probe `pr` of `n` (<= kNA) consecutive subtrees of (nt, size) starting at `rank`, written
// to lo[j] (and hi[j] for the high words unless hi is null); returns the mask of those that are defined there and, in `fits`, of those that fit int32.
// A subtree above the table sizes whose operands are in the tables is unranked one level for
// the first rank only; the following ranks advance the operand ranks like an odometer (right
// operand fastest), so the left operand's value is fetched once per run.
__device__ __noinline__ u32 fill_reg_operands(const GrammarDev* g, const HoleDev* hole, int pr, int nt, int size, u64 rank,
                                              int n, u32* lo, u32* hi, u32& fits) {
    u32 alive = 0;
    fits = 0;
    const int tmax = hole->tab_max_size;
    const u64 pbase = (u64)pr * hole->tab_total;
    for (int j = 0; j < kNA; ++j) { lo[j] = 0; if (hi) hi[j] = 0; }
    if (n <= 0) return 0;
    auto put = [&](int j, i64 v) {
        lo[j] = (u32)(u64)v;
        if (hi) hi[j] = (u32)((u64)v >> 32);
        alive |= 1u << j;
        if (v > -(1ll << 31) && v < (1ll << 31)) fits |= 1u << j;
    };
    int j = 0;
    if (pr == 0 && size == hole->big_size && hole->big_on) {      // tabulated at the first probe: consecutive entries
        const u64 at = hole->big_off[nt] + rank;
        if (n == kNA && (at & 7ull) == 0) {
            // the usual case: eight aligned entries, fetched with five independent loads
            const u64 oks = *reinterpret_cast<const u64*>(hole->big_ok + at);
            const longlong2* src = reinterpret_cast<const longlong2*>(hole->big_val + at);
            longlong2 v[kNA / 2];
#pragma unroll
            for (int k = 0; k < kNA / 2; ++k) v[k] = src[k];
#pragma unroll
            for (int k = 0; k < kNA / 2; ++k) {
                if ((oks >> (16 * k)) & 0xffull) put(2 * k, v[k].x);
                if ((oks >> (16 * k + 8)) & 0xffull) put(2 * k + 1, v[k].y);
            }
            return alive;
        }
        for (; j < n; ++j) if (hole->big_ok[at + j]) put(j, hole->big_val[at + j]);
        return alive;
    }
    if (size > tmax && tmax >= 1 && size >= 3) {
        int op, lnt, rnt, a;
        u64 l, r;
        unrank_root(g, nt, size, rank, op, lnt, rnt, a, l, r);
        bool tables = a <= tmax && size - 1 - a <= tmax;
        while (tables && j < n) {
            const u64 cl = g->cnt[lnt][a], cr = g->cnt[rnt][size - 1 - a];
            const u64 lbase = pbase + hole->tab_off[lnt][a], rbase = pbase + hole->tab_off[rnt][size - 1 - a];
            for (; j < n && l < cl; ++l, r = 0) {
                const bool lok = hole->tab_ok[lbase + l] != 0;
                const i64 lv = hole->tab_val[lbase + l];
                for (; j < n && r < cr; ++r, ++j) {
                    i64 v;
                    if (lok && hole->tab_ok[rbase + r] && apply_op(op, lv, hole->tab_val[rbase + r], v)) put(j, v);
                }
                if (j == n) break;
            }
            if (j < n) {                                  // ran off this (production, left size) block
                unrank_root(g, nt, size, rank + j, op, lnt, rnt, a, l, r);
                tables = a <= tmax && size - 1 - a <= tmax;
            }
        }
    }
    for (; j < n; ++j) {
        i64 v;
        if (operand_value(g, hole, pr, nt, size, rank + j, v)) put(j, v);
    }
    return alive;
}

// Staging of a box domain at load: the coordinates of every point (int32 rows, like a table
// domain) and, per hole with a spec expression, the spec's value at every point.  *bad is set
// if the spec is undefined somewhere (then no candidate can match).
__global__ void __launch_bounds__(256) stage_points_kernel(const SketchDev* sk, i32* coords) {
    const i64 pid = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (pid >= sk->n_points) return;
    const int nv = sk->n_vars;
    u64 rem = (u64)pid;
    for (int d = nv - 1; d >= 0; --d) {
        u64 q, r;
        divmod_u64(rem, (u64)sk->ext[d], q, r);
        coords[pid * nv + d] = (i32)(sk->lo[d] + (i64)r);
        rem = q;
    }
}

// Smallest and largest coordinate of every variable over the rows of a table domain, into the
// sketch (whose vmin / vmax start at the extreme values).  Warp shuffles, then one atomic pair
// per warp and variable.
__global__ void __launch_bounds__(256) coord_bounds_kernel(SketchDev* const* list) {
    SketchDev* sk = list[blockIdx.y];                   // one grid row per sketch of the batch
    if (sk->domain_kind != XP_DOMAIN_TABLE) return;
    const int nv = sk->n_vars;
    const i64 n = sk->n_points;
    for (int v = 0; v < nv; ++v) {
        i64 lo = LLONG_MAX, hi = LLONG_MIN;
        for (i64 pid = (i64)blockIdx.x * blockDim.x + threadIdx.x; pid < n; pid += (i64)gridDim.x * blockDim.x) {
            const i64 x = sk->coords[pid * nv + v];
            lo = x < lo ? x : lo;
            hi = x > hi ? x : hi;
        }
        for (int o = 16; o > 0; o >>= 1) {
            const i64 l2 = __shfl_down_sync(0xffffffffu, lo, o), h2 = __shfl_down_sync(0xffffffffu, hi, o);
            lo = l2 < lo ? l2 : lo;
            hi = h2 > hi ? h2 : hi;
        }
        if ((threadIdx.x & 31) == 0 && lo <= hi) { atomicMin(&sk->vmin[v], lo); atomicMax(&sk->vmax[v], hi); }
    }
}

__global__ void __launch_bounds__(256) stage_spec_kernel(const SketchDev* sk, int hole_index, i64* spec, u32* bad) {
    const i64 pid = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (pid >= sk->n_points) return;
    const HoleDev* hole = &sk->holes[hole_index];
    i64 pt[kMaxVars];
    point_coords(sk, pid, pt);
    i64 v = 0;
    if (!eval_code(hole->spec, hole->spec_len, pt, 0, v)) atomicOr(bad, 1u);
    spec[pid] = v;
}

// Bottom-up construction of one size of a hole's subtree-value tables: thread = (nonterminal,
// rank); the operands' values come from the smaller sizes built by earlier launches.
__global__ void __launch_bounds__(256) subvalue_kernel(const LoadJob* jobs, int size) {
    const SketchDev* sk = jobs[blockIdx.z].s;           // one grid layer per hole of the batch
    const int hole_index = jobs[blockIdx.z].hole;
    const int pr = blockIdx.y;                          // one grid row per probe
    const GrammarDev* g = sk->g;
    HoleDev* hole = &sk->holes[hole_index];
    if (pr >= hole->tab_probes || size > hole->tab_max_size) return;      // (the grid is sized for the most there can be)
    const u64 pbase = (u64)pr * hole->tab_total;
    u64 idx = (u64)blockIdx.x * blockDim.x + threadIdx.x;
    for (int nt = 0; nt < g->n_nt; ++nt) {
        const u64 c = g->cnt[nt][size];
        if (idx >= c) { idx -= c; continue; }
        i64 v = 0;
        bool ok = true;
        u32 vars = 0;
        if (size == 1) {
            const LeafDev lf = g->leaves[g->leaf_begin[nt] + (i32)idx];
            v = lf.var >= 0 ? hole->probe_pt[pr][lf.var] : lf.value;
            vars = lf.var >= 0 ? 1u << lf.var : 0u;
        } else {
            int op, lnt, rnt, a;
            u64 l, r;
            unrank_root(g, nt, size, idx, op, lnt, rnt, a, l, r);
            const u64 la = pbase + hole->tab_off[lnt][a] + l, ra = pbase + hole->tab_off[rnt][size - 1 - a] + r;
            ok = hole->tab_ok[la] && hole->tab_ok[ra] && apply_op(op, hole->tab_val[la], hole->tab_val[ra], v);
            vars = (u32)hole->tab_vars[hole->tab_off[lnt][a] + l] | (u32)hole->tab_vars[hole->tab_off[rnt][size - 1 - a] + r];
        }
        const u64 at = pbase + hole->tab_off[nt][size] + idx;
        hole->tab_val[at] = v;
        hole->tab_ok[at] = ok ? 1 : 0;
        if (pr == 0) hole->tab_vars[hole->tab_off[nt][size] + idx] = (unsigned char)vars;
        return;
    }
}

// The big table: values at probe 0 of every subtree of size big_size, from the smaller sizes'
// tables by one level of unranking.  A thread writes 8 consecutive entries of one nonterminal (the
// nonterminals' ranges start at multiples of 8): the first is unranked, the others follow by
// advancing the operand ranks like an odometer (right operand fastest).  The first thread turns
// the table on for the searches once the launch is under way for a hole whose smaller tables
// exist (the flag is read by later launches only).
constexpr int kBigPerThread = 8;
__global__ void __launch_bounds__(256) bigvalue_kernel(const LoadJob* jobs) {
    const SketchDev* sk = jobs[blockIdx.y].s;
    HoleDev* hole = &sk->holes[jobs[blockIdx.y].hole];
    const int size = hole->big_size;
    if (size <= 0 || hole->tab_probes < 1 || hole->tab_max_size != hole->tab_size_cap || hole->big_val == nullptr) return;
    const GrammarDev* g = sk->g;
    const u64 t = (u64)blockIdx.x * blockDim.x + threadIdx.x;
    if (t == 0) hole->big_on = 1;
    const u64 at0 = t * (u64)kBigPerThread;
    if (at0 >= hole->big_total) return;
    int nt = g->n_nt - 1;                               // the last nonterminal whose range starts at or before at0
    while (nt > 0 && hole->big_off[nt] > at0) --nt;
    const u64 c = g->cnt[nt][size], idx = at0 - hole->big_off[nt];
    if (idx >= c) return;                               // (padding between two nonterminals' ranges)
    const int n = c - idx < (u64)kBigPerThread ? (int)(c - idx) : kBigPerThread;
    // (local copies: the stores below cannot change them, which the compiler cannot know of fields of *hole)
    const i64* __restrict__ tab_val = hole->tab_val;
    const unsigned char* __restrict__ tab_ok = hole->tab_ok;
    i64* __restrict__ out_val = hole->big_val + at0;
    unsigned char* __restrict__ out_ok = hole->big_ok + at0;
    int j = 0;
    while (j < n) {
        int op, lnt, rnt, a;
        u64 l, r;
        unrank_root(g, nt, size, idx + j, op, lnt, rnt, a, l, r);
        const u64 cl = g->cnt[lnt][a], cr = g->cnt[rnt][size - 1 - a];
        const u64 lbase = hole->tab_off[lnt][a], rbase = hole->tab_off[rnt][size - 1 - a];      // (probe 0: first copy of the tables)
        while (j < n && l < cl) {                       // until this (production, left size) block ends
            const bool lok = tab_ok[lbase + l] != 0;
            const i64 lv = tab_val[lbase + l];
            for (; j < n && r < cr; ++r, ++j) {
                i64 v = 0;
                const bool ok = lok && tab_ok[rbase + r] && apply_op(op, lv, tab_val[rbase + r], v);
                out_val[j] = v;
                out_ok[j] = ok ? 1 : 0;
            }
            if (r == cr) { r = 0; ++l; }
        }
    }
}

// Inverse of an odd number modulo 2^32 (Newton: each step doubles the number of correct bits).
__device__ __forceinline__ u32 inv_odd(u32 o) {
    u32 x = o;                       // correct to 3 bits
    x *= 2u - o * x; x *= 2u - o * x; x *= 2u - o * x; x *= 2u - o * x;
    return x;
}

__device__ __forceinline__ u32 rotr32(u32 x, u32 k) { return __funnelshift_r(x, x, k); }

// The register-side operands of a thread for the ticket at hand: low and high words of the values
// at probe 0 and the values at probe 1 (second look).  The loops below are not inlined and get a
// pointer to this record; each copies the low words into registers when it starts and derives what
// it needs of them there (a handful of instructions per operand, once per call).  The record is
// kept this small on purpose: it lives in the thread's local memory, and the records of all
// resident threads together (96 bytes x 768 threads per SM) stay in the L1 cache, where a record
// with every derived array (ten times the size) did not and went through L2 to DRAM on every tile.
struct RegVals { u32 lo[kNA], hi[kNA], p1[kNA]; };

// The second look: the candidate's exact value at probe 1 from its operands' values there,
// through the affine context, against the spec.  Operand values that are not known exactly in
// int32 pass (the exact stages decide).  Runs for filter hits only.
__device__ __noinline__ bool probe1_pass(const EvalShared& sh, int op, bool a_ok, i32 a1, u32 bc_meta, u32 b1, bool swap) {
    if (!sh.p1_on) return true;
    if (!a_ok || !(bc_meta >> 31)) return true;
    const i64 x = swap ? (i64)(i32)b1 : (i64)a1, y = swap ? (i64)a1 : (i64)(i32)b1;
    i64 v;
    if (!apply_op(op, x, y, v)) return false;
    if (sh.p1_rng) return v >= sh.p1_lo && v <= sh.p1_hi;
    return (u64)v * sh.p1_A + sh.p1_B == sh.p1_spec;
}
// (a1ok: bit j says that this thread's operand j is known exactly at probe 1)
#define XP_P1(op, j, s) probe1_pass(sh, op, (a1ok >> (j)) & 1u, (i32)R->p1[j], sh.bc_meta[s].meta, sh.bc_meta[s].pad, SWAP)

// The second look, first cut (dense form of the loops): the hits `m` of operator OP between this
// thread's operands and broadcast slot s are held against the spec at probe 1 in 32-bit arithmetic,
// inline.  It is a necessary condition for the exact test of probe1_pass (the low 32 bits of both
// sides must agree; a zero divisor makes the candidate undefined there), like the filter itself, so
// the few hits it leaves still go through that test.  Where the spec is small at the first probe and
// one candidate in a hundred agrees with it there, this keeps the out-of-line routines rare.
// Operands that are not known exactly at probe 1 are kept.  Returns the bits that remain.
template <int OP, bool SWAP>
__device__ __forceinline__ u32 p1_first_cut(const EvalShared& sh, const RegVals* R, u32 a1ok, int s, u32 m) {
    if (!sh.p1_on || sh.p1_rng) return m;
    const u32 meta = sh.bc_meta[s].meta;
    if (!(meta >> 31)) return m;
    const u32 b1 = sh.bc_meta[s].pad, A1 = (u32)sh.p1_A, t1 = (u32)sh.p1_spec - (u32)sh.p1_B;
    u32 out = m & ~a1ok;
    for (u32 k = m & a1ok; k; k &= k - 1) {
        const int j = __ffs((int)k) - 1;
        const u32 a1 = R->p1[j];
        const u32 x = SWAP ? b1 : a1, y = SWAP ? a1 : b1;
        u32 v;
        bool ok = true;
        if (OP == XP_OP_ADD) v = x + y;
        else if (OP == XP_OP_SUB) v = x - y;
        else if (OP == XP_OP_MUL) v = x * y;
        else {                                          // / and %: exact in int32 but for the one quotient that leaves it
            ok = y != 0u;
            const i32 d = ok ? (i32)y : 1;
            if (OP == XP_OP_DIV) v = y == 0xffffffffu ? 0u - x : (u32)((i32)x / d);
            else v = y == 0xffffffffu ? 0u : (u32)((i32)x % d);
        }
        if (ok && v * A1 == t1) out |= 1u << j;
    }
    return out;
}

// The loops below are separate (not inlined) functions on purpose: each copies the thread's
// register-side operands into registers, derives what it needs of them and runs with a small
// live set, instead of sharing one large frame with the rest of the kernel.
// `opip` packs the index of each operator inside the segment's list, 3 bits per operator.

// Position of a grammar operator among the seven a segment may hold: + - * / % min max.
__device__ __forceinline__ int op_slot(int op) { return op <= XP_OP_MOD ? op : op - XP_OP_MIN + 5; }
constexpr int kSlotMin = 5;                         // (max follows at 6)

// x and -x have the same sign-free form: the smaller of the two as unsigned numbers.
__device__ __forceinline__ u32 signfree(u32 x) { const u32 y = 0u - x; return x < y ? x : y; }

// The rare paths of the loops below: a warp vote said that some lane has a hit among the
// candidates of broadcast slot s.  Each lane repeats its tests from registers and collects bit
// sets of the register operands that hit; a lane with a non-empty set calls one of these
// compact functions, which walks the set bits, looks at each hit once more at probe 1 (when
// the hole has that second look) and queues what is left.  Keeping this part out of line and
// rolled keeps the loops' instruction footprint small, which matters where the filter is not
// selective (small value ranges) and the rare path is not rare.
__device__ __noinline__ void emit_ring(EvalShared& sh, const RegVals* R, u32 a1ok, int s, u32 m_as, u32 m_mul, u32 A, u32 tp, u32 opip,
                                       u32 mask, bool SWAP) {
    const BcRing e = sh.bc_ring[s];
    const u32 t_sub = SWAP ? 0u - e.t_add : 2u * tp - e.t_add;
    for (u32 m = m_as; m; m &= m - 1) {                 // + and -: which of the two (or both) it was
        const int j = __ffs((int)m) - 1;
        const u32 a = R->lo[j] * A;
        const u32 idx = threadIdx.x * (u32)kNA + (u32)j;
        if ((mask & 1u) && a == e.t_add && XP_P1(XP_OP_ADD, j, s)) push_hit(sh, idx, (u32)s, (opip >> (3 * XP_OP_ADD)) & 7u);
        if ((mask & 2u) && a == t_sub && XP_P1(XP_OP_SUB, j, s)) push_hit(sh, idx, (u32)s, (opip >> (3 * XP_OP_SUB)) & 7u);
    }
    for (u32 m = m_mul; m; m &= m - 1) {
        const int j = __ffs((int)m) - 1;
        if (XP_P1(XP_OP_MUL, j, s)) push_hit(sh, threadIdx.x * (u32)kNA + (u32)j, (u32)s, (opip >> (3 * XP_OP_MUL)) & 7u);
    }
}

__device__ __noinline__ void emit_pairs(EvalShared& sh, const RegVals* R, u32 a1ok, int s, u32 m0, int op0, u32 m1, int op1, u32 opip,
                                        bool SWAP) {
    for (u32 m = m0; m; m &= m - 1) {
        const int j = __ffs((int)m) - 1;
        if (XP_P1(op0, j, s)) push_hit(sh, threadIdx.x * (u32)kNA + (u32)j, (u32)s, (opip >> (3 * op_slot(op0))) & 7u);
    }
    for (u32 m = m1; m; m &= m - 1) {
        const int j = __ffs((int)m) - 1;
        if (XP_P1(op1, j, s)) push_hit(sh, threadIdx.x * (u32)kNA + (u32)j, (u32)s, (opip >> (3 * op_slot(op1))) & 7u);
    }
}

// Ring operators on int32-exact operands, mod 2^32, for the broadcast slots [s0, s1).
// MASK: bit0 +, bit1 -, bit2 *.  The comparisons were brought to the register operand's side
// when the tile was filled (tp = low 32 bits of target - B):
//   A*(a + b) == tp  <=>  A*a == tp - A*b  (= t_add);   A*(a * b) == tp  <=>  (A*a) * b == tp;
//   A*(a - b) == tp  <=>  A*a == tp + A*b;              A*(b - a) == tp  <=>  A*a == A*b - tp.
// When + and - are both present they share one comparison: without SWAP the two wanted values
// are tp -+ A*b, i.e. A*a - tp == -+ A*b; with SWAP they are +-(tp - A*b).  Either way the pair
// hits iff the sign-free forms agree: ca == t_pm.  Which of the two hit is settled in the rare
// path, from t_add.
// Broadcast operands per warp vote.  A vote that fires makes every lane repeat the group's tests,
// so the group is large where hits are rare (the vote and the loop control are shared by more
// candidates) and small where they are frequent (DENSE).  The choice is made per launch, not per
// hole: the search kernel exists in both forms and the host launches the dense one when a hole of
// the plan takes the second look.  (Both sets of loops inside one kernel cost the batch workload a
// tenth of its time in instruction-cache misses although only one set ever runs there.)
template <bool DENSE> struct VoteGroup { static constexpr int kRing = DENSE ? 4 : 8, kDiv = DENSE ? 2 : 4; };

template <u32 MASK, bool SWAP, bool DENSE>
__device__ __noinline__ void ring_pass(EvalShared& sh, const RegVals* R, u32 alive, u32 a1ok, u32 A, u32 tp, int s0, int s1, u32 opip) {
    constexpr bool kPair = (MASK & 3u) == 3u;
    constexpr int kRingGroup = VoteGroup<DENSE>::kRing;
    u32 aA[kNA], ca[kNA];                               // A * value, and the sign-free form for the joint +/- test
#pragma unroll
    for (int j = 0; j < kNA; ++j) {
        aA[j] = R->lo[j] * A;
        ca[j] = signfree(SWAP ? aA[j] : aA[j] - tp);
    }
    auto t_sub_of = [&](u32 t_add) { return SWAP ? 0u - t_add : 2u * tp - t_add; };
    // The products' distances from the target (one multiply-add each, mul_nt = -tp) are folded
    // into running minima: a candidate hits iff its distance is zero, so one comparison per vote
    // group replaces one per candidate.
    auto scan = [&](const BcRing& e, bool (&h)[4], u32 (&m)[4]) {
        const u32 t_one = (MASK & 1u) ? e.t_add : t_sub_of(e.t_add);       // used when only one of + - is present
#pragma unroll
        for (int j = 0; j < kNA; ++j) {
            if (kPair) h[j & 3] |= ca[j] == e.t_pm;
            else if (MASK & 3u) h[j & 3] |= aA[j] == t_one;
            if (MASK & 4u) {
                const u32 d = aA[j] * e.mul_b + e.mul_nt;
                m[j & 3] = d < m[j & 3] ? d : m[j & 3];
            }
        }
    };
    auto resolve = [&](int s) {                          // the rare path: which candidates hit
        const BcRing e = sh.bc_ring[s];
        const u32 t_one = (MASK & 1u) ? e.t_add : t_sub_of(e.t_add);
        u32 m_as = 0, m_mul = 0;
#pragma unroll
        for (int j = 0; j < kNA; ++j) {
            if (kPair) m_as |= (u32)(ca[j] == e.t_pm) << j;
            else if (MASK & 3u) m_as |= (u32)(aA[j] == t_one) << j;
            if (MASK & 4u) m_mul |= (u32)(aA[j] * e.mul_b + e.mul_nt == 0u) << j;
        }
        m_as &= alive; m_mul &= alive;
        if (DENSE) {
            if (MASK & 3u) m_as = ((MASK & 1u) ? p1_first_cut<XP_OP_ADD, SWAP>(sh, R, a1ok, s, m_as) : 0u) |
                                  ((MASK & 2u) ? p1_first_cut<XP_OP_SUB, SWAP>(sh, R, a1ok, s, m_as) : 0u);
            if (MASK & 4u) m_mul = p1_first_cut<XP_OP_MUL, SWAP>(sh, R, a1ok, s, m_mul);
        }
        if (m_as | m_mul) emit_ring(sh, R, a1ok, s, m_as, m_mul, A, tp, opip, MASK, SWAP);
    };
    // One warp vote per kRingGroup broadcast operands (fewer at the end of the run).  The rare path has
    // a single, rolled call site: its code is large, and every copy of it competes with the loops
    // for the instruction cache.
    for (int s = s0; s < s1; s += kRingGroup) {
        const int n = s1 - s < kRingGroup ? s1 - s : kRingGroup;
        bool h[4] = {false, false, false, false};       // independent chains of comparisons
        u32 m[4] = {0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu};       // ... and of minima
        if (n == kRingGroup) {
#pragma unroll
            for (int q0 = 0; q0 < kRingGroup; q0 += 4) {
                const BcRing e0 = sh.bc_ring[s + q0], e1 = sh.bc_ring[s + q0 + 1], e2 = sh.bc_ring[s + q0 + 2], e3 = sh.bc_ring[s + q0 + 3];
                scan(e0, h, m);
                scan(e1, h, m);
                scan(e2, h, m);
                scan(e3, h, m);
            }
        } else {
#pragma unroll 1
            for (int q = 0; q < n; ++q) { const BcRing e0 = sh.bc_ring[s + q]; scan(e0, h, m); }
        }
        const u32 mm = (m[0] < m[1] ? m[0] : m[1]) < (m[2] < m[3] ? m[2] : m[3]) ? (m[0] < m[1] ? m[0] : m[1]) : (m[2] < m[3] ? m[2] : m[3]);
        if (__any_sync(0xffffffffu, h[0] | h[1] | h[2] | h[3] | (mm == 0u))) {
#pragma unroll 1
            for (int q = 0; q < n; ++q) resolve(s + q);
        }
    }
}

// The divisors 0 and +-1 among the broadcast operands (register operand / broadcast operand) sit
// in a run of their own: 0 is skipped (invalid), +-1 gives |quotient| = |dividend| and remainder
// 0.  There are at most a few such slots per tile, so this is a small rolled routine rather than
// another instance of the loop below.
__device__ __noinline__ void div_special(EvalShared& sh, const RegVals* R, u32 alive, u32 a1ok, u32 tabs, int s0, int s1, u32 opip, u32 mask) {
    constexpr bool SWAP = false;
    for (int s = s0; s < s1; ++s) {
        if (sh.bc_div[s].ub != 1u) continue;
        u32 mq = 0, mr = 0;
        for (int j = 0; j < kNA; ++j) {
            if ((mask & 1u) && abs_u32((i32)R->lo[j]) == tabs) mq |= 1u << j;
            if ((mask & 2u) && tabs == 0u) mr |= 1u << j;
        }
        mq &= alive; mr &= alive;
        const bool any = (mq | mr) != 0;
        if (__any_sync(0xffffffffu, any) && any) emit_pairs(sh, R, a1ok, s, mq, XP_OP_DIV, mr, XP_OP_MOD, opip, SWAP);
    }
}

// / and % on int32-exact operands with the context factor A == 1.  MASK: bit0 /, bit1 %.
// Only magnitudes are compared (|quotient| or |remainder| against tabs = |target|): still a
// necessary condition, the signs are settled by the exact check.  With n the dividend's and d
// the divisor's magnitude:
//   floor(n / d) == tabs  <=>  n - tabs*d < d            (unsigned; tabs*d precomputed)
//   n mod d == tabs       <=>  d divides n - tabs (and tabs < d, n >= tabs); for d = 2^k * o,
//                              d | x  <=>  rotr(x * o^-1, k) <= floor((2^32-1) / d).
// SWAP = false: register operand / broadcast operand; SWAP = true: broadcast / register.
// SPECIAL (without SWAP only): the slots hold the divisors 0 and +-1: 0 is skipped (invalid),
// +-1 gives |quotient| = |dividend| and remainder 0.
template <u32 MASK, bool SWAP, bool SPECIAL, bool DENSE>
__device__ __noinline__ void div_pass(EvalShared& sh, const RegVals* R, u32 alive, u32 a1ok, u32 tabs, int s0, int s1, u32 opip) {
    constexpr int kDivGroup = VoteGroup<DENSE>::kDiv;
    // ua: |value|.  xa: |value| - tabs as a dividend (register operand / broadcast operand).  With SWAP the
    // register operand is the DIVISOR: low = tabs * |value| (0x80000000 when that is 2^31 or more: never
    // matches), inv = inverse mod 2^32 of the odd part of |value|, kk = its trailing zero bits, cc =
    // floor((2^32-1) / |value|), or 0 when the remainder tabs is impossible.
    u32 ua[kNA], xa[kNA], low[kNA], inv[kNA], kk[kNA], cc[kNA];
#pragma unroll
    for (int j = 0; j < kNA; ++j) {
        ua[j] = abs_u32((i32)R->lo[j]);
        xa[j] = ua[j] >= tabs ? ua[j] - tabs : 1u;      // 1 is a multiple of no divisor >= 2
        if (SWAP) {
            low[j] = 0x80000000u; inv[j] = 1u; kk[j] = 0u; cc[j] = 0u;
            if (ua[j] != 0u) {
                const u64 lw = (u64)tabs * ua[j];
                if (lw < (1ull << 31)) low[j] = (u32)lw;
                kk[j] = (u32)__ffs((int)ua[j]) - 1u;
                inv[j] = inv_odd(ua[j] >> kk[j]);
                cc[j] = tabs < ua[j] ? 0xffffffffu / ua[j] : 0u;
            }
        }
    }
    // hits of register operand j against broadcast entry e (quotient, remainder)
    auto test = [&](const BcDiv& e, u32 ek, int j, bool& hq, bool& hr) {
        if (SWAP) {                 // e.ub: dividend magnitude; e.low: dividend - tabs (or 1)
            hq = (e.ub - low[j]) < ua[j];
            hr = rotr32(e.low * inv[j], kk[j]) <= cc[j];
        } else if (SPECIAL) {
            hq = e.ub == 1u && ua[j] == tabs;
            hr = e.ub == 1u && tabs == 0u;
        } else {                    // e.low: tabs * divisor (or never); e.ub: divisor magnitude
            hq = (ua[j] - e.low) < e.ub;
            hr = rotr32(xa[j] * e.inv, ek) <= e.cmax;
        }
    };
    auto scan = [&](const BcDiv& e, u32 ek, bool& h0, bool& h1, bool& h2, bool& h3) {
#pragma unroll
        for (int j = 0; j < kNA; j += 2) {
            bool q0, r0, q1, r1;
            test(e, ek, j, q0, r0);
            test(e, ek, j + 1, q1, r1);
            if (MASK & 1u) { h0 |= q0; h1 |= q1; }
            if (MASK & 2u) { h2 |= r0; h3 |= r1; }
        }
    };
    const bool need_k = !SWAP && !SPECIAL && (MASK & 2u);
    auto resolve = [&](int s) {
        const BcDiv e = sh.bc_div[s];
        const u32 ek = need_k ? (sh.bc_meta[s].meta >> 16) & 63u : 0u;
        u32 mq = 0, mr = 0, nz = 0;
#pragma unroll
        for (int j = 0; j < kNA; ++j) {
            bool hq, hr;
            test(e, ek, j, hq, hr);
            if (MASK & 1u) mq |= (u32)hq << j;
            if (MASK & 2u) mr |= (u32)hr << j;
            nz |= (u32)(ua[j] != 0u) << j;
        }
        // register operands that are invalid, or (SWAP) zero divisors, are dropped here
        const u32 keep = SWAP ? alive & nz : alive;
        mq &= keep; mr &= keep;
        if (DENSE) {
            if (MASK & 1u) mq = p1_first_cut<XP_OP_DIV, SWAP>(sh, R, a1ok, s, mq);
            if (MASK & 2u) mr = p1_first_cut<XP_OP_MOD, SWAP>(sh, R, a1ok, s, mr);
        }
        if (mq | mr) emit_pairs(sh, R, a1ok, s, mq, XP_OP_DIV, mr, XP_OP_MOD, opip, SWAP);
    };
    for (int s = s0; s < s1; s += kDivGroup) {          // one warp vote per kDivGroup broadcast operands; one rare-path site
        const int n = s1 - s < kDivGroup ? s1 - s : kDivGroup;
        bool h0 = false, h1 = false, h2 = false, h3 = false;
        if (n == kDivGroup) {
#pragma unroll
            for (int q = 0; q < kDivGroup; ++q) {
                const BcDiv e = sh.bc_div[s + q];
                const u32 k = need_k ? (sh.bc_meta[s + q].meta >> 16) & 63u : 0u;
                scan(e, k, h0, h1, h2, h3);
            }
        } else {
#pragma unroll 1
            for (int q = 0; q < n; ++q) {
                const BcDiv e = sh.bc_div[s + q];
                const u32 k = need_k ? (sh.bc_meta[s + q].meta >> 16) & 63u : 0u;
                scan(e, k, h0, h1, h2, h3);
            }
        }
        if (__any_sync(0xffffffffu, h0 | h1 | h2 | h3)) {
#pragma unroll 1
            for (int q = 0; q < n; ++q) resolve(s + q);
        }
    }
}

// min and max of int32-exact operands (exact signed comparison), times the context factor A,
// against tp.  MASK: bit0 min, bit1 max.  Both are symmetric, so SWAP plays no role.
template <u32 MASK, bool HAS_A>
__device__ __noinline__ void minmax_pass(EvalShared& sh, const RegVals* R, u32 alive, u32 a1ok, u32 A, u32 tp, int s0, int s1, u32 opip) {
    i32 av[kNA];
#pragma unroll
    for (int j = 0; j < kNA; ++j) av[j] = (i32)R->lo[j];
    auto test = [&](i32 b, int j, bool& hmin, bool& hmax) {
        u32 lo = (u32)(av[j] < b ? av[j] : b), hi = (u32)(av[j] < b ? b : av[j]);
        if (HAS_A) { lo *= A; hi *= A; }
        hmin = lo == tp;
        hmax = hi == tp;
    };
    for (int s = s0; s < s1; ++s) {
        const i32 b = (i32)sh.bc_meta[s].lo;
        bool h0 = false, h1 = false, h2 = false, h3 = false;
#pragma unroll
        for (int j = 0; j < kNA; j += 2) {
            bool m0, x0, m1, x1;
            test(b, j, m0, x0);
            test(b, j + 1, m1, x1);
            if (MASK & 1u) { h0 |= m0; h1 |= m1; }
            if (MASK & 2u) { h2 |= x0; h3 |= x1; }
        }
        if (__any_sync(0xffffffffu, h0 | h1 | h2 | h3)) {
            u32 mmin = 0, mmax = 0;
#pragma unroll
            for (int j = 0; j < kNA; ++j) {
                bool hmin, hmax;
                test(b, j, hmin, hmax);
                if (MASK & 1u) mmin |= (u32)hmin << j;
                if (MASK & 2u) mmax |= (u32)hmax << j;
            }
            mmin &= alive; mmax &= alive;
            if (mmin | mmax) { constexpr bool SWAP = false; emit_pairs(sh, R, a1ok, s, mmin, XP_OP_MIN, mmax, XP_OP_MAX, opip, SWAP); }
        }
    }
}

// / and % on int32-exact operands under a context factor A != 1: signed results times A are
// compared with tp.  Plain 32-bit division; this form only serves sketches whose hole sits
// under a multiplication (small searches).
template <bool SWAP>
__device__ __noinline__ void div_pass_signed(EvalShared& sh, const RegVals* R, u32 alive, u32 a1ok, u32 mask, u32 A, u32 tp,
                                             int s0, int s1, u32 opip) {
    for (int s = s0; s < s1; ++s) {
        const i32 b = (i32)sh.bc_meta[s].lo;
        for (int j = 0; j < kNA; ++j) {
            if (!((alive >> j) & 1u)) continue;
            const i32 a = (i32)R->lo[j];
            const i32 n = SWAP ? b : a, d = SWAP ? a : b;
            if (d == 0) continue;
            const i32 q = n / d;                         // magnitudes are below 2^31: no overflow case
            const u32 r = (u32)n - (u32)q * (u32)d;
            const u32 idx = threadIdx.x * (u32)kNA + (u32)j;
            if ((mask & 8u) && (u32)q * A == tp && XP_P1(XP_OP_DIV, j, s)) push_hit(sh, idx, (u32)s, (opip >> (3 * XP_OP_DIV)) & 7u);
            if ((mask & 16u) && r * A == tp && XP_P1(XP_OP_MOD, j, s)) push_hit(sh, idx, (u32)s, (opip >> (3 * XP_OP_MOD)) & 7u);
        }
    }
}

// Any operator on int64 operands (tiles with an operand outside int32): exact, slow, rare.
// rng 1: the context compares (HoleDev::rng_lo) and the value must lie in [lo, hi] instead;
// rng 2: every defined value passes.
__device__ __noinline__ void wide_chunk(EvalShared& sh, const RegVals* R, u32 alive, u32 a1ok, bool swap, u64 A, u64 tq,
                                        int rng, i64 lo, i64 hi, int s0, int s1, int n_ops, const i32* ops) {
    const bool SWAP = swap;
    for (int s = s0; s < s1; ++s) {
        const i64 b = (i64)(((u64)sh.bc_meta[s].hi << 32) | sh.bc_meta[s].lo);
        for (int j = 0; j < kNA; ++j) {
            if (!((alive >> j) & 1u)) continue;
            const i64 aj = (i64)(((u64)R->hi[j] << 32) | R->lo[j]);
            for (int o = 0; o < n_ops; ++o) {
                i64 v;
                if (!apply_op(ops[o], swap ? b : aj, swap ? aj : b, v)) continue;
                if ((rng == 0 ? (u64)v * A == tq : (rng == 2 || (v >= lo && v <= hi))) && XP_P1(ops[o], j, s))
                    push_hit(sh, threadIdx.x * (u32)kNA + (u32)j, (u32)s, (u32)o);
            }
        }
    }
}

// Stage 2 over the warp's queue (lane = hit): exact values at the probes that have operand
// tables (two lookups, or one level of unranking over the tables, and one operation each);
// for the remaining probes the candidate is rebuilt by full unranking.  Survivors go to the
// global queue, or are checked by the warp itself when that is full.  Called by all 32 lanes.
__device__ __noinline__ void drain_queue(EvalShared& sh, const PlanDev& plan, const SketchDev* sk, const HoleDev* hole,
                                         u64& my_evals) {
    const GrammarDev* g = sk->g;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncwarp();
    const u32 nq = sh.wq_n[warp] < (u32)kWarpQueue ? sh.wq_n[warp] : (u32)kWarpQueue;
    if (nq == 0) return;
    // probes 0 .. n_tab-1 can be checked from the tables: the spec is defined and the context affine
    // (or a comparison) there
    int n_tab = 0;
    while (n_tab < hole->tab_probes && n_tab < hole->n_probe &&
           ((hole->probe_spec_ok & (hole->aff_okmask | hole->rng_okmask)) >> n_tab & 1u)) ++n_tab;
    u32 passes = 0;
    const int cand_size = sh.mseg[0].size;              // (the members of a family build candidates of one size)
    for (u32 base = 0; base < nq; base += 32) {
        const u32 i = base + lane;
        bool pending = false;
        u64 rank = 0;
        if (i < nq) {
            const u32 e = sh.queue[warp][i];
            const u64 reg_first = sh.wq_first[warp][(e >> 27) & (u32)(kQueueTags - 1)];
            const SegDev& seg = sh.mseg[(e >> 24) & 7u];
            const u32 opi = (e >> 21) & 7u;
            const u64 rr = reg_first + (e & 2047u);
            const u32 q_slot = XP_CHECKED(((e >> 11) & 1023u) < (u32)kBcTile && opi < (u32)seg.n_ops, kChkQueue) ? (e >> 11) & 1023u : 0u;
            const u64 br = sh.mb[(e >> 24) & 7u].bc_first + (sh.bc_meta[q_slot].meta & 0xffffu);
            const u64 l = seg.swap ? br : rr, r = seg.swap ? rr : br;
            rank = seg.op_base[opi] + l * seg.right_count + r;
            bool dead = rank < seg.rank_begin || rank >= seg.rank_end;
            if (!XP_CHECKED(rr < g->cnt[seg.reg_nt][seg.reg_size] && br < g->cnt[seg.bc_nt][seg.bc_size] &&
                            rank < g->cnt[hole->start_nt][seg.size], kChkQueue)) dead = true;
            for (int j = 0; j < n_tab && !dead; ++j) {
                ++my_evals;
                i64 rv, bv, v;
                dead = !operand_value(g, hole, j, seg.reg_nt, seg.reg_size, rr, rv) ||
                       !operand_value(g, hole, j, seg.bc_nt, seg.bc_size, br, bv) ||
                       !apply_op(seg.op[opi], seg.swap ? bv : rv, seg.swap ? rv : bv, v);
                if (dead) break;
                if ((hole->aff_okmask >> j) & 1u) dead = (u64)v * hole->aff_Aj[j] + hole->aff_Bj[j] != (u64)hole->probe_spec[j];
                else if (v > -(1ll << 62) && v < (1ll << 62)) dead = v < hole->rng_lo[j] || v > hole->rng_hi[j];
                // (a value of 2^62 or more in magnitude is left to the whole-domain check)
            }
            if (!dead && n_tab < hole->n_probe) {        // some probes have no tables: rebuild the candidate
                u32 code[kMaxSize];
                const int n = unrank(g, hole->start_nt, seg.size, rank, code);
                dead = !probe_check(g, hole, code, n, my_evals);
            }
            if (!dead) {
                ++passes;
                const u32 vars = sk->project ? operand_vars(g, hole, seg.reg_nt, seg.reg_size, rr) |
                                               operand_vars(g, hole, seg.bc_nt, seg.bc_size, br) : 0xffu;
                pending = !push_survivor(plan, seg, rank, vars);      // (the hit's own segment: the ticket at hand may be another's)
            }
        }
        warp_verify_pending(sh, sk, hole, cand_size, pending, rank, my_evals);
    }
    warp_tally(&sh.probe_survivors, passes);
    if (lane == 0) { atomicAdd(&sh.filter_survivors, (u64)nq); sh.wq_n[warp] = 0; sh.wq_age[warp] = 0; }
    __syncwarp();
}

// The exact check of the hits that wait in the warp's queue, for the hole they belong to.
__device__ __forceinline__ void drain_waiting(EvalShared& sh, const PlanDev& plan, u64& my_evals) {
    const SketchDev* qs = plan.sketches[sh.q_sketch];
    drain_queue(sh, plan, qs, &qs->holes[sh.q_hole], my_evals);
}

// What a piece of a tile needs beyond the member's and the hole's constants in shared memory.
constexpr u32 kPieceSpecial = 1u, kPieceWide = 2u, kPieceSkipMod = 4u;

// One piece of a tile: broadcast slots [s0, s1) of member m against the register operands in `alv`.
// Picks the loops for the member's operators; one copy of this dispatch serves every member and
// both call sites of a tile.
template <bool SWAP, bool DENSE>
__device__ __forceinline__ void run_piece_as(EvalShared& sh, const RegVals* R, u32 alv, u32 a1ok, int m, int s0, int s1, u32 flags) {
    const SegDev& seg = sh.mseg[m];
    const u32 mask = sh.mb[m].mask, opip = sh.mb[m].opip;
    const u64 A64 = sh.h_A, tq = sh.h_tq;
    const bool tile_wide = (flags & kPieceWide) != 0;
    const int rng = sh.h_aff_ok ? 0 : (tile_wide ? 2 : 1);
    if (tile_wide || rng) {
        wide_chunk(sh, R, alv, a1ok, SWAP, A64, tq, rng, sh.h_rng_lo, sh.h_rng_hi, s0, s1, seg.n_ops, seg.op);
        return;
    }
    const u32 A = (u32)A64, tp = (u32)tq;
    switch (mask & 7u) {
#define XP_RING(M) case M: ring_pass<M, SWAP, DENSE>(sh, R, alv, a1ok, A, tp, s0, s1, opip); break;
        XP_RING(1u) XP_RING(2u) XP_RING(3u) XP_RING(4u) XP_RING(5u) XP_RING(6u) XP_RING(7u)
#undef XP_RING
        default: break;
    }
    if (mask >> kSlotMin) switch ((mask >> kSlotMin) & 3u) {
#define XP_MM(M) case M: if (A != 1u) minmax_pass<M, true>(sh, R, alv, a1ok, A, tp, s0, s1, opip); \
                         else minmax_pass<M, false>(sh, R, alv, a1ok, A, tp, s0, s1, opip); break;
        XP_MM(1u) XP_MM(2u) XP_MM(3u)
#undef XP_MM
        default: break;
    }
    if (!(mask & 24u)) return;
    if (A != 1u) { div_pass_signed<SWAP>(sh, R, alv, a1ok, mask, A, tp, s0, s1, opip); return; }
    // With A == 1 a quotient or remainder of int32 operands can only equal a target of
    // magnitude below 2^31; its magnitude is what the unsigned loops compare with.
    const i64 T = (i64)tq;
    if (!(T > -(1ll << 31) && T < (1ll << 31))) return;    // no int32 quotient or remainder can be the target
    const u32 tabs = (u32)(T < 0 ? -T : T);
    const bool special = (flags & kPieceSpecial) != 0;
    switch ((flags & kPieceSkipMod) ? (mask >> 3) & 1u : (mask >> 3) & 3u) {
#define XP_DIV(M) case M: if (special && !SWAP) div_special(sh, R, alv, a1ok, tabs, s0, s1, opip, M); \
                          else div_pass<M, SWAP, false, DENSE>(sh, R, alv, a1ok, tabs, s0, s1, opip); break;
        XP_DIV(1u) XP_DIV(2u) XP_DIV(3u)
#undef XP_DIV
        default: break;
    }
}

template <bool DENSE>
__device__ __noinline__ void run_piece(EvalShared& sh, const RegVals* R, u32 alv, u32 a1ok, int m, int s0, int s1, u32 flags) {
    if (sh.mseg[m].swap) run_piece_as<true, DENSE>(sh, R, alv, a1ok, m, s0, s1, flags);
    else run_piece_as<false, DENSE>(sh, R, alv, a1ok, m, s0, s1, flags);
}

// Member m of the family on the ticket's register operands.
template <bool DENSE>
__device__ __forceinline__ void tile_body(EvalShared& sh, const PlanDev& plan, const SketchDev* sk, const HoleDev* hole, int m,
                                       u64 reg_first, u64 pairs, const RegVals* R, u32 a1ok, u32 alive, bool drain_at_end, u64& my_evals) {
    const SegDev& seg = sh.mseg[m];
    const MemberState& mbs = sh.mb[m];
    const bool SWAP = seg.swap != 0;
    const int nb = (int)mbs.n, bc_lo = mbs.lo, bc_hi = mbs.hi;
    const bool tile_wide = (sh.reg_wide | mbs.wide | seg.generic) != 0;
    const u64 tq = sh.h_tq;
    // a context that compares: interval test on int32-exact operands (results stay below 2^62 in
    // magnitude, where the interval is exact); wider operands are all passed on to the exact stages
    const int rng = sh.h_aff_ok ? 0 : (tile_wide ? 2 : 1);
    const u32 mask = mbs.mask;
    const u32 A = (u32)sh.h_A;
    const i64 T = (i64)tq;
    const bool t_small = T > -(1ll << 31) && T < (1ll << 31);
    // A remainder is smaller in magnitude than its divisor: when no divisor of the tile exceeds the
    // target's magnitude no candidate  a % b  can match, and the loops leave the remainders out.
    const bool skip_mod = !SWAP && (mask & 16u) && !mbs.mod_possible && !tile_wide && !rng && A == 1u && t_small;
    if (skip_mod && threadIdx.x == 0) sh.ops_skipped += pairs * ((mask & 8u) ? 2ull : 9ull);     // (cost model of the host plan)
    // Tests of this member that run: this thread's operands that are defined at the probe, times the
    // member's broadcast operands that are, times the operators whose loop is entered (the 32-bit
    // loops leave / and % out when the target cannot be a quotient or remainder of int32 operands, and
    // the remainders alone when no divisor exceeds the target).
    {
        int tested_ops = seg.n_ops;
        if (!tile_wide && !rng && (mask & 24u) && A == 1u) {
            if (!t_small) tested_ops -= __popc(mask & 24u);
            else if (skip_mod) tested_ops -= 1;
        }
        warp_tally(&sh.filter_tests, (u32)__popc(alive) * (u32)(nb + (int)mbs.nspecial) * (u32)tested_ops);
    }
    const u32 flags = (tile_wide ? kPieceWide : 0u) | (skip_mod ? kPieceSkipMod : 0u);

    // The broadcast operands sit in two runs of slots: the general ones from slot 0 up, the
    // ones of magnitude <= 1 (special as divisors) from the last slot down.  Every warp walks
    // the runs on its own, in chunks of `chunk` slots, and looks at its hit queue after each:
    // no CTA-wide synchronisation happens inside a tile.  A chunk that overflows the queue (a
    // spec that many candidates satisfy at probe 0) is forgotten and redone with a quarter of
    // the chunk size, down to one slot and one register operand per lane at a time (at most
    // 32 * 5 hits, which always fit).  The chunk size is kept per warp from tile to tile and
    // grows back slowly.
    const int warp = threadIdx.x >> 5;
    const int n_special = (int)mbs.nspecial;
    int chunk = sh.chunk_hint[warp];
    bool shrunk = false;
    if ((threadIdx.x & 31) == 0) sh.wmember[warp] = (u32)m | (((sh.wq_tiles[warp] - 1u) & (u32)(kQueueTags - 1)) << 3);
    __syncwarp();
    u32 q_start = sh.wq_n[warp];                        // queue length when the current chunk began (hits of
                                                        // earlier members of the family may still wait there)
    for (int part = 0; part < 2; ++part) {
        const int lo = part == 0 ? bc_lo : bc_hi - n_special, hi = part == 0 ? bc_lo + nb : bc_hi;
        const u32 pflags = flags | (part == 1 ? kPieceSpecial : 0u);
        int s0 = lo;
        while (s0 < hi) {
            const int s1 = s0 + chunk < hi ? s0 + chunk : hi;
            run_piece<DENSE>(sh, R, alive, a1ok, m, s0, s1, pflags);
            __syncwarp();
            const u32 qn = sh.wq_n[warp];
            const bool overflow = sh.wq_over[warp] != 0;
            __syncwarp();
            if (overflow) {
                if ((threadIdx.x & 31) == 0) { sh.wq_n[warp] = q_start; sh.wq_over[warp] = 0; }
                drain_queue(sh, plan, sk, hole, my_evals);
                q_start = 0;
                shrunk = true;
                if (chunk > 1) { chunk = chunk / 4 > 1 ? chunk / 4 : 1; continue; }
                for (int j = 0; j < kNA; ++j) {
                    run_piece<DENSE>(sh, R, alive & (1u << j), a1ok, m, s0, s0 + 1, pflags);
                    drain_queue(sh, plan, sk, hole, my_evals);
                }
            } else if (qn > (u32)(kWarpQueue / 2)) {
                drain_queue(sh, plan, sk, hole, my_evals);
                q_start = 0;
            } else {
                q_start = qn;
            }
            s0 = s1;
        }
    }
    if ((threadIdx.x & 31) == 0) sh.chunk_hint[warp] = shrunk ? chunk : (chunk * 2 < kChunkB ? chunk * 2 : kChunkB);
    if (drain_at_end) drain_queue(sh, plan, sk, hole, my_evals);
}

// Members with a handful of broadcast operands and no operator but + and - (the large typed search:
// `E + v`, `E - v`, `v + E`, `v - E` over 4 variables) have a few dozen candidates per thread and
// tile: the general walk above, with its chunks, votes and choice of loop, spends far more
// instructions around them than on them, and most of those from cold code.  This compact routine
// takes all such members of the family in one call and tests their candidates directly (no votes: a
// lane with a hit goes to the rare path on its own).  Returns the set of members it has done; a
// member is left to the general walk when the warp's queue is too full to be sure of room, or ran
// over (its hits are then forgotten first).
constexpr u32 kTinyOperands = 16;
__device__ __forceinline__ bool tiny_member(const EvalShared& sh, int m) {      // (the same for every thread of the CTA)
    const MemberState& mbs = sh.mb[m];
    return (mbs.mask & ~3u) == 0u && mbs.n + mbs.nspecial <= kTinyOperands && sh.h_aff_ok != 0 &&
           (sh.reg_wide | mbs.wide | sh.mseg[m].generic) == 0;
}
__device__ __noinline__ u32 tiny_ring(EvalShared& sh, const RegVals* R, u32 alive, u32 a1ok, int family) {
    const int warp = threadIdx.x >> 5;
    const u32 A = (u32)sh.h_A, tp = (u32)sh.h_tq;
    u32 aA[kNA];
#pragma unroll
    for (int j = 0; j < kNA; ++j) aA[j] = R->lo[j] * A;
    u32 done = 0;
    for (int m = 0; m < family; ++m) {
        if (!tiny_member(sh, m)) continue;
        const SegDev& seg = sh.mseg[m];
        const MemberState& mbs = sh.mb[m];
        const bool SWAP = seg.swap != 0;
        const u32 mask = mbs.mask;
        __syncwarp();
        const u32 q_start = sh.wq_n[warp];
        if (q_start > (u32)(kWarpQueue / 2)) continue;
        if ((threadIdx.x & 31) == 0) sh.wmember[warp] = (u32)m | (((sh.wq_tiles[warp] - 1u) & (u32)(kQueueTags - 1)) << 3);
        __syncwarp();
        for (int part = 0; part < 2; ++part) {          // the general operands, then those of magnitude <= 1
            const int lo = part == 0 ? mbs.lo : mbs.hi - (int)mbs.nspecial, hi = part == 0 ? mbs.lo + (int)mbs.n : mbs.hi;
            for (int s = lo; s < hi; ++s) {
                const u32 t_add = sh.bc_ring[s].t_add;  // A*a must equal this for +, and t_sub for - (see ring_pass)
                const u32 t_sub = SWAP ? 0u - t_add : 2u * tp - t_add;
                u32 hits = 0;
#pragma unroll
                for (int j = 0; j < kNA; ++j)
                    hits |= (u32)(((mask & 1u) && aA[j] == t_add) || ((mask & 2u) && aA[j] == t_sub)) << j;
                hits &= alive;
                if (hits) emit_ring(sh, R, a1ok, s, hits, 0u, A, tp, mbs.opip, mask, SWAP);
            }
        }
        __syncwarp();
        if (sh.wq_over[warp] != 0) {                    // the queue ran over: this member's hits are forgotten
            __syncwarp();
            if ((threadIdx.x & 31) == 0) { sh.wq_n[warp] = q_start; sh.wq_over[warp] = 0; }
            continue;
        }
        warp_tally(&sh.filter_tests, (u32)__popc(alive) * (mbs.n + mbs.nspecial) * (u32)seg.n_ops);
        done |= 1u << m;
    }
    return done;
}

// Fills the broadcast side of a tile: operand values at probe 0, with everything the loops
// need that depends on them alone.  Returns (per thread) whether a value did not fit int32.
__device__ __noinline__ bool fill_bc_operands(EvalShared& sh, const GrammarDev* g, const HoleDev* hole, int m, int n_bc) {
    const SegDev& seg = sh.mseg[m];
    MemberState& mbs = sh.mb[m];
    const u64 bc_first = mbs.bc_first;
    const bool swap = seg.swap != 0;
    const bool second = hole->second_ok != 0;           // (kept even while the second look is off: the CTA may turn it on)
    const u32 fA = (u32)hole->aff_A;
    const u64 ftq = (u64)hole->probe_spec[0] - hole->aff_B;
    const u32 ftp = (u32)ftq;
    const u32 ftabs = (u32)((i64)ftq < 0 ? 0ull - ftq : ftq);
    bool wide = false;
    for (int i = threadIdx.x; i < n_bc; i += kThreads) {
        i64 v;
        if (!operand_value(g, hole, 0, seg.bc_nt, seg.bc_size, bc_first + i, v)) continue;
        i64 v1 = 0;                                         // second look: value at probe 1 (undefined there: no match)
        if (second && !operand_value(g, hole, 1, seg.bc_nt, seg.bc_size, bc_first + i, v1)) continue;
        const bool v1_exact = second && v1 > -(1ll << 31) && v1 < (1ll << 31);
        const bool special = v >= -1 && v <= 1;
        const u32 slot = special ? (u32)mbs.hi - 1u - atomicAdd(&mbs.nspecial, 1u) : (u32)mbs.lo + atomicAdd(&mbs.n, 1u);
        const bool fits = v > -(1ll << 31) && v < (1ll << 31);
        wide |= !fits;
        if (!XP_CHECKED(slot < (u32)kBcTile && (i32)slot >= mbs.lo && (i32)slot < mbs.hi, kChkSlot)) continue;
        const u32 b = (u32)(u64)v, ub = abs_u32((i32)v);
        const u32 k = ub ? (u32)__ffs((int)ub) - 1u : 0u;
        const u32 io = ub ? inv_odd(ub >> k) : 1u;          // inverse of the odd part of |v|
        BcMeta m;
        m.lo = b; m.hi = (u32)((u64)v >> 32); m.meta = (u32)i | (k << 16) | (v1_exact ? 0x80000000u : 0u); m.pad = (u32)(u64)v1;
        sh.bc_meta[slot] = m;
        // + and -: the value A*a must have; *: the operand and the target
        BcRing r;
        const u32 bA = b * fA;
        r.t_add = ftp - bA;
        r.t_pm = signfree(swap ? r.t_add : bA);
        r.mul_b = b;
        r.mul_nt = 0u - ftp;
        sh.bc_ring[slot] = r;
        // / and %: this operand as divisor (not swap) or as dividend (swap)
        BcDiv d;
        d.ub = ub; d.inv = io;
        if (swap) { d.low = ub >= ftabs ? ub - ftabs : 1u; d.cmax = 0u; }
        else {
            const u64 lw = (u64)ftabs * ub;
            d.low = lw < (1ull << 31) ? (u32)lw : 0x80000000u;
            d.cmax = (ub != 0u && ftabs < ub) ? 0xffffffffu / ub : 0u;
            if (d.cmax != 0u || !fits) mbs.mod_possible = 1;         // (benign race: every writer stores 1)
        }
        sh.bc_div[slot] = d;
    }
    return wide;
}

// Copies segment `index` of the plan into shared memory with the first warp.
__device__ __forceinline__ void load_segment(EvalShared& sh, const PlanDev& plan, int index) {
    if (threadIdx.x < 32) {
        const u32* src = (const u32*)&plan.segs[index];
        u32* dst = (u32*)&sh.seg;
        for (int w = threadIdx.x; w < (int)(sizeof(SegDev) / 4); w += 32) dst[w] = src[w];
    }
}

// Copies the segments of a family (head at `index`) into shared memory, one warp per member.
__device__ __forceinline__ void load_family(EvalShared& sh, const PlanDev& plan, int index, int family) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int m = warp; m < family; m += kWarps) {
        const u32* src = (const u32*)&plan.segs[index + m];
        u32* dst = (u32*)&sh.mseg[m];
        for (int w = lane; w < (int)(sizeof(SegDev) / 4); w += 32) dst[w] = src[w];
    }
}

template <bool DENSE>
__device__ __noinline__ void tile_ticket(EvalShared& sh, const PlanDev& plan, const SketchDev* sk, const HoleDev* hole,
                                            u64 local, u64& my_evals) {
    const GrammarDev* g = sk->g;
    if (!(hole->probe_spec_ok & 1u)) return;            // spec undefined at probe 0: nothing can match
    // the register side: the same for every member of the segment's family
    int family = sh.seg.family > 1 ? sh.seg.family : 1;
    if (family > kMaxFamily) family = kMaxFamily;        // (the host's plan builder stops at kMaxFamily members)
    const int seg_index = sh.seg_index;
    const u64 reg_tile = local / sh.seg.bc_tiles, bc_tile0 = local % sh.seg.bc_tiles;
    const u64 reg_first = sh.seg.reg_begin + reg_tile * (u64)kRegTile;
    const u64 reg_left = sh.seg.reg_begin + sh.seg.reg_count - reg_first;
    const int n_reg = reg_left < (u64)kRegTile ? (int)reg_left : kRegTile;
    const bool keep = sh.seg.bc_keep != 0;
    const bool resident = keep && sh.kept_head == seg_index;       // this family's broadcast operands are in the tile
    const int reg_nt = sh.seg.reg_nt, reg_size = sh.seg.reg_size;
    const bool second = hole->second != 0 || (hole->second_ok != 0 && sh.adapt_second != 0);
    if (!resident) load_family(sh, plan, seg_index, family);       // (a resident family's segments are still in place)
    if ((threadIdx.x & 31) == 0) {                      // the tag that this tile's hits carry in the warp's queue
        const int w = threadIdx.x >> 5;
        sh.wq_first[w][sh.wq_tiles[w] & (u32)(kQueueTags - 1)] = reg_first;
        sh.wq_tiles[w] += 1u;
    }
    if (threadIdx.x == 0) {
        sh.reg_wide = 0;
        sh.p1_on = second ? 1 : 0;
        sh.p1_A = hole->aff_Aj[1]; sh.p1_B = hole->aff_Bj[1]; sh.p1_spec = (u64)hole->probe_spec[1];
        sh.p1_rng = (hole->rng_okmask >> 1) & 1u;
        sh.p1_lo = hole->rng_lo[1]; sh.p1_hi = hole->rng_hi[1];
        sh.h_A = hole->aff_A; sh.h_tq = (u64)hole->probe_spec[0] - hole->aff_B;
        sh.h_rng_lo = hole->rng_lo[0]; sh.h_rng_hi = hole->rng_hi[0]; sh.h_aff_ok = hole->aff_ok;
    }
    // this thread's operands: kNA consecutive ranks
    RegVals RV;
    const int mine = n_reg - (int)threadIdx.x * kNA;
    const int n_mine = mine < 0 ? 0 : (mine > kNA ? kNA : mine);
    u32 fits0 = 0;
    u32 alive = fill_reg_operands(g, hole, 0, reg_nt, reg_size, reg_first + threadIdx.x * (u64)kNA, n_mine,
                                  RV.lo, RV.hi, fits0);
    const bool wide_reg = fits0 != alive;
    // second look: the same operands at probe 1; one that is undefined there can be in no match
    u32 a1ok = 0;
    if (second)
        alive &= fill_reg_operands(g, hole, 1, reg_nt, reg_size, reg_first + threadIdx.x * (u64)kNA, n_mine,
                                   RV.p1, nullptr, a1ok);
    __syncthreads();                                    // the members' segments are in place, reg_wide is clear
    if (wide_reg) sh.reg_wide = 1;
    if (threadIdx.x == 0) { sh.q_sketch = sh.seg.sketch; sh.q_hole = sh.seg.hole; }      // (read at the top of a later ticket)
    // broadcast operands of member m: tile bc_tile0 of the head (a family's other members have one tile)
    auto n_bc_of = [&](int m) {
        const SegDev& seg = sh.mseg[m];
        const u64 first = seg.bc_begin + (m == 0 ? bc_tile0 : 0) * (u64)seg.bc_tile;
        const u64 left = seg.bc_begin + seg.bc_count - first;
        return left < (u64)seg.bc_tile ? (int)left : seg.bc_tile;
    };
    auto start_member = [&](int m) {                    // (one thread) empty slots for member m
        const SegDev& seg = sh.mseg[m];
        MemberState& mbs = sh.mb[m];
        mbs.bc_first = seg.bc_begin + (m == 0 ? bc_tile0 : 0) * (u64)seg.bc_tile;
        mbs.lo = keep ? seg.bc_base : 0;
        mbs.hi = keep ? seg.bc_base + n_bc_of(m) : kBcTile;
        mbs.n = 0; mbs.nspecial = 0; mbs.wide = 0; mbs.mod_possible = 0;
        u32 opip = 0, mask = 0;
        for (int o = 0; o < seg.n_ops; ++o) { opip |= (u32)o << (3 * op_slot(seg.op[o])); mask |= 1u << op_slot(seg.op[o]); }
        mbs.opip = opip; mbs.mask = mask;
    };
    if (keep) {
        // Every member's operands fit the tile side by side.  They are filled once (by the first
        // ticket of the family that this CTA takes); after that the warps go through the members on
        // their own, with no CTA-wide synchronisation, and look at their hit queues when those fill
        // up and once at the end.
        if (!resident) {
            if ((int)threadIdx.x < family) start_member((int)threadIdx.x);
            __syncthreads();
            for (int m = 0; m < family; ++m)
                if (fill_bc_operands(sh, g, hole, m, n_bc_of(m))) sh.mb[m].wide = 1;
            if (threadIdx.x == 0) sh.kept_head = seg_index;
        }
        __syncthreads();
        // (sparse form) the members with next to no work per tile first, all in one compact routine
        const u32 tiny_done = DENSE ? 0u : tiny_ring(sh, &RV, alive, a1ok, family);
        bool first = true;
        for (int m = 0; m < family; ++m) {
            const SegDev& seg = sh.mseg[m];
            const u64 pairs = (u64)n_reg * (u64)n_bc_of(m);
            if (threadIdx.x == 0) sh.tile_cands += pairs * (u64)seg.n_ops;
            const bool tiny = !DENSE && tiny_member(sh, m);
            if (!tiny) {                                // (the same for every thread of the CTA)
                if (!first) __syncthreads();            // keeps the CTA's warps in the same loop from member to member
                first = false;
            }
            if ((tiny_done >> m) & 1u) continue;
            tile_body<DENSE>(sh, plan, sk, hole, m, reg_first, pairs, &RV, a1ok, alive, false, my_evals);
        }
        // In the sparse form of the kernel, when the CTA came to this ticket from another one of the same
        // family (a long run of them is likely), a handful of hits waits for the next (eval_kernel empties the queues before anything
        // else runs); enough of them, or old ones, are checked now.
        const int w = threadIdx.x >> 5;
        __syncwarp();
        const u32 qn = sh.wq_n[w], age = sh.wq_age[w];
        __syncwarp();
        if (DENSE || !resident || qn >= kDrainMin || age + 2u >= (u32)kQueueTags) drain_queue(sh, plan, sk, hole, my_evals);
        else if ((threadIdx.x & 31) == 0) { sh.wq_age[w] = age + 1u; if (qn) sh.q_waiting = 1; }
        return;
    }
    for (int m = 0; m < family; ++m) {                  // members take turns in the tile
        if (m > 0) __syncthreads();                     // every warp is done with the previous member's operands
        if (threadIdx.x == 0) { start_member(m); sh.kept_head = -1; }      // (whatever was resident is overwritten)
        __syncthreads();
        if (fill_bc_operands(sh, g, hole, m, n_bc_of(m))) sh.mb[m].wide = 1;
        __syncthreads();
        const SegDev& seg = sh.mseg[m];
        const u64 pairs = (u64)n_reg * (u64)n_bc_of(m);
        if (threadIdx.x == 0) sh.tile_cands += pairs * (u64)seg.n_ops;
        tile_body<DENSE>(sh, plan, sk, hole, m, reg_first, pairs, &RV, a1ok, alive, true, my_evals);
    }
}

#ifndef XP_MIN_CTAS
#define XP_MIN_CTAS 3
#endif
template <bool DENSE>
__global__ void __launch_bounds__(kThreads, XP_MIN_CTAS) eval_kernel(const PlanDev plan) {
    __shared__ EvalShared sh;
    u64 my_evals = 0;
    if (threadIdx.x <= kMaxSize) { sh.match_count[threadIdx.x] = 0; sh.min_rank[threadIdx.x] = ~0ull; }
    if (threadIdx.x == 0) { sh.cur_acc = -1; sh.kept_head = -1; sh.filter_survivors = 0; sh.probe_survivors = 0; sh.ops_skipped = 0; sh.adapt_second = 0; sh.filter_tests = 0; sh.tile_cands = 0; }
    if (threadIdx.x < kWarps) {
        sh.chunk_hint[threadIdx.x] = kChunkB; sh.wq_n[threadIdx.x] = 0; sh.wq_over[threadIdx.x] = 0; sh.wmember[threadIdx.x] = 0;
        sh.wq_tiles[threadIdx.x] = 0; sh.wq_age[threadIdx.x] = 0;
    }
    if (threadIdx.x == 0) { sh.q_sketch = 0; sh.q_hole = 0; sh.q_waiting = 0; }
    __syncthreads();
    for (;;) {
        if (threadIdx.x == 0) {
            sh.ticket = plan.ticket_base + atomicAdd(plan.ticket, 1ull);
            // many filter hits so far for the hole at hand (this CTA's own counts): second look from now on
            if (!sh.adapt_second && sh.filter_survivors * kAdaptRate > sh.tile_cands) sh.adapt_second = 1;
        }
        __syncthreads();
        const u64 t = sh.ticket;
        if (t >= plan.n_tickets) {
            if (!DENSE && sh.q_waiting && sh.wq_n[threadIdx.x >> 5] != 0) drain_waiting(sh, plan, my_evals);
            break;
        }
        if (threadIdx.x < 32) {
            // last segment with first_ticket <= t: a 32-way search, one probe per lane and round
            int lo = 0, n = plan.n_segs;
            while (n > 1) {
                const int step = (n + 31) / 32;
                const int pos = lo + (int)threadIdx.x * step;
                const bool le = pos < lo + n && plan.segs[pos].first_ticket <= t;
                const u32 mask = __ballot_sync(0xffffffffu, le);          // lane 0 always holds
                const int k = 31 - __clz((int)(mask | 1u));
                const int nlo = lo + k * step;
                n = (lo + n - nlo) < step ? (lo + n - nlo) : step;
                lo = nlo;
            }
            if (!XP_CHECKED(lo >= 0 && lo < plan.n_segs && plan.segs[lo].first_ticket <= t, kChkSegment)) lo = 0;
            if (threadIdx.x == 0) sh.seg_index = lo;
            load_segment(sh, plan, lo);
        }
        __syncthreads();
        // Hits that wait in the warps' queues belong to the family resident in the tile: any ticket but
        // another one of that family has them checked first (their segments and operands are about to go).
        if (!DENSE && sh.q_waiting && !(sh.seg.kind == kSegTile && sh.seg.bc_keep != 0 && sh.kept_head == sh.seg_index)) {
            if (sh.wq_n[threadIdx.x >> 5] != 0) drain_waiting(sh, plan, my_evals);
            __syncthreads();
            if (threadIdx.x == 0) sh.q_waiting = 0;
        }
        if (sh.seg.acc != sh.cur_acc) {
            flush_acc(sh, plan, my_evals);
            if (threadIdx.x == 0) sh.cur_acc = sh.seg.acc;
            __syncthreads();
        }
        const SketchDev* sk = plan.sketches[sh.seg.sketch];
        const HoleDev* hole = &sk->holes[sh.seg.hole];
        const u64 local = t - sh.seg.first_ticket;
        if (sh.seg.kind == kSegTile) tile_ticket<DENSE>(sh, plan, sk, hole, local, my_evals);
        else linear_ticket(sh, plan, sk, hole, local, my_evals);
        __syncthreads();
    }
    flush_acc(sh, plan, my_evals);
}

// ------------------------------------------------------------------------------------------
// verify: whole-domain check of the queued survivors
// ------------------------------------------------------------------------------------------

// Notes, for xp_sketch_refine, that domain point `pid` ended a survivor's whole-domain check.
__device__ __noinline__ void record_killer(const HoleDev* hole, i64 pid) {
    if (hole->kill_pid == nullptr) return;
    u64 x = (u64)pid * 0x9E3779B97F4A7C15ull;
    u32 slot = (u32)(x >> 40) % (u32)kKillSlots;
    for (int k = 0; k < 8; ++k, slot = (slot + 1u) % (u32)kKillSlots) {
        const u64 old = atomicCAS((u64*)&hole->kill_pid[slot], ~0ull, (u64)pid);
        if (old == ~0ull || old == (u64)pid) { atomicAdd(&hole->kill_cnt[slot], 1u); return; }
    }                                                   // (table crowded around this slot: the point goes unrecorded)
}

// ---- survivors in hole order ----
//
// eval_kernel counts the queued survivors per accumulator slot (= per hole of the call); a scan turns
// the counts into offsets and a scatter writes, per slot, the queue indices of its survivors side by
// side.  The verification kernel walks that order, so the survivors a warp takes together mostly
// belong to one hole: same points, same spec values.

// One CTA: exclusive scan of hist[0 .. n_acc) into off[0 .. n_acc]; hist is cleared for the scatter.
__global__ void __launch_bounds__(1024) surv_scan_kernel(u32* hist, u32* off, int n_acc) {
    __shared__ u32 part[1024];
    const int t = threadIdx.x;
    const int per = (n_acc + 1023) / 1024;
    const int lo = t * per < n_acc ? t * per : n_acc, hi = lo + per < n_acc ? lo + per : n_acc;
    u32 sum = 0;
    for (int i = lo; i < hi; ++i) sum += hist[i];
    part[t] = sum;
    __syncthreads();
    for (int d = 1; d < 1024; d <<= 1) {
        const u32 v = t >= d ? part[t - d] : 0u;
        __syncthreads();
        part[t] += v;
        __syncthreads();
    }
    u32 run = part[t] - sum;
    for (int i = lo; i < hi; ++i) { const u32 h = hist[i]; off[i] = run; run += h; hist[i] = 0; }
    if (t == 1023) off[n_acc] = part[1023];
}

__global__ void __launch_bounds__(256) surv_scatter_kernel(const PlanDev plan) {
    const u32 pushed = *plan.surv_n;
    const u32 n = pushed < plan.surv_cap ? pushed : plan.surv_cap;
    const u32 i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int acc = plan.surv[i].acc;
    plan.surv_sorted[plan.surv_off[acc] + atomicAdd(&plan.surv_hist[acc], 1u)] = i;
}

// One thread per queued survivor: those whose (projected) domain has more than one chunk of points
// go on the list of long survivors.
__global__ void __launch_bounds__(256) surv_long_kernel(const PlanDev plan) {
    const u32 pushed = *plan.surv_n;
    const u32 n = pushed < plan.surv_cap ? pushed : plan.surv_cap;
    const u32 i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const SurvDev sv = plan.surv[i];
    const SketchDev* sk = plan.sketches[sv.sketch];
    if (proj_points(sk, &sk->holes[sv.hole], sv.vars, nullptr) > (i64)kVerifyChunk) plan.surv_long[atomicAdd(plan.surv_long_n, 1u)] = i;
}

// ---- whole-domain check of several survivors of one hole together ----
//
// For table domains.  The warp's lanes each stage one survivor (unranking, substitution into the
// context, magnitude bounds, constant-divisor folding: all 32 at once, where one lane used to do it
// for one survivor while 31 waited) as a compact program in the warp's arena.  Then the chunk is
// walked in steps of 128 points (4 per lane): the step's coordinates go to shared memory and its
// spec values to registers ONCE, and every staged survivor still alive is run on them; a survivor
// that fails at some point of the step leaves the set.
constexpr int kVArena = 256;                              // program entries a warp stages at once
constexpr int kVStep = 128;                               // points per step
constexpr int kVBatchVars = 4;                            // most variables a table may have for this form
constexpr int kVBatchDepth = 4;                           // deepest operand stack it takes
// A warp's shared memory: the batch form's arrays and the one-survivor form's share the same bytes
// (a warp is in one form at a time), which keeps three CTAs resident per SM.
struct VerifyBatch {
    i32 pvar[kVArena];                                    // >= 0: variable; -1: constant; -2 - op: operator
    i64 pval[kVArena];
    i32 coords[kVBatchVars][kVStep];                      // the step's points, [variable][point]
    uint4 stack[kVBatchDepth * 32];                       // operand stacks below the top, per level and lane
};
struct VerifySingle {
    uint4 stack[kVecDepth * 32];
    CandShared cand;                                      // the one-survivor form (boxes, long or deep programs, many variables)
};
struct __align__(16) VerifyWarp {
    union { VerifyBatch b; VerifySingle s; };
};

// Length of the program that candidate code of `n` nodes gives in the hole's context; -1 if the
// context never mentions the hole (the one-survivor form handles that).
__device__ __forceinline__ int staged_length(const HoleDev* hole, int n) {
    if (hole->ctx_len == 0) return n;
    int holes = 0;
    for (int i = 0; i < hole->ctx_len; ++i) holes += hole->ctx[i].kind == XP_I_HOLE;
    return holes ? hole->ctx_len + holes * (n - 1) : -1;
}

// One lane: stages survivor (size, rank) at w.pvar / w.pval [off ...).  Returns the final length
// (constant divisors folded when the program is exact in int32), or -1 when the operand stack gets
// deeper than the vectorised check takes.
__device__ __noinline__ int stage_compact(VerifyWarp& w, int off, const SketchDev* sk, const HoleDev* hole, int size, u64 rank,
                                         bool& narrow_out) {
    const GrammarDev* g = sk->g;
    u32 code[kMaxSize];
    const int n = unrank(g, hole->start_nt, size, rank, code);
    int len = 0, sp = 0, depth = 0;
    bool narrow = true;
    constexpr u64 kSat = 1ull << 62;
    u64 mag[kMaxStack + kCandStack + 1];
    auto mag_of = [](i64 v) { return v < 0 ? 0ull - (u64)v : (u64)v; };
    auto emit = [&](i32 var, i64 val) {
        if (sp > kMaxStack + kCandStack - 1) { depth = kVBatchDepth + 1; return; }
        w.b.pvar[off + len] = var; w.b.pval[off + len] = val; ++len;
        u64 m;
        if (var >= -1) {
            if (var >= 0) { const u64 a = mag_of(sk->vmin[var]), b = mag_of(sk->vmax[var]); m = a > b ? a : b; }
            else m = mag_of(val);
            mag[sp] = m < kSat ? m : kSat;
            if (++sp > depth) depth = sp;
        } else {
            --sp;
            const u64 a = mag[sp - 1], b = mag[sp];
            switch (-2 - var) {
                case XP_OP_ADD: case XP_OP_SUB: m = a + b; break;
                case XP_OP_MUL: m = (a >> 31 || b >> 31) ? kSat : a * b; break;
                case XP_OP_DIV: m = a; break;
                case XP_OP_MOD: m = a < b ? a : b; break;
                case XP_OP_MIN: case XP_OP_MAX: m = a > b ? a : b; break;
                case XP_OP_SHL: m = kSat; break;
                case XP_OP_SHR: m = a; break;
                default: m = 1; break;
            }
            mag[sp - 1] = m < kSat ? m : kSat;
        }
        narrow = narrow && (m >> 31) == 0;
    };
    auto emit_cand = [&]() {
        for (int k = 0; k < n; ++k) {
            if (code[k] & kOpBit) emit(-2 - (i32)(code[k] & 0xff), 0);
            else { const LeafDev lf = g->leaves[code[k]]; emit(lf.var >= 0 ? lf.var : -1, lf.value); }
        }
    };
    if (hole->ctx_len == 0) emit_cand();
    else
        for (int i = 0; i < hole->ctx_len; ++i) {
            const xp_instr in = hole->ctx[i];
            if (in.kind == XP_I_HOLE) emit_cand();
            else if (in.kind == XP_I_OP) emit(-2 - in.arg, 0);
            else emit(in.kind == XP_I_VAR ? in.arg : -1, in.value);
        }
    narrow_out = narrow;
    if (depth > kVBatchDepth) return -1;
    if (narrow) {                                         // "push c; x / y" -> one instruction on the top of the stack
        int wr = 0;
        for (int k = 0; k < len; ++k) {
            const i32 cv = w.b.pvar[off + k];
            const bool divmod = cv == -2 - XP_OP_DIV || cv == -2 - XP_OP_MOD;
            if (divmod && wr > 0 && w.b.pvar[off + wr - 1] == -1 && w.b.pval[off + wr - 1] != 0 &&
                w.b.pval[off + wr - 1] > -(1ll << 31) && w.b.pval[off + wr - 1] < (1ll << 31)) {
                const i32 d = (i32)w.b.pval[off + wr - 1];
                const u32 ad = d < 0 ? 0u - (u32)d : (u32)d;
                const u32 M = ad == 1u ? 0xffffffffu : (u32)((1ull << 32) / ad);
                w.b.pvar[off + wr - 1] = -2 - (cv == -2 - XP_OP_DIV ? kOpDivC : kOpModC);
                w.b.pval[off + wr - 1] = (i64)(((u64)M << 32) | (u32)d);
                continue;
            }
            w.b.pvar[off + wr] = cv; w.b.pval[off + wr] = w.b.pval[off + k]; ++wr;
        }
        len = wr;
    }
    return len;
}

// The staged program [off, off + len) on the lane's points of the step (P at a time: points
// lane*4 + half*P + i).  Returns the bit set of the lane's points that fail (a zero divisor: bit 0).
template <typename T, int P>
__device__ __forceinline__ u32 run_staged(VerifyWarp& w, int off, int len, int half, const i64* want, u32 in_mask) {
    typedef VecSlot<T, P> Slot;
    const int lane = threadIdx.x & 31;
    Slot t;
#pragma unroll
    for (int i = 0; i < P; ++i) t.v[i] = 0;
    bool bad = false;
    int below = 0;
    for (int k = 0; k < len; ++k) {
        const i32 cv = w.b.pvar[off + k];
        if (cv >= -1) {
            w.b.stack[below * 32 + lane] = t.q;
            ++below;
            if (cv >= 0) {
                if (sizeof(T) == 4) t.q = *reinterpret_cast<const uint4*>(&w.b.coords[cv][lane * 4]);
                else {
#pragma unroll
                    for (int i = 0; i < P; ++i) t.v[i] = (T)w.b.coords[cv][lane * 4 + half * P + i];
                }
            } else {
                const T v = (T)w.b.pval[off + k];
#pragma unroll
                for (int i = 0; i < P; ++i) t.v[i] = v;
            }
            continue;
        }
        const int op = -2 - cv;
        Slot a;
        a.q = t.q;
        if (!(sizeof(T) == 4 && op >= kOpDivC)) { --below; a.q = w.b.stack[below * 32 + lane]; }
        vec_op<T, P>(op, w.b.pval[off + k], a, t, bad);
    }
    u32 which = 0;
#pragma unroll
    for (int i = 0; i < P; ++i) which |= (u32)(((in_mask >> (half * P + i)) & 1u) && (i64)t.v[i] != want[half * P + i]) << (half * P + i);
    // (points past the end of the chunk repeat its first point, so a zero divisor there is one at a real point too)
    return which | (bad ? 1u : 0u);
}

// The survivors of `now` (bit b = lane b holds one, all of one hole) on chunk `chunk` of the hole's
// table domain.  Each lane ends up with `failed` set if its survivor failed at some point
// (fail_pid), and the warp with the number of candidate-point evaluations it made.
__device__ __noinline__ void verify_batch(VerifyWarp& w, const SketchDev* sk, const HoleDev* hole, u32 now, int my_off, int my_len,
                                          bool my_narrow, i64 first, i64 last, bool& failed, i64& fail_pid, u64& evals) {
    const int lane = threadIdx.x & 31;
    const int nv = sk->n_vars;
    const i32* __restrict__ coords = sk->coords;
    const i64* __restrict__ spec = hole->spec_table;
    u32 alive = now;
    for (i64 base = first; base < last && alive; base += kVStep) {
        const int npts = last - base < kVStep ? (int)(last - base) : kVStep;
        __syncwarp();                                     // everyone is done with the previous step's points
        for (int idx = lane; idx < kVStep * nv; idx += 32) {      // rows are contiguous: coalesced reads
            const int p = idx / nv, v = idx - p * nv;
            const int src = p < npts ? idx : v;           // points past the end repeat the step's first point
            w.b.coords[v][p] = coords[base * nv + src];
        }
        i64 want[4];
        u32 in_mask = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int p = lane * 4 + i;
            if (p < npts) in_mask |= 1u << i;
            want[i] = spec[base + (p < npts ? p : 0)];
        }
        __syncwarp();
        evals += (u64)npts * (u64)__popc(alive);
        for (u32 m = alive; m; m &= m - 1) {
            const int b = __ffs((int)m) - 1;
            const int off = __shfl_sync(0xffffffffu, my_off, b), len = __shfl_sync(0xffffffffu, my_len, b);
            const bool narrow = __shfl_sync(0xffffffffu, (int)my_narrow, b) != 0;
            u32 which;
            if (narrow) which = run_staged<i32, 4>(w, off, len, 0, want, in_mask);
            else which = run_staged<i64, 2>(w, off, len, 0, want, in_mask) | run_staged<i64, 2>(w, off, len, 1, want, in_mask);
            const u32 bm = __ballot_sync(0xffffffffu, which != 0u);
            if (bm) {
                const int src = __ffs((int)bm) - 1;
                const u32 wsrc = __shfl_sync(0xffffffffu, which, src);
                alive &= ~(1u << b);
                if (lane == b) {
                    const int p = src * 4 + (__ffs((int)wsrc) - 1);
                    failed = true;
                    fail_pid = base + (p < npts ? p : 0);
                }
            }
        }
    }
}

// One survivor on one chunk, staged by the warp's first lane (boxes with their sub-box projection,
// programs that do not fit the arena, contexts that never mention the hole).
__device__ __noinline__ void verify_one(const PlanDev& plan, VerifyWarp& w, u32 si, u64 chunk) {
    const int lane = threadIdx.x & 31;
    CandShared& cand = w.s.cand;
    int skip = 1;
    i64 np = 0;
    SurvDev* sv = &plan.surv[si];
    const SketchDev* sk = plan.sketches[sv->sketch];
    const HoleDev* hole = &sk->holes[sv->hole];
    if (lane == 0) {
        const bool failed = (*(volatile const u32*)&sv->state & kSurvFailed) != 0;
        np = proj_points(sk, hole, sv->vars, nullptr);
        if ((i64)chunk * kVerifyChunk < np && !failed) {
            skip = 0;
            stage_candidate(cand, sk, hole, sv->size, sv->rank);
            proj_points(sk, hole, sv->vars, &cand);
            if (cand.narrow && sk->coords != nullptr && hole->spec_table != nullptr && cand.depth >= 1 && cand.depth <= kVecDepth)
                fold_constant_divisors(cand);             // (exactly the case that takes the int32 vectorised check below)
        }
    }
    __syncwarp();
    skip = __shfl_sync(0xffffffffu, skip, 0);
    if (skip) return;
    np = __shfl_sync(0xffffffffu, np, 0);
    const i64 first = (i64)chunk * kVerifyChunk;
    const i64 last = first + kVerifyChunk < np ? first + kVerifyChunk : np;
    u64 evals = 0;
    i64 fail_pid = 0;
    bool ok;
    if (sk->coords != nullptr && hole->spec_table != nullptr && cand.depth >= 1 && cand.depth <= kVecDepth) {
        ok = cand.narrow ? check_points_vec<i32, 4>(cand, w.s.stack, sk, hole, first, last, &fail_pid)
                         : check_points_vec<i64, 2>(cand, w.s.stack, sk, hole, first, last, &fail_pid);
    } else {
        ok = check_points(cand, sk, hole, first, last, evals, &fail_pid);
    }
    if (lane == 0) {
        if (ok) atomicAdd(&sv->state, 1u);
        else if (!(atomicOr(&sv->state, kSurvFailed) & kSurvFailed)) record_killer(hole, fail_pid);   // (once per survivor)
        atomicAdd(&plan.acc[sv->acc].evals, (u64)(last - first));     // points of the chunk (an early exit tries fewer)
    }
    __syncwarp();                                       // the staged candidate is free for the next item
}

// Items are (chunk of points, block of up to 32 survivors), chunk-major: the first chunk of every
// survivor (blocks in hole order) is taken before any second chunk, so candidates that fail early
// cost one chunk; the later chunks exist for the long survivors only (surv_long_kernel), which keeps
// a call whose largest domain has hundreds of chunks from walking hundreds of empty items for every
// survivor of a small (or projected) domain.  Each WARP takes items on its own: nothing in this kernel synchronises a CTA, and no
// warp waits for another.  Within a block the survivors of one hole are handled together when the
// hole's domain is a table (verify_batch), one after the other otherwise (verify_one).  A survivor
// that has already failed is skipped.
constexpr int kVerifyThreads = 256;
constexpr int kVerifyWarps = kVerifyThreads / 32;
__global__ void __launch_bounds__(kVerifyThreads, 3) verify_kernel(const PlanDev plan) {
    extern __shared__ __align__(16) unsigned char verify_smem[];
    VerifyWarp& w = reinterpret_cast<VerifyWarp*>(verify_smem)[threadIdx.x >> 5];
    const int lane = threadIdx.x & 31;
    const u32 pushed = *plan.surv_n;
    const u64 n = pushed < plan.surv_cap ? pushed : plan.surv_cap;
    // Survivors per item: 32 when there are plenty (the batch form then has a full warp to stage and
    // share points with); fewer, down to one, when the call has too few survivors to give every warp
    // of the grid a full block (a search with a few thousand survivors on a large domain spreads
    // better as one survivor per warp).
    const u64 warps = (u64)gridDim.x * kVerifyWarps;
    u32 width = 32;
    while (width > 1 && n < warps * width) width >>= 1;
    const u64 n_blocks = (n + width - 1) / width;
    // The first chunk is walked for every survivor, the later ones for the long survivors only.
    const u64 n_long = plan.max_chunks > 1 ? *plan.surv_long_n : 0u;
    const u64 long_blocks = (n_long + width - 1) / width;
    const u64 total = n_blocks + long_blocks * (plan.max_chunks - 1);
    const u64 kBatch = 2;                               // items a warp takes per atomic
    u64 next = 0, batch_end = 0;
    for (;;) {
        if (next == batch_end) {
            if (lane == 0) next = atomicAdd(plan.verify_ticket, kBatch);
            next = __shfl_sync(0xffffffffu, next, 0);
            batch_end = next + kBatch;
        }
        const u64 t = next++;
        if (t >= total) break;
        const bool later = t >= n_blocks;
        const u64 chunk = later ? 1 + (t - n_blocks) / long_blocks : 0;
        const u64 block = later ? (t - n_blocks) % long_blocks : t;
        const u64 pos = block * width + lane;
        const bool have = (u32)lane < width && pos < (later ? n_long : n);
        const u32 si = !have ? 0u : later ? plan.surv_long[pos] : plan.surv_sorted ? plan.surv_sorted[pos] : (u32)pos;
        const int my_acc = have ? plan.surv[si].acc : -1;
        u32 remaining = __ballot_sync(0xffffffffu, have);
        while (remaining) {
            const int leader = __ffs((int)remaining) - 1;
            const int acc = __shfl_sync(0xffffffffu, my_acc, leader);
            const u32 run = __ballot_sync(0xffffffffu, have && my_acc == acc) & remaining;
            remaining &= ~run;
            const u32 lsi = __shfl_sync(0xffffffffu, si, leader);
            const SketchDev* sk = plan.sketches[plan.surv[lsi].sketch];
            const HoleDev* hole = &sk->holes[plan.surv[lsi].hole];
            const bool table = sk->domain_kind == XP_DOMAIN_TABLE && sk->coords != nullptr && hole->spec_table != nullptr &&
                               sk->n_vars <= kVBatchVars;
            const i64 first = (i64)chunk * kVerifyChunk;
            const bool mine = (run >> lane) & 1u;
            u32 single = 0;                               // survivors of the run that go one by one
            if (!table) single = run;
            else if (first < sk->n_points) {
                const i64 last = first + kVerifyChunk < sk->n_points ? first + kVerifyChunk : sk->n_points;
                SurvDev* sv = &plan.surv[si];
                const bool live = mine && !(*(volatile const u32*)&sv->state & kSurvFailed);
                const int want_len = live ? staged_length(hole, sv->size) : 0;
                single = __ballot_sync(0xffffffffu, live && (want_len < 0 || want_len > kVArena));
                u32 todo = __ballot_sync(0xffffffffu, live) & ~single;
                while (todo) {                            // as many as the arena holds at a time
                    int off = 0, my_off = 0;
                    u32 now = 0;
                    for (u32 m = todo; m; m &= m - 1) {   // (uniform: every lane walks the same set)
                        const int b = __ffs((int)m) - 1;
                        const int len_b = __shfl_sync(0xffffffffu, want_len, b);
                        if (off + len_b > kVArena) break;
                        if (lane == b) my_off = off;
                        now |= 1u << b;
                        off += len_b;
                    }
                    todo &= ~now;
                    __syncwarp();                         // the arena is free (the previous round's programs are done)
                    bool narrow = false, failed = false;
                    int len = 0;
                    if ((now >> lane) & 1u) {
                        len = stage_compact(w, my_off, sk, hole, sv->size, sv->rank, narrow);
                        if (len < 0) { len = 0; }
                    }
                    const u32 deep = __ballot_sync(0xffffffffu, ((now >> lane) & 1u) && len == 0);      // stack too deep: one by one
                    single |= deep;
                    now &= ~deep;
                    __syncwarp();
                    i64 fail_pid = 0;
                    u64 evals = 0;
                    verify_batch(w, sk, hole, now, my_off, len, narrow, first, last, failed, fail_pid, evals);
                    if ((now >> lane) & 1u) {
                        if (!failed) atomicAdd(&sv->state, 1u);
                        else if (!(atomicOr(&sv->state, kSurvFailed) & kSurvFailed)) record_killer(hole, fail_pid);
                    }
                    if (lane == 0 && evals) atomicAdd(&plan.acc[acc].evals, evals);
                }
            }
            for (u32 m = single; m; m &= m - 1) {
                const int b = __ffs((int)m) - 1;
                verify_one(plan, w, __shfl_sync(0xffffffffu, si, b), chunk);
            }
        }
    }
}

// One thread per queued survivor: it is a match if no chunk failed and every chunk passed.
__global__ void count_kernel(const PlanDev plan) {
    const u32 pushed = *plan.surv_n;
    const u32 n = pushed < plan.surv_cap ? pushed : plan.surv_cap;
    const u32 i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const SurvDev sv = plan.surv[i];
    const SketchDev* sk = plan.sketches[sv.sketch];
    const i64 np = proj_points(sk, &sk->holes[sv.hole], sv.vars, nullptr);
    const u32 chunks = (u32)((np + kVerifyChunk - 1) / kVerifyChunk);
    if ((sv.state & kSurvFailed) || sv.state != chunks) return;
    AccDev* a = &plan.acc[sv.acc];
    atomicAdd(&a->match_count[sv.size], 1ull);
    atomicMin(&a->min_rank[sv.size], sv.rank);
}

// ------------------------------------------------------------------------------------------
// finish: least (size, rank) per hole from the per-size minima
// ------------------------------------------------------------------------------------------

// One warp per accumulator: lane = size; ballot finds the smallest size with a match.
__global__ void finish_kernel(AccDev* acc, int n_acc, u32* err) {
    const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
#ifdef XP_CHECKS
    if (blockIdx.x == 0 && threadIdx.x == 0) *err = atomicExch(&g_check_word, 0u);     // what the checks recorded, if anything
#else
    (void)err;
#endif
    if (w >= n_acc) return;
    AccDev* a = &acc[w];
    const bool has = lane <= kMaxSize && a->match_count[lane] > 0;
    const u32 m = __ballot_sync(0xffffffffu, has);
    if (lane == 0) a->pad = m ? (u64)(__ffs(m) - 1) : 0ull;     // least size (0 = unsolved)
}

// ------------------------------------------------------------------------------------------
// integer peak
// ------------------------------------------------------------------------------------------

// Two groups of four independent chains per thread, 128 32-bit operations per loop iteration.
__global__ void __launch_bounds__(256) int32_peak_add_kernel(u32* out, int iters, u32 seed) {
    u32 a0 = threadIdx.x + seed, a1 = a0 * 3 + 1, a2 = a0 * 5 + 2, a3 = a0 * 7 + 3;
    u32 a4 = a0 * 11 + 4, a5 = a0 * 13 + 5, a6 = a0 * 17 + 6, a7 = a0 * 19 + 7;
#pragma unroll 1
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int u = 0; u < 16; ++u) {
            a0 += a4; a1 += a5; a2 += a6; a3 += a7;
            a4 += a0; a5 += a1; a6 += a2; a7 += a3;
        }
    }
    const u32 r = a0 ^ a1 ^ a2 ^ a3 ^ a4 ^ a5 ^ a6 ^ a7;
    if (r == 0x12345678u) out[0] = r;
}

__global__ void __launch_bounds__(256) int32_peak_mad_kernel(u32* out, int iters, u32 seed) {
    u32 a0 = threadIdx.x + seed, a1 = a0 * 3 + 1, a2 = a0 * 5 + 2, a3 = a0 * 7 + 3;
    u32 a4 = a0 * 11 + 4, a5 = a0 * 13 + 5, a6 = a0 * 17 + 6, a7 = a0 * 19 + 7;
    const u32 k = blockIdx.x | 1u;
#pragma unroll 1
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int u = 0; u < 16; ++u) {
            a0 = a0 * k + a4; a1 = a1 * k + a5; a2 = a2 * k + a6; a3 = a3 * k + a7;
            a4 = a4 * k + a0; a5 = a5 * k + a1; a6 = a6 * k + a2; a7 = a7 * k + a3;
        }
    }
    const u32 r = a0 ^ a1 ^ a2 ^ a3 ^ a4 ^ a5 ^ a6 ^ a7;
    if (r == 0x12345678u) out[0] = r;
}

// Cost of a division in thread-operations: four independent chains per thread of (a) int64
// truncating division by a divisor that is not known in advance, (b) int32 division by a
// constant through a precomputed reciprocal (multiply-high, multiply-subtract, one correction),
// the form the whole-domain check uses.  64 divisions per chain and loop iteration.
__global__ void __launch_bounds__(256) int_div_general_kernel(long long* out, int iters, long long seed) {
    long long a0 = seed + threadIdx.x, a1 = a0 * 3 + 1, a2 = a0 * 5 + 2, a3 = a0 * 7 + 3;
    const long long d0 = (seed & 1023) + 3 + (threadIdx.x & 7), big = 0x3fffffffffffll;
#pragma unroll 1
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int u = 0; u < 16; ++u) {
            a0 = (a0 | big) / (d0 + u); a1 = (a1 | big) / (d0 + u + 1); a2 = (a2 | big) / (d0 + u + 2); a3 = (a3 | big) / (d0 + u + 3);
        }
    }
    if ((a0 ^ a1 ^ a2 ^ a3) == 0x12345678) out[0] = a0;
}

__global__ void __launch_bounds__(256) int_div_reciprocal_kernel(u32* out, int iters, u32 seed) {
    u32 a0 = seed + threadIdx.x, a1 = a0 * 3 + 1, a2 = a0 * 5 + 2, a3 = a0 * 7 + 3;
    const u32 d = (seed & 127u) + 3u, M = (u32)((1ull << 32) / d);
#pragma unroll 1
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int u = 0; u < 16; ++u) {
#define XP_RDIV(a) { const u32 x = a | 0x40000000u; u32 q = __umulhi(x, M); u32 r = x - q * d; if (r >= d) ++q; a = q + u; }
            XP_RDIV(a0) XP_RDIV(a1) XP_RDIV(a2) XP_RDIV(a3)
#undef XP_RDIV
        }
    }
    if ((a0 ^ a1 ^ a2 ^ a3) == 0x12345678u) out[0] = a0;
}

// ------------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------------

cudaError_t launch_prepare(const LoadJob* jobs, int n_jobs, cudaStream_t stream) {
    if (n_jobs <= 0) return cudaSuccess;
    prepare_kernel<<<n_jobs, kPrepThreads, 0, stream>>>(jobs);
    return cudaGetLastError();
}

cudaError_t launch_bigvalues(const LoadJob* jobs, int n_jobs, u64 most_entries, cudaStream_t stream) {
    if (most_entries == 0 || n_jobs <= 0) return cudaSuccess;
    bigvalue_kernel<<<dim3((unsigned)((most_entries / kBigPerThread + 255) / 256 + 1), (unsigned)n_jobs), 256, 0, stream>>>(jobs);
    return cudaGetLastError();
}

cudaError_t launch_reprobe(const LoadJob* jobs, int n_jobs, cudaStream_t stream) {
    if (n_jobs <= 0) return cudaSuccess;
    reprobe_kernel<<<n_jobs, 32, 0, stream>>>(jobs);
    return cudaGetLastError();
}

cudaError_t launch_coord_bounds(SketchDev* const* list, int n_sketches, i64 most_points, cudaStream_t stream) {
    if (most_points <= 0 || n_sketches <= 0) return cudaSuccess;
    const i64 blocks = (most_points + 255) / 256;
    coord_bounds_kernel<<<dim3((unsigned)(blocks < 64 ? blocks : 64), (unsigned)n_sketches), 256, 0, stream>>>(list);
    return cudaGetLastError();
}

cudaError_t launch_stage_points(const SketchDev* s, i64 n_points, i32* coords, cudaStream_t stream) {
    stage_points_kernel<<<(unsigned)((n_points + 255) / 256), 256, 0, stream>>>(s, coords);
    return cudaGetLastError();
}

cudaError_t launch_stage_spec(const SketchDev* s, int hole_index, i64 n_points, i64* spec, u32* bad, cudaStream_t stream) {
    stage_spec_kernel<<<(unsigned)((n_points + 255) / 256), 256, 0, stream>>>(s, hole_index, spec, bad);
    return cudaGetLastError();
}

cudaError_t launch_subvalues(const LoadJob* jobs, int n_jobs, int size, int most_probes, u64 most_entries, cudaStream_t stream) {
    if (most_entries == 0 || most_probes <= 0 || n_jobs <= 0) return cudaSuccess;
    subvalue_kernel<<<dim3((unsigned)((most_entries + 255) / 256), (unsigned)most_probes, (unsigned)n_jobs), 256, 0, stream>>>(jobs, size);
    return cudaGetLastError();
}

static int resident_ctas(const void* kernel, size_t dynamic_smem = 0) {
    int dev = 0, sms = 1, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 1;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, dynamic_smem) != cudaSuccess || per_sm < 1) per_sm = 1;
    return sms * per_sm;
}

static PlanDev plan_on(char* base, const SearchLayout& L, int n_segs, int n_sketches, u32 max_chunks) {
    PlanDev pd;
    pd.ticket_base = 0;
    pd.n_tickets = 0;
    pd.n_segs = n_segs;
    pd.n_sketches = n_sketches;
    pd.ticket = (u64*)base;
    pd.verify_ticket = (u64*)(base + 8);
    pd.surv_n = (u32*)(base + 16);
    pd.err = (u32*)(base + 20);
    pd.segs = (const SegDev*)(base + L.segs);
    pd.sketches = (const SketchDev* const*)(base + L.sketches);
    pd.acc = (AccDev*)(base + L.acc);
    pd.surv = (SurvDev*)(base + L.surv);
    pd.surv_cap = L.surv_cap;
    pd.max_chunks = max_chunks;
    pd.n_acc = L.n_acc;
    const bool order = L.n_acc > 1;                       // (one hole: the queue is in hole order as it is)
    pd.surv_hist = order ? (u32*)(base + L.hist) : nullptr;
    pd.surv_off = order ? (u32*)(base + L.sort_off) : nullptr;
    pd.surv_sorted = order ? (u32*)(base + L.sorted) : nullptr;
    pd.surv_long = (u32*)(base + L.longs);
    pd.surv_long_n = (u32*)(base + 24);
    return pd;
}

// Stages 1 and 2 for the tickets [t_begin, t_end) of the plan staged at `base`.  A search is one
// such launch, or several in a row when the host wants to look at a cancel word or a clock in
// between; `restart` says that the ticket counter has to be set back to zero first (every launch
// but the first, whose counter the staged copy has just zeroed).
cudaError_t launch_search_part(char* base, const SearchLayout& L, u64 t_begin, u64 t_end, bool restart, int n_segs,
                               int n_sketches, u32 max_chunks, cudaStream_t stream, int* n_launches) {
    if (t_end <= t_begin) return cudaSuccess;
    cudaError_t e;
    if (restart && (e = cudaMemsetAsync(base, 0, 8, stream)) != cudaSuccess) return e;
    PlanDev pd = plan_on(base, L, n_segs, n_sketches, max_chunks);
    pd.ticket_base = t_begin;
    pd.n_tickets = t_end;
    const void* kernel = L.dense ? (const void*)eval_kernel<true> : (const void*)eval_kernel<false>;
    u64 ctas = (u64)resident_ctas(kernel, 0);             // persistent CTAs: one wave
    if (ctas > t_end - t_begin) ctas = t_end - t_begin;
    if (L.dense) eval_kernel<true><<<(unsigned)ctas, kThreads, 0, stream>>>(pd);
    else eval_kernel<false><<<(unsigned)ctas, kThreads, 0, stream>>>(pd);
    *n_launches += 1;
    return cudaGetLastError();
}

// Stage 3 and the reductions, after every part of the search has been queued.
cudaError_t launch_search_end(char* base, const SearchLayout& L, bool any_tickets, int n_segs, int n_sketches, int n_acc,
                              u32 max_chunks, cudaStream_t stream, int* n_launches) {
    PlanDev pd = plan_on(base, L, n_segs, n_sketches, max_chunks);
    cudaError_t e;
    if (any_tickets) {
        if (pd.surv_sorted) {
            surv_scan_kernel<<<1, 1024, 0, stream>>>(pd.surv_hist, pd.surv_off, pd.n_acc);
            if ((e = cudaGetLastError()) != cudaSuccess) return e;
            surv_scatter_kernel<<<(L.surv_cap + 255) / 256, 256, 0, stream>>>(pd);
            if ((e = cudaGetLastError()) != cudaSuccess) return e;
            *n_launches += 2;
        }
        if (max_chunks > 1) {
            surv_long_kernel<<<(L.surv_cap + 255) / 256, 256, 0, stream>>>(pd);
            if ((e = cudaGetLastError()) != cudaSuccess) return e;
            *n_launches += 1;
        }
        const size_t vsmem = sizeof(VerifyWarp) * kVerifyWarps;
        if ((e = cudaFuncSetAttribute((const void*)verify_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)vsmem)) != cudaSuccess) return e;
        verify_kernel<<<resident_ctas((const void*)verify_kernel, vsmem), kVerifyThreads, vsmem, stream>>>(pd);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        count_kernel<<<(L.surv_cap + 255) / 256, 256, 0, stream>>>(pd);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
        *n_launches += 2;
    }
    const int warps_per_block = 8;
    finish_kernel<<<(n_acc + warps_per_block - 1) / warps_per_block, warps_per_block * 32, 0, stream>>>(pd.acc, n_acc, pd.err);
    *n_launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_search(char* base, const SearchLayout& L, u64 n_tickets, int n_segs, int n_sketches, int n_acc,
                          u32 max_chunks, cudaStream_t stream, int* n_launches) {
    cudaError_t e = launch_search_part(base, L, 0, n_tickets, false, n_segs, n_sketches, max_chunks, stream, n_launches);
    if (e != cudaSuccess) return e;
    return launch_search_end(base, L, n_tickets > 0, n_segs, n_sketches, n_acc, max_chunks, stream, n_launches);
}

// ------------------------------------------------------------------------------------------
// search with the scratch in a fixed device array (no allocation at call time)
// ------------------------------------------------------------------------------------------

// Scratch of the allocation-free entry point: counters, segment table, sketch pointer,
// accumulators and survivor queue of ONE call.  Every GPU that loads the library holds these
// bytes until the process exits.  In host code the name below is only a stand-in for the
// symbol; the device address comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

static void* g_static_scratch_addr[64];      // per device, filled on the first call made on it

// Copies the staged head of the plan (counters and accumulators in their start state, which
// also wipes what the last call left) into the fixed array, runs the search on it, and queues
// the copy of the accumulators back to `acc_out`.  Allocates nothing.
cudaError_t launch_search_static(const void* stage, const SearchLayout& L, u64 n_tickets, int n_segs, int n_acc,
                                 u32 max_chunks, AccDev* acc_out, cudaStream_t stream) {
    if (L.total > kStaticScratchBytes) return cudaErrorInvalidValue;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!g_static_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_static_scratch_addr[dev] = p;
    }
    char* base = (char*)g_static_scratch_addr[dev];
    e = cudaMemcpyAsync(base, stage, L.head, cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) return e;
    int launches = 0;
    e = launch_search(base, L, n_tickets, n_segs, 1, n_acc, max_chunks, stream, &launches);
    if (e != cudaSuccess) return e;
    return cudaMemcpyAsync(acc_out, base + L.acc, sizeof(AccDev) * (size_t)n_acc, cudaMemcpyDeviceToHost, stream);
}

cudaError_t launch_int32_peak(int which, u32* out, int blocks, int iters, cudaStream_t stream) {
    if (which == 0) int32_peak_add_kernel<<<blocks, 256, 0, stream>>>(out, iters, 1u);
    else if (which == 1) int32_peak_mad_kernel<<<blocks, 256, 0, stream>>>(out, iters, 1u);
    else if (which == 2) int_div_general_kernel<<<blocks, 256, 0, stream>>>((long long*)out, iters, 12345);
    else int_div_reciprocal_kernel<<<blocks, 256, 0, stream>>>(out, iters, 12345u);
    return cudaGetLastError();
}

}  // namespace xp
