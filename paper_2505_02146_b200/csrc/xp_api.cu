// Host side of libxpiler_repair: grammar tables, sketch encoding, launch planning, result
// decoding and the C ABI declared in include/xp.h.
#include <cuda_runtime.h>

#include <algorithm>
#include <climits>
#include <chrono>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <thread>
#include <vector>

#include "xp_dev.h"
#include "xp_launch.h"

using namespace xp;

// ------------------------------------------------------------------------------------------
// errors
// ------------------------------------------------------------------------------------------

static thread_local std::string g_last_error;

static xp_status fail(xp_status st, const std::string& msg) {
    g_last_error = msg;
    return st;
}

namespace xp {
xp_status set_error(xp_status st, const char* msg) { return fail(st, msg); }      // for the library's other source files
}

#define XP_CUDA(call)                                                                          \
    do {                                                                                       \
        cudaError_t e_ = (call);                                                               \
        if (e_ != cudaSuccess)                                                                 \
            return fail(e_ == cudaErrorMemoryAllocation ? XP_ERR_NOMEM : XP_ERR_CUDA,          \
                        std::string(#call) + ": " + cudaGetErrorString(e_));                   \
    } while (0)

// ------------------------------------------------------------------------------------------
// device memory of grammars and sketches
// ------------------------------------------------------------------------------------------
//
// Blocks up to kPoolBigBytes are carved from 64 MiB slabs and, when released, kept in a
// free list by size for the next load (a loop that loads and destroys the same sketch never
// reaches cudaMalloc or cudaFree, whose cost and device-wide synchronisation would otherwise
// dominate small searches).  Larger blocks come from cudaMalloc; released ones are kept too,
// up to kPoolBigKeep bytes in all, and handed out again to a request of the same size.  Slabs
// and kept blocks are returned to the driver when the process ends.  One pool per device.
namespace {
constexpr size_t kPoolSlabBytes = 64ull << 20, kPoolBigBytes = 16ull << 20, kPoolBigKeep = 24ull << 30;
struct DevPool {
    std::multimap<size_t, char*> free_blocks;
    std::multimap<size_t, char*> big_blocks;
    size_t big_kept = 0;
    char* slab = nullptr;
    size_t slab_left = 0;
};
std::mutex g_pool_mu;
std::map<int, DevPool> g_pools;

// *granted receives the size of the block handed out (>= bytes): it is what pool_release must be given.
cudaError_t pool_alloc(void** out, size_t bytes, int* device_out, size_t* granted) {
    const size_t need = ((bytes ? bytes : 1) + 255) & ~(size_t)255;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    *device_out = dev;
    *granted = need;
    std::lock_guard<std::mutex> lock(g_pool_mu);
    DevPool& p = g_pools[dev];
    // a kept block fits a request when it wastes at most an eighth of itself (sketches of varying
    // sizes then reuse each other's blocks instead of growing the pool without bound)
    auto fits = [&](std::multimap<size_t, char*>& m) {
        auto it = m.lower_bound(need);
        return (it != m.end() && it->first - need <= it->first / 8) ? it : m.end();
    };
    if (need > kPoolBigBytes) {
        auto big = fits(p.big_blocks);
        if (big == p.big_blocks.end()) return cudaMalloc(out, need);
        *out = big->second;
        *granted = big->first;
        p.big_kept -= big->first;
        p.big_blocks.erase(big);
        return cudaSuccess;
    }
    auto it = fits(p.free_blocks);
    if (it != p.free_blocks.end()) { *out = it->second; *granted = it->first; p.free_blocks.erase(it); return cudaSuccess; }
    if (p.slab_left < need) {
        if (p.slab_left >= 256) p.free_blocks.insert({p.slab_left, p.slab});      // the old slab's tail stays usable
        char* slab = nullptr;
        e = cudaMalloc((void**)&slab, kPoolSlabBytes);
        if (e != cudaSuccess) { p.slab = nullptr; p.slab_left = 0; return e; }
        p.slab = slab;
        p.slab_left = kPoolSlabBytes;
    }
    *out = p.slab;
    p.slab += need;
    p.slab_left -= need;
    return cudaSuccess;
}

void pool_release(void* ptr, size_t bytes, int device) {
    if (!ptr) return;
    const size_t need = ((bytes ? bytes : 1) + 255) & ~(size_t)255;
    std::lock_guard<std::mutex> lock(g_pool_mu);
    DevPool& p = g_pools[device];
    if (need > kPoolBigBytes) {
        if (p.big_kept + need > kPoolBigKeep) { cudaFree(ptr); return; }
        p.big_blocks.insert({need, (char*)ptr});
        p.big_kept += need;
        return;
    }
    p.free_blocks.insert({need, (char*)ptr});
}
}  // namespace

struct xp_sketch;
static xp_status check_device(const xp_sketch* const* sk, size_t n);

// Page-locked host memory for the staged copies of a load (what goes to the device and what comes
// back), kept by the library from load to load: copies from and to page-locked memory are queued
// without the extra pass through the driver's own staging buffer that a copy from ordinary memory
// takes, which for a batch of thousands of sketches was most of the load's time.  One load uses it
// at a time (a concurrent load falls back to ordinary memory).
namespace {
constexpr size_t kPinnedChunk = 64ull << 20, kPinnedMost = 1ull << 30;
struct PinnedArena {
    std::mutex mu;
    std::vector<char*> chunks;
    size_t chunk = 0, used = 0;
    std::mutex take_mu;               // (the threads of one batch load share the arena)
    void reset() { chunk = 0; used = 0; }
    char* take(size_t bytes) {
        std::lock_guard<std::mutex> lock(take_mu);
        const size_t need = (bytes + 255) & ~(size_t)255;
        if (need > kPinnedChunk) return nullptr;
        if (chunk < chunks.size() && used + need > kPinnedChunk) { ++chunk; used = 0; }
        if (chunk >= chunks.size()) {
            if ((chunks.size() + 1) * kPinnedChunk > kPinnedMost) return nullptr;
            void* p = nullptr;
            if (cudaHostAlloc(&p, kPinnedChunk, cudaHostAllocDefault) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
            chunks.push_back((char*)p);
        }
        char* out = chunks[chunk] + used;
        used += need;
        return out;
    }
};
PinnedArena g_pinned;
}  // namespace

static const char* const kOpText[] = {"+", "-", "*", "/", "%", "<", "<=", "==", "!=", "min", "max", "&&", "||", "<<", ">>"};

// ------------------------------------------------------------------------------------------
// grammar
// ------------------------------------------------------------------------------------------

struct xp_grammar {
    int n_vars = 0, n_nt = 0;
    std::vector<std::string> names;
    std::vector<i64> lo, hi;
    std::vector<xp_production> prods;
    std::vector<LeafDev> leaves;
    std::vector<BinDev> bins;
    int leaf_begin[kMaxNt + 1] = {0};
    int bin_begin[kMaxNt + 1] = {0};
    u64 cnt[kMaxNt][kMaxSize + 1] = {{0}};
    int ok_size = kMaxSize;          // counts are exact (< 2^63) up to this size
    // device copy, made on first use
    std::mutex mu;
    GrammarDev* d_g = nullptr;       // one block: header, leaves, binary productions
    size_t d_bytes = 0;
    int d_device = 0;
};

// cnt[nt][s] by the recurrence over productions and left sizes; off[s] of a binary production
// is the number of size-s trees of its nonterminal that come before it.  Sizes from the first
// one at which a count reaches 2^63 are marked unusable (ok_size).
static void build_counts(xp_grammar* g) {
    for (int s = 1; s <= kMaxSize; ++s) {
        bool overflow = g->ok_size < s;
        for (int nt = 0; nt < g->n_nt && !overflow; ++nt) {
            unsigned __int128 total = 0;
            if (s == 1) total = (unsigned)(g->leaf_begin[nt + 1] - g->leaf_begin[nt]);
            for (int b = g->bin_begin[nt]; b < g->bin_begin[nt + 1] && !overflow; ++b) {
                BinDev& bd = g->bins[b];
                bd.off[s] = (u64)total;
                for (int a = 1; a <= s - 2 && !overflow; ++a) {
                    total += (unsigned __int128)g->cnt[bd.lnt][a] * g->cnt[bd.rnt][s - 1 - a];
                    overflow = (total >> 63) != 0;
                }
            }
            g->cnt[nt][s] = (u64)total;
        }
        if (overflow) {
            if (g->ok_size >= s) g->ok_size = s - 1;
            for (int nt = 0; nt < g->n_nt; ++nt) g->cnt[nt][s] = 0;
        }
    }
}

extern "C" xp_status xp_grammar_create(const xp_grammar_desc* d, xp_grammar** out) {
    if (!d || !out) return fail(XP_ERR_INVALID_ARG, "xp_grammar_create: null argument");
    *out = nullptr;
    if (d->n_vars < 0 || d->n_vars > kMaxVars) return fail(XP_ERR_GRAMMAR, "n_vars out of range");
    if (d->n_nonterminals < 1 || d->n_nonterminals > kMaxNt) return fail(XP_ERR_GRAMMAR, "n_nonterminals out of range");
    if (d->n_productions < 1 || !d->productions) return fail(XP_ERR_GRAMMAR, "no productions");
    if (d->n_vars > 0 && !d->vars) return fail(XP_ERR_GRAMMAR, "vars is null");
    xp_grammar* g = new (std::nothrow) xp_grammar;
    if (!g) return fail(XP_ERR_NOMEM, "out of host memory");
    g->n_vars = d->n_vars;
    g->n_nt = d->n_nonterminals;
    for (int i = 0; i < d->n_vars; ++i) {
        if (d->vars[i].hi < d->vars[i].lo) { delete g; return fail(XP_ERR_GRAMMAR, "variable range with hi < lo"); }
        g->names.push_back(d->vars[i].name ? d->vars[i].name : ("v" + std::to_string(i)));
        g->lo.push_back(d->vars[i].lo);
        g->hi.push_back(d->vars[i].hi);
    }
    for (int i = 0; i < d->n_productions; ++i) {
        const xp_production& p = d->productions[i];
        bool ok = p.lhs >= 0 && p.lhs < g->n_nt;
        if (p.kind == XP_PROD_VAR) ok = ok && p.var >= 0 && p.var < g->n_vars;
        else if (p.kind == XP_PROD_BIN) ok = ok && ((p.op >= XP_OP_ADD && p.op <= XP_OP_MOD) || p.op == XP_OP_MIN || p.op == XP_OP_MAX || p.op == XP_OP_SHL || p.op == XP_OP_SHR) && p.left >= 0 && p.left < g->n_nt && p.right >= 0 && p.right < g->n_nt;
        else if (p.kind != XP_PROD_CONST) ok = false;
        if (!ok) { delete g; return fail(XP_ERR_GRAMMAR, "production " + std::to_string(i) + " is malformed"); }
        g->prods.push_back(p);
    }
    for (int nt = 0; nt < g->n_nt; ++nt) {          // leaves and binaries grouped per nonterminal, order kept
        g->leaf_begin[nt] = (int)g->leaves.size();
        g->bin_begin[nt] = (int)g->bins.size();
        for (const xp_production& p : g->prods) {
            if (p.lhs != nt) continue;
            if (p.kind == XP_PROD_BIN) {
                BinDev b;
                memset(&b, 0, sizeof(b));
                b.op = p.op; b.lnt = p.left; b.rnt = p.right;
                g->bins.push_back(b);
            } else {
                LeafDev l;
                l.var = p.kind == XP_PROD_VAR ? p.var : -1;
                l.pad = 0;
                l.value = p.kind == XP_PROD_CONST ? p.value : 0;
                g->leaves.push_back(l);
            }
        }
    }
    g->leaf_begin[g->n_nt] = (int)g->leaves.size();
    g->bin_begin[g->n_nt] = (int)g->bins.size();
    build_counts(g);
    *out = g;
    return XP_OK;
}

extern "C" void xp_grammar_destroy(xp_grammar* g) {
    if (!g) return;
    pool_release(g->d_g, g->d_bytes, g->d_device);
    delete g;
}

extern "C" xp_status xp_grammar_count(const xp_grammar* g, int32_t nt, int32_t max_size, uint64_t* out) {
    if (!g || !out || nt < 0 || nt >= g->n_nt || max_size < 0 || max_size > kMaxSize)
        return fail(XP_ERR_INVALID_ARG, "xp_grammar_count: bad argument");
    if (max_size > g->ok_size) return fail(XP_ERR_TOO_LARGE, "a candidate count reaches 2^63");
    out[0] = 0;
    for (int s = 1; s <= max_size; ++s) out[s] = g->cnt[nt][s];
    return XP_OK;
}

// rank -> tree, appended to `code` in postfix and to `text` in infix.
static bool host_unrank(const xp_grammar* g, int nt, int size, u64 rank, std::vector<xp_instr>* code, std::string* text) {
    if (size < 1 || size > g->ok_size || rank >= g->cnt[nt][size]) return false;
    if (size == 1) {
        const LeafDev& l = g->leaves[g->leaf_begin[nt] + (int)rank];
        xp_instr in;
        in.kind = l.var >= 0 ? XP_I_VAR : XP_I_CONST;
        in.arg = l.var >= 0 ? l.var : 0;
        in.value = l.value;
        code->push_back(in);
        *text += l.var >= 0 ? g->names[l.var] : std::to_string((long long)l.value);
        return true;
    }
    int p = g->bin_begin[nt];
    const int pe = g->bin_begin[nt + 1];
    while (p + 1 < pe && g->bins[p + 1].off[size] <= rank) ++p;
    const BinDev& b = g->bins[p];
    u64 rem = rank - b.off[size];
    for (int a = 1; a <= size - 2; ++a) {
        const u64 cr = g->cnt[b.rnt][size - 1 - a];
        const u64 block = g->cnt[b.lnt][a] * cr;
        if (rem >= block) { rem -= block; continue; }
        const bool call = b.op == XP_OP_MIN || b.op == XP_OP_MAX;      // printed min(l,r) / max(l,r)
        *text += call ? std::string(kOpText[b.op]) + "(" : std::string("(");
        if (!host_unrank(g, b.lnt, a, rem / cr, code, text)) return false;
        *text += call ? "," : kOpText[b.op];
        if (!host_unrank(g, b.rnt, size - 1 - a, rem % cr, code, text)) return false;
        *text += ")";
        xp_instr in;
        in.kind = XP_I_OP; in.arg = b.op; in.value = 0;
        code->push_back(in);
        return true;
    }
    return false;
}

extern "C" xp_status xp_grammar_unrank(const xp_grammar* g, int32_t nt, int32_t size, uint64_t rank,
                                       xp_instr* code, int32_t code_cap, char* text, size_t text_cap) {
    if (!g || nt < 0 || nt >= g->n_nt || size < 1 || size > kMaxSize)
        return fail(XP_ERR_INVALID_ARG, "xp_grammar_unrank: bad argument");
    std::vector<xp_instr> c;
    std::string t;
    if (!host_unrank(g, nt, size, rank, &c, &t)) return fail(XP_ERR_INVALID_ARG, "xp_grammar_unrank: rank out of range");
    if (code) {
        if (code_cap < (int)c.size()) return fail(XP_ERR_INVALID_ARG, "xp_grammar_unrank: code buffer too small");
        memcpy(code, c.data(), c.size() * sizeof(xp_instr));
    }
    if (text) {
        if (text_cap < t.size() + 1) return fail(XP_ERR_INVALID_ARG, "xp_grammar_unrank: text buffer too small");
        memcpy(text, t.c_str(), t.size() + 1);
    }
    return XP_OK;
}

// (staging: page-locked memory of the load at hand, or null; with it the copy is queued on the
// load's stream like the sketch's own copies and nobody waits for it here)
static xp_status grammar_to_device(xp_grammar* g, size_t* copied, PinnedArena* staging) {
    *copied = 0;
    std::lock_guard<std::mutex> lock(g->mu);
    if (g->d_g) {
        // the device copy was made on the device that was current at the first load and serves that device only
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess || dev != g->d_device)
            return fail(XP_ERR_INVALID_ARG, "the grammar's tables live on device " + std::to_string(g->d_device) +
                        ", the current device is " + std::to_string(dev) + ": use one grammar handle per device");
        return XP_OK;
    }
    GrammarDev h;
    memset(&h, 0, sizeof(h));
    h.n_vars = g->n_vars; h.n_nt = g->n_nt;
    h.n_leaves = (int)g->leaves.size(); h.n_bins = (int)g->bins.size();
    memcpy(h.leaf_begin, g->leaf_begin, sizeof(h.leaf_begin));
    memcpy(h.bin_begin, g->bin_begin, sizeof(h.bin_begin));
    memcpy(h.cnt, g->cnt, sizeof(h.cnt));
    // one device block and one copy: header | leaves | binary productions
    const size_t off_leaves = (sizeof(GrammarDev) + 255) & ~(size_t)255;
    const size_t off_bins = off_leaves + ((sizeof(LeafDev) * (g->leaves.size() + 1) + 255) & ~(size_t)255);
    const size_t total = off_bins + sizeof(BinDev) * (g->bins.size() + 1);
    char* block = nullptr;
    size_t granted = 0;
    XP_CUDA(pool_alloc((void**)&block, total, &g->d_device, &granted));
    g->d_bytes = granted;
    h.leaves = (const LeafDev*)(block + off_leaves);
    h.bins = (const BinDev*)(block + off_bins);
    std::vector<char> stage_own;
    char* stage = staging ? staging->take(total) : nullptr;
    const bool queued = stage != nullptr;
    if (!stage) { stage_own.resize(total); stage = stage_own.data(); }
    memset(stage, 0, total);
    memcpy(stage, &h, sizeof(h));
    if (!g->leaves.empty()) memcpy(stage + off_leaves, g->leaves.data(), sizeof(LeafDev) * g->leaves.size());
    if (!g->bins.empty()) memcpy(stage + off_bins, g->bins.data(), sizeof(BinDev) * g->bins.size());
    cudaError_t e = queued ? cudaMemcpyAsync(block, stage, total, cudaMemcpyHostToDevice, nullptr)
                           : cudaMemcpy(block, stage, total, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) { pool_release(block, g->d_bytes, g->d_device); return fail(XP_ERR_CUDA, std::string("cudaMemcpy: ") + cudaGetErrorString(e)); }
    g->d_g = (GrammarDev*)block;
    *copied = total;
    return XP_OK;
}

// ------------------------------------------------------------------------------------------
// sketch
// ------------------------------------------------------------------------------------------

struct HoleHost {
    int start_nt = 0, max_size = 0;
    bool filter_ok = false;          // the probe filter applies (probe 0 exists, context affine there)
    bool never = false;              // the spec is undefined at some point: no candidate can match
    bool compares = false;           // the filter works on an interval of hole values (the context compares)
    bool second = false;             // filter hits are looked at once more at probe 1 from the start (hits are frequent)
};

struct xp_sketch {
    xp_grammar* g = nullptr;
    int n_holes = 0;
    i64 n_points = 0;
    std::vector<HoleHost> holes;
    SketchDev* d_s = nullptr;
    HoleDev* d_holes = nullptr;
    // Device memory of the sketch: one block laid out at load for everything (sketch and hole
    // records, copies of host tables, staged points and specs, subtree-value tables).
    char* arena = nullptr;
    size_t arena_bytes = 0, arena_used = 0;
    int arena_device = 0;
    size_t load_h2d = 0, load_d2h = 0;               // bytes the load moved
    std::vector<int> n_probes;                       // per hole, as the load (or the last refinement) left them
    int n_refined = 0;                               // points promoted to probes by xp_sketch_refine
    std::vector<size_t> off_kill;                    // per hole: offset of its table of whole-domain failures in the arena
    size_t off_holes = 0;
    int tab_size_cap = 0, tab_probes_cap = 0;        // most sizes / probes that the subtree tables of a hole cover
    u64 entries_at[kMaxSize + 1] = {0};              // subtree-table entries per size (all nonterminals)
    u64 big_entries = 0;                             // most entries of a hole's first-probe table of the next size
    // The sketch's part of a launch plan under default options (every size, no rank window, no flag), as
    // if it were the only sketch of the call: built on the first such call and copied, with ticket, sketch
    // and accumulator numbers shifted, into the plan of every later one (a batch of thousands of small
    // sketches would otherwise spend longer planning than some of its searches take).
    mutable std::mutex plan_mu;
    mutable bool plan_cached = false;
    mutable std::vector<SegDev> plan_segs;
    mutable std::vector<u64> plan_ops;
    mutable u64 plan_tickets = 0;
};

// Checks a postfix expression; returns false when malformed or too deep.
static bool check_code(const xp_instr* code, int n, int n_vars, bool hole_allowed) {
    if (n < 0 || n > kMaxCode || (n > 0 && !code)) return false;
    int sp = 0;
    for (int i = 0; i < n; ++i) {
        const xp_instr& c = code[i];
        if (c.kind == XP_I_OP) {
            if (c.arg < XP_OP_ADD || c.arg > XP_OP_SHR || sp < 2) return false;
            --sp;
        } else {
            if (c.kind == XP_I_VAR) { if (c.arg < 0 || c.arg >= n_vars) return false; }
            else if (c.kind == XP_I_HOLE) { if (!hole_allowed) return false; }
            else if (c.kind != XP_I_CONST) return false;
            if (++sp > kMaxStack) return false;
        }
    }
    return n == 0 || sp == 1;
}

static u64 mix64(u64 x) {            // SplitMix64 finaliser: spreads sample ids over the domain
    x += 0x9E3779B97F4A7C15ull;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}

extern "C" void xp_sketch_destroy(xp_sketch* s) {
    if (!s) return;
    pool_release(s->arena, s->arena_bytes, s->arena_device);
    delete s;
}

// Entries of the subtree-value tables of a hole with size bound max_size: sizes 1, 2, ... while
// every nonterminal has at most kTabMaxEntries trees of that size, and never the sizes that only
// occur as whole candidates (operands have at most max_size - 2 nodes).
static u64 table_entries(const xp_grammar* g, int max_size, u64 (*off)[kMaxSize + 1], int* tmax_out) {
    u64 total = 0;
    int tmax = 0;
    for (int k = 1; k <= max_size - 2; ++k) {
        bool fits = true;
        for (int nt = 0; nt < g->n_nt; ++nt) fits = fits && g->cnt[nt][k] <= kTabMaxEntries;
        if (!fits) break;
        for (int nt = 0; nt < g->n_nt; ++nt) { if (off) off[nt][k] = total; total += g->cnt[nt][k]; }
        tmax = k;
    }
    if (tmax_out) *tmax_out = tmax;
    return total;
}

// One sketch on its way through a load: everything between its description and the moment the
// load's kernels have run.
struct LoadState {
    xp_sketch* s = nullptr;
    std::vector<HoleDev> hh;
    std::vector<char> back_own;      // holes and flags as the kernels left them (ordinary memory, when no page-locked
    char* back = nullptr;            //   memory could be had); back points at whichever holds them
    size_t back_bytes = 0;
    PinnedArena* pinned = nullptr;   // page-locked staging memory of this load, or null
    size_t off_holes = 0;
    i64 table_points = 0;            // rows of a table domain (0 for a box)
    u64 entries_at[kMaxSize + 1] = {0};      // subtree-table entries per size (all nonterminals)
    int size_cap = 0, probes_cap = 0;        // over the holes
    u64 big_entries = 0;                     // most entries of a hole's first-probe table of the next size
};

// First half of a load: checks the description, lays out and allocates the sketch's device
// block, queues the copies of what the host provides and, for a box, the kernels that stage its
// points and spec values.  Nothing here waits for the device.
static xp_status load_begin(const xp_grammar* gc, const xp_sketch_desc* d, LoadState* L) {
    if (!gc || !d) return fail(XP_ERR_INVALID_ARG, "xp_sketch_load: null argument");
    xp_grammar* g = const_cast<xp_grammar*>(gc);
    if (d->n_holes < 1 || !d->holes) return fail(XP_ERR_SKETCH, "a sketch needs at least one hole");
    if (d->domain_kind != XP_DOMAIN_BOX && d->domain_kind != XP_DOMAIN_TABLE) return fail(XP_ERR_SKETCH, "bad domain_kind");
    const int nv = g->n_vars;
    i64 n_points = 0;
    if (d->domain_kind == XP_DOMAIN_BOX) {
        unsigned __int128 n = 1;
        for (int v = 0; v < nv; ++v) {
            n *= (unsigned __int128)(u64)(g->hi[v] - g->lo[v]);
            if (n >> 62) return fail(XP_ERR_TOO_LARGE, "box domain has 2^62 points or more");
        }
        n_points = (i64)n;
    } else {
        if (d->n_points < 0 || (d->n_points > 0 && !d->coords)) return fail(XP_ERR_SKETCH, "table domain without coords");
        n_points = d->n_points;
    }
    for (int h = 0; h < d->n_holes; ++h) {
        const xp_hole_desc& hd = d->holes[h];
        if (hd.start_nt < 0 || hd.start_nt >= g->n_nt) return fail(XP_ERR_SKETCH, "hole start_nt out of range");
        if (hd.max_size < 1 || hd.max_size > kMaxSize) return fail(XP_ERR_SKETCH, "hole max_size out of range");
        if (hd.max_size > g->ok_size) return fail(XP_ERR_TOO_LARGE, "a candidate count reaches 2^63 within the size bound");
        if (!check_code(hd.ctx, hd.ctx_len, nv, true)) return fail(XP_ERR_SKETCH, "malformed context expression");
        if (hd.spec_kind == XP_SPEC_EXPR) {
            if (hd.spec_len < 1 || !check_code(hd.spec_expr, hd.spec_len, nv, false)) return fail(XP_ERR_SKETCH, "malformed spec expression");
        } else if (hd.spec_kind == XP_SPEC_TABLE) {
            if (n_points > 0 && !hd.spec_table) return fail(XP_ERR_SKETCH, "spec table is null");
        } else return fail(XP_ERR_SKETCH, "bad spec_kind");
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) return fail(XP_ERR_CUDA, "no CUDA device is usable");
    size_t grammar_bytes = 0;
    xp_status st = grammar_to_device(g, &grammar_bytes, L->pinned);
    if (st != XP_OK) return st;

    xp_sketch* s = new (std::nothrow) xp_sketch;
    if (!s) return fail(XP_ERR_NOMEM, "out of host memory");
    s->g = g; s->n_holes = d->n_holes; s->n_points = n_points;
#define XP_CUDA_S(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { xp_sketch_destroy(s); \
        return fail(e_ == cudaErrorMemoryAllocation ? XP_ERR_NOMEM : XP_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e_)); } } while (0)

    // One device block for the whole sketch, laid out here before anything runs: first what the
    // host provides (sketch, holes, flags, small tables: one staged copy), then what the load's
    // kernels produce (staged points and specs, subtree tables).  The host then looks at the
    // device once more, at the end, to read back what the kernels decided.
    const int nh = d->n_holes;
    const size_t np = (size_t)n_points, row = (size_t)(nv ? nv : 1);
    auto al = [](size_t b) { return (b + 255) & ~(size_t)255; };
    constexpr size_t kPackMax = 256u << 10;              // host tables up to this size travel in the staged copy
    bool i32_ok = true;
    for (int v = 0; v < nv; ++v) i32_ok = i32_ok && g->lo[v] >= INT32_MIN && g->hi[v] <= (i64)INT32_MAX + 1;
    const bool stage = n_points > 0 && (u64)n_points <= kStageMaxPoints;
    const bool stage_box = d->domain_kind == XP_DOMAIN_BOX && stage && i32_ok && nv > 0;
    const bool copy_coords = d->domain_kind == XP_DOMAIN_TABLE && np > 0 && !d->coords_on_device;
    const size_t coords_bytes = sizeof(i32) * np * row, spec_bytes = sizeof(i64) * np;
    size_t off = 0;
    const size_t off_sketch = off;  off += al(sizeof(SketchDev));
    const size_t off_holes = off;   off += al(sizeof(HoleDev) * nh + sizeof(u32) * nh);       // holes, then one flag each
    const size_t off_bad = off_holes + sizeof(HoleDev) * nh;
    size_t off_coords = 0;
    std::vector<size_t> off_spec(nh, 0), off_tabv(nh, 0), off_tabk(nh, 0), off_tabm(nh, 0), off_bigv(nh, 0), off_bigk(nh, 0);
    if (copy_coords && coords_bytes <= kPackMax) { off_coords = off; off += al(coords_bytes); }
    for (int h = 0; h < nh; ++h)
        if (d->holes[h].spec_kind == XP_SPEC_TABLE && np > 0 && !d->holes[h].spec_table_on_device && spec_bytes <= kPackMax) {
            off_spec[h] = off; off += al(spec_bytes);
        }
    s->off_kill.assign(nh, 0);
    for (int h = 0; h < nh; ++h) { s->off_kill[h] = off; off += al((sizeof(i64) + sizeof(u32)) * kKillSlots); }
    const size_t head = off;                              // [0, head): staged on the host and copied in one piece
    if ((copy_coords && coords_bytes > kPackMax) || stage_box) { off_coords = off; off += al(coords_bytes); }
    std::vector<HoleDev>& hh = L->hh;
    hh.resize(nh);
    for (int h = 0; h < nh; ++h) {
        const xp_hole_desc& hd = d->holes[h];
        HoleDev& o = hh[h];
        memset(&o, 0, sizeof(o));
        if (np > 0 && off_spec[h] == 0 &&
            ((hd.spec_kind == XP_SPEC_TABLE && !hd.spec_table_on_device) || (hd.spec_kind == XP_SPEC_EXPR && stage))) {
            off_spec[h] = off; off += al(spec_bytes);
        }
        const u64 entries = table_entries(g, hd.max_size, o.tab_off, &o.tab_size_cap);
        u64 probes = kMaxProbe;
        while (probes > 1 && entries * 9 * probes > kTabBudgetBytes) --probes;
        o.tab_total = entries;
        o.tab_probes_cap = entries > 0 ? (i32)probes : 0;
        if (entries > 0) {
            off_tabv[h] = off; off += al(sizeof(i64) * entries * probes);
            off_tabk[h] = off; off += al(entries * probes);
            off_tabm[h] = off; off += al(entries);
        }
        // one size further at the first probe only (see HoleDev::big_size): the register-side operands of the largest candidates
        int big = o.tab_size_cap + 1;                     // the next size that has trees at all
        while (big <= hd.max_size - 2) {
            bool any = false;
            for (int nt = 0; nt < g->n_nt; ++nt) any = any || g->cnt[nt][big] > 0;
            if (any) break;
            ++big;
        }
        if (entries > 0 && o.tab_size_cap >= 1 && big <= hd.max_size - 2) {
            u64 total = 0;
            for (int nt = 0; nt < g->n_nt; ++nt) { o.big_off[nt] = total; total += (g->cnt[nt][big] + 7) & ~7ull; }     // (ranges start at multiples of 8: bigvalue_kernel)
            size_t free_b = 0, total_b = 0;
            const bool room = cudaMemGetInfo(&free_b, &total_b) == cudaSuccess && (u64)free_b > 3 * total * 9;
            if (total > 0 && total <= kBigMaxEntries && total * 9 <= kBigBudgetBytes && room) {
                o.big_size = big; o.big_total = total;
                off_bigv[h] = off; off += al(sizeof(i64) * total);
                off_bigk[h] = off; off += al(total);
                if (total > L->big_entries) L->big_entries = total;
            }
        }
    }
    size_t arena_granted = 0;
    if (pool_alloc((void**)&s->arena, off, &s->arena_device, &arena_granted) != cudaSuccess) {
        (void)cudaGetLastError();
        delete s;
        return fail(XP_ERR_NOMEM, "device memory for the sketch (" + std::to_string(off) + " bytes)");
    }
    s->arena_bytes = arena_granted;
    s->arena_used = off;
    char* base = s->arena;
    s->d_s = (SketchDev*)(base + off_sketch);
    s->d_holes = (HoleDev*)(base + off_holes);

    SketchDev hs;
    memset(&hs, 0, sizeof(hs));
    hs.g = g->d_g; hs.n_vars = nv; hs.n_holes = nh; hs.domain_kind = d->domain_kind; hs.n_points = n_points;
    hs.holes = s->d_holes;
    for (int v = 0; v < nv; ++v) {
        hs.lo[v] = g->lo[v]; hs.ext[v] = g->hi[v] - g->lo[v];
        const bool table = d->domain_kind == XP_DOMAIN_TABLE;      // a table's bounds are reduced over its rows below
        hs.vmin[v] = table ? LLONG_MAX : g->lo[v];
        hs.vmax[v] = table ? LLONG_MIN : g->hi[v] - 1;
    }
    if (d->domain_kind == XP_DOMAIN_TABLE && np > 0) hs.coords = d->coords_on_device ? d->coords : (const i32*)(base + off_coords);
    if (stage_box) { hs.coords = (const i32*)(base + off_coords); hs.project = 1; }
    // Sample points the probes are chosen from: box corners first (they expose bound and
    // padding mistakes), then ids spread over the domain by a fixed hash.
    int ns = 0;
    if (n_points > 0) {
        if (d->domain_kind == XP_DOMAIN_BOX) {
            const int ncorner = 1 << (nv < 5 ? nv : 5);
            for (int m = 0; m < ncorner && ns < kProbeSamples / 2; ++m) {
                i64 id = 0;
                for (int v = 0; v < nv; ++v) {
                    const i64 ext = hs.ext[v];
                    const i64 c = (v < 5 && ((m >> v) & 1)) ? ext - 1 : 0;
                    id = id * ext + c;
                }
                bool dup = false;
                for (int k = 0; k < ns; ++k) dup = dup || hs.sample_id[k] == id;
                if (!dup) hs.sample_id[ns++] = id;
            }
        } else {
            for (i64 id = 0; id < n_points && ns < 4; ++id) hs.sample_id[ns++] = id;
        }
        for (u64 k = 0; ns < kProbeSamples && k < 4 * kProbeSamples; ++k) {
            const i64 id = (i64)(mix64(k) % (u64)n_points);
            bool dup = false;
            for (int j = 0; j < ns; ++j) dup = dup || hs.sample_id[j] == id;
            if (!dup) hs.sample_id[ns++] = id;
        }
    }
    hs.n_samples = ns;
    u64 most = 0;                                         // small searches get a cheaper probe choice: the load
    for (int h = 0; h < nh; ++h) {                        // should not outweigh the search
        u64 c = 0;
        for (int k = 1; k <= d->holes[h].max_size; ++k) c += g->cnt[d->holes[h].start_nt][k];
        most = c > most ? c : most;
        hh[h].small_search = c <= 100000000ull ? 1 : 0;
    }
    hs.prep_cands = most <= 100000000ull ? 256 : 1024;

    for (int h = 0; h < nh; ++h) {
        const xp_hole_desc& hd = d->holes[h];
        HoleDev& o = hh[h];
        o.start_nt = hd.start_nt; o.max_size = hd.max_size; o.ctx_len = hd.ctx_len;
        if (hd.ctx_len) memcpy(o.ctx, hd.ctx, sizeof(xp_instr) * hd.ctx_len);
        if (hd.spec_kind == XP_SPEC_EXPR) {
            o.spec_len = hd.spec_len;
            memcpy(o.spec, hd.spec_expr, sizeof(xp_instr) * hd.spec_len);
            if (off_spec[h]) o.spec_table = (const i64*)(base + off_spec[h]);       // staged below, before anything reads it
        } else if (np > 0) {
            o.spec_table = hd.spec_table_on_device ? (const i64*)hd.spec_table : (const i64*)(base + off_spec[h]);
        }
        if (o.tab_total > 0) {
            o.tab_val = (i64*)(base + off_tabv[h]);
            o.tab_ok = (unsigned char*)(base + off_tabk[h]);
            o.tab_vars = (unsigned char*)(base + off_tabm[h]);
        }
        if (o.big_size > 0) {
            o.big_val = (i64*)(base + off_bigv[h]);
            o.big_ok = (unsigned char*)(base + off_bigk[h]);
        }
        // variables the context and the spec mention (a caller's spec table may depend on all)
        u32 fv = hd.spec_kind == XP_SPEC_EXPR ? 0u : 0xffffffffu;
        for (int i = 0; i < hd.ctx_len; ++i) if (hd.ctx[i].kind == XP_I_VAR) fv |= 1u << hd.ctx[i].arg;
        if (hd.spec_kind == XP_SPEC_EXPR)
            for (int i = 0; i < hd.spec_len; ++i) if (hd.spec_expr[i].kind == XP_I_VAR) fv |= 1u << hd.spec_expr[i].arg;
        o.fixed_vars = fv;
        o.kill_pid = (i64*)(base + s->off_kill[h]);
        o.kill_cnt = (u32*)(base + s->off_kill[h] + sizeof(i64) * kKillSlots);
        HoleHost ho;
        ho.start_nt = hd.start_nt; ho.max_size = hd.max_size;
        s->holes.push_back(ho);
    }

    // the staged copy, then the tables too large for it
    std::vector<char> stg_own;
    char* stg = L->pinned ? L->pinned->take(head) : nullptr;
    if (!stg) { stg_own.resize(head); stg = stg_own.data(); }
    memset(stg, 0, head);
    memcpy(&stg[off_sketch], &hs, sizeof(hs));
    memcpy(&stg[off_holes], hh.data(), sizeof(HoleDev) * nh);
    if (copy_coords && coords_bytes <= kPackMax) memcpy(&stg[off_coords], d->coords, coords_bytes);
    for (int h = 0; h < nh; ++h) {
        const xp_hole_desc& hd = d->holes[h];
        if (hd.spec_kind == XP_SPEC_TABLE && np > 0 && !hd.spec_table_on_device && spec_bytes <= kPackMax)
            memcpy(&stg[off_spec[h]], hd.spec_table, spec_bytes);
        memset(&stg[s->off_kill[h]], 0xff, sizeof(i64) * kKillSlots);           // no point noted yet (ids -1, counts 0)
    }
    s->load_h2d = grammar_bytes + head;
    XP_CUDA_S(cudaMemcpyAsync(base, stg, head, cudaMemcpyHostToDevice, nullptr));
    if (copy_coords && coords_bytes > kPackMax) {
        XP_CUDA_S(cudaMemcpyAsync(base + off_coords, d->coords, coords_bytes, cudaMemcpyHostToDevice, nullptr));
        s->load_h2d += coords_bytes;
    }
    for (int h = 0; h < nh; ++h) {
        const xp_hole_desc& hd = d->holes[h];
        if (hd.spec_kind == XP_SPEC_TABLE && np > 0 && !hd.spec_table_on_device && spec_bytes > kPackMax) {
            XP_CUDA_S(cudaMemcpyAsync(base + off_spec[h], hd.spec_table, spec_bytes, cudaMemcpyHostToDevice, nullptr));
            s->load_h2d += spec_bytes;
        }
    }
    // The load's kernels, in stream order: points of a box and values of spec expressions (so that
    // the whole-domain check, and the probe choice, read tables for every kind of domain); bounds of a
    // table's coordinates; the probe choice; the subtree tables, bottom-up, for as many sizes and
    // probes as there can be (launches beyond what the probe choice settled on return at once).
    if (stage_box) XP_CUDA_S(launch_stage_points(s->d_s, n_points, (i32*)(base + off_coords), nullptr));
    if (stage)
        for (int h = 0; h < nh; ++h)
            if (hh[h].spec_len != 0)
                XP_CUDA_S(launch_stage_spec(s->d_s, h, n_points, (i64*)(base + off_spec[h]), (u32*)(base + off_bad) + h, nullptr));
    L->s = s;
    L->off_holes = off_holes;
    s->off_holes = off_holes;
    L->table_points = d->domain_kind == XP_DOMAIN_TABLE ? n_points : 0;
    for (int h = 0; h < nh; ++h) {
        if (hh[h].tab_size_cap > L->size_cap) L->size_cap = hh[h].tab_size_cap;
        if (hh[h].tab_probes_cap > L->probes_cap) L->probes_cap = hh[h].tab_probes_cap;
    }
    for (int k = 1; k <= kMaxSize; ++k)
        for (int nt = 0; nt < g->n_nt; ++nt) L->entries_at[k] += g->cnt[nt][k];
    s->tab_size_cap = L->size_cap; s->tab_probes_cap = L->probes_cap; s->big_entries = L->big_entries;
    memcpy(s->entries_at, L->entries_at, sizeof(s->entries_at));
#undef XP_CUDA_S
    return XP_OK;
}

extern "C" xp_status xp_sketch_load_batch(const xp_grammar* const* grammars, const xp_sketch_desc* descs, size_t n,
                                          xp_sketch** outs) {
    if (!grammars || !descs || !outs || n == 0) return fail(XP_ERR_INVALID_ARG, "xp_sketch_load_batch: null argument");
    for (size_t i = 0; i < n; ++i) outs[i] = nullptr;
    std::vector<LoadState> st(n);
    std::unique_lock<std::mutex> pin(g_pinned.mu, std::try_to_lock);
    if (pin.owns_lock()) {
        g_pinned.reset();
        for (size_t i = 0; i < n; ++i) st[i].pinned = &g_pinned;
    }
    char* jobs_dev = nullptr;
    size_t jobs_bytes = 0;
    int jobs_device = 0;
    auto undo = [&]() {
        cudaStreamSynchronize(nullptr);                   // nothing may still be writing into the blocks
        for (size_t i = 0; i < n; ++i) if (st[i].s) xp_sketch_destroy(st[i].s);
        pool_release(jobs_dev, jobs_bytes, jobs_device);
    };
    size_t n_jobs = 0;
    {
        // The host part of a load (checks, layout, staging of the tables, queueing of the copies) is
        // independent from sketch to sketch: large batches spread it over a few threads, each with
        // the caller's device current.  Everything is queued on the same stream; the batch's kernels
        // follow once the threads are done.
        std::vector<xp_status> status(n, XP_OK);
        std::vector<std::string> message(n);
        int dev = 0;
        cudaGetDevice(&dev);
        unsigned hw = std::thread::hardware_concurrency();
        size_t n_threads = n / 128;
        if (n_threads > 8) n_threads = 8;
        if (hw > 0 && n_threads > hw) n_threads = hw;
        auto work = [&](size_t t, size_t step) {
            if (step > 1) cudaSetDevice(dev);
            for (size_t i = t; i < n; i += step) {
                status[i] = load_begin(grammars[i], &descs[i], &st[i]);
                if (status[i] != XP_OK) message[i] = g_last_error;
            }
        };
        if (n_threads < 2) work(0, 1);
        else {
            std::vector<std::thread> pool;
            for (size_t t = 0; t < n_threads; ++t) pool.emplace_back(work, t, n_threads);
            for (std::thread& th : pool) th.join();
        }
        for (size_t i = 0; i < n; ++i)
            if (status[i] != XP_OK) { undo(); return fail(status[i], "sketch " + std::to_string(i) + ": " + message[i]); }
        for (size_t i = 0; i < n; ++i) n_jobs += (size_t)st[i].s->n_holes;
    }
#define XP_CUDA_B(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { undo(); \
        return fail(e_ == cudaErrorMemoryAllocation ? XP_ERR_NOMEM : XP_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e_)); } } while (0)
    // the batch's kernels: one list of sketches, one list of (sketch, hole) jobs
    const size_t list_bytes = (sizeof(SketchDev*) * n + 255) & ~(size_t)255;
    std::vector<char> stage(list_bytes + sizeof(LoadJob) * n_jobs, 0);
    {
        size_t j = 0;
        for (size_t i = 0; i < n; ++i) {
            ((SketchDev**)stage.data())[i] = st[i].s->d_s;
            for (int h = 0; h < st[i].s->n_holes; ++h, ++j) {
                LoadJob job;
                job.s = st[i].s->d_s; job.hole = h; job.pad = 0;
                memcpy(&stage[list_bytes + sizeof(LoadJob) * j], &job, sizeof(job));
            }
        }
    }
    XP_CUDA_B(pool_alloc((void**)&jobs_dev, stage.size(), &jobs_device, &jobs_bytes));
    XP_CUDA_B(cudaMemcpyAsync(jobs_dev, stage.data(), stage.size(), cudaMemcpyHostToDevice, nullptr));
    SketchDev* const* d_list = (SketchDev* const*)jobs_dev;
    const LoadJob* d_jobs = (const LoadJob*)(jobs_dev + list_bytes);
    // In stream order after the copies and the boxes' staging: bounds of the tables' coordinates;
    // the probe choice; the subtree tables, bottom-up, for as many sizes and probes as there can be
    // (blocks beyond what the probe choice settled on for their hole return at once).  Grids are
    // cut into pieces of at most kPiece jobs (a grid dimension holds 65 535).
    constexpr size_t kPiece = 32768;
    i64 most_points = 0;
    int size_cap = 0, probes_cap = 0;
    u64 most_entries[kMaxSize + 1] = {0};
    for (size_t i = 0; i < n; ++i) {
        most_points = st[i].table_points > most_points ? st[i].table_points : most_points;
        size_cap = st[i].size_cap > size_cap ? st[i].size_cap : size_cap;
        probes_cap = st[i].probes_cap > probes_cap ? st[i].probes_cap : probes_cap;
        for (int k = 1; k <= st[i].size_cap; ++k) most_entries[k] = st[i].entries_at[k] > most_entries[k] ? st[i].entries_at[k] : most_entries[k];
    }
    for (size_t at = 0; at < n; at += kPiece)
        XP_CUDA_B(launch_coord_bounds(d_list + at, (int)(n - at < kPiece ? n - at : kPiece), most_points, nullptr));
    for (size_t at = 0; at < n_jobs; at += kPiece)
        XP_CUDA_B(launch_prepare(d_jobs + at, (int)(n_jobs - at < kPiece ? n_jobs - at : kPiece), nullptr));
    for (int k = 1; k <= size_cap; ++k)
        for (size_t at = 0; at < n_jobs; at += kPiece)
            XP_CUDA_B(launch_subvalues(d_jobs + at, (int)(n_jobs - at < kPiece ? n_jobs - at : kPiece), k, probes_cap, most_entries[k], nullptr));
    {
        u64 big = 0;
        for (size_t i = 0; i < n; ++i) big = st[i].big_entries > big ? st[i].big_entries : big;
        for (size_t at = 0; at < n_jobs && big > 0; at += 32768)
            XP_CUDA_B(launch_bigvalues(d_jobs + at, (int)(n_jobs - at < 32768 ? n_jobs - at : 32768), big, nullptr));
    }
    // what the kernels decided, per hole
    for (size_t i = 0; i < n; ++i) {
        const int nh = st[i].s->n_holes;
        st[i].back_bytes = sizeof(HoleDev) * nh + sizeof(u32) * nh;
        st[i].back = st[i].pinned ? st[i].pinned->take(st[i].back_bytes) : nullptr;
        if (!st[i].back) { st[i].back_own.resize(st[i].back_bytes); st[i].back = st[i].back_own.data(); }
        XP_CUDA_B(cudaMemcpyAsync(st[i].back, st[i].s->arena + st[i].off_holes, st[i].back_bytes, cudaMemcpyDeviceToHost, nullptr));
        st[i].s->load_d2h = st[i].back_bytes;
        st[i].s->load_h2d += sizeof(SketchDev*) + sizeof(LoadJob) * (size_t)nh;       // its lines of the batch's job lists
    }
    XP_CUDA_B(cudaStreamSynchronize(nullptr));
#undef XP_CUDA_B
    pool_release(jobs_dev, jobs_bytes, jobs_device);
    for (size_t i = 0; i < n; ++i) {
        xp_sketch* s = st[i].s;
        const int nh = s->n_holes;
        for (int h = 0; h < nh; ++h) {
            HoleDev o;
            memcpy(&o, &st[i].back[sizeof(HoleDev) * h], sizeof(o));
            u32 bad = 0;
            memcpy(&bad, &st[i].back[sizeof(HoleDev) * nh + sizeof(u32) * h], sizeof(bad));
            // the filter applies where the context at probe 0 is affine in the hole, or a comparison
            s->holes[h].filter_ok = o.filter_ok != 0;
            s->holes[h].compares = o.filter_ok != 0 && o.aff_ok == 0;
            s->holes[h].never = bad != 0;                 // the spec is undefined at some point
            s->holes[h].second = o.second != 0;
            s->n_probes.push_back(o.n_probe);
        }
        outs[i] = s;
    }
    return XP_OK;
}

extern "C" xp_status xp_sketch_load(const xp_grammar* g, const xp_sketch_desc* d, xp_sketch** out) {
    if (!g || !d || !out) return fail(XP_ERR_INVALID_ARG, "xp_sketch_load: null argument");
    return xp_sketch_load_batch(&g, d, 1, out);
}

namespace xp {
SketchInternals sketch_internals(const xp_sketch* s) { return SketchInternals{s->d_s, s->g, s->n_points, s->arena_device, s->g->n_vars}; }
u64 grammar_cnt(const xp_grammar* g, int nt, int size) { return g->cnt[nt][size]; }
int grammar_nonterminals(const xp_grammar* g) { return g->n_nt; }
int grammar_ok_size(const xp_grammar* g) { return g->ok_size; }
GrammarHost grammar_host(const xp_grammar* g) {
    static thread_local std::vector<const char*> names;
    names.clear();
    for (const std::string& n : g->names) names.push_back(n.c_str());
    return GrammarHost{g->n_nt, g->n_vars, g->leaf_begin, g->bin_begin, g->leaves.data(), g->bins.data(), names.data()};
}
HoleSpec sketch_hole(const xp_sketch* s, int hole) {
    if (hole < 0 || hole >= s->n_holes) return HoleSpec{-1, 0};
    return HoleSpec{s->holes[hole].start_nt, s->holes[hole].max_size};
}
const HoleDev* sketch_hole_dev(const xp_sketch* s, int hole) { return s->d_holes + hole; }
cudaError_t device_alloc(void** out, size_t bytes, int* device, size_t* granted) { return pool_alloc(out, bytes, device, granted); }
void device_release(void* ptr, size_t granted, int device) { pool_release(ptr, granted, device); }
}  // namespace xp

extern "C" xp_status xp_sketch_info_get(const xp_sketch* s, xp_sketch_info* out) {
    if (!s || !out) return fail(XP_ERR_INVALID_ARG, "xp_sketch_info_get: null argument");
    memset(out, 0, sizeof(*out));
    out->n_holes = s->n_holes; out->device = s->arena_device; out->n_points = s->n_points;
    out->device_bytes = s->arena_bytes; out->load_h2d_bytes = s->load_h2d; out->load_d2h_bytes = s->load_d2h;
    for (int h = 0; h < s->n_holes && h < 8; ++h) out->n_probes[h] = s->n_probes[h];
    out->n_refined = s->n_refined;
    return XP_OK;
}

// Promotes the points that ended whole-domain checks to probes (see include/xp.h).  The hole
// records and the tables of noted points are read back; per hole the new probe list is
// [probe 0, promoted points by how many survivors each ended, the other old probes]; the records
// go back with the new ids, one small kernel derives coordinates, spec values and context forms
// of the probes again, and the subtree tables are rebuilt for them.
extern "C" xp_status xp_sketch_refine(xp_sketch* s, int32_t max_promote, int32_t* n_promoted) {
    if (n_promoted) *n_promoted = 0;
    if (!s || max_promote < 0) return fail(XP_ERR_INVALID_ARG, "xp_sketch_refine: bad argument");
    const xp_sketch* cs = s;
    xp_status st = check_device(&cs, 1);
    if (st != XP_OK) return st;
    const int nh = s->n_holes;
    const int most = max_promote == 0 ? 4 : max_promote;
    const size_t kill_bytes = (sizeof(i64) + sizeof(u32)) * kKillSlots;
    std::vector<HoleDev> hh(nh);
    std::vector<char> kills(kill_bytes * nh);
    XP_CUDA(cudaStreamSynchronize(nullptr));
    XP_CUDA(cudaMemcpy(hh.data(), s->arena + s->off_holes, sizeof(HoleDev) * nh, cudaMemcpyDeviceToHost));
    for (int h = 0; h < nh; ++h)
        XP_CUDA(cudaMemcpy(&kills[kill_bytes * h], s->arena + s->off_kill[h], kill_bytes, cudaMemcpyDeviceToHost));
    int promoted = 0;
    std::vector<LoadJob> jobs;
    for (int h = 0; h < nh; ++h) {
        HoleDev& o = hh[h];
        const i64* pid = (const i64*)&kills[kill_bytes * h];
        const u32* cnt = (const u32*)(&kills[kill_bytes * h] + sizeof(i64) * kKillSlots);
        std::vector<std::pair<u32, i64>> found;          // (survivors ended, point), most frequent first
        for (int k = 0; k < kKillSlots; ++k)
            if (pid[k] >= 0 && pid[k] < s->n_points && cnt[k] > 0) found.push_back({cnt[k], pid[k]});
        std::sort(found.begin(), found.end(), [](const std::pair<u32, i64>& a, const std::pair<u32, i64>& b) {
            return a.first != b.first ? a.first > b.first : a.second < b.second; });
        if (found.empty() || o.n_probe < 1) continue;
        std::vector<i64> ids;
        ids.push_back(o.probe_id[0]);
        int taken = 0;
        for (size_t k = 0; k < found.size() && taken < most && (int)ids.size() < kMaxProbe; ++k) {
            bool dup = false;
            for (int j = 0; j < o.n_probe; ++j) dup = dup || o.probe_id[j] == found[k].second;
            if (!dup) { ids.push_back(found[k].second); ++taken; }
        }
        if (taken == 0) continue;
        for (int j = 1; j < o.n_probe && (int)ids.size() < kMaxProbe; ++j) ids.push_back(o.probe_id[j]);
        o.n_probe = (i32)ids.size();
        for (int j = 0; j < o.n_probe; ++j) o.probe_id[j] = ids[j];
        promoted += taken;
        LoadJob job;
        job.s = s->d_s; job.hole = h; job.pad = 0;
        jobs.push_back(job);
    }
    // the notes start afresh whether or not anything was promoted
    std::vector<char> fresh(kill_bytes, 0);
    memset(fresh.data(), 0xff, sizeof(i64) * kKillSlots);
    for (int h = 0; h < nh; ++h) XP_CUDA(cudaMemcpyAsync(s->arena + s->off_kill[h], fresh.data(), kill_bytes, cudaMemcpyHostToDevice, nullptr));
    if (!jobs.empty()) {
        char* jobs_dev = nullptr;
        size_t jobs_bytes = 0;
        int jobs_device = 0;
        XP_CUDA(pool_alloc((void**)&jobs_dev, sizeof(LoadJob) * jobs.size(), &jobs_device, &jobs_bytes));
        cudaError_t e = cudaMemcpyAsync(s->arena + s->off_holes, hh.data(), sizeof(HoleDev) * nh, cudaMemcpyHostToDevice, nullptr);
        if (e == cudaSuccess) e = cudaMemcpyAsync(jobs_dev, jobs.data(), sizeof(LoadJob) * jobs.size(), cudaMemcpyHostToDevice, nullptr);
        if (e == cudaSuccess) e = launch_reprobe((const LoadJob*)jobs_dev, (int)jobs.size(), nullptr);
        for (int k = 1; k <= s->tab_size_cap && e == cudaSuccess; ++k)
            e = launch_subvalues((const LoadJob*)jobs_dev, (int)jobs.size(), k, s->tab_probes_cap, s->entries_at[k], nullptr);
        if (e == cudaSuccess) e = launch_bigvalues((const LoadJob*)jobs_dev, (int)jobs.size(), s->big_entries, nullptr);
        if (e == cudaSuccess) e = cudaMemcpyAsync(hh.data(), s->arena + s->off_holes, sizeof(HoleDev) * nh, cudaMemcpyDeviceToHost, nullptr);
        const cudaError_t e2 = cudaStreamSynchronize(nullptr);
        pool_release(jobs_dev, jobs_bytes, jobs_device);
        if (e != cudaSuccess || e2 != cudaSuccess)
            return fail(XP_ERR_CUDA, std::string("xp_sketch_refine: ") + cudaGetErrorString(e != cudaSuccess ? e : e2));
        for (int h = 0; h < nh; ++h) {
            s->holes[h].filter_ok = hh[h].filter_ok != 0;
            s->holes[h].compares = hh[h].filter_ok != 0 && hh[h].aff_ok == 0;
            s->holes[h].second = hh[h].second != 0;
            s->n_probes[h] = hh[h].n_probe;
        }
        std::lock_guard<std::mutex> lock(s->plan_mu);
        s->plan_cached = false;                           // (the plan depends on which holes the filter serves)
    } else {
        XP_CUDA(cudaStreamSynchronize(nullptr));
    }
    s->n_refined += promoted;
    if (n_promoted) *n_promoted = promoted;
    return XP_OK;
}

// ------------------------------------------------------------------------------------------
// repair
// ------------------------------------------------------------------------------------------

struct HoleResult {
    int max_size = 0, solved = 0, least_size = 0;
    u64 cand_count[kMaxSize + 1] = {0};
    u64 match_count[kMaxSize + 1] = {0};
    u64 least_rank = 0;
    std::vector<xp_instr> code;
    std::string text;
    u64 evals = 0, filter_survivors = 0, probe_survivors = 0, nominal_ops = 0;
    u64 filter_tests = 0, skipped = 0;
};

struct xp_result {
    std::vector<HoleResult> holes;
    double kernel_ms = 0, total_ms = 0;
    int n_launches = 0;
    u64 h2d_bytes = 0, d2h_bytes = 0;
};

struct Plan {
    std::vector<SegDev> segs;
    std::vector<AccDev> acc;
    std::vector<u64> nominal_ops;    // per accumulator: cost-model operations of the filter stage
    u64 n_tickets = 0;
};

// Scratch of calls that bring no workspace: one block per process, reused while no other call
// is using it (a concurrent call allocates its own).
static std::mutex g_ws_mu;
static char* g_ws = nullptr;
static size_t g_ws_bytes = 0;
static int g_ws_device = -1;

static const xp_repair_opts kDefaultOpts = {0, 0, 0, nullptr, nullptr, nullptr, 0, 0u, nullptr, 0};

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

static void add_linear(Plan* plan, int sketch, int hole, int acc, int k, u64 lo, u64 hi) {
    SegDev sg;
    memset(&sg, 0, sizeof(sg));
    sg.first_ticket = plan->n_tickets;
    sg.rank_begin = lo; sg.rank_end = hi;
    sg.sketch = sketch; sg.hole = hole; sg.size = k; sg.kind = kSegLinear; sg.acc = acc;
    plan->segs.push_back(sg);
    plan->n_tickets += (hi - lo + (u64)kLinearChunk - 1) / (u64)kLinearChunk;
}

constexpr u64 kFamilyMaxWork = 512;          // candidates per register operand below which segments share a fill

// Tile segments of (start nonterminal, size k) restricted to ranks [lo, hi): one per
// (left size, group of productions with the same operand nonterminals and the same rows).
static void add_tiles(Plan* plan, const xp_grammar* g, int nt, int sketch, int hole, int acc, int k, u64 lo, u64 hi, int bc_tile) {
    const size_t first_seg = plan->segs.size();
    for (int b = g->bin_begin[nt]; b < g->bin_begin[nt + 1]; ++b) {
        const BinDev& bd = g->bins[b];
        u64 base = bd.off[k];
        for (int a = 1; a <= k - 2; ++a) {
            const u64 cl = g->cnt[bd.lnt][a], cr = g->cnt[bd.rnt][k - 1 - a];
            const u64 block = cl * cr;
            if (block == 0) continue;
            const u64 this_base = base;
            base += block;
            if (this_base + block <= lo || this_base >= hi) continue;
            const u64 wlo = lo > this_base ? lo - this_base : 0;
            const u64 whi = hi - this_base < block ? hi - this_base : block;
            const u64 l0 = wlo / cr, l1 = (whi + cr - 1) / cr;
            const bool reg_left = (l1 - l0) >= cr;
            SegDev* sg = nullptr;
            for (size_t i = first_seg; i < plan->segs.size() && !sg; ++i) {       // an open group this production fits in
                SegDev& c = plan->segs[i];
                const int c_lnt = c.swap ? c.bc_nt : c.reg_nt, c_rnt = c.swap ? c.reg_nt : c.bc_nt;
                const int c_a = c.swap ? c.bc_size : c.reg_size;
                const u64 c_l0 = c.swap ? c.bc_begin : c.reg_begin, c_l1 = c_l0 + (c.swap ? c.bc_count : c.reg_count);
                bool has_op = false;
                for (int o = 0; o < c.n_ops; ++o) has_op = has_op || c.op[o] == bd.op;
                if (c_lnt == bd.lnt && c_rnt == bd.rnt && c_a == a && c_l0 == l0 && c_l1 == l1 && !has_op && c.n_ops < 5) sg = &c;
            }
            if (!sg) {
                SegDev n;
                memset(&n, 0, sizeof(n));
                n.rank_begin = lo; n.rank_end = hi;
                n.sketch = sketch; n.hole = hole; n.size = k; n.kind = kSegTile; n.acc = acc;
                n.swap = reg_left ? 0 : 1;
                n.reg_nt = reg_left ? bd.lnt : bd.rnt;  n.reg_size = reg_left ? a : k - 1 - a;
                n.bc_nt = reg_left ? bd.rnt : bd.lnt;   n.bc_size = reg_left ? k - 1 - a : a;
                n.reg_begin = reg_left ? l0 : 0;        n.reg_count = reg_left ? l1 - l0 : cr;
                n.bc_begin = reg_left ? 0 : l0;         n.bc_count = reg_left ? cr : l1 - l0;
                n.right_count = cr;
                n.reg_tiles = (u32)((n.reg_count + kRegTile - 1) / kRegTile);
                n.bc_tile = bc_tile;
                n.bc_tiles = (u32)((n.bc_count + bc_tile - 1) / bc_tile);
                plan->segs.push_back(n);
                sg = &plan->segs.back();
            }
            sg->op[sg->n_ops] = bd.op;
            sg->op_base[sg->n_ops] = this_base;
            sg->n_ops += 1;
            if (bd.op == XP_OP_DIV || bd.op == XP_OP_MOD) sg->has_div = 1;
            if (bd.op == XP_OP_SHL || bd.op == XP_OP_SHR) sg->generic = 1;
        }
    }
    // Families: segments with the same register-side operands and a single broadcast tile are
    // put next to each other; the first takes the tickets (one per register tile) and visits
    // the others, so the register operands are fetched once for all of them.
    std::vector<SegDev> ordered;
    std::vector<char> placed(plan->segs.size() - first_seg, 0);
    for (size_t i = first_seg; i < plan->segs.size(); ++i) {
        if (placed[i - first_seg]) continue;
        const SegDev head = plan->segs[i];
        placed[i - first_seg] = 1;
        const size_t at = ordered.size();
        ordered.push_back(head);
        int members = 1;
        // (worth it only for segments with little work per register operand: the fill is then a large share)
        if (head.bc_tiles == 1 && head.bc_count * (u64)head.n_ops < kFamilyMaxWork)
            for (size_t j = i + 1; j < plan->segs.size(); ++j) {
                const SegDev& c = plan->segs[j];
                if (members == kMaxFamily) break;               // the rest head families of their own
                if (placed[j - first_seg] || c.bc_tiles != 1 || c.bc_count * (u64)c.n_ops >= kFamilyMaxWork || c.reg_nt != head.reg_nt || c.reg_size != head.reg_size ||
                    c.reg_begin != head.reg_begin || c.reg_count != head.reg_count) continue;
                placed[j - first_seg] = 1;
                ordered.push_back(c);
                ordered.back().family = 0;
                ++members;
            }
        ordered[at].family = members;
        // broadcast slots side by side when the whole family fits the tile and has one tile each
        u64 slots = 0;
        bool one_tile = true;
        for (int m = 0; m < members; ++m) { slots += ordered[at + m].bc_count; one_tile = one_tile && ordered[at + m].bc_tiles == 1; }
        if (one_tile && slots <= (u64)kBcTile) {
            u64 base = 0;
            for (int m = 0; m < members; ++m) { ordered[at + m].bc_base = (i32)base; base += ordered[at + m].bc_count; }
            ordered[at].bc_keep = 1;
        }
    }
    for (size_t i = 0; i < ordered.size(); ++i) plan->segs[first_seg + i] = ordered[i];
    for (size_t i = first_seg; i < plan->segs.size(); ++i) {
        SegDev& c = plan->segs[i];
        c.first_ticket = plan->n_tickets;                          // members: where the next head starts
        if (c.family >= 1) plan->n_tickets += (u64)c.reg_tiles * c.bc_tiles;
        // cost model: operation + comparison per evaluation; / and % share one reciprocal division
        u64 per_pair = 0;
        bool div = false, mod = false;
        for (int o = 0; o < c.n_ops; ++o) {
            if (c.op[o] == XP_OP_DIV) div = true;
            else if (c.op[o] == XP_OP_MOD) mod = true;
            else per_pair += 2;
        }
        if (div || mod) per_pair += 7 + (div ? 1 : 0) + (mod ? 2 : 0);
        plan->nominal_ops[acc] += c.reg_count * c.bc_count * per_pair;
    }
}

constexpr u64 kTileMinRanks = 4096;          // smaller windows are searched rank by rank

static void plan_sketch(const xp_sketch* s, size_t i, const xp_repair_opts* o, Plan* plan);

// A sketch's tables, and the library's scratch, live on the device that was current when the sketch was
// loaded: a call made with another device current would hand the kernels pointers of the wrong GPU.
static xp_status check_device(const xp_sketch* const* sk, size_t n) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return fail(XP_ERR_CUDA, "no CUDA device is usable");
    for (size_t i = 0; i < n; ++i)
        if (sk[i] && sk[i]->arena_device != dev)
            return fail(XP_ERR_INVALID_ARG, "sketch " + std::to_string(i) + " was loaded on device " + std::to_string(sk[i]->arena_device) +
                        ", the current device is " + std::to_string(dev));
    return XP_OK;
}

static xp_status build_plan(const xp_sketch* const* sk, size_t n, const xp_repair_opts* o, Plan* plan) {
    const bool plain = o->size_min <= 0 && o->size_max <= 0 && o->n_rank_ranges == 0 && o->flags == 0;
    if (n > 16) { plan->segs.reserve(n * 8); plan->acc.reserve(n * 2); plan->nominal_ops.reserve(n * 2); }
    for (size_t i = 0; i < n; ++i) {
        const xp_sketch* s = sk[i];
        if (!s) return fail(XP_ERR_INVALID_ARG, "null sketch in batch");
        if (!plain) { plan_sketch(s, i, o, plan); continue; }
        {
            std::lock_guard<std::mutex> lock(s->plan_mu);
            if (!s->plan_cached) {
                Plan own;
                plan_sketch(s, 0, o, &own);
                s->plan_segs = std::move(own.segs);
                s->plan_ops = std::move(own.nominal_ops);
                s->plan_tickets = own.n_tickets;
                s->plan_cached = true;
            }
        }
        const int acc_base = (int)plan->acc.size();
        AccDev a;
        memset(&a, 0, sizeof(a));
        for (int k = 0; k <= kMaxSize; ++k) a.min_rank[k] = ~0ull;
        for (int h = 0; h < s->n_holes; ++h) { plan->acc.push_back(a); plan->nominal_ops.push_back(s->plan_ops[h]); }
        const size_t at = plan->segs.size();
        plan->segs.insert(plan->segs.end(), s->plan_segs.begin(), s->plan_segs.end());
        for (size_t j = at; j < plan->segs.size(); ++j) {
            SegDev& c = plan->segs[j];
            c.first_ticket += plan->n_tickets;
            c.sketch = (i32)i;
            c.acc += acc_base;
        }
        plan->n_tickets += s->plan_tickets;
    }
    return XP_OK;
}

// One sketch's segments, accumulators and tickets, appended to the plan as sketch number i.
static void plan_sketch(const xp_sketch* s, size_t i, const xp_repair_opts* o, Plan* plan) {
    {
        for (int h = 0; h < s->n_holes; ++h) {
            const HoleHost& ho = s->holes[h];
            AccDev a;
            memset(&a, 0, sizeof(a));
            for (int k = 0; k <= kMaxSize; ++k) a.min_rank[k] = ~0ull;
            const int acc = (int)plan->acc.size();
            plan->acc.push_back(a);
            plan->nominal_ops.push_back(0);
            int kmin = 1, kmax = ho.max_size;
            if (o->size_min > 0) kmin = o->size_min;
            if (o->size_max > 0 && o->size_max < kmax) kmax = o->size_max;
            for (int k = kmin; k <= kmax && !ho.never; ++k) {
                u64 lo = 0, hi = s->g->cnt[ho.start_nt][k];
                for (int r = 0; r < o->n_rank_ranges; ++r) {
                    const xp_rank_range& rr = o->rank_ranges[r];
                    if ((rr.hole == -1 || rr.hole == h) && rr.size == k) {
                        if (rr.begin > lo) lo = rr.begin;
                        if (rr.end < hi) hi = rr.end;
                    }
                }
                if (lo >= hi) continue;
                const bool forced = (o->flags & XP_FLAG_ALWAYS_FILTER) != 0;
                const bool tiles = k >= 3 && ho.filter_ok && !(o->flags & XP_FLAG_NO_FILTER) &&
                                   (forced || hi - lo >= kTileMinRanks);
                if (tiles) add_tiles(plan, s->g, ho.start_nt, (int)i, h, acc, k, lo, hi, ho.compares ? kBcTileSlow : kBcTile);
                else add_linear(plan, (int)i, h, acc, k, lo, hi);
            }
        }
    }
}

constexpr u32 kSurvCap = 65536;              // survivor queue entries of a call with its own workspace (at least)

// Batches get 256 entries per sketch, up to 2^20.
static u32 surv_cap_for(size_t n_sketches) {
    const size_t want = n_sketches * 256;
    return (u32)(want < kSurvCap ? kSurvCap : (want > (1u << 20) ? (1u << 20) : want));
}
constexpr u32 kSurvCapStatic = 8192;         // ... of a call on the library's fixed scratch

static SearchLayout ws_layout(size_t n_segs, size_t n_sketches, size_t n_acc, u32 surv_cap) {
    SearchLayout w;
    w.segs = 256;
    w.sketches = w.segs + align256(sizeof(SegDev) * (n_segs + 1));
    w.acc = w.sketches + align256(sizeof(SketchDev*) * (n_sketches + 1));
    w.hist = w.acc + align256(sizeof(AccDev) * (n_acc + 1));
    w.head = w.hist + align256(sizeof(u32) * (n_acc + 1));
    w.surv = w.head;
    w.sort_off = w.surv + align256(sizeof(SurvDev) * (size_t)surv_cap);
    w.sorted = w.sort_off + align256(sizeof(u32) * (n_acc + 2));
    w.longs = w.sorted + align256(sizeof(u32) * (size_t)surv_cap);
    w.total = w.longs + align256(sizeof(u32) * (size_t)surv_cap);
    w.n_acc = (int)n_acc;
    w.dense = 0;
    w.surv_cap = surv_cap;
    return w;
}

// Does some hole among the sketches take the second look (frequent filter hits)?
static int any_dense(const xp_sketch* const* sk, size_t n) {
    for (size_t i = 0; i < n; ++i)
        for (const HoleHost& h : sk[i]->holes) if (h.second) return 1;
    return 0;
}

// Chunks of the whole-domain check that the largest domain among the sketches needs.
static u32 max_chunks_of(const xp_sketch* const* sk, size_t n) {
    i64 most = 0;
    for (size_t i = 0; i < n; ++i) most = sk[i]->n_points > most ? sk[i]->n_points : most;
    return (u32)((most + kVerifyChunk - 1) / kVerifyChunk);
}

extern "C" size_t xp_workspace_bytes(const xp_sketch* const* sketches, size_t n, const xp_repair_opts* opts) {
    if (!sketches || n == 0) return 0;
    Plan plan;
    if (build_plan(sketches, n, opts ? opts : &kDefaultOpts, &plan) != XP_OK) return 0;
    return ws_layout(plan.segs.size(), n, plan.acc.size(), surv_cap_for(n)).total;
}

extern "C" xp_status xp_repair_batch(const xp_sketch* const* sketches, size_t n, const xp_repair_opts* opts,
                                     xp_result** outs) {
    if (!sketches || !outs || n == 0) return fail(XP_ERR_INVALID_ARG, "xp_repair_batch: null argument");
    for (size_t i = 0; i < n; ++i) outs[i] = nullptr;
    const xp_repair_opts* o = opts ? opts : &kDefaultOpts;
    if (o->n_rank_ranges < 0 || (o->n_rank_ranges > 0 && !o->rank_ranges)) return fail(XP_ERR_INVALID_ARG, "bad rank_ranges");
    if (o->cancel && *o->cancel) return fail(XP_ERR_CANCELLED, "cancelled before launch");
    const auto t0 = std::chrono::steady_clock::now();
    Plan plan;
    xp_status st = build_plan(sketches, n, o, &plan);
    if (st == XP_OK) st = check_device(sketches, n);
    if (st != XP_OK) return st;
    cudaStream_t stream = (cudaStream_t)o->stream;

    SearchLayout w = ws_layout(plan.segs.size(), n, plan.acc.size(), surv_cap_for(n));
    w.dense = any_dense(sketches, n);
    char* ws = (char*)o->workspace;
    bool own_ws = false, cached_ws = false;
    if (ws) {
        if (o->workspace_bytes < w.total || ((uintptr_t)ws & 255)) return fail(XP_ERR_NOMEM, "workspace too small or misaligned");
    } else if (g_ws_mu.try_lock()) {
        // the library's own scratch, kept from call to call (grown when a call needs more)
        cached_ws = true;
        int dev = -1;
        cudaGetDevice(&dev);
        if (g_ws_bytes < w.total || g_ws_device != dev) {
            if (g_ws) cudaFree(g_ws);                // (a block of another device is freed from here as well)
            g_ws_device = dev;
            g_ws = nullptr; g_ws_bytes = 0;
            cudaError_t e = cudaMalloc((void**)&g_ws, w.total);
            if (e != cudaSuccess) { g_ws_mu.unlock(); return fail(XP_ERR_NOMEM, std::string("cudaMalloc: ") + cudaGetErrorString(e)); }
            g_ws_bytes = w.total;
        }
        ws = g_ws;
    } else {                                       // another call holds the kept scratch
        XP_CUDA(cudaMalloc((void**)&ws, w.total));
        own_ws = true;
    }
    std::vector<char> stage(w.head, 0);
    if (!plan.segs.empty()) memcpy(&stage[w.segs], plan.segs.data(), sizeof(SegDev) * plan.segs.size());
    for (size_t i = 0; i < n; ++i) ((const SketchDev**)&stage[w.sketches])[i] = sketches[i]->d_s;
    memcpy(&stage[w.acc], plan.acc.data(), sizeof(AccDev) * plan.acc.size());

    cudaEvent_t e0 = nullptr, e1 = nullptr;
    float ms = 0.f;
    int launches = 0;
    std::vector<AccDev> acc(plan.acc.size());
    u32 check_word = 0;
#define XP_CUDA_R(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { if (own_ws) cudaFree(ws); if (cached_ws) g_ws_mu.unlock(); \
        if (e0) cudaEventDestroy(e0); if (e1) cudaEventDestroy(e1); \
        return fail(e_ == cudaErrorMemoryAllocation ? XP_ERR_NOMEM : XP_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e_)); } } while (0)
    XP_CUDA_R(cudaEventCreate(&e0));
    XP_CUDA_R(cudaEventCreate(&e1));
    XP_CUDA_R(cudaMemcpyAsync(ws, stage.data(), w.head, cudaMemcpyHostToDevice, stream));
    XP_CUDA_R(cudaEventRecord(e0, stream));
    const int n_segs = (int)plan.segs.size(), n_acc = (int)plan.acc.size();
    const u32 max_chunks = max_chunks_of(sketches, n);
    xp_status stopped = XP_OK;
    if (!o->cancel && o->timeout_ms <= 0) {
        XP_CUDA_R(launch_search_part(ws, w, 0, plan.n_tickets, false, n_segs, (int)n, max_chunks, stream, &launches));
    } else {
        // Bounded launches: the host waits for each and then looks at the cancel word and the clock.
        // Nothing on the device waits for either, and when the call gives up no kernel is in flight.
        const u64 n_items = plan.n_tickets;
        for (u64 t = 0; t < n_items && stopped == XP_OK; t += (u64)XP_CANCEL_TICKETS) {
            const u64 t_end = t + (u64)XP_CANCEL_TICKETS < n_items ? t + (u64)XP_CANCEL_TICKETS : n_items;
            XP_CUDA_R(launch_search_part(ws, w, t, t_end, t > 0, n_segs, (int)n, max_chunks, stream, &launches));
            XP_CUDA_R(cudaStreamSynchronize(stream));
            if (o->cancel && *o->cancel) stopped = XP_ERR_CANCELLED;
            else if (o->timeout_ms > 0 && t_end < n_items &&
                     std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t0).count() >= (double)o->timeout_ms)
                stopped = XP_ERR_TIMEOUT;
        }
    }
    if (stopped == XP_OK) {
        XP_CUDA_R(launch_search_end(ws, w, plan.n_tickets > 0, n_segs, (int)n, n_acc, max_chunks, stream, &launches));
        XP_CUDA_R(cudaEventRecord(e1, stream));
        XP_CUDA_R(cudaMemcpyAsync(acc.data(), ws + w.acc, sizeof(AccDev) * acc.size(), cudaMemcpyDeviceToHost, stream));
        XP_CUDA_R(cudaMemcpyAsync(&check_word, ws + 20, sizeof(check_word), cudaMemcpyDeviceToHost, stream));
        XP_CUDA_R(cudaStreamSynchronize(stream));
        XP_CUDA_R(cudaEventElapsedTime(&ms, e0, e1));
    }
#undef XP_CUDA_R
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (own_ws) cudaFree(ws);
    if (cached_ws) g_ws_mu.unlock();
    if (stopped == XP_ERR_CANCELLED) return fail(stopped, "cancelled between launches (" + std::to_string(launches) + " done)");
    if (stopped == XP_ERR_TIMEOUT) return fail(stopped, "time limit of " + std::to_string((long long)o->timeout_ms) + " ms reached between launches (" + std::to_string(launches) + " done)");
    if (check_word != 0) return fail(XP_ERR_CUDA, "an index check of the checked build failed (code " + std::to_string(check_word) + ")");

    size_t ai = 0;
    for (size_t i = 0; i < n; ++i) {
        const xp_sketch* s = sketches[i];
        xp_result* r = new (std::nothrow) xp_result;
        if (!r) {
            for (size_t j = 0; j < i; ++j) { delete outs[j]; outs[j] = nullptr; }
            return fail(XP_ERR_NOMEM, "out of host memory");
        }
        r->holes.resize(s->n_holes);
        for (int h = 0; h < s->n_holes; ++h, ++ai) {
            HoleResult& hr = r->holes[h];
            const AccDev& a = acc[ai];
            hr.max_size = s->holes[h].max_size;
            for (int k = 1; k <= hr.max_size; ++k) {
                hr.cand_count[k] = s->g->cnt[s->holes[h].start_nt][k];
                hr.match_count[k] = a.match_count[k];
            }
            hr.evals = a.evals + a.filter_tests; hr.filter_survivors = a.filter_survivors; hr.probe_survivors = a.probe_survivors;
            hr.filter_tests = a.filter_tests;
            hr.skipped = a.tile_cands > a.filter_tests ? a.tile_cands - a.filter_tests : 0;
            hr.nominal_ops = plan.nominal_ops[ai] - (a.ops_skipped < plan.nominal_ops[ai] ? a.ops_skipped : plan.nominal_ops[ai]);
            const int ls = (int)a.pad;
            if (ls >= 1 && ls <= hr.max_size && a.match_count[ls] > 0) {
                hr.solved = 1; hr.least_size = ls; hr.least_rank = a.min_rank[ls];
                host_unrank(s->g, s->holes[h].start_nt, ls, hr.least_rank, &hr.code, &hr.text);
            }
        }
        r->kernel_ms = ms;
        r->n_launches = launches;
        r->h2d_bytes = w.head;
        r->d2h_bytes = sizeof(AccDev) * acc.size() + sizeof(check_word);
        outs[i] = r;
    }
    const double total = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t0).count();
    for (size_t i = 0; i < n; ++i) outs[i]->total_ms = total;
    return XP_OK;
}

extern "C" xp_status xp_repair(const xp_sketch* sketch, const xp_repair_opts* opts, xp_result** out) {
    if (!sketch || !out) return fail(XP_ERR_INVALID_ARG, "xp_repair: null argument");
    return xp_repair_batch(&sketch, 1, opts, out);
}

// The search of one sketch with every byte of device scratch taken from a fixed array inside
// the library: no device memory is allocated or freed, no event or stream is created.
extern "C" xp_status xp_repair_static(const xp_sketch* sketch, const xp_repair_opts* opts, xp_hole_summary* out,
                                      int32_t out_cap) {
    if (!sketch || !out) return fail(XP_ERR_INVALID_ARG, "xp_repair_static: null argument");
    if (out_cap < sketch->n_holes) return fail(XP_ERR_INVALID_ARG, "xp_repair_static: out has fewer entries than the sketch has holes");
    const xp_repair_opts* o = opts ? opts : &kDefaultOpts;
    if (o->n_rank_ranges < 0 || (o->n_rank_ranges > 0 && !o->rank_ranges)) return fail(XP_ERR_INVALID_ARG, "bad rank_ranges");
    if (o->cancel && *o->cancel) return fail(XP_ERR_CANCELLED, "cancelled before launch");
    Plan plan;
    xp_status st = build_plan(&sketch, 1, o, &plan);
    if (st == XP_OK) st = check_device(&sketch, 1);
    if (st != XP_OK) return st;
    SearchLayout w = ws_layout(plan.segs.size(), 1, plan.acc.size(), kSurvCapStatic);
    w.dense = any_dense(&sketch, 1);
    if (plan.acc.size() > 64)
        return fail(XP_ERR_TOO_LARGE, "xp_repair_static: the sketch has more than 64 holes; use xp_repair with a workspace");
    if (w.total > kStaticScratchBytes)
        return fail(XP_ERR_TOO_LARGE, "xp_repair_static: the call needs " + std::to_string(w.total) +
                    " bytes of scratch, the fixed array holds " + std::to_string(kStaticScratchBytes) +
                    "; use xp_repair with a workspace");
    static thread_local char stage[kStaticScratchBytes];          // no heap use that grows with the call
    memset(stage, 0, w.head);
    if (!plan.segs.empty()) memcpy(&stage[w.segs], plan.segs.data(), sizeof(SegDev) * plan.segs.size());
    ((const SketchDev**)&stage[w.sketches])[0] = sketch->d_s;
    memcpy(&stage[w.acc], plan.acc.data(), sizeof(AccDev) * plan.acc.size());
    AccDev acc[64];
    cudaStream_t stream = (cudaStream_t)o->stream;
    XP_CUDA(launch_search_static(stage, w, plan.n_tickets, (int)plan.segs.size(), (int)plan.acc.size(),
                                 max_chunks_of(&sketch, 1), acc, stream));
    XP_CUDA(cudaStreamSynchronize(stream));
    for (int h = 0; h < sketch->n_holes; ++h) {
        xp_hole_summary& r = out[h];
        memset(&r, 0, sizeof(r));
        const AccDev& a = acc[h];
        r.max_size = sketch->holes[h].max_size;
        for (int k = 1; k <= r.max_size; ++k) {
            r.cand_count[k] = sketch->g->cnt[sketch->holes[h].start_nt][k];
            r.match_count[k] = a.match_count[k];
        }
        r.evals_executed = a.evals + a.filter_tests;
        const int ls = (int)a.pad;
        if (ls >= 1 && ls <= r.max_size && a.match_count[ls] > 0) {
            r.solved = 1; r.least_size = ls; r.least_rank = a.min_rank[ls];
            std::vector<xp_instr> code;
            std::string text;
            host_unrank(sketch->g, sketch->holes[h].start_nt, ls, r.least_rank, &code, &text);
            snprintf(r.least_text, sizeof(r.least_text), "%s", text.c_str());
        }
    }
    return XP_OK;
}

extern "C" xp_status xp_result_get(const xp_result* r, int32_t hole, xp_result_view* v) {
    if (!r || !v || hole < 0 || hole >= (int)r->holes.size()) return fail(XP_ERR_INVALID_ARG, "xp_result_get: bad argument");
    const HoleResult& h = r->holes[hole];
    v->solved = h.solved;
    v->max_size = h.max_size;
    v->cand_count = (const uint64_t*)h.cand_count;
    v->match_count = (const uint64_t*)h.match_count;
    v->least_size = h.least_size;
    v->least_rank = h.least_rank;
    v->least_code = h.code.data();
    v->least_len = (int)h.code.size();
    v->least_text = h.text.c_str();
    v->evals_executed = h.evals;
    v->filter_survivors = h.filter_survivors;
    v->probe_survivors = h.probe_survivors;
    v->nominal_ops = h.nominal_ops;
    v->kernel_ms = r->kernel_ms;
    v->total_ms = r->total_ms;
    v->n_launches = r->n_launches;
    v->filter_tests = h.filter_tests;
    v->candidates_skipped = h.skipped;
    v->h2d_bytes = r->h2d_bytes;
    v->d2h_bytes = r->d2h_bytes;
    return XP_OK;
}

extern "C" xp_status xp_result_pack(const xp_result* const* results, size_t n, xp_hole_summary* out, size_t out_cap, size_t* n_out) {
    if (n_out) *n_out = 0;
    if (!results || !out) return fail(XP_ERR_INVALID_ARG, "xp_result_pack: null argument");
    size_t at = 0;
    for (size_t i = 0; i < n; ++i) {
        if (!results[i]) return fail(XP_ERR_INVALID_ARG, "xp_result_pack: result " + std::to_string(i) + " is null");
        for (const HoleResult& h : results[i]->holes) {
            if (at >= out_cap) return fail(XP_ERR_INVALID_ARG, "xp_result_pack: out holds fewer entries than the results have holes");
            xp_hole_summary& r = out[at++];
            memset(&r, 0, sizeof(r));
            r.solved = h.solved; r.max_size = h.max_size; r.least_size = h.least_size; r.least_rank = h.least_rank;
            memcpy(r.cand_count, h.cand_count, sizeof(r.cand_count));
            memcpy(r.match_count, h.match_count, sizeof(r.match_count));
            r.evals_executed = h.evals;
            snprintf(r.least_text, sizeof(r.least_text), "%s", h.text.c_str());
        }
    }
    if (n_out) *n_out = at;
    return XP_OK;
}

extern "C" void xp_result_free(xp_result* r) { delete r; }

extern "C" const char* xp_last_error(void) { return g_last_error.c_str(); }

// ------------------------------------------------------------------------------------------
// integer peak
// ------------------------------------------------------------------------------------------

// Divisions per second of the two division forms (see the kernels): 64 per chain, 4 chains per thread.
extern "C" xp_status xp_int_div_rate(double* out_divs) {
    if (!out_divs) return fail(XP_ERR_INVALID_ARG, "xp_int_div_rate: null argument");
    int dev = 0, sms = 1;
    XP_CUDA(cudaGetDevice(&dev));
    XP_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    u32* d = nullptr;
    XP_CUDA(cudaMalloc(&d, 256));
    cudaEvent_t e0, e1;
    XP_CUDA(cudaEventCreate(&e0));
    XP_CUDA(cudaEventCreate(&e1));
    const int blocks = sms * 8;
    for (int which = 2; which < 4; ++which) {
        const int iters = which == 2 ? 64 : 2048;
        float best = 1e30f;
        for (int rep = 0; rep < 4; ++rep) {
            XP_CUDA(cudaEventRecord(e0, nullptr));
            XP_CUDA(launch_int32_peak(which, d, blocks, iters, nullptr));
            XP_CUDA(cudaEventRecord(e1, nullptr));
            XP_CUDA(cudaEventSynchronize(e1));
            float ms = 0.f;
            XP_CUDA(cudaEventElapsedTime(&ms, e0, e1));
            if (rep > 0 && ms < best) best = ms;
        }
        out_divs[which - 2] = (double)blocks * 256.0 * (double)iters * 64.0 / (best * 1e-3);
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(d);
    return XP_OK;
}

extern "C" xp_status xp_int32_peak(double* out_ops, double* out_ms) {
    if (!out_ops) return fail(XP_ERR_INVALID_ARG, "xp_int32_peak: null argument");
    int dev = 0, sms = 1;
    XP_CUDA(cudaGetDevice(&dev));
    XP_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    u32* d = nullptr;
    XP_CUDA(cudaMalloc(&d, 256));
    cudaEvent_t e0, e1;
    XP_CUDA(cudaEventCreate(&e0));
    XP_CUDA(cudaEventCreate(&e1));
    const int blocks = sms * 8, iters = 4096;
    for (int which = 0; which < 2; ++which) {
        float best = 1e30f;
        for (int rep = 0; rep < 4; ++rep) {
            XP_CUDA(cudaEventRecord(e0, nullptr));
            XP_CUDA(launch_int32_peak(which, d, blocks, iters, nullptr));
            XP_CUDA(cudaEventRecord(e1, nullptr));
            XP_CUDA(cudaEventSynchronize(e1));
            float ms = 0.f;
            XP_CUDA(cudaEventElapsedTime(&ms, e0, e1));
            if (rep > 0 && ms < best) best = ms;
        }
        const double ops = (double)blocks * 256.0 * (double)iters * 128.0;
        out_ops[which] = ops / (best * 1e-3);
        if (out_ms) out_ms[which] = best;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(d);
    return XP_OK;
}
