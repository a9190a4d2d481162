// The behaviour mode of include/xp.h (xp_behaviours): bottom-up enumeration with
// observational-equivalence pruning on signature points.
//
// Representatives of every (nonterminal, size) live side by side in device memory: their
// signatures (n_sig int64 values each) and a 16-byte record (operator or leaf, the two operand
// representatives).  One pass per (size, nonterminal), in chunks of kChunk candidates:
//   beh_sig_kernel     -- thread = candidate of the pruned space: finds its (production, left size)
//                         block, reads the operands' signatures, writes its own to the chunk buffer;
//   beh_insert_kernel  -- puts the candidate into the nonterminal's hash table (open addressing, one
//                         64-bit word per class: 24 bits of the signature's hash, a kind bit, an id).
//                         A word with the same 24 bits is confirmed by comparing the signatures
//                         themselves.  A class that a representative already owns drops the candidate;
//                         among the chunk's candidates the smallest index takes the word (compare-and-
//                         swap that only ever lowers it: no thread waits for another);
//   beh_flag_kernel    -- a candidate is new iff its class's word carries its own index; counts per block;
//   beh_scan_kernel    -- exclusive scan of the block counts (one CTA);
//   beh_append_kernel  -- the new ones, in candidate order, become representatives: signature and
//                         record are appended, and the class's word now names the representative.
// Then the representatives of the hole's nonterminal are held against the constraint at the
// signature points (beh_match_kernel) and the few that satisfy it are checked on the whole domain,
// in order (beh_verify_kernel: thread = point, the representative's tree walked with a small stack).
// The passes are bound by memory traffic: a candidate moves about 2 * 8 * n_sig + 16 bytes.
#include <cuda_runtime.h>

#include <algorithm>
#include <chrono>
#include <cstddef>
#include <cstring>
#include <functional>
#include <string>
#include <vector>

#include "xp_device.cuh"
#include "xp_launch.h"

namespace xp {

constexpr int kBehBlocks = 64;                            // (production, left size) blocks of one pass
constexpr u64 kBehChunk = 1ull << 22;                     // candidates per chunk
constexpr int kBehThreads = 256;
constexpr u64 kEmpty = ~0ull;
constexpr u64 kKindCand = 1ull << 39;
constexpr u64 kIdMask = (1ull << 39) - 1;
constexpr int kMatchCap = 256;                            // representatives that satisfy the signature, kept for the whole-domain check
constexpr u32 kLeafBit = 0x80000000u;

struct RepDesc { u32 op_or_leaf, left, right, size; };    // leaf: kLeafBit | index into the grammar's leaves; else operator and operand ids

struct BehDev {
    const SketchDev* sk;
    const HoleDev* hole;
    i32 n_sig, n_nt;
    u32 spec_ok, err;                                     // err: a probe sequence ran its limit (table too full)
    i64 sig_id[XP_MAX_SIG];
    i64 sig_pt[XP_MAX_SIG][kMaxVars];
    i64 sig_spec[XP_MAX_SIG];
    i64* rep_sig;                                         // [max_reps][n_sig]
    RepDesc* rep_desc;
    u64* table;                                           // [n_nt][table_size]
    u64 table_size;                                       // a power of two
    i64* buf_sig;                                         // chunk buffers: [kBehChunk][n_sig]
    unsigned char* buf_def;
    u32* buf_flag;
    u64* buf_slot;
    u32* block_count;                                     // per block of the chunk: new candidates, then their exclusive scan
    u64 chunk_new;                                        // new representatives of the chunk at hand
    u64 match_count;
    u32 match_n, verify_fail;
    u32 match_id[kMatchCap];
};

struct BehBlock { u64 first, cr, lbase, rbase; i32 op, pad; };
struct BehPass {
    i32 nt, size, n_blocks, leaf_first;                   // size 1: candidates are the leaves leaf_first ...
    u64 n_cand;
    BehBlock blocks[kBehBlocks];
};

__device__ __forceinline__ u64 sig_hash(const i64* s, int n) {
    u64 h = 0x243F6A8885A308D3ull;
    for (int j = 0; j < n; ++j) { h = (h ^ (u64)s[j]) * 0x9E3779B97F4A7C15ull; h ^= h >> 29; }
    return h;
}

__device__ __forceinline__ bool sig_equal(const i64* a, const i64* b, int n) {
    bool eq = true;
    for (int j = 0; j < n; ++j) eq = eq && a[j] == b[j];
    return eq;
}

__global__ void beh_points_kernel(BehDev* B) {
    const int t = threadIdx.x;
    const SketchDev* sk = B->sk;
    bool ok = false;
    if (t < B->n_sig) {
        i64 pt[kMaxVars];
        point_coords(sk, B->sig_id[t], pt);
        for (int d = 0; d < sk->n_vars; ++d) B->sig_pt[t][d] = pt[d];
        i64 v = 0;
        ok = true;
        // (a spec expression is evaluated here even when the load staged its values: the staged table does
        // not say where the expression is undefined)
        if (B->hole->spec_len > 0) ok = eval_code(B->hole->spec, B->hole->spec_len, pt, 0, v);
        else v = B->hole->spec_table[B->sig_id[t]];
        B->sig_spec[t] = v;
    }
    const u32 m = __ballot_sync(0xffffffffu, ok);
    if (t == 0) B->spec_ok = m;
}

__global__ void __launch_bounds__(kBehThreads) beh_sig_kernel(BehDev* B, const BehPass P, u64 chunk_first, u32 chunk_n) {
    const u32 c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= chunk_n) return;
    const u64 idx = chunk_first + c;
    const int ns = B->n_sig;
    i64* out = B->buf_sig + (u64)c * ns;
    bool defined = true;
    if (P.size == 1) {
        const LeafDev lf = B->sk->g->leaves[P.leaf_first + (i32)idx];
        for (int j = 0; j < ns; ++j) out[j] = lf.var >= 0 ? B->sig_pt[j][lf.var] : lf.value;
    } else {
        int b = 0;
        while (b + 1 < P.n_blocks && P.blocks[b + 1].first <= idx) ++b;
        const BehBlock& k = P.blocks[b];
        const u64 rem = idx - k.first, l = rem / k.cr, r = rem - l * k.cr;
        const i64* ls = B->rep_sig + (k.lbase + l) * ns;
        const i64* rs = B->rep_sig + (k.rbase + r) * ns;
        for (int j = 0; j < ns; ++j) {
            i64 v = 0;
            defined = apply_op(k.op, ls[j], rs[j], v) && defined;
            out[j] = v;
        }
    }
    B->buf_def[c] = defined ? 1 : 0;
}

// Signature behind a table word: a representative's, or a candidate's of the chunk at hand.
__device__ __forceinline__ const i64* sig_of(const BehDev* B, u64 word, u64 chunk_first) {
    const u64 id = word & kIdMask;
    return (word & kKindCand) ? B->buf_sig + (id - chunk_first) * B->n_sig : B->rep_sig + id * B->n_sig;
}

__global__ void __launch_bounds__(kBehThreads) beh_insert_kernel(BehDev* B, int nt, u64 chunk_first, u32 chunk_n) {
    const u32 c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= chunk_n || !B->buf_def[c]) return;
    const int ns = B->n_sig;
    const i64* mine = B->buf_sig + (u64)c * ns;
    const u64 h = sig_hash(mine, ns), mask = B->table_size - 1;
    const u64 me = ((h & 0xffffffull) << 40) | kKindCand | (chunk_first + c);
    u64* tab = B->table + (u64)nt * B->table_size;
    u64 slot = (h >> 24) & mask;
    for (u64 step = 0; step <= mask; ++step, slot = (slot + 1) & mask) {
        u64 w = tab[slot];
        bool other_class = false;
        // A failed compare-and-swap means that another thread has just changed the word (claimed it,
        // or lowered it within this class), never that one must be waited for; the limit only guards
        // against a mistake in this routine.
        for (int tries = 0; tries < (1 << 20) && !other_class; ++tries) {
            if (w == kEmpty) {
                const u64 old = atomicCAS((unsigned long long*)&tab[slot], kEmpty, me);
                if (old == kEmpty) return;
                w = old;
                continue;
            }
            if ((w >> 40) != (me >> 40) || !sig_equal(mine, sig_of(B, w, chunk_first), ns)) { other_class = true; break; }
            if (!(w & kKindCand) || w <= me) return;      // a representative, or an earlier candidate, owns the class
            const u64 old = atomicCAS((unsigned long long*)&tab[slot], w, me);
            if (old == w) return;
            w = old;
        }
        if (!other_class) break;                          // (the limit ran out)
    }
    atomicOr(&B->err, 1u);
}

__global__ void __launch_bounds__(kBehThreads) beh_flag_kernel(BehDev* B, int nt, u64 chunk_first, u32 chunk_n) {
    const u32 c = blockIdx.x * blockDim.x + threadIdx.x;
    bool is_new = false;
    if (c < chunk_n && B->buf_def[c]) {
        const int ns = B->n_sig;
        const i64* mine = B->buf_sig + (u64)c * ns;
        const u64 h = sig_hash(mine, ns), mask = B->table_size - 1;
        const u64 me = ((h & 0xffffffull) << 40) | kKindCand | (chunk_first + c);
        const u64* tab = B->table + (u64)nt * B->table_size;
        u64 slot = (h >> 24) & mask;
        for (u64 step = 0; step <= mask; ++step, slot = (slot + 1) & mask) {
            const u64 w = tab[slot];
            if (w == kEmpty) { atomicOr(&B->err, 2u); break; }          // (cannot happen: the class was inserted)
            if ((w >> 40) == (me >> 40) && sig_equal(mine, sig_of(B, w, chunk_first), ns)) {
                is_new = w == me;
                B->buf_slot[c] = slot;
                break;
            }
        }
    }
    if (c < chunk_n) B->buf_flag[c] = is_new ? 1u : 0u;
    const int n = __syncthreads_count(is_new);
    if (threadIdx.x == 0) B->block_count[blockIdx.x] = (u32)n;
}

__global__ void __launch_bounds__(1024) beh_scan_kernel(BehDev* B, int n_blocks) {
    __shared__ u32 part[1024];
    const int t = threadIdx.x;
    const int per = (n_blocks + 1023) / 1024;
    const int lo = t * per < n_blocks ? t * per : n_blocks, hi = lo + per < n_blocks ? lo + per : n_blocks;
    u32 sum = 0;
    for (int i = lo; i < hi; ++i) sum += B->block_count[i];
    part[t] = sum;
    __syncthreads();
    for (int d = 1; d < 1024; d <<= 1) {
        const u32 v = t >= d ? part[t - d] : 0u;
        __syncthreads();
        part[t] += v;
        __syncthreads();
    }
    u32 run = part[t] - sum;
    for (int i = lo; i < hi; ++i) { const u32 h = B->block_count[i]; B->block_count[i] = run; run += h; }
    if (t == 1023) B->chunk_new = part[1023];
}

__global__ void __launch_bounds__(kBehThreads) beh_append_kernel(BehDev* B, const BehPass P, u64 chunk_first, u32 chunk_n, u64 rep_base) {
    __shared__ u32 warp_sum[kBehThreads / 32];
    const u32 c = blockIdx.x * blockDim.x + threadIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool is_new = c < chunk_n && B->buf_flag[c] != 0;
    const u32 bal = __ballot_sync(0xffffffffu, is_new);
    if (lane == 0) warp_sum[warp] = (u32)__popc(bal);
    __syncthreads();
    if (!is_new) return;
    u32 pos = B->block_count[blockIdx.x] + (u32)__popc(bal & ((1u << lane) - 1u));
    for (int w = 0; w < warp; ++w) pos += warp_sum[w];
    const u64 gid = rep_base + pos;
    const int ns = B->n_sig;
    const i64* mine = B->buf_sig + (u64)c * ns;
    i64* dst = B->rep_sig + gid * ns;
    for (int j = 0; j < ns; ++j) dst[j] = mine[j];
    const u64 idx = chunk_first + c;
    RepDesc d;
    d.size = (u32)P.size;
    if (P.size == 1) { d.op_or_leaf = kLeafBit | (u32)(P.leaf_first + (i32)idx); d.left = d.right = 0; }
    else {
        int b = 0;
        while (b + 1 < P.n_blocks && P.blocks[b + 1].first <= idx) ++b;
        const BehBlock& k = P.blocks[b];
        const u64 rem = idx - k.first, l = rem / k.cr, r = rem - l * k.cr;
        d.op_or_leaf = (u32)k.op; d.left = (u32)(k.lbase + l); d.right = (u32)(k.rbase + r);
    }
    B->rep_desc[gid] = d;
    u64* tab = B->table + (u64)P.nt * B->table_size;
    const u64 slot = B->buf_slot[c];
    tab[slot] = (tab[slot] & ~((1ull << 40) - 1)) | gid;  // the class's word now names the representative
}

// Representatives [first, first + n) of the hole's nonterminal against the constraint at the signature points.
__global__ void __launch_bounds__(kBehThreads) beh_match_kernel(BehDev* B, u64 first, u64 n) {
    const u64 i = (u64)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int ns = B->n_sig;
    const u32 all = ns >= 32 ? 0xffffffffu : (1u << ns) - 1u;
    if ((B->spec_ok & all) != all) return;                // the spec is undefined at a signature point: nothing satisfies it
    const i64* s = B->rep_sig + (first + i) * ns;
    bool ok = true;
    for (int j = 0; j < ns && ok; ++j) ok = ctx_matches(B->hole, B->sig_pt[j], s[j], B->sig_spec[j]);
    if (!ok) return;
    atomicAdd((unsigned long long*)&B->match_count, 1ull);
    const u32 at = atomicAdd(&B->match_n, 1u);
    if (at < (u32)kMatchCap) B->match_id[at] = (u32)(first + i);
}

// Value of representative `gid` at one point: its tree is walked with an explicit stack.
__device__ bool rep_value(const BehDev* B, u32 gid, const i64* pt, i64& out) {
    u32 todo[2 * kMaxSize + 2];                           // node ids; kLeafBit set: "apply this node's operator now"
    i64 val[kCandStack + 1];
    int nt = 0, nv = 0;
    todo[nt++] = gid;
    const LeafDev* leaves = B->sk->g->leaves;
    while (nt > 0) {
        const u32 x = todo[--nt];
        if (x & kLeafBit) {                               // operator of node x & ~kLeafBit: operands are on the value stack
            const RepDesc d = B->rep_desc[x & ~kLeafBit];
            const i64 b = val[--nv], a = val[nv - 1];
            i64 r;
            if (!apply_op((int)d.op_or_leaf, a, b, r)) return false;
            val[nv - 1] = r;
            continue;
        }
        const RepDesc d = B->rep_desc[x];
        if (d.op_or_leaf & kLeafBit) {
            const LeafDev lf = leaves[d.op_or_leaf & ~kLeafBit];
            if (!XP_CHECKED(nv <= kCandStack, kChkStack)) return false;
            val[nv++] = lf.var >= 0 ? pt[lf.var] : lf.value;
        } else {
            if (!XP_CHECKED(nt + 3 <= 2 * kMaxSize + 2, kChkStack)) return false;
            todo[nt++] = x | kLeafBit;
            todo[nt++] = d.right;
            todo[nt++] = d.left;
        }
    }
    out = val[0];
    return true;
}

__global__ void __launch_bounds__(kBehThreads) beh_verify_kernel(BehDev* B, u32 gid) {
    const SketchDev* sk = B->sk;
    const HoleDev* hole = B->hole;
    for (i64 pid = (i64)blockIdx.x * blockDim.x + threadIdx.x; pid < sk->n_points; pid += (i64)gridDim.x * blockDim.x) {
        if (*(volatile u32*)&B->verify_fail) return;
        i64 pt[kMaxVars];
        point_coords(sk, pid, pt);
        i64 want = 0, h;
        bool ok = true;
        if (hole->spec_len > 0) ok = eval_code(hole->spec, hole->spec_len, pt, 0, want);
        else want = hole->spec_table[pid];
        ok = ok && rep_value(B, gid, pt, h) && ctx_matches(hole, pt, h, want);
        if (!ok) { atomicOr(&B->verify_fail, 1u); return; }
    }
}

}  // namespace xp

using namespace xp;

namespace {
struct Cuda { cudaError_t e = cudaSuccess; void operator()(cudaError_t x) { if (e == cudaSuccess) e = x; } bool ok() const { return e == cudaSuccess; } };
}

extern "C" xp_status xp_behaviours(const xp_sketch* sketch, const xp_behaviour_desc* d, const xp_repair_opts* opts,
                                   xp_behaviour_summary* out) {
    if (!sketch || !d || !out) return set_error(XP_ERR_INVALID_ARG, "xp_behaviours: null argument");
    memset(out, 0, sizeof(*out));
    const auto t0 = std::chrono::steady_clock::now();
    const SketchInternals si = sketch_internals(sketch);
    const HoleSpec hs = sketch_hole(sketch, d->hole);
    if (hs.start_nt < 0) return set_error(XP_ERR_INVALID_ARG, "xp_behaviours: hole out of range");
    if (d->n_sig < 1 || d->n_sig > XP_MAX_SIG || !d->sig_points) return set_error(XP_ERR_INVALID_ARG, "xp_behaviours: n_sig must be 1..16");
    for (int j = 0; j < d->n_sig; ++j)
        if (d->sig_points[j] < 0 || d->sig_points[j] >= si.n_points) return set_error(XP_ERR_INVALID_ARG, "xp_behaviours: a signature point lies outside the domain");
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return set_error(XP_ERR_CUDA, "no CUDA device is usable");
    if (dev != si.device) return set_error(XP_ERR_INVALID_ARG, "xp_behaviours: the sketch was loaded on another device than the current one");
    const GrammarHost gh = grammar_host(si.g);
    const int ns = d->n_sig, K = hs.max_size, n_nt = gh.n_nt;
    const u64 max_reps = d->max_representatives ? d->max_representatives : (1ull << 22);
    if (max_reps >= (1ull << 31)) return set_error(XP_ERR_TOO_LARGE, "xp_behaviours: max_representatives must stay below 2^31");
    u64 tsize = 1024;
    while (tsize < 2 * max_reps + 2 * kBehChunk) tsize <<= 1;
    // one device block
    auto al = [](size_t b) { return (b + 255) & ~(size_t)255; };
    size_t off = al(sizeof(BehDev));
    const size_t o_sig = off;   off += al(sizeof(i64) * max_reps * ns);
    const size_t o_desc = off;  off += al(sizeof(RepDesc) * max_reps);
    const size_t o_tab = off;   off += al(sizeof(u64) * tsize * n_nt);
    const size_t o_bsig = off;  off += al(sizeof(i64) * kBehChunk * ns);
    const size_t o_bdef = off;  off += al(kBehChunk);
    const size_t o_bflag = off; off += al(sizeof(u32) * kBehChunk);
    const size_t o_bslot = off; off += al(sizeof(u64) * kBehChunk);
    const size_t o_bcnt = off;  off += al(sizeof(u32) * (kBehChunk / kBehThreads + 1));
    char* block = nullptr;
    size_t granted = 0;
    int bdev = 0;
    if (device_alloc((void**)&block, off, &bdev, &granted) != cudaSuccess) {
        (void)cudaGetLastError();
        return set_error(XP_ERR_NOMEM, ("xp_behaviours: device memory (" + std::to_string(off) + " bytes)").c_str());
    }
    BehDev h;
    memset(&h, 0, sizeof(h));
    h.sk = si.d_s; h.hole = sketch_hole_dev(sketch, d->hole); h.n_sig = ns; h.n_nt = n_nt;
    for (int j = 0; j < ns; ++j) h.sig_id[j] = d->sig_points[j];
    h.rep_sig = (i64*)(block + o_sig); h.rep_desc = (RepDesc*)(block + o_desc);
    h.table = (u64*)(block + o_tab); h.table_size = tsize;
    h.buf_sig = (i64*)(block + o_bsig); h.buf_def = (unsigned char*)(block + o_bdef);
    h.buf_flag = (u32*)(block + o_bflag); h.buf_slot = (u64*)(block + o_bslot); h.block_count = (u32*)(block + o_bcnt);
    BehDev* dB = (BehDev*)block;
    cudaStream_t stream = opts ? (cudaStream_t)opts->stream : nullptr;
    Cuda cu;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cu(cudaEventCreate(&e0));
    cu(cudaEventCreate(&e1));
    cu(cudaMemcpyAsync(dB, &h, sizeof(h), cudaMemcpyHostToDevice, stream));
    cu(cudaMemsetAsync(block + o_tab, 0xff, sizeof(u64) * tsize * n_nt, stream));
    cu(cudaEventRecord(e0, stream));
    int launches = 0;
    if (cu.ok()) { beh_points_kernel<<<1, 32, 0, stream>>>(dB); ++launches; cu(cudaGetLastError()); }
    std::vector<std::vector<u64>> count(n_nt, std::vector<u64>(K + 1, 0)), base(n_nt, std::vector<u64>(K + 1, 0));
    u64 n_reps = 0, bytes = 0;
    xp_status st = XP_OK;
    std::string why;
    for (int s = 1; s <= K && cu.ok() && st == XP_OK; ++s)
        for (int nt = 0; nt < n_nt && cu.ok() && st == XP_OK; ++nt) {
            BehPass P;
            memset(&P, 0, sizeof(P));
            P.nt = nt; P.size = s;
            if (s == 1) { P.leaf_first = gh.leaf_begin[nt]; P.n_cand = (u64)(gh.leaf_begin[nt + 1] - gh.leaf_begin[nt]); }
            else
                for (int b = gh.bin_begin[nt]; b < gh.bin_begin[nt + 1] && st == XP_OK; ++b)
                    for (int a = 1; a <= s - 2; ++a) {
                        const u64 cl = count[gh.bins[b].lnt][a], cr = count[gh.bins[b].rnt][s - 1 - a];
                        if (cl == 0 || cr == 0) continue;
                        if (P.n_blocks == kBehBlocks) { st = XP_ERR_TOO_LARGE; why = "xp_behaviours: more than 64 (production, left size) blocks in one pass"; break; }
                        BehBlock& k = P.blocks[P.n_blocks++];
                        k.first = P.n_cand; k.cr = cr; k.lbase = base[gh.bins[b].lnt][a]; k.rbase = base[gh.bins[b].rnt][s - 1 - a]; k.op = gh.bins[b].op;
                        P.n_cand += cl * cr;
                        if (P.n_cand >= kKindCand) { st = XP_ERR_TOO_LARGE; why = "xp_behaviours: 2^39 candidates or more in one pass"; break; }
                    }
            base[nt][s] = n_reps;
            if (st != XP_OK) break;
            if (nt == hs.start_nt) out->enumerated[s] = P.n_cand;
            bytes += P.n_cand * (u64)(2 * 8 * ns + 16);
            for (u64 first = 0; first < P.n_cand && cu.ok() && st == XP_OK; first += kBehChunk) {
                const u32 n = (u32)(P.n_cand - first < kBehChunk ? P.n_cand - first : kBehChunk);
                const int nb = (int)((n + kBehThreads - 1) / kBehThreads);
                beh_sig_kernel<<<nb, kBehThreads, 0, stream>>>(dB, P, first, n);
                beh_insert_kernel<<<nb, kBehThreads, 0, stream>>>(dB, nt, first, n);
                beh_flag_kernel<<<nb, kBehThreads, 0, stream>>>(dB, nt, first, n);
                beh_scan_kernel<<<1, 1024, 0, stream>>>(dB, nb);
                launches += 4;
                cu(cudaGetLastError());
                BehDev back;
                cu(cudaMemcpyAsync(&back, dB, offsetof(BehDev, match_count), cudaMemcpyDeviceToHost, stream));
                cu(cudaStreamSynchronize(stream));
                if (!cu.ok()) break;
                if (back.err) { st = XP_ERR_TOO_LARGE; why = "xp_behaviours: the hash table is too full (raise max_representatives)"; break; }
                if (n_reps + back.chunk_new > max_reps) {
                    st = XP_ERR_TOO_LARGE;
                    why = "xp_behaviours: more than " + std::to_string(max_reps) + " representatives (size " + std::to_string(s) + ")";
                    break;
                }
                beh_append_kernel<<<nb, kBehThreads, 0, stream>>>(dB, P, first, n, n_reps);
                ++launches;
                cu(cudaGetLastError());
                n_reps += back.chunk_new;
                count[nt][s] += back.chunk_new;
                bytes += back.chunk_new * (u64)(2 * 8 * ns + 24);
            }
            if (nt == hs.start_nt) out->distinct[s] = count[nt][s];
        }
    // the hole's representatives against the constraint, then the whole-domain checks in order
    std::vector<u32> ids;
    if (cu.ok() && st == XP_OK) {
        for (int s = 1; s <= K; ++s)
            if (count[hs.start_nt][s] > 0) {
                const u64 n = count[hs.start_nt][s];
                beh_match_kernel<<<(unsigned)((n + kBehThreads - 1) / kBehThreads), kBehThreads, 0, stream>>>(dB, base[hs.start_nt][s], n);
                ++launches;
            }
        cu(cudaGetLastError());
        BehDev back;
        cu(cudaMemcpyAsync(&back, dB, sizeof(back), cudaMemcpyDeviceToHost, stream));
        cu(cudaStreamSynchronize(stream));
        if (cu.ok()) {
            out->sig_matches = back.match_count;
            const u32 n = back.match_n < (u32)kMatchCap ? back.match_n : (u32)kMatchCap;
            ids.assign(back.match_id, back.match_id + n);
            std::sort(ids.begin(), ids.end());            // ids grow with (size, order found) within a nonterminal
            if (back.match_n > (u32)kMatchCap) { st = XP_ERR_TOO_LARGE; why = "xp_behaviours: more than 256 representatives satisfy the signature points"; }
        }
    }
    auto locate = [&](u32 gid, int* size, u64* index) {
        for (int s = 1; s <= K; ++s)
            if (gid >= base[hs.start_nt][s] && gid < base[hs.start_nt][s] + count[hs.start_nt][s]) { *size = s; *index = gid - base[hs.start_nt][s]; }
    };
    std::function<bool(u32, std::string&)> text_of = [&](u32 gid, std::string& t) -> bool {
        RepDesc r;
        if (cudaMemcpy(&r, (char*)block + o_desc + sizeof(RepDesc) * gid, sizeof(r), cudaMemcpyDeviceToHost) != cudaSuccess) return false;
        if (r.op_or_leaf & kLeafBit) {
            const LeafDev& lf = gh.leaves[r.op_or_leaf & ~kLeafBit];
            t += lf.var >= 0 ? std::string(gh.var_names[lf.var]) : std::to_string((long long)lf.value);
            return true;
        }
        static const char* const kText[] = {"+", "-", "*", "/", "%", "<", "<=", "==", "!=", "min", "max", "&&", "||", "<<", ">>"};
        const bool call = r.op_or_leaf == XP_OP_MIN || r.op_or_leaf == XP_OP_MAX;
        t += call ? std::string(kText[r.op_or_leaf]) + "(" : std::string("(");
        if (!text_of(r.left, t)) return false;
        t += call ? "," : kText[r.op_or_leaf];
        if (!text_of(r.right, t)) return false;
        t += ")";
        return true;
    };
    for (size_t k = 0; k < ids.size() && cu.ok() && st == XP_OK && !out->solved; ++k) {
        cu(cudaMemsetAsync((char*)dB + offsetof(BehDev, verify_fail), 0, sizeof(u32), stream));
        int sms = 148;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const i64 want = (si.n_points + kBehThreads - 1) / kBehThreads;
        if (want > 0) { beh_verify_kernel<<<(unsigned)(want < sms * 8 ? want : sms * 8), kBehThreads, 0, stream>>>(dB, ids[k]); ++launches; }
        cu(cudaGetLastError());
        u32 fail = 0;
        cu(cudaMemcpyAsync(&fail, (char*)dB + offsetof(BehDev, verify_fail), sizeof(fail), cudaMemcpyDeviceToHost, stream));
        cu(cudaStreamSynchronize(stream));
        if (!cu.ok()) break;
        std::string t;
        int size = 0;
        u64 index = 0;
        locate(ids[k], &size, &index);
        if (k == 0 || !fail) text_of(ids[k], t);
        if (k == 0) {
            out->hit = 1; out->hit_size = size; out->hit_index = index; out->hit_verified = fail ? 0 : 1;
            snprintf(out->hit_text, sizeof(out->hit_text), "%s", t.c_str());
        }
        if (!fail) {
            out->solved = 1; out->solution_size = size; out->solution_index = index;
            snprintf(out->solution_text, sizeof(out->solution_text), "%s", t.c_str());
        }
    }
    float ms = 0.f;
    if (cu.ok()) { cu(cudaEventRecord(e1, stream)); cu(cudaEventSynchronize(e1)); cu(cudaEventElapsedTime(&ms, e0, e1)); }
    else cudaStreamSynchronize(stream);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    device_release(block, granted, bdev);
    if (!cu.ok()) return set_error(XP_ERR_CUDA, (std::string("xp_behaviours: ") + cudaGetErrorString(cu.e)).c_str());
    if (st != XP_OK) return set_error(st, why.c_str());
    out->max_size = K;
    out->representatives = n_reps;
    out->bytes_moved = bytes;
    out->kernel_ms = ms;
    out->n_launches = launches;
    out->total_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t0).count();
    return XP_OK;
}
