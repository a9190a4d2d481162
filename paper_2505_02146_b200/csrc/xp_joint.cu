// Two holes inside one constraint: the product search of xp_repair_joint (include/xp.h).
//
//   joint_probe_kernel   -- coordinates and spec values of the probe points (the first sample points
//                           of the sketch: box corners first, then ids spread by a fixed hash).
//   joint_values_kernel  -- value at every probe of every candidate of either part (every size up
//                           to its bound): thread = (table entry, probe).
//   joint_pairs_kernel   -- one (size of part 0, size of part 1) block of the pair space: thread =
//                           pair, rank of part 1 fastest; the constraint is evaluated at the probes
//                           from the tables, first failure ends the pair; the pairs of a warp that
//                           pass every probe are checked on the whole domain by the warp together
//                           (lane = point, vote exit).  Matches go into per-total-size counts (sum)
//                           and least keys (min) by atomics.
// No CTA or warp waits for another.
#include <cuda_runtime.h>

#include <chrono>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "xp_device.cuh"
#include "xp_launch.h"

namespace xp {

constexpr int kJointProbes = 16;
constexpr int kJointTotal = 2 * kMaxSize;                 // largest total size of a pair
constexpr u64 kJointMaxEntries = 1ull << 22;              // candidates of one part and size
constexpr u64 kJointMaxPairs = 1ull << 40;

struct JointDev {
    const SketchDev* sk;
    i32 n_probe, ctx_len, spec_len, pad;
    u32 spec_ok, pad2;                                    // bit j: the spec is defined at probe j
    i32 start_nt[2], max_size[2];
    i64 probe_id[kJointProbes];
    i64 probe_pt[kJointProbes][kMaxVars];
    i64 probe_spec[kJointProbes];
    xp_instr ctx[kMaxCode], spec[kMaxCode];
    const i64* spec_table;                                // device, or null: evaluate `spec`
    u64 tab_off[2][kMaxSize + 1];                         // first entry of each size in a part's table
    u64 tab_total[2];
    i64* tab_val[2];                                      // device, [probe][entry]
    unsigned char* tab_ok[2];
    u64 match_count[kJointTotal + 1];
    u64 min_key[kJointTotal + 1];                         // size of part 0 << 48 | rank 0 << 24 | rank 1 (all-ones: none)
    u64 evals, survivors;
};

// Value of the joint context at one point from the values of its two parts.
__device__ __forceinline__ bool eval_joint(const xp_instr* code, int n, const i64* pt, i64 h0, i64 h1, i64& out) {
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
            st[sp++] = c.kind == XP_I_VAR ? pt[c.arg] : (c.kind == XP_I_CONST ? c.value : (c.arg == 0 ? h0 : h1));
        }
    }
    out = st[0];
    return true;
}

__global__ void joint_probe_kernel(JointDev* J) {
    const int t = threadIdx.x;
    const SketchDev* sk = J->sk;
    bool ok = false;
    if (t < J->n_probe) {
        i64 pt[kMaxVars];
        const i64 pid = sk->sample_id[t];
        point_coords(sk, pid, pt);
        for (int d = 0; d < sk->n_vars; ++d) J->probe_pt[t][d] = pt[d];
        J->probe_id[t] = pid;
        i64 v = 0;
        ok = true;
        if (J->spec_table != nullptr) v = J->spec_table[pid];
        else ok = eval_code(J->spec, J->spec_len, pt, 0, v);
        J->probe_spec[t] = v;
    }
    const u32 m = __ballot_sync(0xffffffffu, ok);
    if (t == 0) J->spec_ok = m;
}

__global__ void __launch_bounds__(256) joint_values_kernel(JointDev* J, int part, int size) {
    const SketchDev* sk = J->sk;
    const GrammarDev* g = sk->g;
    const int nt = J->start_nt[part];
    const u64 rank = (u64)blockIdx.x * blockDim.x + threadIdx.x;
    const int pr = blockIdx.y;
    if (rank >= g->cnt[nt][size] || pr >= J->n_probe) return;
    u32 code[kMaxSize];
    const int n = unrank(g, nt, size, rank, code);
    i64 v = 0;
    const bool ok = eval_cand(code, n, g->leaves, J->probe_pt[pr], v);
    const u64 at = (u64)pr * J->tab_total[part] + J->tab_off[part][size] + rank;
    J->tab_val[part][at] = v;
    J->tab_ok[part][at] = ok ? 1 : 0;
}

// The pair (tree r0 of size s0, tree r1 of size s1) on every domain point; called by all 32
// lanes of a warp together.  Adds the points tried to evals.
__device__ __noinline__ bool joint_check_domain(const JointDev* J, int s0, u64 r0, int s1, u64 r1, u64& evals) {
    const SketchDev* sk = J->sk;
    const GrammarDev* g = sk->g;
    const int lane = threadIdx.x & 31;
    u32 c0[kMaxSize], c1[kMaxSize];
    const int n0 = unrank(g, J->start_nt[0], s0, r0, c0);
    const int n1 = unrank(g, J->start_nt[1], s1, r1, c1);
    for (i64 base = 0; base < sk->n_points; base += 32) {
        bool bad = false;
        const i64 pid = base + lane;
        if (pid < sk->n_points) {
            ++evals;
            i64 pt[kMaxVars];
            point_coords(sk, pid, pt);
            i64 want = 0, h0, h1, v;
            bool ok = true;
            if (J->spec_table != nullptr) want = J->spec_table[pid];
            else ok = eval_code(J->spec, J->spec_len, pt, 0, want);
            ok = ok && eval_cand(c0, n0, g->leaves, pt, h0) && eval_cand(c1, n1, g->leaves, pt, h1) &&
                 eval_joint(J->ctx, J->ctx_len, pt, h0, h1, v) && v == want;
            bad = !ok;
        }
        if (__any_sync(0xffffffffu, bad)) return false;
    }
    return true;
}

__global__ void __launch_bounds__(256) joint_pairs_kernel(JointDev* J, int s0, int s1, u64 n0, u64 n1) {
    const int lane = threadIdx.x & 31;
    const u64 pairs = n0 * n1;
    const u64 stride = (u64)gridDim.x * blockDim.x;
    const int np = J->n_probe;
    const u32 spec_ok = J->spec_ok;
    const u64 all_ok = np >= 32 ? 0xffffffffu : (1u << np) - 1u;
    u64 evals = 0, survivors = 0;
    // (whole warps walk the loop together: the bound is rounded up to a multiple of the warp's 32 pairs)
    for (u64 q0 = ((u64)blockIdx.x * blockDim.x + threadIdx.x) & ~31ull; q0 < pairs; q0 += stride) {
        const u64 q = q0 + lane;
        bool pass = q < pairs && (spec_ok & all_ok) == all_ok;          // a spec undefined at a probe: nothing matches
        u64 r0 = 0, r1 = 0;
        if (pass) {
            r0 = q / n1; r1 = q - r0 * n1;
            const u64 e0 = J->tab_off[0][s0] + r0, e1 = J->tab_off[1][s1] + r1;
            for (int j = 0; j < np && pass; ++j) {
                ++evals;
                const u64 a0 = (u64)j * J->tab_total[0] + e0, a1 = (u64)j * J->tab_total[1] + e1;
                i64 v;
                pass = J->tab_ok[0][a0] && J->tab_ok[1][a1] &&
                       eval_joint(J->ctx, J->ctx_len, J->probe_pt[j], J->tab_val[0][a0], J->tab_val[1][a1], v) && v == J->probe_spec[j];
            }
        }
        u32 m = __ballot_sync(0xffffffffu, pass);
        survivors += (u64)__popc(m) * (lane == 0);
        while (m) {                                       // the warp checks its survivors on the whole domain, one by one
            const int src = __ffs((int)m) - 1;
            m &= m - 1;
            const u64 x0 = __shfl_sync(0xffffffffu, r0, src), x1 = __shfl_sync(0xffffffffu, r1, src);
            if (joint_check_domain(J, s0, x0, s1, x1, evals) && lane == 0) {
                atomicAdd(&J->match_count[s0 + s1], 1ull);
                atomicMin(&J->min_key[s0 + s1], ((u64)s0 << 48) | (x0 << 24) | x1);
            }
        }
    }
    for (int o = 16; o > 0; o >>= 1) evals += __shfl_down_sync(0xffffffffu, evals, o);
    if (lane == 0) {
        if (evals) atomicAdd(&J->evals, evals);
        if (survivors) atomicAdd(&J->survivors, survivors);
    }
}

}  // namespace xp

using namespace xp;

struct xp_joint_result {
    int solved = 0, max_total = 0, least_total = 0, least_size[2] = {0, 0};
    u64 cand[kJointTotal + 1] = {0}, match[kJointTotal + 1] = {0};
    u64 least_rank[2] = {0, 0};
    std::string text[2];
    u64 evals = 0, survivors = 0;
    double kernel_ms = 0, total_ms = 0;
    int n_launches = 0;
};

extern "C" xp_status xp_joint_result_get(const xp_joint_result* r, xp_joint_view* v) {
    if (!r || !v) return set_error(XP_ERR_INVALID_ARG, "xp_joint_result_get: null argument");
    v->solved = r->solved; v->max_total = r->max_total;
    v->cand_count = (const uint64_t*)r->cand; v->match_count = (const uint64_t*)r->match;
    v->least_total = r->least_total;
    for (int k = 0; k < 2; ++k) { v->least_size[k] = r->least_size[k]; v->least_rank[k] = r->least_rank[k]; v->least_text[k] = r->text[k].c_str(); }
    v->evals_executed = r->evals; v->probe_survivors = r->survivors;
    v->kernel_ms = r->kernel_ms; v->total_ms = r->total_ms; v->n_launches = r->n_launches;
    return XP_OK;
}

extern "C" void xp_joint_result_free(xp_joint_result* r) { delete r; }

static bool joint_code_ok(const xp_instr* code, int n, int n_vars, bool holes, int* parts_seen) {
    if (n < 1 || n > kMaxCode || !code) return false;
    int sp = 0;
    for (int i = 0; i < n; ++i) {
        const xp_instr& c = code[i];
        if (c.kind == XP_I_OP) { if (c.arg < XP_OP_ADD || c.arg > XP_OP_SHR || sp < 2) return false; --sp; continue; }
        if (c.kind == XP_I_VAR) { if (c.arg < 0 || c.arg >= n_vars) return false; }
        else if (c.kind == XP_I_HOLE) { if (!holes || c.arg < 0 || c.arg > 1) return false; *parts_seen |= 1 << c.arg; }
        else if (c.kind != XP_I_CONST) return false;
        if (++sp > kMaxStack) return false;
    }
    return sp == 1;
}

extern "C" xp_status xp_repair_joint(const xp_sketch* sketch, const xp_joint_desc* d, const xp_repair_opts* opts, xp_joint_result** out) {
    if (!sketch || !d || !out) return set_error(XP_ERR_INVALID_ARG, "xp_repair_joint: null argument");
    *out = nullptr;
    const auto t0 = std::chrono::steady_clock::now();
    const SketchInternals si = sketch_internals(sketch);
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return set_error(XP_ERR_CUDA, "no CUDA device is usable");
    if (dev != si.device) return set_error(XP_ERR_INVALID_ARG, "xp_repair_joint: the sketch was loaded on another device than the current one");
    int parts = 0, none = 0;
    if (!joint_code_ok(d->ctx, d->ctx_len, si.n_vars, true, &parts) || parts != 3)
        return set_error(XP_ERR_SKETCH, "xp_repair_joint: malformed context, or one that does not mention both parts");
    if (d->spec_kind == XP_SPEC_EXPR) {
        if (!joint_code_ok(d->spec_expr, d->spec_len, si.n_vars, false, &none)) return set_error(XP_ERR_SKETCH, "xp_repair_joint: malformed spec expression");
    } else if (d->spec_kind != XP_SPEC_TABLE || (si.n_points > 0 && !d->spec_table)) return set_error(XP_ERR_SKETCH, "xp_repair_joint: bad spec");
    xp_joint_result* r = new (std::nothrow) xp_joint_result;
    if (!r) return set_error(XP_ERR_NOMEM, "out of host memory");
    JointDev h;
    memset(&h, 0, sizeof(h));
    u64 entries[2] = {0, 0};
    for (int k = 0; k < 2; ++k) {
        const int nt = d->start_nt[k], K = d->max_size[k];
        if (nt < 0 || nt >= grammar_nonterminals(si.g) || K < 1 || K > kMaxSize) { delete r; return set_error(XP_ERR_SKETCH, "xp_repair_joint: start_nt or max_size out of range"); }
        if (K > grammar_ok_size(si.g)) { delete r; return set_error(XP_ERR_TOO_LARGE, "a candidate count reaches 2^63 within the size bound"); }
        h.start_nt[k] = nt; h.max_size[k] = K;
        for (int s = 1; s <= K; ++s) {
            const u64 c = grammar_cnt(si.g, nt, s);
            if (c >= kJointMaxEntries) { delete r; return set_error(XP_ERR_TOO_LARGE, "xp_repair_joint: a part has 2^22 candidates or more of one size"); }
            h.tab_off[k][s] = entries[k];
            entries[k] += c;
        }
        h.tab_total[k] = entries[k];
    }
    r->max_total = d->max_size[0] + d->max_size[1];
    u64 all_pairs = 0;
    for (int s0 = 1; s0 <= d->max_size[0]; ++s0)
        for (int s1 = 1; s1 <= d->max_size[1]; ++s1) {
            const u64 p = grammar_cnt(si.g, d->start_nt[0], s0) * grammar_cnt(si.g, d->start_nt[1], s1);      // (< 2^44)
            r->cand[s0 + s1] += p;
            all_pairs += p;
        }
    if (all_pairs > kJointMaxPairs) { delete r; return set_error(XP_ERR_TOO_LARGE, "xp_repair_joint: more than 2^40 pairs"); }
    if (si.n_points == 0) {                                 // no constraint at all: every pair satisfies it
        for (int t = 2; t <= r->max_total; ++t) r->match[t] = r->cand[t];
        for (int t = 2; t <= r->max_total && !r->solved; ++t)
            for (int s0 = 1; s0 < t && !r->solved; ++s0)
                if (s0 <= d->max_size[0] && t - s0 <= d->max_size[1] && grammar_cnt(si.g, d->start_nt[0], s0) * grammar_cnt(si.g, d->start_nt[1], t - s0) > 0) {
                    r->solved = 1; r->least_total = t; r->least_size[0] = s0; r->least_size[1] = t - s0;
                    for (int k = 0; k < 2; ++k) {
                        char buf[1024];
                        if (xp_grammar_unrank(si.g, d->start_nt[k], r->least_size[k], 0, nullptr, 0, buf, sizeof(buf)) == XP_OK) r->text[k] = buf;
                    }
                }
        r->total_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t0).count();
        *out = r;
        return XP_OK;
    }
    const int n_probe = (int)(si.n_points < kJointProbes ? si.n_points : kJointProbes);
    // one device block: the record, the spec table (if it is the host's), the value tables
    auto al = [](size_t b) { return (b + 255) & ~(size_t)255; };
    const bool copy_spec = d->spec_kind == XP_SPEC_TABLE && si.n_points > 0 && !d->spec_table_on_device;
    size_t off = al(sizeof(JointDev));
    const size_t off_spec = off;
    if (copy_spec) off += al(sizeof(i64) * (size_t)si.n_points);
    size_t off_val[2], off_ok[2];
    for (int k = 0; k < 2; ++k) {
        off_val[k] = off; off += al(sizeof(i64) * entries[k] * (size_t)(n_probe ? n_probe : 1));
        off_ok[k] = off; off += al(entries[k] * (size_t)(n_probe ? n_probe : 1));
    }
    char* block = nullptr;
    size_t granted = 0;
    int bdev = 0;
    if (device_alloc((void**)&block, off, &bdev, &granted) != cudaSuccess) {
        (void)cudaGetLastError();
        delete r;
        return set_error(XP_ERR_NOMEM, "xp_repair_joint: device memory for the value tables");
    }
    h.sk = si.d_s; h.n_probe = n_probe; h.ctx_len = d->ctx_len;
    memcpy(h.ctx, d->ctx, sizeof(xp_instr) * d->ctx_len);
    if (d->spec_kind == XP_SPEC_EXPR) { h.spec_len = d->spec_len; memcpy(h.spec, d->spec_expr, sizeof(xp_instr) * d->spec_len); }
    else if (si.n_points > 0) h.spec_table = copy_spec ? (const i64*)(block + off_spec) : (const i64*)d->spec_table;
    for (int k = 0; k < 2; ++k) { h.tab_val[k] = (i64*)(block + off_val[k]); h.tab_ok[k] = (unsigned char*)(block + off_ok[k]); }
    for (int t = 0; t <= kJointTotal; ++t) h.min_key[t] = ~0ull;
    JointDev* dJ = (JointDev*)block;
    cudaStream_t stream = opts ? (cudaStream_t)opts->stream : nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaError_t e = cudaMemcpyAsync(dJ, &h, sizeof(h), cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess && copy_spec) e = cudaMemcpyAsync(block + off_spec, d->spec_table, sizeof(i64) * (size_t)si.n_points, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    if (e == cudaSuccess) e = cudaEventRecord(e0, stream);
    int launches = 0;
    if (e == cudaSuccess && n_probe > 0) {
        joint_probe_kernel<<<1, 32, 0, stream>>>(dJ);
        ++launches;
        e = cudaGetLastError();
        for (int k = 0; k < 2 && e == cudaSuccess; ++k)
            for (int s = 1; s <= d->max_size[k] && e == cudaSuccess; ++s) {
                const u64 c = grammar_cnt(si.g, d->start_nt[k], s);
                if (c == 0) continue;
                joint_values_kernel<<<dim3((unsigned)((c + 255) / 256), (unsigned)n_probe), 256, 0, stream>>>(dJ, k, s);
                ++launches;
                e = cudaGetLastError();
            }
        int sms = 148;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        for (int t = 2; t <= r->max_total && e == cudaSuccess; ++t)          // total size ascending (any order gives the same sums and minima)
            for (int s0 = 1; s0 < t && e == cudaSuccess; ++s0) {
                const int s1 = t - s0;
                if (s0 > d->max_size[0] || s1 > d->max_size[1]) continue;
                const u64 n0 = grammar_cnt(si.g, d->start_nt[0], s0), n1 = grammar_cnt(si.g, d->start_nt[1], s1);
                if (n0 == 0 || n1 == 0) continue;
                const u64 want = (n0 * n1 + 255) / 256, most = (u64)sms * 8;
                joint_pairs_kernel<<<(unsigned)(want < most ? want : most), 256, 0, stream>>>(dJ, s0, s1, n0, n1);
                ++launches;
                e = cudaGetLastError();
            }
    }
    JointDev back;
    if (e == cudaSuccess) e = cudaEventRecord(e1, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(&back, dJ, sizeof(back), cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream); else cudaStreamSynchronize(stream);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    device_release(block, granted, bdev);
    if (e != cudaSuccess) { delete r; return set_error(XP_ERR_CUDA, (std::string("xp_repair_joint: ") + cudaGetErrorString(e)).c_str()); }
    for (int t = 2; t <= r->max_total; ++t) {
        r->match[t] = back.match_count[t];
        if (!r->solved && back.match_count[t] > 0) {
            r->solved = 1; r->least_total = t;
            const u64 key = back.min_key[t];
            r->least_size[0] = (int)(key >> 48); r->least_size[1] = t - r->least_size[0];
            r->least_rank[0] = (key >> 24) & 0xffffffull; r->least_rank[1] = key & 0xffffffull;
            for (int k = 0; k < 2; ++k) {
                char buf[1024];
                if (xp_grammar_unrank(si.g, d->start_nt[k], r->least_size[k], r->least_rank[k], nullptr, 0, buf, sizeof(buf)) == XP_OK) r->text[k] = buf;
            }
        }
    }
    r->evals = back.evals; r->survivors = back.survivors;
    r->kernel_ms = ms; r->n_launches = launches;
    r->total_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t0).count();
    *out = r;
    return XP_OK;
}
