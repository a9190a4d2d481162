// Device kernels of libxpiler_repair (sm_100a).
//
//   prepare_kernel  -- per sketch, once at load: coordinates and spec values of the sample
//                      points, choice and order of each hole's probe points.
//   eval_kernel     -- the search.  Persistent CTAs take tickets (pieces of the rank space)
//                      from an atomic counter; no CTA ever waits for another.
//                        stage 1 (tile segments): probe-point filter over a product of operand tiles;
//                        stage 2: exact int64 check of a candidate on the probe points (lane = candidate);
//                        stage 3: check on the whole domain (lane = point, block-wide early exit).
//   finish_kernel   -- reduction of the per-size results to the least solution per hole.
//   int32_peak_*    -- integer-ALU peak microbenchmarks.
#include <cuda_runtime.h>

#include "xp_device.cuh"
#include "xp_launch.h"

namespace xp {

// ------------------------------------------------------------------------------------------
// prepare
// ------------------------------------------------------------------------------------------

// One CTA of kProbeSamples threads per sketch.  Thread t evaluates sample point t; thread 0
// then orders each hole's probes: the sample with the largest |spec| + sum |coordinate|
// first (large, distinct operand values make coincidental matches rare), the rest in sample
// order (box corners come first there).
__global__ void __launch_bounds__(kProbeSamples) prepare_kernel(SketchDev* s) {
    __shared__ i64 s_pt[kProbeSamples][kMaxVars];
    __shared__ i64 s_spec[kProbeSamples];
    __shared__ int s_ok[kProbeSamples];
    __shared__ u64 s_score[kProbeSamples];
    const int t = threadIdx.x;
    const int ns = s->n_samples;
    const int nv = s->n_vars;
    i64 pt[kMaxVars];
    u64 coord_mag = 0;
    if (t < ns) {
        point_coords(s, s->sample_id[t], pt);
        for (int d = 0; d < nv; ++d) {
            s_pt[t][d] = pt[d];
            coord_mag += (u64)(pt[d] < 0 ? -pt[d] : pt[d]);
        }
    }
    for (int h = 0; h < s->n_holes; ++h) {
        HoleDev* hole = &s->holes[h];
        __syncthreads();
        if (t < ns) {
            i64 v = 0;
            bool ok = true;
            if (hole->spec_len == 0) v = hole->spec_table[s->sample_id[t]];
            else ok = eval_code(hole->spec, hole->spec_len, pt, 0, v);
            s_spec[t] = v;
            s_ok[t] = ok;
            const u64 mag = (u64)(v < 0 ? -v : v);
            s_score[t] = ok ? (mag > (1ull << 62) ? (1ull << 62) : mag) + coord_mag : 0;
        }
        __syncthreads();
        if (t == 0) {
            int best = 0;
            for (int i = 1; i < ns; ++i) if (s_score[i] > s_score[best]) best = i;
            int n = 0;
            u32 okmask = 0;
            for (int j = -1; j < ns && n < kMaxProbe; ++j) {
                const int i = j < 0 ? best : j;
                if (j >= 0 && i == best) continue;
                if (ns == 0) break;
                hole->probe_id[n] = s->sample_id[i];
                for (int d = 0; d < nv; ++d) hole->probe_pt[n][d] = s_pt[i][d];
                hole->probe_spec[n] = s_spec[i];
                if (s_ok[i]) okmask |= 1u << n;
                ++n;
            }
            hole->n_probe = n;
            hole->probe_spec_ok = okmask;
            hole->chain_len = -1;
        }
    }
}

// ------------------------------------------------------------------------------------------
// eval
// ------------------------------------------------------------------------------------------

constexpr int kLinearPerThread = 4;                       // ranks per thread per linear ticket
constexpr int kLinearChunk = kThreads * kLinearPerThread; // ranks per linear ticket
constexpr int kMaxSurvivors = kLinearChunk;

struct EvalShared {
    u64 ticket;
    SegDev seg;
    // survivors of the probe stage, waiting for the whole-domain check
    u32 n_surv;
    u64 surv_rank[kMaxSurvivors];
    // the candidate under whole-domain check, leaves resolved
    i32 cand_len;
    i32 cand_var[kMaxSize];      // >= 0: variable; -1: constant; -2 - op: operator
    i64 cand_val[kMaxSize];
    // results of the (sketch, hole) the CTA is working on
    i32 cur_acc;
    u64 match_count[kMaxSize + 1];
    u64 min_rank[kMaxSize + 1];
    u64 filter_survivors, probe_survivors;
    u64 warp_evals[kThreads / 32];
};

// Moves the CTA's private results of one (sketch, hole) into the global accumulators.
// Counts are sums and ranks are minima, so the order of flushes cannot change the result.
__device__ void flush_acc(EvalShared& sh, const PlanDev& plan, u64& my_evals) {
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
        }
    }
    __syncthreads();
    if (threadIdx.x <= kMaxSize) { sh.match_count[threadIdx.x] = 0; sh.min_rank[threadIdx.x] = ~0ull; }
    if (threadIdx.x == 0) { sh.filter_survivors = 0; sh.probe_survivors = 0; }
    my_evals = 0;
    __syncthreads();
}

// Stage 2: exact check of one candidate on the hole's probe points, first failure ends it.
__device__ __forceinline__ bool probe_check(const GrammarDev* g, const HoleDev* hole, const u32* code, int n,
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

// Stage 3: the whole CTA checks one candidate on every domain point, kThreads points at a
// time; a failing point anywhere ends the scan at the next block-wide vote.
__device__ void verify_survivors(EvalShared& sh, const SketchDev* sk, const HoleDev* hole, int size, u64& my_evals) {
    const GrammarDev* g = sk->g;
    const u32 ns = sh.n_surv;
    for (u32 i = 0; i < ns; ++i) {
        const u64 rank = sh.surv_rank[i];
        if (threadIdx.x == 0) {
            u32 code[kMaxSize];
            const int n = unrank(g, hole->start_nt, size, rank, code);
            sh.cand_len = n;
            for (int k = 0; k < n; ++k) {
                if (code[k] & kOpBit) { sh.cand_var[k] = -2 - (i32)(code[k] & 0xff); sh.cand_val[k] = 0; }
                else { const LeafDev lf = g->leaves[code[k]]; sh.cand_var[k] = lf.var >= 0 ? lf.var : -1; sh.cand_val[k] = lf.value; }
            }
        }
        __syncthreads();
        const int n = sh.cand_len;
        bool failed = false;
        for (i64 base = 0; base < sk->n_points; base += kThreads) {
            const i64 pid = base + threadIdx.x;
            bool bad = false;
            if (pid < sk->n_points) {
                ++my_evals;
                i64 pt[kMaxVars];
                point_coords(sk, pid, pt);
                i64 want = 0;
                bool ok = true;
                if (hole->spec_len == 0) want = hole->spec_table[pid];
                else ok = eval_code(hole->spec, hole->spec_len, pt, 0, want);
                i64 st[kCandStack];
                int sp = 0;
                for (int k = 0; k < n && ok; ++k) {
                    const i32 cv = sh.cand_var[k];
                    if (cv >= -1) st[sp++] = cv >= 0 ? pt[cv] : sh.cand_val[k];
                    else {
                        const i64 b = st[--sp];
                        i64 r;
                        ok = apply_op(-2 - cv, st[sp - 1], b, r);
                        st[sp - 1] = r;
                    }
                }
                bad = !ok || !ctx_matches(hole, pt, st[0], want);
            }
            if (__syncthreads_or(bad)) { failed = true; break; }
        }
        if (!failed && threadIdx.x == 0) {
            sh.match_count[size] += 1;
            if (rank < sh.min_rank[size]) sh.min_rank[size] = rank;
        }
        __syncthreads();
    }
    __syncthreads();
    if (threadIdx.x == 0) sh.n_surv = 0;
    __syncthreads();
}

// A linear ticket: kLinearChunk consecutive ranks, each unranked and checked on its own.
__device__ void linear_ticket(EvalShared& sh, const SketchDev* sk, const HoleDev* hole, u64 local, u64& my_evals) {
    const SegDev& seg = sh.seg;
    const GrammarDev* g = sk->g;
    const u64 first = seg.rank_begin + local * (u64)kLinearChunk;
    for (int i = 0; i < kLinearPerThread; ++i) {
        const u64 rank = first + (u64)i * kThreads + threadIdx.x;
        if (rank < seg.rank_end) {
            u32 code[kMaxSize];
            const int n = unrank(g, hole->start_nt, seg.size, rank, code);
            if (probe_check(g, hole, code, n, my_evals)) {
                const u32 slot = atomicAdd(&sh.n_surv, 1u);
                sh.surv_rank[slot] = rank;
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) { sh.filter_survivors += sh.n_surv; sh.probe_survivors += sh.n_surv; }
    verify_survivors(sh, sk, hole, seg.size, my_evals);
}

__global__ void __launch_bounds__(kThreads) eval_kernel(const PlanDev plan) {
    __shared__ EvalShared sh;
    u64 my_evals = 0;
    if (threadIdx.x <= kMaxSize) { sh.match_count[threadIdx.x] = 0; sh.min_rank[threadIdx.x] = ~0ull; }
    if (threadIdx.x == 0) { sh.cur_acc = -1; sh.n_surv = 0; sh.filter_survivors = 0; sh.probe_survivors = 0; }
    __syncthreads();
    for (;;) {
        if (threadIdx.x == 0) {
            const u64 t = atomicAdd(plan.ticket, 1ull);
            sh.ticket = t;
            if (t < plan.n_tickets) {
                int lo = 0, hi = plan.n_segs - 1;             // last segment with first_ticket <= t
                while (lo < hi) {
                    const int mid = (lo + hi + 1) >> 1;
                    if (plan.segs[mid].first_ticket <= t) lo = mid; else hi = mid - 1;
                }
                sh.seg = plan.segs[lo];
            }
        }
        __syncthreads();
        const u64 t = sh.ticket;
        if (t >= plan.n_tickets) break;
        if (sh.seg.acc != sh.cur_acc) {
            flush_acc(sh, plan, my_evals);
            if (threadIdx.x == 0) sh.cur_acc = sh.seg.acc;
            __syncthreads();
        }
        const SketchDev* sk = plan.sketches[sh.seg.sketch];
        const HoleDev* hole = &sk->holes[sh.seg.hole];
        const u64 local = t - sh.seg.first_ticket;
        linear_ticket(sh, sk, hole, local, my_evals);
        __syncthreads();
    }
    flush_acc(sh, plan, my_evals);
}

// ------------------------------------------------------------------------------------------
// finish: least (size, rank) per hole from the per-size minima
// ------------------------------------------------------------------------------------------

// One warp per accumulator: lane = size; ballot finds the smallest size with a match.
__global__ void finish_kernel(AccDev* acc, int n_acc) {
    const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
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

// ------------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------------

cudaError_t launch_prepare(SketchDev* s, cudaStream_t stream) {
    prepare_kernel<<<1, kProbeSamples, 0, stream>>>(s);
    return cudaGetLastError();
}

cudaError_t launch_eval(const PlanDev& plan, int n_ctas, cudaStream_t stream) {
    eval_kernel<<<n_ctas, kThreads, 0, stream>>>(plan);
    return cudaGetLastError();
}

cudaError_t launch_finish(AccDev* acc, int n_acc, cudaStream_t stream) {
    const int warps_per_block = 8;
    const int blocks = (n_acc + warps_per_block - 1) / warps_per_block;
    finish_kernel<<<blocks, warps_per_block * 32, 0, stream>>>(acc, n_acc);
    return cudaGetLastError();
}

int eval_ctas_per_sm() {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, eval_kernel, kThreads, 0) != cudaSuccess || n < 1) n = 1;
    return n;
}

cudaError_t launch_int32_peak(int which, u32* out, int blocks, int iters, cudaStream_t stream) {
    if (which == 0) int32_peak_add_kernel<<<blocks, 256, 0, stream>>>(out, iters, 1u);
    else int32_peak_mad_kernel<<<blocks, 256, 0, stream>>>(out, iters, 1u);
    return cudaGetLastError();
}

}  // namespace xp
