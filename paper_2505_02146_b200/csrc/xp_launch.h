// Host-callable launchers of the kernels in xp_kernels.cu.
#pragma once

#include <cuda_runtime.h>

#include "xp_dev.h"

namespace xp {

cudaError_t launch_prepare(const LoadJob* jobs, int n_jobs, cudaStream_t stream);
cudaError_t launch_reprobe(const LoadJob* jobs, int n_jobs, cudaStream_t stream);
cudaError_t launch_coord_bounds(SketchDev* const* list, int n_sketches, i64 most_points, cudaStream_t stream);
cudaError_t launch_stage_points(const SketchDev* s, i64 n_points, i32* coords, cudaStream_t stream);
cudaError_t launch_stage_spec(const SketchDev* s, int hole_index, i64 n_points, i64* spec, u32* bad, cudaStream_t stream);
cudaError_t launch_subvalues(const LoadJob* jobs, int n_jobs, int size, int most_probes, u64 most_entries, cudaStream_t stream);
cudaError_t launch_bigvalues(const LoadJob* jobs, int n_jobs, u64 most_entries, cudaStream_t stream);
// Layout of one call's device scratch (byte offsets from its 256-byte aligned base):
//   0: eval ticket (u64), 8: verify ticket (u64), 16: survivor pushes (u32), 20: failed-check word (u32; checked
//      build only)   -- zero at launch
//   segs, sketches, acc: staged from the host;  [0, head) is what the host copies in
//   hist: survivors per accumulator slot, zero at launch (staged);
//   surv: the survivor queue (surv_cap entries); sort_off, sorted: its hole order -- written by the kernels only
struct SearchLayout { size_t segs, sketches, acc, hist, head, surv, sort_off, sorted, longs, total; u32 surv_cap; int n_acc;
                      int dense; /* some hole of the plan takes the second look: launch the search kernel's dense form */ };

// The whole search on a staged scratch: eval_kernel, verify_kernel, count_kernel, finish_kernel;
// or the same in pieces: eval_kernel over one range of tickets at a time, then the rest.
cudaError_t launch_search_part(char* base, const SearchLayout& L, u64 t_begin, u64 t_end, bool restart, int n_segs,
                               int n_sketches, u32 max_chunks, cudaStream_t stream, int* n_launches);
cudaError_t launch_search_end(char* base, const SearchLayout& L, bool any_tickets, int n_segs, int n_sketches, int n_acc,
                              u32 max_chunks, cudaStream_t stream, int* n_launches);
cudaError_t launch_search(char* base, const SearchLayout& L, u64 n_tickets, int n_segs, int n_sketches, int n_acc,
                          u32 max_chunks, cudaStream_t stream, int* n_launches);
constexpr size_t kStaticScratchBytes = 1u << 20;     // fixed scratch of the allocation-free entry point
cudaError_t launch_search_static(const void* stage, const SearchLayout& L, u64 n_tickets, int n_segs, int n_acc,
                                 u32 max_chunks, AccDev* acc_out, cudaStream_t stream);
cudaError_t launch_int32_peak(int which, u32* out, int blocks, int iters, cudaStream_t stream);

// What the library's other source files may know of a grammar and a loaded sketch (defined in xp_api.cu).
struct SketchInternals { const SketchDev* d_s; const xp_grammar* g; i64 n_points; int device, n_vars; };
SketchInternals sketch_internals(const xp_sketch* s);
u64 grammar_cnt(const xp_grammar* g, int nt, int size);      // trees of nt with exactly `size` nodes
int grammar_nonterminals(const xp_grammar* g);
int grammar_ok_size(const xp_grammar* g);                    // counts are exact (< 2^63) up to this size
// The grammar as the kernels see it (host copy of the tables): leaves and binary productions grouped by nonterminal.
struct GrammarHost { int n_nt, n_vars; const int* leaf_begin; const int* bin_begin; const LeafDev* leaves; const BinDev* bins;
                     const char* const* var_names; };
GrammarHost grammar_host(const xp_grammar* g);
struct HoleSpec { int start_nt, max_size; };
HoleSpec sketch_hole(const xp_sketch* s, int hole);           // hole < 0 or >= n_holes: start_nt = -1
const HoleDev* sketch_hole_dev(const xp_sketch* s, int hole); // device pointer
cudaError_t device_alloc(void** out, size_t bytes, int* device, size_t* granted);     // the library's device pool
void device_release(void* ptr, size_t granted, int device);
xp_status set_error(xp_status st, const char* msg);

}  // namespace xp
