// Host-callable launchers of the kernels in xp_kernels.cu.
#pragma once

#include <cuda_runtime.h>

#include "xp_dev.h"

namespace xp {

cudaError_t launch_prepare(SketchDev* s, cudaStream_t stream);
cudaError_t launch_subvalues(const SketchDev* s, int hole_index, int size, u64 n_entries, cudaStream_t stream);
cudaError_t launch_eval(const PlanDev& plan, int n_ctas, cudaStream_t stream);
cudaError_t launch_finish(AccDev* acc, int n_acc, cudaStream_t stream);
int eval_ctas_per_sm();
constexpr size_t kStaticScratchBytes = 1u << 20;     // fixed scratch of the allocation-free entry point
cudaError_t launch_search_static(const void* stage, size_t total, size_t off_segs, size_t off_sketches, size_t off_acc,
                                 u64 n_tickets, int n_segs, int n_acc, int n_ctas, AccDev* acc_out, cudaStream_t stream);
cudaError_t launch_int32_peak(int which, u32* out, int blocks, int iters, cudaStream_t stream);

}  // namespace xp
