// Host-callable launchers of the kernels in xp_kernels.cu.
#pragma once

#include <cuda_runtime.h>

#include "xp_dev.h"

namespace xp {

cudaError_t launch_prepare(SketchDev* s, cudaStream_t stream);
cudaError_t launch_eval(const PlanDev& plan, int n_ctas, cudaStream_t stream);
cudaError_t launch_finish(AccDev* acc, int n_acc, cudaStream_t stream);
int eval_ctas_per_sm();
cudaError_t launch_int32_peak(int which, u32* out, int blocks, int iters, cudaStream_t stream);

}  // namespace xp
