// Host-side entry to the fit kernels.  The kernels are templates on the class count; each
// class count is compiled in its own translation unit (fit_inst.cu with -DBBO_CT=<n>) so the
// library builds in parallel, and this dispatcher picks the instance at run time.
#pragma once
#include <cuda_runtime.h>

#include "fit_common.cuh"

namespace bbo {

constexpr int kMaxClasses = 16;

// Launches `grid` CTAs of `threads` threads (one per fit of a.fits) with `smem` bytes of
// dynamic shared memory.  vreg: second moments of W1 kept in registers.
template <int CT>
cudaError_t launch_fit_ct(const FitArgs& a, bool vreg, int threads, int grid, size_t smem, cudaStream_t s);

cudaError_t launch_fit(int C, const FitArgs& a, bool vreg, int threads, int grid, size_t smem, cudaStream_t s);

}  // namespace bbo
