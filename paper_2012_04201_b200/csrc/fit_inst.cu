// Instantiates the fit kernel for one class count (BBO_CT) and its launch-bound classes.
#include "fit_kernel.cuh"
#include "fit_launch.h"

#ifndef BBO_CT
#error "compile with -DBBO_CT=<class count>"
#endif

namespace bbo {

namespace {

template <typename Kern>
cudaError_t launch_one(Kern kern, const FitArgs& a, int threads, int grid, size_t smem, cudaStream_t s) {
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  // every fit kernel asks for the full shared-memory carve-out so that CTAs of launches with
  // different footprints can share an SM
  e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  if (e != cudaSuccess) return e;
  kern<<<grid, threads, smem, s>>>(a);
  return cudaGetLastError();
}

template <int CT, bool VR>
cudaError_t launch_class(const FitArgs& a, int threads, int grid, size_t smem, cudaStream_t s) {
  if (threads <= 128) return launch_one(mlp_cv_fit_kernel<CT, VR, 128, 4>, a, threads, grid, smem, s);
  if (threads <= 256) return launch_one(mlp_cv_fit_kernel<CT, VR, 256, 2>, a, threads, grid, smem, s);
  if (threads <= 448) return launch_one(mlp_cv_fit_kernel<CT, VR, 448, 1>, a, threads, grid, smem, s);
  return launch_one(mlp_cv_fit_kernel<CT, VR, 512, 1>, a, threads, grid, smem, s);
}

}  // namespace

template <>
cudaError_t launch_fit_ct<BBO_CT>(const FitArgs& a, bool vreg, int threads, int grid, size_t smem, cudaStream_t s) {
  if (vreg) return launch_class<BBO_CT, true>(a, threads, grid, smem, s);
  return launch_class<BBO_CT, false>(a, threads, grid, smem, s);
}

}  // namespace bbo
