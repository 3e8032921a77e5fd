// Instantiates the run-time-stride fit kernels for one class count (BBO_CT).
#include "fit_kernel.cuh"
#include "fit_launch.h"

#ifndef BBO_CT
#error "compile with -DBBO_CT=<class count>"
#endif

namespace bbo {

template <>
const void* generic_fit_kernel<BBO_CT>() {
  return reinterpret_cast<const void*>(&mlp_cv_fit_kernel<BBO_CT, 0, 0, kMaxFitThreads, 1>);
}

}  // namespace bbo
