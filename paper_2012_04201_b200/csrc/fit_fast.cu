// Instantiates the compile-time-stride fit kernels (64 padded features, 10 classes) for one
// padded hidden width (BBO_HSC).
#include "fit_kernel.cuh"
#include "fit_launch.h"

#ifndef BBO_HSC
#error "compile with -DBBO_HSC=<padded hidden width>"
#endif

namespace bbo {

template <>
const void* fast_fit_kernel<BBO_HSC>(bool pipe) {
  constexpr int NT = fast_threads(BBO_HSC);
#if BBO_HSC >= 184
  constexpr int NTP = NT + 64 <= kMaxFitThreads ? NT + 64 : NT + 32;  // one or two extra warps for the output layer
  if (pipe) return reinterpret_cast<const void*>(&mlp_cv_fit_kernel<kFastClasses, BBO_HSC, kFastDp, NTP, 1, true>);
#else
  if (pipe) return nullptr;
#endif
  return reinterpret_cast<const void*>(&mlp_cv_fit_kernel<kFastClasses, BBO_HSC, kFastDp, NT, fast_min_blocks(BBO_HSC)>);
}

}  // namespace bbo
