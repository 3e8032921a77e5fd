// Instantiates the run-time-stride fit kernels for one class count (BBO_CT).
#include "fit_kernel.cuh"
#include "fit_roles.cuh"
#include "fit_launch.h"

#ifndef BBO_CT
#error "compile with -DBBO_CT=<class count>"
#endif

namespace bbo {

template <>
const void* generic_fit_kernel<BBO_CT>(bool vreg) {
  if (vreg) return reinterpret_cast<const void*>(&mlp_cv_fit_kernel<BBO_CT, true, 0, 0, kMaxFitThreads, 1>);
  return reinterpret_cast<const void*>(&mlp_cv_fit_kernel<BBO_CT, false, 0, 0, kMaxFitThreads, 1>);
}

template <>
const void* generic_roles_kernel<BBO_CT>(bool wide) {
  if (wide) return reinterpret_cast<const void*>(&mlp_cv_fit_roles_kernel<BBO_CT, 0, 0, 32 * kWideRoleWarps.total(), 1, true>);
  return reinterpret_cast<const void*>(&mlp_cv_fit_roles_kernel<BBO_CT, 0, 0, 32 * kCompactRoleWarps, 1, false>);
}

}  // namespace bbo
