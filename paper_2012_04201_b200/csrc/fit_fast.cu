// Instantiates the compile-time-stride fit kernels (64 padded features, 10 classes) for one
// padded hidden width (BBO_HSC).
#include "fit_kernel.cuh"
#include "fit_roles.cuh"
#include "fit_launch.h"

#ifndef BBO_HSC
#error "compile with -DBBO_HSC=<padded hidden width>"
#endif

namespace bbo {

template <>
const void* fast_fit_kernel<BBO_HSC>(bool vreg, bool pipe) {
  constexpr int NT = (BBO_HSC + 31) / 32 * 32;
#if BBO_HSC >= 128
  constexpr int NTP = NT + 64 <= kMaxFitThreads ? NT + 64 : NT + 32;  // one or two extra warps for the output layer
  if (pipe) {
    if (vreg) return reinterpret_cast<const void*>(&mlp_cv_fit_kernel<kFastClasses, true, BBO_HSC, kFastDp, NTP, 1, true>);
    return reinterpret_cast<const void*>(&mlp_cv_fit_kernel<kFastClasses, false, BBO_HSC, kFastDp, NTP, 1, true>);
  }
#else
  if (pipe) return nullptr;
#endif
  if (vreg) return reinterpret_cast<const void*>(&mlp_cv_fit_kernel<kFastClasses, true, BBO_HSC, kFastDp, NT, 1>);
  return reinterpret_cast<const void*>(&mlp_cv_fit_kernel<kFastClasses, false, BBO_HSC, kFastDp, NT, 1>);
}

template <>
const void* fast_roles_kernel<BBO_HSC>() {
  constexpr RoleWarps r = role_warps(kFastDp, BBO_HSC, kFastClasses, 32);
  constexpr bool wide = wide_layout(r);
  constexpr int NT = wide ? 32 * kWideRoleWarps.total() : 32 * r.total();
  return reinterpret_cast<const void*>(&mlp_cv_fit_roles_kernel<kFastClasses, BBO_HSC, kFastDp, NT, 1, wide>);
}

}  // namespace bbo
