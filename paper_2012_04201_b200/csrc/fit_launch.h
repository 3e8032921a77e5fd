// Host-side access to the fit kernels.  The kernels are templates on the class count (and,
// for the 64-feature / 10-class shape, on the padded hidden width); every instance is
// compiled in its own translation unit so the library builds in parallel, and this table
// returns the instance for a launch at run time.
#pragma once
#include <cuda_runtime.h>

#include "fit_common.cuh"

namespace bbo {

constexpr int kMaxClasses = 16;
constexpr int kMaxFitThreads = 256;  // launch bound of every fit kernel

// Fast-path shape: compile-time strides for dp == kFastDp, C == kFastClasses and
// Hs in [kFastHsMin, kFastHsMax] (multiples of 8).
constexpr int kFastDp = 64, kFastClasses = 10, kFastHsMin = 56, kFastHsMax = 200;

// Pipelined schedule (gradient tiles of one sub-tile overlap the output layer of the next, run by
// extra warps): built for the fast-path widths that sit alone on an SM.
constexpr int kPipeHsMin = 128;
inline int pipe_extra_warps(int Hs) { return (Hs + 31) / 32 * 32 + 64 <= kMaxFitThreads ? 2 : 1; }

// Warp-specialised schedule: warps per role for a fit of padded width Hs on dp padded features,
// C classes, sub-tiles of TB rows.  G: one thread per 8x8 tile of W1; H: one thread per 8x8 tile
// of a sub-tile's activations; O: a lane pair per row, sixteen rows per warp; U: one
// thread per group of units_per_thread(C) hidden units plus C threads for the output biases.
struct RoleWarps {
  int nG, nH, nO, nU;
  constexpr int total() const { return nG + nH + nO + nU; }
};
constexpr RoleWarps role_warps(int dp, int Hs, int C, int TB) {
  return RoleWarps{ceil_div((dp / 8) * (Hs / 8), 32), ceil_div(((TB + 7) / 8) * (Hs / 8), 32), TB > 16 ? 2 : 1,
                   ceil_div(Hs / units_per_thread(C) + C, 32)};
}
constexpr int kMaxGradWarps = 8;    // tensor memory holds the W1 moments of at most eight G warps
// Up to twelve warps the roles are packed one after the other and every thread has 168 registers.
// Wider fits run the 512-thread layout with the roles on warp-group boundaries (8 / 4 / 2 / 2
// warps) and the registers re-divided between the groups.
constexpr int kCompactRoleWarps = 12;
constexpr RoleWarps kWideRoleWarps{8, 4, 2, 2};
constexpr bool wide_layout(const RoleWarps& r) { return r.total() > kCompactRoleWarps; }
constexpr bool fits_wide_layout(const RoleWarps& r) {
  return r.nG <= kWideRoleWarps.nG && r.nH <= kWideRoleWarps.nH && r.nO <= kWideRoleWarps.nO && r.nU <= kWideRoleWarps.nU;
}

template <int CT> const void* generic_roles_kernel(bool wide);  // warp-specialised, run-time strides
template <int HSC> const void* fast_roles_kernel();            // warp-specialised, compile-time strides (layout follows from the width)
const void* roles_kernel_for(int C, int Hs, int dp, bool wide);

template <int CT> const void* generic_fit_kernel(bool vreg);   // run-time strides
template <int HSC> const void* fast_fit_kernel(bool vreg, bool pipe);  // compile-time strides; pipe: pipelined schedule

// Kernel for a launch of fits with C classes, padded width Hs, padded feature count dp;
// vreg: second moments of W1 in registers.  Null when C is out of range.
const void* fit_kernel_for(int C, int Hs, int dp, bool vreg, bool pipe = false);

}  // namespace bbo
