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
constexpr int kPipeHsMin = 184;
inline int pipe_extra_warps(int Hs) { return (Hs + 31) / 32 * 32 + 64 <= kMaxFitThreads ? 2 : 1; }

// Resident CTAs per SM the compile-time-width instances are built for: the launch bound caps
// their registers at 65,536 / (CTAs x threads), and shared memory admits that many (the row
// buffers and parameters of a fit of that width, moments of W1 in tensor memory).  Four fits per
// SM up to width 64 and two up to 128 keep about 250 registers per thread.  Widths 136..176 (five
// or six warps) also run two per SM, at 168 registers with the lean forms of the tile loops
// (fit_kernel.cuh) and about two hundred bytes of spills: a lone CTA is then slower, but two of
// them share an SM at a cost of 10 %, which beats one CTA with the pipelined schedule.  Three CTAs of widths 72..96 at 168 registers were 12 %
// slower than two at 250.  Widths from 184 sit alone on their SM (shared memory) and take the
// pipelined schedule.
constexpr int fast_threads(int Hs) { return (Hs + 31) / 32 * 32; }
constexpr int fast_min_blocks(int Hs) { return fast_threads(Hs) <= 64 ? 4 : (Hs <= 176 ? 2 : 1); }

template <int CT> const void* generic_fit_kernel();            // run-time strides
template <int HSC> const void* fast_fit_kernel(bool pipe);     // compile-time strides; pipe: pipelined schedule

// Kernel for a launch of fits with C classes, padded width Hs, padded feature count dp.
// Null when C is out of range or the pipelined schedule is not built for the shape.
const void* fit_kernel_for(int C, int Hs, int dp, bool pipe = false);

}  // namespace bbo
