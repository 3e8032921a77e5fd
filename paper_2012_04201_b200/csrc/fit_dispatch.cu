// Run-time dispatch over the class count to the per-class translation units.
#include "fit_launch.h"

namespace bbo {

#define BBO_DECLARE(N) \
  template <> cudaError_t launch_fit_ct<N>(const FitArgs&, bool, int, int, size_t, cudaStream_t);
BBO_DECLARE(1) BBO_DECLARE(2) BBO_DECLARE(3) BBO_DECLARE(4) BBO_DECLARE(5) BBO_DECLARE(6) BBO_DECLARE(7)
BBO_DECLARE(8) BBO_DECLARE(9) BBO_DECLARE(10) BBO_DECLARE(11) BBO_DECLARE(12) BBO_DECLARE(13)
BBO_DECLARE(14) BBO_DECLARE(15) BBO_DECLARE(16)
#undef BBO_DECLARE

cudaError_t launch_fit(int C, const FitArgs& a, bool vreg, int threads, int grid, size_t smem, cudaStream_t s) {
  switch (C) {
#define BBO_CASE(N) case N: return launch_fit_ct<N>(a, vreg, threads, grid, smem, s);
    BBO_CASE(1) BBO_CASE(2) BBO_CASE(3) BBO_CASE(4) BBO_CASE(5) BBO_CASE(6) BBO_CASE(7) BBO_CASE(8)
    BBO_CASE(9) BBO_CASE(10) BBO_CASE(11) BBO_CASE(12) BBO_CASE(13) BBO_CASE(14) BBO_CASE(15) BBO_CASE(16)
#undef BBO_CASE
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace bbo
