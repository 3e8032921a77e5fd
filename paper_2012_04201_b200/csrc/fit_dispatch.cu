// Run-time lookup of the fit kernel instance (see fit_launch.h).
#include "fit_launch.h"

namespace bbo {

#define BBO_DECLARE(N) template <> const void* generic_fit_kernel<N>();
BBO_DECLARE(1) BBO_DECLARE(2) BBO_DECLARE(3) BBO_DECLARE(4) BBO_DECLARE(5) BBO_DECLARE(6) BBO_DECLARE(7)
BBO_DECLARE(8) BBO_DECLARE(9) BBO_DECLARE(10) BBO_DECLARE(11) BBO_DECLARE(12) BBO_DECLARE(13)
BBO_DECLARE(14) BBO_DECLARE(15) BBO_DECLARE(16)
#undef BBO_DECLARE
#define BBO_DECLARE(N) template <> const void* fast_fit_kernel<N>(bool);
BBO_DECLARE(56) BBO_DECLARE(64) BBO_DECLARE(72) BBO_DECLARE(80) BBO_DECLARE(88) BBO_DECLARE(96)
BBO_DECLARE(104) BBO_DECLARE(112) BBO_DECLARE(120) BBO_DECLARE(128) BBO_DECLARE(136) BBO_DECLARE(144)
BBO_DECLARE(152) BBO_DECLARE(160) BBO_DECLARE(168) BBO_DECLARE(176) BBO_DECLARE(184) BBO_DECLARE(192)
BBO_DECLARE(200)
#undef BBO_DECLARE

const void* fit_kernel_for(int C, int Hs, int dp, bool pipe) {
  if (C == kFastClasses && dp == kFastDp && Hs >= kFastHsMin && Hs <= kFastHsMax && Hs % 8 == 0) {
    switch (Hs) {
#define BBO_CASE(N) case N: return fast_fit_kernel<N>(pipe);
      BBO_CASE(56) BBO_CASE(64) BBO_CASE(72) BBO_CASE(80) BBO_CASE(88) BBO_CASE(96) BBO_CASE(104)
      BBO_CASE(112) BBO_CASE(120) BBO_CASE(128) BBO_CASE(136) BBO_CASE(144) BBO_CASE(152) BBO_CASE(160)
      BBO_CASE(168) BBO_CASE(176) BBO_CASE(184) BBO_CASE(192) BBO_CASE(200)
#undef BBO_CASE
      default: break;
    }
  }
  if (pipe) return nullptr;  // the run-time-stride kernels have no pipelined variant
  switch (C) {
#define BBO_CASE(N) case N: return generic_fit_kernel<N>();
    BBO_CASE(1) BBO_CASE(2) BBO_CASE(3) BBO_CASE(4) BBO_CASE(5) BBO_CASE(6) BBO_CASE(7) BBO_CASE(8)
    BBO_CASE(9) BBO_CASE(10) BBO_CASE(11) BBO_CASE(12) BBO_CASE(13) BBO_CASE(14) BBO_CASE(15) BBO_CASE(16)
#undef BBO_CASE
    default: return nullptr;
  }
}

}  // namespace bbo
