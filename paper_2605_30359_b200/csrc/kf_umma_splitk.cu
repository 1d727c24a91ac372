// Instantiations of the split-K cluster kernel (tile width x cluster size).
#include "kf_internal.h"
#include "kf_splitk.cuh"

namespace kf {

cudaError_t launch_umma_splitk(int bn, int s, int act, const UmmaMaps& tm, const UmmaParams& p,
                               cudaStream_t st, bool two_per_sm) {
  if (bn == 128 && s == 4 && two_per_sm) return launch_splitk_instance<128, 4, 3>(tm.a, tm.b, p, act, st);
  if (bn == 256 && s == 8) return launch_splitk_instance<256, 8>(tm.a, tm.b, p, act, st);
  if (bn == 256 && s == 4) return launch_splitk_instance<256, 4>(tm.a, tm.b, p, act, st);
  if (bn == 128 && s == 4) return launch_splitk_instance<128, 4>(tm.a, tm.b, p, act, st);
  if (bn == 128 && s == 2) return launch_splitk_instance<128, 2>(tm.a, tm.b, p, act, st);
  return cudaErrorInvalidValue;
}

}  // namespace kf
