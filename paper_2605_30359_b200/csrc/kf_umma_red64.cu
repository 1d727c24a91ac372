// Instantiations of the softmax first pass with 64-column tiles (one-wave problems: more CTAs,
// and an epilogue of two pieces instead of eight).
#include "kf_internal.h"

namespace kf {

cudaError_t launch_umma_softmax_narrow(int act, int out_dt, const UmmaMaps& tm, const UmmaParams& p,
                                       int grid, cudaStream_t st) {
  cudaError_t e = cudaErrorInvalidValue;
  dispatch_act(act, [&](auto A) {
    constexpr int ACT = decltype(A)::value;
    if (out_dt == DT_BF16) e = launch_umma_instance<kRowReduceNarrowBN, EPI_SOFTMAX, ACT, __nv_bfloat16>(tm, p, grid, st);
    else e = launch_umma_instance<kRowReduceNarrowBN, EPI_SOFTMAX, ACT, float>(tm, p, grid, st);
  });
  return e;
}

}  // namespace kf
