// Instantiations of the tensor-core kernel with the softmax first-pass epilogue
// (numerators + per-tile (max, sum) statistics).
#include "kf_internal.h"

namespace kf {

cudaError_t launch_umma_softmax(int bn, int act, int out_dt, int pair, const UmmaMaps& tm,
                                const UmmaParams& p, int grid, cudaStream_t st) {
  if (bn == kRowReduceNarrowBN) return launch_umma_softmax_narrow(act, out_dt, tm, p, grid, st);
  cudaError_t e = cudaErrorInvalidValue;
  dispatch_act(act, [&](auto A) {
    constexpr int ACT = decltype(A)::value;
    if (pair) {
      if (out_dt == DT_BF16) e = launch_umma_instance<kRowReduceBN, EPI_SOFTMAX, ACT, __nv_bfloat16, true>(tm, p, grid, st);
      else e = launch_umma_instance<kRowReduceBN, EPI_SOFTMAX, ACT, float, true>(tm, p, grid, st);
    } else {
      if (out_dt == DT_BF16) e = launch_umma_instance<kRowReduceBN, EPI_SOFTMAX, ACT, __nv_bfloat16>(tm, p, grid, st);
      else e = launch_umma_instance<kRowReduceBN, EPI_SOFTMAX, ACT, float>(tm, p, grid, st);
    }
  });
  return e;
}

}  // namespace kf
