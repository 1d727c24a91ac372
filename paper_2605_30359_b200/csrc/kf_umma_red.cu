// Instantiations of the tensor-core kernel with the row-reduction first-pass epilogues
// (softmax numerators + per-tile statistics; per-tile row sums).
#include "kf_internal.h"

namespace kf {

cudaError_t launch_umma_softmax(int act, int out_dt, const UmmaMaps& tm, const UmmaParams& p,
                                int grid, cudaStream_t st) {
  cudaError_t e = cudaErrorInvalidValue;
  dispatch_act(act, [&](auto A) {
    constexpr int ACT = decltype(A)::value;
    if (out_dt == DT_BF16) e = launch_umma_instance<kRowReduceBN, EPI_SOFTMAX, ACT, __nv_bfloat16>(tm, p, grid, st);
    else e = launch_umma_instance<kRowReduceBN, EPI_SOFTMAX, ACT, float>(tm, p, grid, st);
  });
  return e;
}

cudaError_t launch_umma_rowsum(int act, const UmmaMaps& tm, const UmmaParams& p, int grid,
                               cudaStream_t st) {
  cudaError_t e = cudaErrorInvalidValue;
  dispatch_act(act, [&](auto A) {
    constexpr int ACT = decltype(A)::value;
    e = launch_umma_instance<kRowReduceBN, EPI_ROWSUM, ACT, float>(tm, p, grid, st);
  });
  return e;
}

}  // namespace kf
