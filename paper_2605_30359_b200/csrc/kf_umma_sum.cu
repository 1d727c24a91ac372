// Instantiations of the tensor-core kernel with the row-sum first-pass epilogue
// (per-tile sums of act(XW^T + b) along each row).
#include "kf_internal.h"

namespace kf {

cudaError_t launch_umma_rowsum(int act, int pair, const UmmaMaps& tm, const UmmaParams& p,
                               int grid, cudaStream_t st) {
  cudaError_t e = cudaErrorInvalidValue;
  dispatch_act(act, [&](auto A) {
    constexpr int ACT = decltype(A)::value;
    if (pair) e = launch_umma_instance<kRowReduceBN, EPI_ROWSUM, ACT, float, true>(tm, p, grid, st);
    else e = launch_umma_instance<kRowReduceBN, EPI_ROWSUM, ACT, float>(tm, p, grid, st);
  });
  return e;
}

}  // namespace kf
