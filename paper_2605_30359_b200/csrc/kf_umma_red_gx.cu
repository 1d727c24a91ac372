// Instantiations of the GEMM + row softmax in one kernel for rows of several 256-column tiles: the
// tiles of a row block are held by neighbouring CTAs of a cooperative grid, which exchange per-row
// (maximum, sum) through global memory.
#include "kf_internal.h"

namespace kf {

cudaError_t launch_umma_softmax_gx(int act, int pair, const UmmaMaps& tm, const UmmaParams& p, int grid,
                                   cudaStream_t st) {
  cudaError_t e = cudaErrorInvalidValue;
  dispatch_act(act, [&](auto A) {
    constexpr int ACT = decltype(A)::value;
    if (pair) e = launch_umma_instance<kRowReduceBN, EPI_SOFTMAX_GX, ACT, __nv_bfloat16, true>(tm, p, grid, st, 0, true);
    else e = launch_umma_instance<kRowReduceBN, EPI_SOFTMAX_GX, ACT, __nv_bfloat16>(tm, p, grid, st, 0, true);
  });
  return e;
}

}  // namespace kf
