// Instantiations of the tensor-core kernel with the elementwise epilogue
// Y = scale*act(XW^T + b) + R, one per activation, tile width and CTA grouping.
#include "kf_internal.h"

namespace kf {

cudaError_t launch_umma_elementwise(int bn, int act, int pair, const UmmaMaps& tm,
                                    const UmmaParams& p, int grid, cudaStream_t st) {
  cudaError_t e = cudaErrorInvalidValue;
  dispatch_act(act, [&](auto A) {
    constexpr int ACT = decltype(A)::value;
    if (pair) {
      if (bn == 256) e = launch_umma_instance<256, EPI_ELEMENTWISE, ACT, __nv_bfloat16, true>(tm, p, grid, st);
    } else {
      if (bn == 256) e = launch_umma_instance<256, EPI_ELEMENTWISE, ACT, __nv_bfloat16>(tm, p, grid, st);
      else if (bn == 128) e = launch_umma_instance<128, EPI_ELEMENTWISE, ACT, __nv_bfloat16>(tm, p, grid, st);
      else if (bn == 64) e = launch_umma_instance<64, EPI_ELEMENTWISE, ACT, __nv_bfloat16>(tm, p, grid, st);
      else if (bn == 32) e = launch_umma_instance<32, EPI_ELEMENTWISE, ACT, __nv_bfloat16>(tm, p, grid, st);
    }
  });
  return e;
}

}  // namespace kf
