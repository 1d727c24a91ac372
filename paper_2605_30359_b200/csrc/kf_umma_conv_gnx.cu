// Instantiations of the implicit-GEMM 3x3 convolution with GroupNorm finished inside the epilogue
// on every SM: the tiles of an image are held by neighbouring CTAs of a cooperative grid, which
// exchange the group statistics through global memory.
#include "kf_internal.h"

namespace kf {

cudaError_t launch_umma_conv_gnx(int bn, int act, const UmmaMaps& tm, const UmmaParams& p, int grid,
                                 cudaStream_t st) {
  cudaError_t e = cudaErrorInvalidValue;
  dispatch_act(act, [&](auto A) {
    constexpr int ACT = decltype(A)::value;
    if (bn == 128)
      e = launch_umma_instance<128, EPI_CONV_GNX, ACT, __nv_bfloat16>(tm, p, grid, st, 0, true);
    else if (bn == 256)
      e = launch_umma_instance<256, EPI_CONV_GNX, ACT, __nv_bfloat16>(tm, p, grid, st, 0, true);
  });
  return e;
}

}  // namespace kf
