// Instantiations of the implicit-GEMM 3x3 convolution with GroupNorm finished inside the epilogue:
// the CTAs that hold one image's tiles form a cluster and exchange the group statistics through
// distributed shared memory.
#include "kf_internal.h"

namespace kf {

cudaError_t launch_umma_conv_gn(int bn, int act, const UmmaMaps& tm, const UmmaParams& p, int images,
                                cudaStream_t st) {
  cudaError_t e = cudaErrorInvalidValue;
  dispatch_act(act, [&](auto A) {
    constexpr int ACT = decltype(A)::value;
    if (bn == 128)
      e = launch_umma_instance<128, EPI_CONV_GN, ACT, __nv_bfloat16>(tm, p, images, st, p.gn_cluster);
    else if (bn == 256)
      e = launch_umma_instance<256, EPI_CONV_GN, ACT, __nv_bfloat16>(tm, p, images, st, p.gn_cluster);
  });
  return e;
}

}  // namespace kf
