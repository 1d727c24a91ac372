// Instantiations of the tensor-core kernel as an implicit-GEMM 3x3 convolution
// (A tiles fetched per tap from the NHWC copy with out-of-image zero fill).
#include "kf_internal.h"

namespace kf {

cudaError_t launch_umma_conv(int bn, int act, const CUtensorMap& a, const CUtensorMap& b,
                             const UmmaParams& p, int grid, cudaStream_t st) {
  cudaError_t e = cudaErrorInvalidValue;
  dispatch_act(act, [&](auto A) {
    constexpr int ACT = decltype(A)::value;
    if (bn == 64) e = launch_umma_instance<64, EPI_CONV, ACT, __nv_bfloat16>(a, b, p, grid, st);
    else if (bn == 128) e = launch_umma_instance<128, EPI_CONV, ACT, __nv_bfloat16>(a, b, p, grid, st);
    else if (bn == 256) e = launch_umma_instance<256, EPI_CONV, ACT, __nv_bfloat16>(a, b, p, grid, st);
  });
  return e;
}

}  // namespace kf
