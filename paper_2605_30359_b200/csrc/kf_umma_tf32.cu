// Launchers of the fp32 "3xTF32" kernels: operand split prepasses, the GEMM chain and the
// 3x3 convolution.
#include "kf_internal.h"
#include "kf_tf32_conv.cuh"

namespace kf {

cudaError_t launch_tf32_split(long long rows, int K, int kp, const float* in, long long ld, float* hi,
                              float* lo, cudaStream_t st) {
  const long long total = rows * (kp / 4);
  long long blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;          // grid-stride: a few waves of 256 threads
  const int vec_in = (reinterpret_cast<uintptr_t>(in) % 16 == 0 && ld % 4 == 0) ? 1 : 0;
  tf32_split_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(rows, K, kp, in, ld, vec_in, hi, lo);
  return cudaGetLastError();
}

cudaError_t launch_tf32_chain(int bn, const CUtensorMap& ah, const CUtensorMap& al,
                              const CUtensorMap& bh, const CUtensorMap& bl, const Tf32Params& p,
                              int grid, cudaStream_t st) {
  if (bn == 256) return launch_tf32_instance<256>(ah, al, bh, bl, p, grid, st);
  if (bn == 128) return launch_tf32_instance<128>(ah, al, bh, bl, p, grid, st);
  return cudaErrorInvalidValue;
}

cudaError_t launch_conv_prep_tf32(int Nb, int Cin, int Cp, long long hw, int Cout, const float* x,
                                  const float* w, float* xh, float* xl, float* wh, float* wl,
                                  cudaStream_t st) {
  const long long x_items = static_cast<long long>(Nb) * hw * (Cp / 4);
  const long long total = x_items + 9ll * Cout * Cp;
  const long long grid = (total + 255) / 256;
  if (grid > 0x7fffffffLL) return cudaErrorInvalidValue;
  conv_prep_tf32_kernel<<<static_cast<unsigned>(grid), 256, 0, st>>>(Nb, Cin, Cp, hw, Cout, x, w, xh, xl,
                                                                     wh, wl, x_items);
  return cudaGetLastError();
}

cudaError_t launch_tf32_conv(int bn, const CUtensorMap& ah, const CUtensorMap& al, const CUtensorMap& bh,
                             const CUtensorMap& bl, const Tf32ConvParams& p, int grid, cudaStream_t st) {
  if (bn == 256) return launch_tf32_conv_instance<256>(ah, al, bh, bl, p, grid, st);
  if (bn == 128) return launch_tf32_conv_instance<128>(ah, al, bh, bl, p, grid, st);
  return cudaErrorInvalidValue;
}

}  // namespace kf
