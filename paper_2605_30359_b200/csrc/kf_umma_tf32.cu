// Launchers of the fp32 "3xTF32" chain: operand split prepass and the tensor-core kernel.
#include "kf_internal.h"
#include "kf_tf32.cuh"

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

}  // namespace kf
