// Instantiations of the cluster softmax: 64-column tiles, the column tiles of a row block held
// by the CTAs of one cluster, (maximum, sum) pairs exchanged through distributed shared memory.
#include "kf_internal.h"

namespace kf {

cudaError_t launch_umma_softmax_cluster(int bn, int act, int out_dt, const UmmaMaps& tm, const UmmaParams& p,
                                        int row_blocks, cudaStream_t st) {
  cudaError_t e = cudaErrorInvalidValue;
  dispatch_act(act, [&](auto A) {
    constexpr int ACT = decltype(A)::value;
    if (bn == 128) {       // 128-column tiles, clusters of 2..8 (bf16 output)
      e = launch_umma_instance<128, EPI_SOFTMAX_CL, ACT, __nv_bfloat16>(tm, p, row_blocks, st, p.gn_cluster);
      return;
    }
    if (out_dt == DT_BF16)
      e = launch_umma_instance<kRowReduceNarrowBN, EPI_SOFTMAX_CL, ACT, __nv_bfloat16>(tm, p, row_blocks, st, p.gn_cluster);
    else
      e = launch_umma_instance<kRowReduceNarrowBN, EPI_SOFTMAX_CL, ACT, float>(tm, p, row_blocks, st, p.gn_cluster);
  });
  return e;
}

}  // namespace kf
