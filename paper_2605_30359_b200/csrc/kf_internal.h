// kf_internal.h -- host-side launcher interface between the C ABI (kf_api.cu) and the files
// that instantiate the kernels.  Every launcher enqueues on `st` and returns the launch's
// cudaError_t; none synchronises.
#pragma once
#include <cstdlib>
#include <mutex>

#include <cuda.h>
#include <cuda_runtime.h>

#include "kf_umma.cuh"

namespace kf {

// The four tensor maps of one tensor-core launch: A and B operands, residual in, output out
// (unused ones are copies of a valid map; the kernel never touches them).
struct UmmaMaps {
  CUtensorMap a, b, r, y;
};

// tensor-core chains (bf16)
// pair != 0: CTA-pair kernel (256-row tiles, `grid` = number of pairs, p.tiles_m counts 256-row
// tiles); otherwise one CTA per 128-row tile
cudaError_t launch_umma_elementwise(int bn, int act, int pair, const UmmaMaps& tm,
                                    const UmmaParams& p, int grid, cudaStream_t st);
cudaError_t launch_umma_softmax(int bn, int act, int out_dt, int pair, const UmmaMaps& tm,
                                const UmmaParams& p, int grid, cudaStream_t st);
cudaError_t launch_umma_softmax_narrow(int act, int out_dt, const UmmaMaps& tm, const UmmaParams& p,
                                       int grid, cudaStream_t st);
// the one-kernel softmax of wide rows: per-row (maximum, sum) exchanged through global memory,
// cooperative launch (bf16 out, 256-column tiles)
cudaError_t launch_umma_softmax_gx(int act, int pair, const UmmaMaps& tm, const UmmaParams& p, int grid,
                                   cudaStream_t st);
cudaError_t launch_umma_rowsum(int act, int pair, const UmmaMaps& tm, const UmmaParams& p,
                               int grid, cudaStream_t st);
cudaError_t launch_umma_conv(int bn, int act, const UmmaMaps& tm, const UmmaParams& p, int grid,
                             cudaStream_t st);
// the cluster form with GroupNorm in the epilogue: `images` units, p.gn_cluster CTAs per cluster
// the cluster softmax: `row_blocks` units, p.gn_cluster (= column tiles per row) CTAs per cluster
cudaError_t launch_umma_softmax_cluster(int bn, int act, int out_dt, const UmmaMaps& tm, const UmmaParams& p,
                                        int row_blocks, cudaStream_t st);
cudaError_t launch_umma_conv_gn(int bn, int act, const UmmaMaps& tm, const UmmaParams& p, int images,
                                cudaStream_t st);
// the same chain on every SM: statistics exchanged through global memory, cooperative launch of
// `grid` CTAs (at most one per SM)
cudaError_t launch_umma_conv_gnx(int bn, int act, const UmmaMaps& tm, const UmmaParams& p, int grid,
                                 cudaStream_t st);
constexpr int kRowReduceBN = 256;   // tile width of the row-reduce first pass
constexpr int kRowReduceNarrowBN = 64;   // ... of the softmax first pass of one-wave problems

// second passes of the tensor-core row reductions
cudaError_t launch_softmax_finalize(int out_dt, int M, int N, int bn, int tiles_n, const float* partial,
                                    void* out, long long ldo, int vec_ok, cudaStream_t st, bool overlap);
cudaError_t launch_rowsum_finalize(int M, int tiles_n, const float* partial, float* out, float scale,
                                   cudaStream_t st, bool overlap);
cudaError_t launch_rowstat_finalize(int red, int M, int slices, const float* partial, float* out,
                                    cudaStream_t st, bool overlap);

// scalar chains (fp32, and bf16 shapes the tensor-core kernels do not take)
cudaError_t launch_simt_gemm(int dt, int mode, int act, int M, int N, int K, const void* X,
                             long long ldx, const void* W, long long ldw, const void* bias,
                             float scale, const void* R, long long ldr, void* out, long long ldo,
                             cudaStream_t st);
cudaError_t launch_row_softmax(int out_dt, int M, int N, const float* A, long long lda, void* out,
                               long long ldo, cudaStream_t st);
cudaError_t launch_row_reduce(int red, int M, int N, const float* A, long long lda, float* out,
                              cudaStream_t st);

// convolution helpers
// (also sets `ones_bytes` bytes at `ones` to 0xff: the empty exchange buffer of EPI_CONV_GNX)
cudaError_t launch_conv_prep(int Nb, int Cin, int Cp, int H, int Wd, int Cout, const void* x,
                             const void* w, void* xt, void* wr, cudaStream_t st, void* ones = nullptr,
                             size_t ones_bytes = 0);
cudaError_t launch_conv_direct(int dt, int act, int Nb, int Cin, int H, int Wd, int Cout,
                               const void* x, const void* w, const void* bias, void* y,
                               cudaStream_t st);
cudaError_t launch_groupnorm(int dt, int Nb, int Cout, int groups, long long hw, float eps,
                             const void* gamma, const void* beta, void* y, cudaStream_t st);
// GroupNorm from the per-tile channel statistics the convolution epilogue wrote (bf16 only)
cudaError_t launch_groupnorm_apply(int Nb, int Cout, int groups, long long hw, int tiles_per_image,
                                   float eps, const float* stats, const void* gamma,
                                   const void* beta, void* y, cudaStream_t st, bool overlap);

// GroupNorm over column groups of an fp32 matrix + activation (scalar path of kf_gemm_groupnorm)
cudaError_t launch_row_groupnorm(int dt, int M, int N, int gs, float eps, const float* A, long long lda,
                                 const void* gamma, const void* beta, int act, void* Y, long long ldy,
                                 cudaStream_t st);

cudaError_t launch_row_groupnorm_inplace(int M, int N, int gs, float eps, const void* gamma,
                                         const void* beta, int act, void* Y, long long ldy,
                                         cudaStream_t st);
cudaError_t launch_row_groupnorm_apply(int M, int N, int gs, int tiles_n, float eps, const float* stats,
                                       const void* gamma, const void* beta, int act, void* Y,
                                       long long ldy, cudaStream_t st, bool overlap);

// max / average pooling (kernel = stride = pool) of an NCHW tensor
cudaError_t launch_pool2d(int dt, long long planes, int H, int Wd, int pool, int kind, const void* in,
                          void* out, cudaStream_t st);

// global average pooling: from the convolution's statistics, or from a stored NCHW tensor
cudaError_t launch_gap_finalize(int Nb, int Cout, int parts, long long hw, const float* stats, float* out,
                                cudaStream_t st, bool overlap);
cudaError_t launch_plane_mean(int dt, long long rows, long long len, const void* in, float* out,
                              cudaStream_t st);

// bf16 operand repack (any pitch / alignment -> dense rows padded to 8 columns)
cudaError_t launch_pad_rows_bf16(long long rows, int K, int kp, const void* in, long long ld, void* out,
                                 cudaStream_t st);

// fp32 chain on the tensor cores (3xTF32): split prepass and GEMM kernel
struct Tf32Params {
  int M, N, K;
  int tiles_m, tiles_n, num_tiles, k_blocks;
  const float* bias;             // [N] or null
  const float* R;                // [M, ldr] or null
  long long ldr;
  float* out;                    // [M, ldo]
  long long ldo;
  float scale;
  int act;
  int vec_ok;                    // rows of out (and R) start on 16 bytes
  uint32_t* status;
};
struct Tf32ConvParams {
  int Cout, H, Wd;
  int tiles_m, tiles_n, num_tiles;     // output-channel tiles, pixel tiles, both
  int tiles_per_image, rows_per_tile, w_segs, tile_px;
  int kb_per_tap, k_blocks;            // K blocks of 16 channels per tap; 9 * kb_per_tap
  const float* bias;                   // [Cout] or null
  float* out;                          // NCHW
  int act;
  int vec_ok;                          // out is 16-byte aligned and H*W is a multiple of 4
  uint32_t* status;
};
cudaError_t launch_conv_prep_tf32(int Nb, int Cin, int Cp, long long hw, int Cout, const float* x,
                                  const float* w, float* xh, float* xl, float* wh, float* wl,
                                  cudaStream_t st);
cudaError_t launch_tf32_conv(int bn, const CUtensorMap& ah, const CUtensorMap& al, const CUtensorMap& bh,
                             const CUtensorMap& bl, const Tf32ConvParams& p, int grid, cudaStream_t st);
cudaError_t launch_tf32_split(long long rows, int K, int kp, const float* in, long long ld, float* hi,
                              float* lo, cudaStream_t st);
cudaError_t launch_tf32_chain(int bn, const CUtensorMap& ah, const CUtensorMap& al,
                              const CUtensorMap& bh, const CUtensorMap& bl, const Tf32Params& p,
                              int grid, cudaStream_t st);

// split-K cluster kernel of the elementwise chain: bn in {128, 256}, s CTAs per tile
cudaError_t launch_umma_splitk(int bn, int s, int act, const UmmaMaps& tm, const UmmaParams& p,
                               cudaStream_t st, bool two_per_sm = false);

// softmax over channels + pool x pool max-pool of an NCHW tensor (pool <= 4)
cudaError_t launch_channel_softmax_pool(int dt, int Nb, int C, int H, int Wd, int pool, const void* a,
                                        void* y, cudaStream_t st);

// Generic launcher for one instantiation of the tensor-core kernel.
// `grid` counts scheduled CTAs for the single-CTA kernel and CTA PAIRS for the pair kernel
// (which launches 2*grid CTAs in clusters of two).
template <int BN, int EPI, int ACT, typename OutT, bool CTA2 = false>
// `cluster` > 0 (EPI_CONV_GN): `grid` counts the images; the launch uses as many clusters of that
// many CTAs as can be resident at once (at most one per image).
// `coop`: a cooperative launch (every CTA of the grid resident together; `grid` must not exceed
// what the device holds at once), for the kernels whose CTAs wait for one another.
inline cudaError_t launch_umma_instance(const UmmaMaps& tm, const UmmaParams& p, int grid,
                                        cudaStream_t st, int cluster = 0, bool coop = false) {
  using C = UmmaCfg<BN, EPI, CTA2>;
  constexpr int smem = C::kTotal;
  static_assert(smem <= kMaxDynSmem, "shared-memory plan exceeds the per-CTA limit");
  auto kern = umma_chain_kernel<BN, EPI, ACT, OutT, CTA2>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  if (cluster > 0) {
    if (cluster > 8) {
      e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
      if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cluster, 1, 1);
    cfg.blockDim = dim3(num_threads(EPI, BN, CTA2), 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // clusters of this size that fit on the device: asked once per device and kernel instance
    static std::mutex mu;
    static int resident[64][17] = {};
    int dev = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    int fit = 0;
    {
      std::lock_guard<std::mutex> lk(mu);
      if (resident[dev][cluster] == 0) {
        int n = 0;
        e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
        if (e != cudaSuccess) return e;
        if (n < 1) return cudaErrorInvalidConfiguration;
        resident[dev][cluster] = n;
      }
      fit = resident[dev][cluster];
    }
    const int clusters = grid < fit ? grid : fit;
    cfg.gridDim = dim3(clusters * cluster, 1, 1);
    static const bool pdl_cl = getenv("KF_NO_PDL") == nullptr;
    cfg.numAttrs = pdl_cl ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kern, tm.a, tm.b, tm.r, tm.y, p);
  }
  if constexpr (CTA2) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * grid, 1, 1);
    cfg.blockDim = dim3(num_threads(EPI, BN, CTA2), 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeCooperative;
    attr[1].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = coop ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kern, tm.a, tm.b, tm.r, tm.y, p);
  } else {
    // programmatic dependent launch: with few CTAs the next launch of the stream starts on the
    // idle SMs and has its prologue behind it when this kernel ends (see griddep_wait)
    static const bool pdl = getenv("KF_NO_PDL") == nullptr;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(num_threads(EPI, BN, CTA2), 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (coop) {
      attr[0].id = cudaLaunchAttributeCooperative;
      attr[0].val.cooperative = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      return cudaLaunchKernelEx(&cfg, kern, tm.a, tm.b, tm.r, tm.y, p);
    }
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, tm.a, tm.b, tm.r, tm.y, p);
  }
}

}  // namespace kf
