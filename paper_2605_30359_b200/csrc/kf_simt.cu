// Launchers for the CUDA-core kernels.
#include <type_traits>
#include <cstdlib>
#include "kf_internal.h"
#include "kf_simt.cuh"

namespace kf {

// Launch of a second-pass kernel.  With `overlap` it is launched with programmatic stream
// serialization: it may be scheduled while the kernel before it (which has called
// griddepcontrol.launch_dependents) is still running, and waits in its first instruction
// (griddep_wait) until that kernel has completed.  That saves 1.5-2 us when the first pass left
// SMs idle (a partial wave).  After a first pass that filled every SM it was measured neutral to
// harmful (the waiting CTAs were released 5-7 us after the first pass ended: 4096x4096x1024
// row sum 34.3 -> 39.2 us, conv + channel softmax + pool 148 -> 155 us), so callers pass
// overlap = false there and the launch is an ordinary one.
template <typename... KArgs, typename... Args>
static cudaError_t launch_after(bool overlap, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                cudaStream_t st, Args... args) {
  static const bool pdl = getenv("KF_NO_PDL") == nullptr;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (pdl && overlap) ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}


template <typename T>
static cudaError_t simt_gemm_t(int mode, int act, int M, int N, int K, const void* X,
                               long long ldx, const void* W, long long ldw, const void* bias,
                               float scale, const void* R, long long ldr, void* out, long long ldo,
                               cudaStream_t st) {
  // 16 x 16 tiles when 32 x 32 tiles would occupy less than half of a B200's SMs
  const bool small = static_cast<long long>((M + 31) / 32) * ((N + 31) / 32) < 74;
  const int t = small ? 16 : 32;
  const dim3 grid((M + t - 1) / t, (N + t - 1) / t), block(256);   // rows on x: up to 2^31-1 tiles
  if (grid.y > 65535u) return cudaErrorInvalidValue;
  cudaError_t err = cudaSuccess;
  bool ok = dispatch_act(act, [&](auto A) {
    constexpr int ACT = decltype(A)::value;
    auto go = [&](auto kern) {
      err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSimtSmemBytes);
      if (err != cudaSuccess) return;
      static const bool pdl = getenv("KF_NO_PDL") == nullptr;
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = grid;
      cfg.blockDim = block;
      cfg.dynamicSmemBytes = kSimtSmemBytes;
      cfg.stream = st;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[0].val.programmaticStreamSerializationAllowed = 1;
      cfg.attrs = attr;
      cfg.numAttrs = pdl ? 1 : 0;
      err = cudaLaunchKernelEx(&cfg, kern, M, N, K, static_cast<const T*>(X), ldx, static_cast<const T*>(W), ldw,
                               static_cast<const T*>(bias), scale, static_cast<const T*>(R), ldr, out, ldo, act);
    };
    if (small) {
      if (mode == 0) go(simt_gemm_kernel<T, 0, ACT, 16, 16>);
      else go(simt_gemm_kernel<T, 1, ACT, 16, 16>);
    } else {
      if (mode == 0) go(simt_gemm_kernel<T, 0, ACT, 32, 32>);
      else go(simt_gemm_kernel<T, 1, ACT, 32, 32>);
    }
  });
  return ok ? err : cudaErrorInvalidValue;
}

cudaError_t launch_simt_gemm(int dt, int mode, int act, int M, int N, int K, const void* X,
                             long long ldx, const void* W, long long ldw, const void* bias,
                             float scale, const void* R, long long ldr, void* out, long long ldo,
                             cudaStream_t st) {
  if (dt == DT_F32)
    return simt_gemm_t<float>(mode, act, M, N, K, X, ldx, W, ldw, bias, scale, R, ldr, out, ldo, st);
  return simt_gemm_t<__nv_bfloat16>(mode, act, M, N, K, X, ldx, W, ldw, bias, scale, R, ldr, out, ldo, st);
}

cudaError_t launch_row_softmax(int out_dt, int M, int N, const float* A, long long lda, void* out,
                               long long ldo, cudaStream_t st) {
  if (out_dt == DT_F32)
    row_softmax_kernel<float><<<M, 256, 0, st>>>(N, A, lda, static_cast<float*>(out), ldo);
  else
    row_softmax_kernel<__nv_bfloat16><<<M, 256, 0, st>>>(N, A, lda, static_cast<__nv_bfloat16*>(out), ldo);
  return cudaGetLastError();
}

cudaError_t launch_row_reduce(int red, int M, int N, const float* A, long long lda, float* out,
                              cudaStream_t st) {
  row_reduce_kernel<<<M, 256, 0, st>>>(N, A, lda, out, red);
  return cudaGetLastError();
}

cudaError_t launch_softmax_finalize(int out_dt, int M, int N, int bn, int tiles_n, const float* partial,
                                    void* out, long long ldo, int vec_ok, cudaStream_t st, bool overlap) {
  int bn_shift = 0;                      // slices are powers of two (half a first-pass tile)
  while ((1 << bn_shift) < bn) ++bn_shift;
  if (tiles_n <= 32) {
    const unsigned grid = static_cast<unsigned>((M + 7) / 8);
    const float2* pw = reinterpret_cast<const float2*>(partial);
    if (out_dt == DT_F32)
      return launch_after(overlap, softmax_finalize_warp_kernel<float>, dim3(grid), dim3(256), 0, st, M, N, bn_shift,
                          tiles_n, pw, static_cast<float*>(out), ldo, vec_ok);
    return launch_after(overlap, softmax_finalize_warp_kernel<__nv_bfloat16>, dim3(grid), dim3(256), 0, st, M, N,
                        bn_shift, tiles_n, pw, static_cast<__nv_bfloat16*>(out), ldo, vec_ok);
  }
  const size_t smem = static_cast<size_t>(tiles_n) * sizeof(float);
  const float2* part = reinterpret_cast<const float2*>(partial);
  if (out_dt == DT_F32)
    return launch_after(overlap, softmax_finalize_kernel<float>, dim3(M), dim3(256), smem, st, N, bn_shift, tiles_n,
                        part, static_cast<float*>(out), ldo, vec_ok);
  return launch_after(overlap, softmax_finalize_kernel<__nv_bfloat16>, dim3(M), dim3(256), smem, st, N, bn_shift,
                      tiles_n, part, static_cast<__nv_bfloat16*>(out), ldo, vec_ok);
}

cudaError_t launch_rowsum_finalize(int M, int tiles_n, const float* partial, float* out, float scale,
                                   cudaStream_t st, bool overlap) {
  return launch_after(overlap, rowsum_finalize_kernel, dim3((M + 255) / 256), dim3(256), 0, st, M, tiles_n, partial, out,
                      scale);
}

cudaError_t launch_rowstat_finalize(int red, int M, int slices, const float* partial, float* out,
                                    cudaStream_t st, bool overlap) {
  return launch_after(overlap, rowstat_finalize_kernel, dim3((M + 255) / 256), dim3(256), 0, st, M, slices,
                      reinterpret_cast<const float2*>(partial), out, red);
}

cudaError_t launch_row_groupnorm(int dt, int M, int N, int gs, float eps, const float* A, long long lda,
                                 const void* gamma, const void* beta, int act, void* Y, long long ldy,
                                 cudaStream_t st) {
  if (dt == DT_F32)
    row_groupnorm_kernel<float, float><<<M, 256, 0, st>>>(N, gs, eps, A, lda, static_cast<const float*>(gamma),
                                                          static_cast<const float*>(beta), act,
                                                          static_cast<float*>(Y), ldy);
  else
    row_groupnorm_kernel<__nv_bfloat16, float><<<M, 256, 0, st>>>(
        N, gs, eps, A, lda, static_cast<const __nv_bfloat16*>(gamma),
        static_cast<const __nv_bfloat16*>(beta), act, static_cast<__nv_bfloat16*>(Y), ldy);
  return cudaGetLastError();
}

// in place on a bf16 matrix that holds z
cudaError_t launch_row_groupnorm_inplace(int M, int N, int gs, float eps, const void* gamma,
                                         const void* beta, int act, void* Y, long long ldy,
                                         cudaStream_t st) {
  __nv_bfloat16* y = static_cast<__nv_bfloat16*>(Y);
  row_groupnorm_kernel<__nv_bfloat16, __nv_bfloat16><<<M, 256, 0, st>>>(
      N, gs, eps, y, ldy, static_cast<const __nv_bfloat16*>(gamma), static_cast<const __nv_bfloat16*>(beta),
      act, y, ldy);
  return cudaGetLastError();
}

cudaError_t launch_row_groupnorm_apply(int M, int N, int gs, int tiles_n, float eps, const float* stats,
                                       const void* gamma, const void* beta, int act, void* Y,
                                       long long ldy, cudaStream_t st, bool overlap) {
  const size_t smem = static_cast<size_t>(N / gs) * sizeof(float2);
  return launch_after(overlap, row_groupnorm_apply_kernel, dim3(M), dim3(256), smem, st, N, gs, tiles_n, eps,
                      reinterpret_cast<const float2*>(stats), static_cast<const __nv_bfloat16*>(gamma),
                      static_cast<const __nv_bfloat16*>(beta), act, static_cast<__nv_bfloat16*>(Y), ldy);
}

cudaError_t launch_pool2d(int dt, long long planes, int H, int Wd, int pool, int kind, const void* in,
                          void* out, cudaStream_t st) {
  const long long total = planes * (H / pool) * (Wd / pool);
  if (total == 0) return cudaSuccess;
  const long long grid = (total + 255) / 256;
  if (grid > 0x7fffffffLL) return cudaErrorInvalidValue;
  if (dt == DT_F32)
    pool2d_kernel<float><<<static_cast<unsigned>(grid), 256, 0, st>>>(
        planes, H, Wd, pool, kind, static_cast<const float*>(in), static_cast<float*>(out));
  else
    pool2d_kernel<__nv_bfloat16><<<static_cast<unsigned>(grid), 256, 0, st>>>(
        planes, H, Wd, pool, kind, static_cast<const __nv_bfloat16*>(in), static_cast<__nv_bfloat16*>(out));
  return cudaGetLastError();
}

cudaError_t launch_gap_finalize(int Nb, int Cout, int parts, long long hw, const float* stats, float* out,
                                cudaStream_t st, bool overlap) {
  const long long total = static_cast<long long>(Nb) * Cout;
  return launch_after(overlap, gap_finalize_kernel, dim3(static_cast<unsigned>((total + 255) / 256)), dim3(256), 0, st, Nb,
                      Cout, parts, hw, reinterpret_cast<const float2*>(stats), out);
}

cudaError_t launch_plane_mean(int dt, long long rows, long long len, const void* in, float* out,
                              cudaStream_t st) {
  if (rows > 0x7fffffffLL) return cudaErrorInvalidValue;
  if (dt == DT_F32)
    plane_mean_kernel<float><<<static_cast<unsigned>(rows), 256, 0, st>>>(len, static_cast<const float*>(in), out);
  else
    plane_mean_kernel<__nv_bfloat16><<<static_cast<unsigned>(rows), 256, 0, st>>>(
        len, static_cast<const __nv_bfloat16*>(in), out);
  return cudaGetLastError();
}

cudaError_t launch_pad_rows_bf16(long long rows, int K, int kp, const void* in, long long ld, void* out,
                                 cudaStream_t st) {
  const long long total = rows * (kp / 8);
  long long blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  pad_rows_bf16_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(
      rows, K, kp, static_cast<const __nv_bfloat16*>(in), ld, static_cast<__nv_bfloat16*>(out));
  return cudaGetLastError();
}

cudaError_t launch_conv_prep(int Nb, int Cin, int Cp, int H, int Wd, int Cout, const void* x,
                             const void* w, void* xt, void* wr, cudaStream_t st, void* ones, size_t ones_bytes) {
  const __nv_bfloat16* xs = static_cast<const __nv_bfloat16*>(x);
  const __nv_bfloat16* ws = static_cast<const __nv_bfloat16*>(w);
  __nv_bfloat16* xd = static_cast<__nv_bfloat16*>(xt);
  __nv_bfloat16* wd = static_cast<__nv_bfloat16*>(wr);
  uint4* od = static_cast<uint4*>(ones);                    // (256-byte aligned, a multiple of 256 bytes)
  const long long ones16 = ones != nullptr ? static_cast<long long>(ones_bytes / 16) : 0;
  if (Cp == Cin && Cin % 8 == 0 && Wd % 8 == 0 && reinterpret_cast<uintptr_t>(x) % 16 == 0) {
    const long long x_blocks = static_cast<long long>(Nb) * H * (Cin / 8) * (Wd / 8);
    long long total = x_blocks + 9ll * Cout * Cin;
    if (total < ones16) total = ones16;
    const long long grid = (total + 255) / 256;
    if (grid > 0x7fffffffLL) return cudaErrorInvalidValue;
    conv_prep_kernel<<<static_cast<unsigned>(grid), 256, 0, st>>>(Nb, Cin, H, Wd, Cout, xs, ws, xd, wd,
                                                                  x_blocks, od, ones16);
  } else {
    const long long x_items = static_cast<long long>(Nb) * H * Wd * (Cp / 8);
    long long total = x_items + 9ll * Cout * Cp;
    if (total < ones16) total = ones16;
    const long long grid = (total + 255) / 256;
    if (grid > 0x7fffffffLL) return cudaErrorInvalidValue;
    conv_prep_general_kernel<<<static_cast<unsigned>(grid), 256, 0, st>>>(Nb, Cin, Cp, H, Wd, Cout, xs, ws,
                                                                          xd, wd, x_items, od, ones16);
  }
  return cudaGetLastError();
}

template <typename T>
static cudaError_t conv_direct_t(int act, int Nb, int Cin, int H, int Wd, int Cout, const void* x,
                                 const void* w, const void* bias, void* y, cudaStream_t st) {
  const long long total = static_cast<long long>(Nb) * Cout * H * Wd;
  const unsigned grid = static_cast<unsigned>((total + 255) / 256);
  bool ok = dispatch_act(act, [&](auto A) {
    constexpr int ACT = decltype(A)::value;
    conv_direct_kernel<T, ACT><<<grid, 256, 0, st>>>(Nb, Cin, H, Wd, Cout, static_cast<const T*>(x),
                                                     static_cast<const T*>(w),
                                                     static_cast<const T*>(bias),
                                                     static_cast<T*>(y), act);
  });
  return ok ? cudaGetLastError() : cudaErrorInvalidValue;
}

cudaError_t launch_conv_direct(int dt, int act, int Nb, int Cin, int H, int Wd, int Cout,
                               const void* x, const void* w, const void* bias, void* y,
                               cudaStream_t st) {
  if (dt == DT_F32) return conv_direct_t<float>(act, Nb, Cin, H, Wd, Cout, x, w, bias, y, st);
  return conv_direct_t<__nv_bfloat16>(act, Nb, Cin, H, Wd, Cout, x, w, bias, y, st);
}

cudaError_t launch_groupnorm(int dt, int Nb, int Cout, int groups, long long hw, float eps,
                             const void* gamma, const void* beta, void* y, cudaStream_t st) {
  const unsigned grid = static_cast<unsigned>(Nb) * static_cast<unsigned>(groups);
  if (dt == DT_F32)
    groupnorm_kernel<float><<<grid, 512, 0, st>>>(Cout, groups, hw, eps,
                                                  static_cast<const float*>(gamma),
                                                  static_cast<const float*>(beta),
                                                  static_cast<float*>(y));
  else
    groupnorm_kernel<__nv_bfloat16><<<grid, 512, 0, st>>>(
        Cout, groups, hw, eps, static_cast<const __nv_bfloat16*>(gamma),
        static_cast<const __nv_bfloat16*>(beta), static_cast<__nv_bfloat16*>(y));
  return cudaGetLastError();
}

cudaError_t launch_groupnorm_apply(int Nb, int Cout, int groups, long long hw, int tiles_per_image,
                                   float eps, const float* stats, const void* gamma,
                                   const void* beta, void* y, cudaStream_t st, bool overlap) {
  const unsigned grid = static_cast<unsigned>(Nb) * static_cast<unsigned>(groups);
  return launch_after(overlap, groupnorm_apply_kernel, dim3(grid), dim3(512), 0, st, Cout, groups, hw, tiles_per_image, eps,
                      reinterpret_cast<const float2*>(stats), static_cast<const __nv_bfloat16*>(gamma),
                      static_cast<const __nv_bfloat16*>(beta), static_cast<__nv_bfloat16*>(y));
}

namespace {
constexpr size_t kPoolStripBytes = 32 * 1024;   // shared-memory strip per block (6 blocks per SM)
// plus one float per strip pixel for the log-sum-exp: at most kPoolStripBytes / sizeof(T) / C * 4

template <typename T>
cudaError_t channel_softmax_pool_typed(int Nb, int C, int H, int Wd, int pool, const T* a, T* y,
                                       cudaStream_t st) {
  const int Ho = H / pool, Wo = Wd / pool;
  const size_t per_col = static_cast<size_t>(C) * pool * pool * sizeof(T);   // one pooled column
  if (per_col > kPoolStripBytes) {
    // strip does not fit: one thread per pooled pixel straight from global memory
    const long long total = static_cast<long long>(Nb) * Ho * Wo;
    channel_softmax_pool_kernel<T><<<static_cast<unsigned>((total + 255) / 256), 256, 0, st>>>(
        Nb, C, H, Wd, pool, a, y);
    return cudaGetLastError();
  }
  int tw = static_cast<int>(kPoolStripBytes / per_col);
  if (tw > Wo) tw = Wo;
  constexpr int kVec = 16 / sizeof(T);
  // vector loads need every row segment to start on 16 bytes and to be whole vectors
  bool vec = (reinterpret_cast<uintptr_t>(a) % 16 == 0) && (Wd % kVec == 0);
  if (vec) {
    // shrink tw until tw*pool is a multiple of the vector (the ragged last tile must be too)
    int t = tw;
    while (t > 0 && ((t * pool) % kVec != 0)) --t;
    if (t > 0 && ((Wo % t) * pool) % kVec == 0) tw = t; else vec = false;
  }
  const size_t px = static_cast<size_t>(pool) * pool * tw;
  const size_t smem = ((static_cast<size_t>(C) * px * sizeof(T) + 15) & ~static_cast<size_t>(15)) +
                      ((px + 3) & ~static_cast<size_t>(3)) * sizeof(float) +
                      kPoolPartials * sizeof(float2);
  const long long blocks = static_cast<long long>(Nb) * Ho * ((Wo + tw - 1) / tw);
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
  auto launch = [&](auto kern) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(kPoolStripBytes * 3 + 8192));
    if (e != cudaSuccess) return e;
    return launch_after(false, kern, dim3(static_cast<unsigned>(blocks)), dim3(256), smem, st, Nb, C, H, Wd, tw, a, y);
  };
  auto by_pool = [&](auto vec_tag) -> cudaError_t {
    constexpr int V = decltype(vec_tag)::value;
    switch (pool) {
      case 1: return launch(channel_softmax_pool_tiled_kernel<T, V, 1>);
      case 2: return launch(channel_softmax_pool_tiled_kernel<T, V, 2>);
      case 3: return launch(channel_softmax_pool_tiled_kernel<T, V, 3>);
      default: return launch(channel_softmax_pool_tiled_kernel<T, V, 4>);
    }
  };
  return vec ? by_pool(std::integral_constant<int, kVec>{}) : by_pool(std::integral_constant<int, 1>{});
}
}  // namespace

cudaError_t launch_channel_softmax_pool(int dt, int Nb, int C, int H, int Wd, int pool, const void* a,
                                        void* y, cudaStream_t st) {
  if (static_cast<long long>(Nb) * (H / pool) * (Wd / pool) == 0) return cudaSuccess;
  if (dt == DT_F32)
    return channel_softmax_pool_typed<float>(Nb, C, H, Wd, pool, static_cast<const float*>(a),
                                             static_cast<float*>(y), st);
  return channel_softmax_pool_typed<__nv_bfloat16>(Nb, C, H, Wd, pool,
                                                   static_cast<const __nv_bfloat16*>(a),
                                                   static_cast<__nv_bfloat16*>(y), st);
}

}  // namespace kf
