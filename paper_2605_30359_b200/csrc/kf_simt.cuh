// kf_simt.cuh -- CUDA-core kernels: the fp32 chains (plain FMA, no TF32), the bf16 chains on
// shapes the tensor-core kernel does not take, the streaming second passes of the row
// reductions, the convolution's layout prepass and GroupNorm.
#pragma once

#include <cuda_runtime.h>

#include "kf_act.cuh"

namespace kf {

// ---------------------------------------------------------------- block reductions
// Fixed tree order: results are bit-identical from run to run.
template <bool IS_MAX>
__device__ __forceinline__ float block_reduce(float v, float* scratch /*[32]*/) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float u = __shfl_xor_sync(0xffffffffu, v, o);
    v = IS_MAX ? fmaxf(v, u) : v + u;
  }
  __syncthreads();                 // scratch may still be read from a previous reduction
  if (lane == 0) scratch[warp] = v;
  __syncthreads();
  float r = IS_MAX ? -INFINITY : 0.0f;
  if (lane < nwarps) r = scratch[lane];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float u = __shfl_xor_sync(0xffffffffu, r, o);
    r = IS_MAX ? fmaxf(r, u) : r + u;
  }
  return r;                        // every thread holds the result
}

// ---------------------------------------------------------------- scalar GEMM + epilogue
// TM x TN output tile per CTA of eight warps (32 x 32 below unless said otherwise).  The warps split K: in each pass over 256 values of
// k, warp w owns k in [32w, 32w+32), loads its 32x32 slabs of X and W with coalesced reads
// (lane = k), stages them k-major in its private shared memory and accumulates the whole 32x32
// tile with an 8x4 register block per lane (32 FMAs per three 16-byte shared loads).  The next
// slab is fetched into registers while the current one is consumed; there is no block-wide
// barrier inside the K loop.  The eight partial tiles are then added in a fixed order.
//   MODE 0: out = T,     Y[m,n] = scale*act(z+b) + R[m,n]
//   MODE 1: out = float, A[m,n] = act(z+b) (pre-reduction values for the row kernels)
constexpr int kSimtLd = 36;                                   // staged row pitch in floats
constexpr int kSimtSmemBytes = 8 * 2 * 32 * kSimtLd * 4;      // 73,728 bytes of dynamic smem

// TM x TN = 32 x 32, or 16 x 16 for problems whose 32 x 32 tiles would leave most SMs idle (the
// register block is (TM/4) x (TN/8) per lane; staging pitch and shared memory are the same).
template <typename T, int MODE, int ACT, int TM, int TN>
__global__ void __launch_bounds__(256)
simt_gemm_kernel(int M, int N, int K, const T* __restrict__ X, long long ldx,
                 const T* __restrict__ W, long long ldw, const T* __restrict__ bias, float scale,
                 const T* R, long long ldr, void* out, long long ldo, int act_code) {
  constexpr int RM = TM / 4, RN = TN / 8;             // register block of a lane
  extern __shared__ float sm[];
  // launched with programmatic stream serialization: wait for the kernel before this one, let
  // the one after it be scheduled
  griddep_wait();
  griddep_launch_dependents();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * TM, n0 = blockIdx.y * TN;
  float* As = sm + warp * (2 * 32 * kSimtLd);
  float* Bs = As + 32 * kSimtLd;
  const int ly = lane >> 3, lx = lane & 7;
  float acc[RM][RN];
#pragma unroll
  for (int i = 0; i < RM; ++i)
#pragma unroll
    for (int j = 0; j < RN; ++j) acc[i][j] = 0.0f;
  float ra[TM], rb[TN];
  auto load_slab = [&](int kw) {
    const int k = kw + lane;
    const bool k_ok = k < K;
#pragma unroll
    for (int i = 0; i < TM; ++i) {
      const long long m = m0 + i;
      ra[i] = (k_ok && m < M) ? to_f32(X[m * ldx + k]) : 0.0f;
    }
#pragma unroll
    for (int i = 0; i < TN; ++i) {
      const long long n = n0 + i;
      rb[i] = (k_ok && n < N) ? to_f32(W[n * ldw + k]) : 0.0f;
    }
  };
  int kw = warp * 32;
  if (kw < K) load_slab(kw);
  for (; kw < K; kw += 256) {
#pragma unroll
    for (int i = 0; i < TM; ++i) As[lane * kSimtLd + i] = ra[i];
#pragma unroll
    for (int i = 0; i < TN; ++i) Bs[lane * kSimtLd + i] = rb[i];
    __syncwarp();
    if (kw + 256 < K) load_slab(kw + 256);
#pragma unroll 8
    for (int kk = 0; kk < 32; ++kk) {
      float a[RM], bb[RN];
#pragma unroll
      for (int i = 0; i < RM; i += 4)
        *reinterpret_cast<float4*>(&a[i]) = *reinterpret_cast<const float4*>(&As[kk * kSimtLd + ly * RM + i]);
      if constexpr (RN == 4) {
        *reinterpret_cast<float4*>(&bb[0]) = *reinterpret_cast<const float4*>(&Bs[kk * kSimtLd + lx * 4]);
      } else {
        *reinterpret_cast<float2*>(&bb[0]) = *reinterpret_cast<const float2*>(&Bs[kk * kSimtLd + lx * 2]);
      }
#pragma unroll
      for (int i = 0; i < RM; ++i)
#pragma unroll
        for (int j = 0; j < RN; ++j) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
    }
    __syncwarp();
  }
  __syncthreads();                       // staging is dead: reuse it for the partial tiles
  float* red = sm;                       // [8 warps][TM rows][TN cols]
#pragma unroll
  for (int i = 0; i < RM; ++i)
#pragma unroll
    for (int j = 0; j < RN; ++j) red[(warp * TM + ly * RM + i) * TN + lx * RN + j] = acc[i][j];
  __syncthreads();
  constexpr int VEC = TM * TN / 256;     // outputs per thread, consecutive columns
  const int r = threadIdx.x / (TN / VEC), c0 = (threadIdx.x % (TN / VEC)) * VEC;
  float zs[VEC];
#pragma unroll
  for (int j = 0; j < VEC; ++j) zs[j] = 0.0f;
#pragma unroll
  for (int w = 0; w < 8; ++w)
#pragma unroll
    for (int j = 0; j < VEC; ++j) zs[j] += red[(w * TM + r) * TN + c0 + j];
  const long long m = m0 + r;
  if (m < M) {
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
      const int n = n0 + c0 + j;
      if (n < N) {
        float z = zs[j];
        if (bias != nullptr) z += to_f32(bias[n]);
        if constexpr (MODE == 0) {
          float y = scale * act_f<ACT, false>(z, act_code);
          if (R != nullptr) y += to_f32(R[m * ldr + n]);
          reinterpret_cast<T*>(out)[m * ldo + n] = from_f32<T>(y);
        } else {
          reinterpret_cast<float*>(out)[m * ldo + n] = act_f<ACT, false>(z, act_code);
        }
      }
    }
  }
}

// ---------------------------------------------------------------- row kernels, scalar path
// One CTA per row over fp32 pre-reduction values A[M,N]: the three-pass softmax (max, sum of
// exp(a-max), quotient) or the plain sum.
template <typename OutT>
__global__ void __launch_bounds__(256)
row_softmax_kernel(int N, const float* __restrict__ A, long long lda, OutT* out, long long ldo) {
  __shared__ float scratch[32];
  const float* a = A + static_cast<long long>(blockIdx.x) * lda;
  OutT* o = out + static_cast<long long>(blockIdx.x) * ldo;
  float mx = -INFINITY;
  for (int n = threadIdx.x; n < N; n += blockDim.x) mx = fmaxf(mx, a[n]);
  mx = block_reduce<true>(mx, scratch);
  float s = 0.0f;
  for (int n = threadIdx.x; n < N; n += blockDim.x) s += expf(a[n] - mx);
  s = block_reduce<false>(s, scratch);
  for (int n = threadIdx.x; n < N; n += blockDim.x) o[n] = from_f32<OutT>(expf(a[n] - mx) / s);
}

// Scalar-valued row reductions of a materialised fp32 matrix: sum, mean, max, log-sum-exp.
__global__ void __launch_bounds__(256)
row_reduce_kernel(int N, const float* __restrict__ A, long long lda, float* out, int red) {
  __shared__ float scratch[32];
  const float* a = A + static_cast<long long>(blockIdx.x) * lda;
  if (red == RED_SUM || red == RED_MEAN) {
    float s = 0.0f;
    for (int n = threadIdx.x; n < N; n += blockDim.x) s += a[n];
    s = block_reduce<false>(s, scratch);
    if (threadIdx.x == 0) out[blockIdx.x] = red == RED_MEAN ? s / static_cast<float>(N) : s;
    return;
  }
  float mx = -INFINITY;
  for (int n = threadIdx.x; n < N; n += blockDim.x) mx = fmaxf(mx, a[n]);
  mx = block_reduce<true>(mx, scratch);
  if (red == RED_MAX) {
    if (threadIdx.x == 0) out[blockIdx.x] = mx;
    return;
  }
  float s = 0.0f;
  for (int n = threadIdx.x; n < N; n += blockDim.x) s += expf(a[n] - mx);
  s = block_reduce<false>(s, scratch);
  if (threadIdx.x == 0) out[blockIdx.x] = mx + logf(s);
}

// GroupNorm over groups of gs consecutive columns of a materialised fp32 matrix A[M,N] (the
// pre-normalisation values), then the activation: one CTA per row, one warp per group at a
// time; mean and biased variance in two passes over the group.
// (TA = float: the fp32 matrix from the workspace; TA = T with A == Y: in place on a stored bf16 z.)
template <typename T, typename TA>
__global__ void __launch_bounds__(256)
row_groupnorm_kernel(int N, int gs, float eps, const TA* A, long long lda,
                     const T* __restrict__ gamma, const T* __restrict__ beta, int act_code,
                     T* Y, long long ldy) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const TA* a = A + static_cast<long long>(blockIdx.x) * lda;
  T* y = Y + static_cast<long long>(blockIdx.x) * ldy;
  for (int g = warp; g < N / gs; g += 8) {
    const int n0 = g * gs;
    float s = 0.0f;
    for (int i = lane; i < gs; i += 32) s += to_f32(a[n0 + i]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const float mu = s / static_cast<float>(gs);
    float v = 0.0f;
    for (int i = lane; i < gs; i += 32) { const float d = to_f32(a[n0 + i]) - mu; v = fmaf(d, d, v); }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const float rstd = rsqrtf(v / static_cast<float>(gs) + eps);
    for (int i = lane; i < gs; i += 32) {
      const int n = n0 + i;
      const float ga = gamma != nullptr ? to_f32(gamma[n]) : 1.0f;
      const float be = beta != nullptr ? to_f32(beta[n]) : 0.0f;
      y[n] = from_f32<T>(act_any<false>(act_code, (to_f32(a[n]) - mu) * rstd * ga + be));
    }
  }
}

// Second pass of a GroupNorm whose groups span whole 256-column tiles: the first pass left
// z (rounded to bf16) in Y and per (row, slice) the exact fp32 (sum, sum of squares) of z, a
// slice being a 256-column tile or half of one; `tiles_n` counts the slices of a row.  One CTA per row: the group
// statistics from the entries (added in increasing order), then the row normalised in place,
// 16 bytes per thread and step.
__global__ void __launch_bounds__(256)
row_groupnorm_apply_kernel(int N, int gs, int tiles_n, float eps, const float2* __restrict__ stats,
                           const __nv_bfloat16* __restrict__ gamma,
                           const __nv_bfloat16* __restrict__ beta, int act_code, __nv_bfloat16* Y,
                           long long ldy) {
  griddep_wait();      // may have been scheduled before the kernel it depends on finished
  extern __shared__ float2 mr[];            // [groups] (mu, rstd)
  const int groups = N / gs, tpg = static_cast<int>(static_cast<long long>(gs) * tiles_n / N);   // entries per group
  const float2* part = stats + static_cast<long long>(blockIdx.x) * tiles_n;
  for (int g = threadIdx.x; g < groups; g += blockDim.x) {
    float s1 = 0.0f, s2 = 0.0f;
    for (int t = 0; t < tpg; ++t) { const float2 q = part[g * tpg + t]; s1 += q.x; s2 += q.y; }
    const float mu = s1 / static_cast<float>(gs);
    mr[g] = make_float2(mu, rsqrtf(fmaxf(s2 / static_cast<float>(gs) - mu * mu, 0.0f) + eps));
  }
  __syncthreads();
  uint4* row = reinterpret_cast<uint4*>(Y + static_cast<long long>(blockIdx.x) * ldy);
  for (int i = threadIdx.x; i < N / 8; i += blockDim.x) {
    const int n0 = i * 8;
    const float2 st = mr[n0 / gs];
    uint4 w = row[i];
    uint32_t* u = reinterpret_cast<uint32_t*>(&w);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + 2 * j;
      const float g0 = gamma != nullptr ? __bfloat162float(gamma[n]) : 1.0f;
      const float g1 = gamma != nullptr ? __bfloat162float(gamma[n + 1]) : 1.0f;
      const float b0 = beta != nullptr ? __bfloat162float(beta[n]) : 0.0f;
      const float b1 = beta != nullptr ? __bfloat162float(beta[n + 1]) : 0.0f;
      const float y0 = act_any<true>(act_code, fmaf((bf16_lo(u[j]) - st.x) * st.y, g0, b0));
      const float y1 = act_any<true>(act_code, fmaf((bf16_hi(u[j]) - st.x) * st.y, g1, b1));
      u[j] = pack_bf16x2(y0, y1);
    }
    row[i] = w;
  }
}

// ---------------------------------------------------------------- second passes, tensor path
// Softmax: the first pass left e[m,n] = exp(a[m,n] - mx_t) in `out` and (mx_t, sum_t) per
// slice t of 2^bn_shift columns (one first-pass tile) in `partial`.  Row maximum mx = max_t mx_t, denominator
// S = sum_t sum_t*exp(mx_t - mx); the output is e * exp(mx_t - mx) / S, in place.
template <typename OutT>
__global__ void __launch_bounds__(256)
softmax_finalize_kernel(int N, int bn_shift, int tiles_n, const float2* __restrict__ partial,
                        OutT* out, long long ldo, int vec_ok) {
  griddep_wait();      // may have been scheduled before the kernel it depends on finished
  extern __shared__ float fac[];   // [tiles_n]
  __shared__ float scratch[32];
  // The first pass wrote the rows in increasing order, so its last rows are the ones still in
  // L2: the blocks that start first take those.
  const long long m = static_cast<long long>(gridDim.x) - 1 - blockIdx.x;
  const float2* part = partial + m * tiles_n;
  float mx = -INFINITY;
  for (int t = threadIdx.x; t < tiles_n; t += blockDim.x) mx = fmaxf(mx, part[t].x);
  mx = block_reduce<true>(mx, scratch);
  float s = 0.0f;
  for (int t = threadIdx.x; t < tiles_n; t += blockDim.x) {
    const float2 pt = part[t];
    const float f = __expf(pt.x - mx);
    fac[t] = f;
    s += pt.y * f;
  }
  s = block_reduce<false>(s, scratch);   // contains the __syncthreads that publishes fac[]
  const float inv = 1.0f / s;
  OutT* o = out + m * ldo;
  if (vec_ok && (N % 8) == 0) {
    constexpr int V = 16 / sizeof(OutT);               // elements per 16-byte vector
    const int nvec = N / V;
    uint4* ov = reinterpret_cast<uint4*>(o);
    for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
      const float f = fac[(i * V) >> bn_shift] * inv;
      uint4 w = ov[i];
      if constexpr (sizeof(OutT) == 2) {
        w.x = pack_bf16x2(bf16_lo(w.x) * f, bf16_hi(w.x) * f);
        w.y = pack_bf16x2(bf16_lo(w.y) * f, bf16_hi(w.y) * f);
        w.z = pack_bf16x2(bf16_lo(w.z) * f, bf16_hi(w.z) * f);
        w.w = pack_bf16x2(bf16_lo(w.w) * f, bf16_hi(w.w) * f);
      } else {
        w.x = __float_as_uint(__uint_as_float(w.x) * f);
        w.y = __float_as_uint(__uint_as_float(w.y) * f);
        w.z = __float_as_uint(__uint_as_float(w.z) * f);
        w.w = __float_as_uint(__uint_as_float(w.w) * f);
      }
      ov[i] = w;
    }
  } else {
    // Rows that do not start on 16 bytes: scalar head up to the first aligned element, 16-byte
    // vectors for the body (a vector may straddle two slices, so each element looks its factor
    // up), scalar tail.
    constexpr int V = 16 / sizeof(OutT);
    const int mis = static_cast<int>((reinterpret_cast<uintptr_t>(o) & 15u) / sizeof(OutT));
    const int head = min(N, (V - mis) % V);
    const int nvec = (N - head) / V;
    for (int n = threadIdx.x; n < head; n += blockDim.x)
      o[n] = from_f32<OutT>(to_f32(o[n]) * fac[n >> bn_shift] * inv);
    uint4* ov = reinterpret_cast<uint4*>(o + head);
    for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
      const int n0 = head + i * V;
      uint4 w = ov[i];
      if constexpr (sizeof(OutT) == 2) {
        uint32_t* u = reinterpret_cast<uint32_t*>(&w);
#pragma unroll
        for (int j = 0; j < 4; ++j)
          u[j] = pack_bf16x2(bf16_lo(u[j]) * (fac[(n0 + 2 * j) >> bn_shift] * inv),
                             bf16_hi(u[j]) * (fac[(n0 + 2 * j + 1) >> bn_shift] * inv));
      } else {
        float* u = reinterpret_cast<float*>(&w);
#pragma unroll
        for (int j = 0; j < 4; ++j) u[j] *= fac[(n0 + j) >> bn_shift] * inv;
      }
      ov[i] = w;
    }
    for (int n = head + nvec * V + threadIdx.x; n < N; n += blockDim.x)
      o[n] = from_f32<OutT>(to_f32(o[n]) * fac[n >> bn_shift] * inv);
  }
}

// The same second pass for rows of at most 32 slices: one WARP per row (eight rows per block),
// statistics combined with shuffles, lane t keeping slice t's factor.  Short rows leave most of
// a 256-thread block idle in the kernel above and pay two block reductions per row.
template <typename OutT>
__global__ void __launch_bounds__(256)
softmax_finalize_warp_kernel(int M, int N, int bn_shift, int tiles_n,
                             const float2* __restrict__ partial, OutT* out, long long ldo,
                             int vec_ok) {
  griddep_wait();      // may have been scheduled before the kernel it depends on finished
  const int lane = threadIdx.x & 31;
  // last-written rows first (they are the ones still in L2)
  const long long m = static_cast<long long>(gridDim.x - 1 - blockIdx.x) * 8 + (threadIdx.x >> 5);
  if (m >= M) return;
  float2 pt = make_float2(-INFINITY, 0.0f);
  if (lane < tiles_n) pt = partial[m * tiles_n + lane];
  float mx = pt.x;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  const float fac = lane < tiles_n ? __expf(pt.x - mx) : 0.0f;
  float s = pt.y * fac;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  const float scale = fac / s;                         // lane t: factor of slice t
  OutT* o = out + m * ldo;
  if (vec_ok && (N % 8) == 0) {
    constexpr int V = 16 / sizeof(OutT);
    const int nvec = N / V;
    uint4* ov = reinterpret_cast<uint4*>(o);
    for (int i0 = 0; i0 < nvec; i0 += 32) {            // uniform trip count: shuffles need all lanes
      const int i = i0 + lane;
      const float f = __shfl_sync(0xffffffffu, scale, (min(i, nvec - 1) * V) >> bn_shift);
      if (i < nvec) {
        uint4 w = ov[i];
        if constexpr (sizeof(OutT) == 2) {
          w.x = pack_bf16x2(bf16_lo(w.x) * f, bf16_hi(w.x) * f);
          w.y = pack_bf16x2(bf16_lo(w.y) * f, bf16_hi(w.y) * f);
          w.z = pack_bf16x2(bf16_lo(w.z) * f, bf16_hi(w.z) * f);
          w.w = pack_bf16x2(bf16_lo(w.w) * f, bf16_hi(w.w) * f);
        } else {
          w.x = __float_as_uint(__uint_as_float(w.x) * f);
          w.y = __float_as_uint(__uint_as_float(w.y) * f);
          w.z = __float_as_uint(__uint_as_float(w.z) * f);
          w.w = __float_as_uint(__uint_as_float(w.w) * f);
        }
        ov[i] = w;
      }
    }
  } else {
    for (int n0 = 0; n0 < N; n0 += 32) {
      const int n = n0 + lane;
      const float f = __shfl_sync(0xffffffffu, scale, min(n, N - 1) >> bn_shift);
      if (n < N) o[n] = from_f32<OutT>(to_f32(o[n]) * f);
    }
  }
}

// Row sum: out[m] = scale * sum_t partial[m,t] in increasing t (scale = 1/N for the mean).
__global__ void __launch_bounds__(256)
rowsum_finalize_kernel(int M, int tiles_n, const float* __restrict__ partial, float* out, float scale) {
  griddep_wait();      // may have been scheduled before the kernel it depends on finished
  const long long m = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (m >= M) return;
  float s = 0.0f;
  for (int t = 0; t < tiles_n; ++t) s += partial[m * tiles_n + t];
  out[m] = s * scale;
}

// Row maximum / log-sum-exp from the softmax first pass's per-slice (max, sum of exp) run in
// statistics-only mode: mx = max_t mx_t; lse = mx + log sum_t sum_t * exp(mx_t - mx).
__global__ void __launch_bounds__(256)
rowstat_finalize_kernel(int M, int slices, const float2* __restrict__ partial, float* out, int red) {
  griddep_wait();      // may have been scheduled before the kernel it depends on finished
  const long long m = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (m >= M) return;
  const float2* part = partial + m * slices;
  float mx = -INFINITY;
  for (int t = 0; t < slices; ++t) mx = fmaxf(mx, part[t].x);
  if (red == RED_MAX) { out[m] = mx; return; }
  float s = 0.0f;
  for (int t = 0; t < slices; ++t) {
    const float2 q = part[t];
    s += q.y * expf(q.x - mx);          // an empty slice holds (-inf, 0) and adds 0
  }
  out[m] = mx + logf(s);
}

// ---------------------------------------------------------------- operand repack for TMA
// in [rows, ld] bf16 with any pitch and alignment -> out dense [rows, kp] (kp = K rounded up to
// 8, padding columns zero): what the tensor-core kernels' TMA loads need.  One thread per group
// of eight columns.
__global__ void __launch_bounds__(256)
pad_rows_bf16_kernel(long long rows, int K, int kp, const __nv_bfloat16* __restrict__ in, long long ld,
                     __nv_bfloat16* __restrict__ out) {
  const int gpr = kp / 8;
  const long long total = rows * gpr;
  for (long long g = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; g < total;
       g += static_cast<long long>(gridDim.x) * blockDim.x) {
    const long long r = g / gpr;
    const int k = static_cast<int>(g - r * gpr) * 8;
    const __nv_bfloat16* src = in + r * ld + k;
    unsigned short e[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) e[j] = (k + j < K) ? __bfloat16_as_ushort(src[j]) : static_cast<unsigned short>(0);
    uint4 o;
    o.x = e[0] | (static_cast<uint32_t>(e[1]) << 16);
    o.y = e[2] | (static_cast<uint32_t>(e[3]) << 16);
    o.z = e[4] | (static_cast<uint32_t>(e[5]) << 16);
    o.w = e[6] | (static_cast<uint32_t>(e[7]) << 16);
    reinterpret_cast<uint4*>(out)[g] = o;
  }
}

// ---------------------------------------------------------------- conv: layout prepass
// x NCHW bf16 -> xt NHWC bf16 (so a pixel's channels are one contiguous, K-major row for the
// implicit GEMM), and w OIHW -> wr[tap][o][c].  Each thread moves an 8-channel x 8-pixel block:
// eight 16-byte reads along w, an in-register transpose, eight 16-byte writes along c.
// Requires Cin % 8 == 0 and Wd % 8 == 0.
__global__ void __launch_bounds__(256)
conv_prep_kernel(int Nb, int Cin, int H, int Wd, int Cout, const __nv_bfloat16* __restrict__ x,
                 const __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ xt,
                 __nv_bfloat16* __restrict__ wr, long long x_blocks, uint4* __restrict__ ones, long long ones16) {
  const long long gid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  // (the first ones16 threads also set 16 bytes each of `ones` to all ones: the empty exchange
  // buffer of the all-SM GroupNorm kernel, which would otherwise cost a memset of its own)
  if (gid < ones16) ones[gid] = make_uint4(~0u, ~0u, ~0u, ~0u);
  const int wb = Wd / 8, cbk = Cin / 8;
  if (gid < x_blocks) {
    // gid -> (n, h, wblk, cblk) with cblk fastest: the lanes that hold one pixel's channel blocks
    // write whole 128-byte stretches of its NHWC row (L2 takes a 16-byte write request as long as
    // a 128-byte one); the reads still cover 64-byte runs of a row of x
    const int cblk = static_cast<int>(gid % cbk);
    long long t = gid / cbk;
    const int wblk = static_cast<int>(t % wb); t /= wb;
    const int h = static_cast<int>(t % H);
    const long long n = t / H;
    const long long hw = static_cast<long long>(H) * Wd;
    const __nv_bfloat16* src = x + ((n * Cin + cblk * 8) * H + h) * Wd + wblk * 8;
    uint4 rows[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) rows[i] = __ldg(reinterpret_cast<const uint4*>(src + i * hw));
    const unsigned short* e = reinterpret_cast<const unsigned short*>(rows);   // e[c*8 + p]
    __nv_bfloat16* dst = xt + ((n * H + h) * Wd + wblk * 8) * Cin + cblk * 8;
#pragma unroll
    for (int p = 0; p < 8; ++p) {
      uint4 o;
      o.x = static_cast<uint32_t>(e[0 * 8 + p]) | (static_cast<uint32_t>(e[1 * 8 + p]) << 16);
      o.y = static_cast<uint32_t>(e[2 * 8 + p]) | (static_cast<uint32_t>(e[3 * 8 + p]) << 16);
      o.z = static_cast<uint32_t>(e[4 * 8 + p]) | (static_cast<uint32_t>(e[5 * 8 + p]) << 16);
      o.w = static_cast<uint32_t>(e[6 * 8 + p]) | (static_cast<uint32_t>(e[7 * 8 + p]) << 16);
      *reinterpret_cast<uint4*>(dst + static_cast<long long>(p) * Cin) = o;
    }
  } else {
    const long long i = gid - x_blocks;                 // index into wr[tap][o][c]
    const long long total = 9ll * Cout * Cin;
    if (i < total) {
      const int c = static_cast<int>(i % Cin);
      const int o = static_cast<int>((i / Cin) % Cout);
      const int tap = static_cast<int>(i / (static_cast<long long>(Cin) * Cout));
      wr[i] = w[(static_cast<long long>(o) * Cin + c) * 9 + tap];
    }
  }
}

// General form of the prepass: any Cin and Wd, channels padded with zeros to Cp (a multiple of
// 64, the K block of the implicit GEMM).  One thread per pixel and block of eight channels,
// pixels fastest across threads: reads run along w, each thread writes one 16-byte vector.
__global__ void __launch_bounds__(256)
conv_prep_general_kernel(int Nb, int Cin, int Cp, int H, int Wd, int Cout,
                         const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w,
                         __nv_bfloat16* __restrict__ xt, __nv_bfloat16* __restrict__ wr,
                         long long x_items, uint4* __restrict__ ones, long long ones16) {
  const long long gid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (gid < ones16) ones[gid] = make_uint4(~0u, ~0u, ~0u, ~0u);   // (see conv_prep_kernel)
  const long long hw = static_cast<long long>(H) * Wd;
  const int cbk = Cp / 8;
  if (gid < x_items) {
    const long long px = gid % hw;                       // pixel inside the image
    long long t = gid / hw;
    const int cblk = static_cast<int>(t % cbk);
    const long long n = t / cbk;
    unsigned short e[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int c = cblk * 8 + i;
      e[i] = c < Cin ? __bfloat16_as_ushort(x[(n * Cin + c) * hw + px]) : static_cast<unsigned short>(0);
    }
    uint4 o;
    o.x = e[0] | (static_cast<uint32_t>(e[1]) << 16);
    o.y = e[2] | (static_cast<uint32_t>(e[3]) << 16);
    o.z = e[4] | (static_cast<uint32_t>(e[5]) << 16);
    o.w = e[6] | (static_cast<uint32_t>(e[7]) << 16);
    *reinterpret_cast<uint4*>(xt + (n * hw + px) * Cp + cblk * 8) = o;
  } else {
    const long long i = gid - x_items;                   // index into wr[tap][o][Cp]
    const long long total = 9ll * Cout * Cp;
    if (i < total) {
      const int c = static_cast<int>(i % Cp);
      const int o = static_cast<int>((i / Cp) % Cout);
      const int tap = static_cast<int>(i / (static_cast<long long>(Cp) * Cout));
      wr[i] = c < Cin ? w[(static_cast<long long>(o) * Cin + c) * 9 + tap] : __float2bfloat16_rn(0.0f);
    }
  }
}

// ---------------------------------------------------------------- conv: scalar path
// One thread per output element, taps with an explicit bounds test; stores act(c) in T.
template <typename T, int ACT>
__global__ void __launch_bounds__(256)
conv_direct_kernel(int Nb, int Cin, int H, int Wd, int Cout, const T* __restrict__ x,
                   const T* __restrict__ w, const T* __restrict__ bias, T* __restrict__ y, int act_code) {
  const long long total = static_cast<long long>(Nb) * Cout * H * Wd;
  const long long gid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (gid >= total) return;
  const int wq = static_cast<int>(gid % Wd);
  const int h = static_cast<int>((gid / Wd) % H);
  const int o = static_cast<int>((gid / (static_cast<long long>(Wd) * H)) % Cout);
  const long long n = gid / (static_cast<long long>(Wd) * H * Cout);
  float acc = bias != nullptr ? to_f32(bias[o]) : 0.0f;
  for (int c = 0; c < Cin; ++c) {
    const T* xp = x + (n * Cin + c) * H * Wd;
    const T* wp = w + (static_cast<long long>(o) * Cin + c) * 9;
#pragma unroll
    for (int r = 0; r < 3; ++r) {
      const int hh = h + r - 1;
      if (hh < 0 || hh >= H) continue;
#pragma unroll
      for (int s = 0; s < 3; ++s) {
        const int ww = wq + s - 1;
        if (ww < 0 || ww >= Wd) continue;
        acc = fmaf(to_f32(xp[hh * Wd + ww]), to_f32(wp[r * 3 + s]), acc);
      }
    }
  }
  y[gid] = from_f32<T>(act_f<ACT, false>(acc, act_code));
}

// ---------------------------------------------------------------- GroupNorm, in place
// One CTA per (image, group): the group's cpg*H*W activations are contiguous in NCHW.  Mean,
// then the biased variance about that mean (two passes: no cancellation), then
// y = (a-mu)*rstd*gamma[o]+beta[o].  The group is re-read from cache, not from HBM, when it
// fits (32 KB for the benchmark's groups).
template <typename T>
__global__ void __launch_bounds__(512)
groupnorm_kernel(int Cout, int groups, long long hw, float eps, const T* __restrict__ gamma,
                 const T* __restrict__ beta, T* y) {
  __shared__ float scratch[32];
  const int cpg = Cout / groups;
  const long long cnt = static_cast<long long>(cpg) * hw;
  const int g = blockIdx.x % groups;
  const long long n = blockIdx.x / groups;
  T* blk = y + (n * Cout + static_cast<long long>(g) * cpg) * hw;
  constexpr int V = 16 / sizeof(T);
  const bool vec = (cnt % V) == 0 && (hw % V) == 0 &&
                   (reinterpret_cast<uintptr_t>(blk) & 15u) == 0;
  float s = 0.0f;
  if (vec) {
    const uint4* bv = reinterpret_cast<const uint4*>(blk);
    for (long long i = threadIdx.x; i < cnt / V; i += blockDim.x) {
      const uint4 w = bv[i];
      if constexpr (sizeof(T) == 2) {
        s += (bf16_lo(w.x) + bf16_hi(w.x)) + (bf16_lo(w.y) + bf16_hi(w.y)) +
             (bf16_lo(w.z) + bf16_hi(w.z)) + (bf16_lo(w.w) + bf16_hi(w.w));
      } else {
        s += (__uint_as_float(w.x) + __uint_as_float(w.y)) +
             (__uint_as_float(w.z) + __uint_as_float(w.w));
      }
    }
  } else {
    for (long long i = threadIdx.x; i < cnt; i += blockDim.x) s += to_f32(blk[i]);
  }
  const float mu = block_reduce<false>(s, scratch) / static_cast<float>(cnt);
  float q = 0.0f;
  if (vec) {
    const uint4* bv = reinterpret_cast<const uint4*>(blk);
    for (long long i = threadIdx.x; i < cnt / V; i += blockDim.x) {
      const uint4 w = bv[i];
      float d[8];
      int nv;
      if constexpr (sizeof(T) == 2) {
        d[0] = bf16_lo(w.x); d[1] = bf16_hi(w.x); d[2] = bf16_lo(w.y); d[3] = bf16_hi(w.y);
        d[4] = bf16_lo(w.z); d[5] = bf16_hi(w.z); d[6] = bf16_lo(w.w); d[7] = bf16_hi(w.w);
        nv = 8;
      } else {
        d[0] = __uint_as_float(w.x); d[1] = __uint_as_float(w.y);
        d[2] = __uint_as_float(w.z); d[3] = __uint_as_float(w.w);
        nv = 4;
      }
      float part = 0.0f;
#pragma unroll
      for (int j = 0; j < 8; ++j) if (j < nv) part = fmaf(d[j] - mu, d[j] - mu, part);
      q += part;
    }
  } else {
    for (long long i = threadIdx.x; i < cnt; i += blockDim.x) {
      const float d = to_f32(blk[i]) - mu;
      q = fmaf(d, d, q);
    }
  }
  const float var = block_reduce<false>(q, scratch) / static_cast<float>(cnt);
  const float rstd = rsqrtf(var + eps);
  if (vec) {
    uint4* bv = reinterpret_cast<uint4*>(blk);
    for (long long i = threadIdx.x; i < cnt / V; i += blockDim.x) {
      const int o = g * cpg + static_cast<int>((i * V) / hw);   // a vector never straddles channels
      const float ga = gamma != nullptr ? to_f32(gamma[o]) : 1.0f;
      const float be = beta != nullptr ? to_f32(beta[o]) : 0.0f;
      const float a = rstd * ga, b = fmaf(-mu, rstd * ga, be);
      uint4 w = bv[i];
      if constexpr (sizeof(T) == 2) {
        w.x = pack_bf16x2(fmaf(bf16_lo(w.x), a, b), fmaf(bf16_hi(w.x), a, b));
        w.y = pack_bf16x2(fmaf(bf16_lo(w.y), a, b), fmaf(bf16_hi(w.y), a, b));
        w.z = pack_bf16x2(fmaf(bf16_lo(w.z), a, b), fmaf(bf16_hi(w.z), a, b));
        w.w = pack_bf16x2(fmaf(bf16_lo(w.w), a, b), fmaf(bf16_hi(w.w), a, b));
      } else {
        w.x = __float_as_uint(fmaf(__uint_as_float(w.x), a, b));
        w.y = __float_as_uint(fmaf(__uint_as_float(w.y), a, b));
        w.z = __float_as_uint(fmaf(__uint_as_float(w.z), a, b));
        w.w = __float_as_uint(fmaf(__uint_as_float(w.w), a, b));
      }
      bv[i] = w;
    }
  } else {
    for (long long i = threadIdx.x; i < cnt; i += blockDim.x) {
      const int o = g * cpg + static_cast<int>(i / hw);
      const float ga = gamma != nullptr ? to_f32(gamma[o]) : 1.0f;
      const float be = beta != nullptr ? to_f32(beta[o]) : 0.0f;
      blk[i] = from_f32<T>((to_f32(blk[i]) - mu) * rstd * ga + be);
    }
  }
}

// ---------------------------------------------------------------- GroupNorm from tile statistics
// The convolution epilogue left, per pixel tile t and channel c, stats[t][c] = (sum, sum of
// squares) of the stored activations.  One CTA per (image, group): add the group's entries in a
// fixed order, mean = S1/cnt, var = S2/cnt - mean^2 (biased), then normalise the group's
// contiguous NCHW block in place: one read and one write of the activations.
__global__ void __launch_bounds__(512)
groupnorm_apply_kernel(int Cout, int groups, long long hw, int tiles_per_image, float eps,
                       const float2* __restrict__ stats, const __nv_bfloat16* __restrict__ gamma,
                       const __nv_bfloat16* __restrict__ beta, __nv_bfloat16* y) {
  griddep_wait();      // may have been scheduled before the kernel it depends on finished
  const int cpg = Cout / groups;
  const long long cnt = static_cast<long long>(cpg) * hw;
  // increasing image order: the convolution wrote the first images last, they are still in L2
  const int g = blockIdx.x % groups;
  const long long n = blockIdx.x / groups;
  __nv_bfloat16* blk = y + (n * Cout + static_cast<long long>(g) * cpg) * hw;
  const bool vec = (hw % 8) == 0 && (reinterpret_cast<uintptr_t>(blk) & 15u) == 0;
  // Fetch this thread's first vectors before the statistics are known: the loads do not depend
  // on them, so their latency hides behind the reduction.
  constexpr int PRE = 4;
  uint4 pre[PRE];
  const long long nvec = cnt / 8;
  if (vec) {
    const uint4* bv = reinterpret_cast<const uint4*>(blk);
#pragma unroll
    for (int k = 0; k < PRE; ++k) {
      const long long i = threadIdx.x + static_cast<long long>(k) * blockDim.x;
      if (i < nvec) pre[k] = bv[i];
    }
  }
  // Every warp adds the group's entries itself (lane-strided, then a shuffle tree): the same
  // order in every warp, so all warps hold bit-identical statistics, and no block-wide barrier
  // sits between the prefetch and the stores.
  float s1 = 0.0f, s2 = 0.0f;
  for (int i = threadIdx.x & 31; i < tiles_per_image * cpg; i += 32) {
    const int t = i / cpg, c = g * cpg + i % cpg;
    const float2 v = stats[(n * tiles_per_image + t) * Cout + c];
    s1 += v.x;
    s2 += v.y;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    s1 += __shfl_xor_sync(0xffffffffu, s1, o);
    s2 += __shfl_xor_sync(0xffffffffu, s2, o);
  }
  const float mu = s1 / static_cast<float>(cnt);
  const float var = fmaxf(s2 / static_cast<float>(cnt) - mu * mu, 0.0f);
  const float rstd = rsqrtf(var + eps);
  if (vec) {
    uint4* bv = reinterpret_cast<uint4*>(blk);
    for (long long i = threadIdx.x, k = 0; i < nvec; i += blockDim.x, ++k) {
      const int o = g * cpg + static_cast<int>((i * 8) / hw);
      const float ga = gamma != nullptr ? to_f32(gamma[o]) : 1.0f;
      const float be = beta != nullptr ? to_f32(beta[o]) : 0.0f;
      const float a = rstd * ga, b = fmaf(-mu, rstd * ga, be);
      uint4 w;
      if (k == 0) w = pre[0];
      else if (k == 1) w = pre[1];
      else if (k == 2) w = pre[2];
      else if (k == 3) w = pre[3];
      else w = bv[i];
      w.x = pack_bf16x2(fmaf(bf16_lo(w.x), a, b), fmaf(bf16_hi(w.x), a, b));
      w.y = pack_bf16x2(fmaf(bf16_lo(w.y), a, b), fmaf(bf16_hi(w.y), a, b));
      w.z = pack_bf16x2(fmaf(bf16_lo(w.z), a, b), fmaf(bf16_hi(w.z), a, b));
      w.w = pack_bf16x2(fmaf(bf16_lo(w.w), a, b), fmaf(bf16_hi(w.w), a, b));
      bv[i] = w;
    }
  } else {
    for (long long i = threadIdx.x; i < cnt; i += blockDim.x) {
      const int o = g * cpg + static_cast<int>(i / hw);
      const float ga = gamma != nullptr ? to_f32(gamma[o]) : 1.0f;
      const float be = beta != nullptr ? to_f32(beta[o]) : 0.0f;
      blk[i] = __float2bfloat16_rn((to_f32(blk[i]) - mu) * rstd * ga + be);
    }
  }
}

// ---------------------------------------------------------------- spatial pooling of an NCHW tensor
// out[plane, i, j] = max (kind 0) or mean (kind 1) over the pool x pool window at (i*pool, j*pool)
// of in[plane, :, :]; one thread per output element, consecutive threads along j.
template <typename T>
__global__ void __launch_bounds__(256)
pool2d_kernel(long long planes, int H, int Wd, int pool, int kind, const T* __restrict__ in,
              T* __restrict__ out) {
  const int Ho = H / pool, Wo = Wd / pool;
  const long long total = planes * Ho * Wo;
  const long long gid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (gid >= total) return;
  const int j = static_cast<int>(gid % Wo);
  const int i = static_cast<int>((gid / Wo) % Ho);
  const long long pl = gid / (static_cast<long long>(Wo) * Ho);
  const T* src = in + (pl * H + static_cast<long long>(i) * pool) * Wd + static_cast<long long>(j) * pool;
  float best = -INFINITY, sum = 0.0f;
  for (int r = 0; r < pool; ++r)
    for (int q = 0; q < pool; ++q) {
      const float v = to_f32(src[static_cast<long long>(r) * Wd + q]);
      best = fmaxf(best, v);
      sum += v;
    }
  out[gid] = from_f32<T>(kind == 0 ? best : sum / static_cast<float>(pool * pool));
}

// ---------------------------------------------------------------- global average pooling
// From the convolution epilogue's statistics: out[n,c] = (sum over the image's pixel tiles of the
// per-tile channel sums) / (H*W), tiles added in increasing order.
__global__ void __launch_bounds__(256)
gap_finalize_kernel(int Nb, int Cout, int parts, long long hw, const float2* __restrict__ stats,
                    float* __restrict__ out) {
  griddep_wait();      // may have been scheduled before the kernel it depends on finished
  const long long gid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (gid >= static_cast<long long>(Nb) * Cout) return;
  const long long n = gid / Cout;
  const int c = static_cast<int>(gid - n * Cout);
  float s = 0.0f;
  for (int t = 0; t < parts; ++t) s += stats[(n * parts + t) * Cout + c].x;
  out[gid] = s / static_cast<float>(hw);
}

// From a stored NCHW tensor: out[row] = mean of the row's `len` contiguous elements (a row is
// one image plane).  One CTA per row.
template <typename T>
__global__ void __launch_bounds__(256)
plane_mean_kernel(long long len, const T* __restrict__ in, float* __restrict__ out) {
  __shared__ float scratch[32];
  const T* a = in + static_cast<long long>(blockIdx.x) * len;
  float s = 0.0f;
  for (long long i = threadIdx.x; i < len; i += blockDim.x) s += to_f32(a[i]);
  s = block_reduce<false>(s, scratch);
  if (threadIdx.x == 0) out[blockIdx.x] = s / static_cast<float>(len);
}

// ---------------------------------------------------------------- channel softmax + max-pool
// Second pass of conv -> softmax over channels -> max-pool.  `a` holds the convolution output
// NCHW.  One thread per pooled output pixel: for each of the pool x pool input pixels the
// three-pass softmax over the channel dimension (max, sum of exp, quotient), then per channel
// the maximum of the window's probabilities.  pool <= 4 (the window's statistics live in
// registers); the second and third reads of `a` come from cache.
template <typename T>
__global__ void __launch_bounds__(256)
channel_softmax_pool_kernel(int Nb, int C, int H, int Wd, int pool, const T* __restrict__ a,
                            T* __restrict__ y) {
  const int Ho = H / pool, Wo = Wd / pool;
  const long long total = static_cast<long long>(Nb) * Ho * Wo;
  const long long gid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (gid >= total) return;
  const int j = static_cast<int>(gid % Wo);
  const int i = static_cast<int>((gid / Wo) % Ho);
  const long long n = gid / (static_cast<long long>(Wo) * Ho);
  const long long hw = static_cast<long long>(H) * Wd;
  const T* an = a + n * C * hw;
  const int pp = pool * pool;
  float mx[16], inv[16];
  for (int q = 0; q < pp; ++q) {
    const T* px = an + static_cast<long long>(i * pool + q / pool) * Wd + (j * pool + q % pool);
    float m = -INFINITY;
    for (int c = 0; c < C; ++c) m = fmaxf(m, to_f32(px[c * hw]));
    float s = 0.0f;
    for (int c = 0; c < C; ++c) s += expf(to_f32(px[c * hw]) - m);
    mx[q] = m;
    inv[q] = 1.0f / s;
  }
  T* yo = y + (n * C * Ho + i) * Wo + j;
  for (int c = 0; c < C; ++c) {
    float best = 0.0f;
    for (int q = 0; q < pp; ++q) {
      const float v = to_f32(an[c * hw + static_cast<long long>(i * pool + q / pool) * Wd +
                                (j * pool + q % pool)]);
      best = fmaxf(best, expf(v - mx[q]) * inv[q]);
    }
    yo[static_cast<long long>(c) * Ho * Wo] = from_f32<T>(best);
  }
}

// 2^x in one MUFU op (relative error about 2^-22; flushes results below 2^-126 to zero).
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Helpers of the tiled pass: N adjacent elements of shared memory as floats, with the widest
// load the alignment allows (the caller guarantees alignment to N * sizeof(T) when that is a
// power of two).
template <int N>
__device__ __forceinline__ void ld_row(const float* p, float (&o)[N]) {
  if constexpr (N == 4) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
  } else if constexpr (N == 2) {
    const float2 v = *reinterpret_cast<const float2*>(p);
    o[0] = v.x; o[1] = v.y;
  } else {
#pragma unroll
    for (int i = 0; i < N; ++i) o[i] = p[i];
  }
}
template <int N>
__device__ __forceinline__ void ld_row(const __nv_bfloat16* p, float (&o)[N]) {
  if constexpr (N == 4) {
    const uint2 v = *reinterpret_cast<const uint2*>(p);
    o[0] = __uint_as_float(v.x << 16); o[1] = __uint_as_float(v.x & 0xffff0000u);
    o[2] = __uint_as_float(v.y << 16); o[3] = __uint_as_float(v.y & 0xffff0000u);
  } else if constexpr (N == 2) {
    const uint32_t v = *reinterpret_cast<const uint32_t*>(p);
    o[0] = __uint_as_float(v << 16); o[1] = __uint_as_float(v & 0xffff0000u);
  } else {
#pragma unroll
    for (int i = 0; i < N; ++i) o[i] = __bfloat162float(p[i]);
  }
}

// Tiled form of the same pass: one block owns, for one image, one pooled output row and `tw`
// pooled columns, i.e. a strip of POOL rows x tw*POOL columns x C channels, held in shared
// memory as s[c][p] (p = row*tw*POOL + column, storage type T).
//   phase 1  loads the strip with VEC-element vectors (coalesced along w);
//   phase 2  computes per pixel the log-sum-exp L over c: a thread owns two adjacent pixels and
//            a slice of the channels (max pass, then sum of exp2), slices are merged through
//            shared memory; strips with an odd row pitch take one thread per pixel instead;
//   phase 3  has one thread per (c, pooled column) take the window maximum of z - L and store
//            its exponential: softmax = exp(z - L) and exp is monotone, so one exponential per
//            OUTPUT replaces one per input of the third softmax pass.
// The intermediate is read from DRAM exactly once.  Shared memory: the strip, P floats of L,
// and up to 512 float2 of per-slice partials.
constexpr int kPoolPartials = 512;
template <typename T, int VEC, int POOL>
__global__ void __launch_bounds__(256)
channel_softmax_pool_tiled_kernel(int Nb, int C, int H, int Wd, int tw, const T* __restrict__ a,
                                  T* __restrict__ y) {
  griddep_wait();      // may have been scheduled before the kernel it depends on finished
  extern __shared__ __align__(16) unsigned char smem_raw[];
  T* s = reinterpret_cast<T*>(smem_raw);
  const int Ho = H / POOL, Wo = Wd / POOL;
  const int col_tiles = (Wo + tw - 1) / tw;
  long long b = blockIdx.x;    // first images first: the convolution wrote those last (still in L2)
  const int jt = static_cast<int>(b % col_tiles); b /= col_tiles;
  const int i = static_cast<int>(b % Ho);
  const long long n = b / Ho;
  const int j0 = jt * tw;
  const int twb = min(tw, Wo - j0);          // pooled columns this block owns
  const int rowlen = tw * POOL;              // shared-memory row pitch (elements)
  const int cols = twb * POOL;               // valid input columns
  const int P = POOL * rowlen;
  const long long hw = static_cast<long long>(H) * Wd;
  const T* src = a + n * C * hw + static_cast<long long>(i) * POOL * Wd + static_cast<long long>(j0) * POOL;
  float* lse = reinterpret_cast<float*>(
      smem_raw + ((static_cast<size_t>(C) * P * sizeof(T) + 15) & ~static_cast<size_t>(15)));
  float2* part = reinterpret_cast<float2*>(lse + ((P + 3) & ~3));
  const int tid = threadIdx.x;

  // phase 1: strip -> shared memory.  When one channel's POOL row segments take at most 256
  // vectors, a thread keeps its (row, vector) slot and strides over channels: one load, one
  // store and two pointer bumps per vector.  Otherwise threads form a (rows x vectors) grid.
  {
    const int vrow = cols / VEC;             // VEC divides cols when VEC > 1 (checked by the host)
    const int per_c = POOL * vrow;
    if (per_c <= 256) {
      const int cstep = 256 / per_c;
      const int c_first = tid / per_c;
      const int rv = tid - c_first * per_c;
      const int r = rv / vrow, v = rv - r * vrow;
      if (c_first < cstep) {
        const T* g = src + c_first * hw + static_cast<long long>(r) * Wd + v * VEC;
        T* d = s + c_first * P + r * rowlen + v * VEC;
        const long long gstep = cstep * hw;
        const int dstep = cstep * P;
#pragma unroll 4
        for (int c = c_first; c < C; c += cstep, g += gstep, d += dstep) {
          if constexpr (VEC * sizeof(T) == 16) {
            *reinterpret_cast<uint4*>(d) = __ldg(reinterpret_cast<const uint4*>(g));
          } else {
            *d = *g;
          }
        }
      }
    } else {
      int vl = 1;
      while (vl < vrow && vl < 256) vl <<= 1;
      const int v0 = tid & (vl - 1);
      const int rstep = 256 / vl;
      for (int row = tid / vl; row < C * POOL; row += rstep) {
        const int c = row / POOL, r = row - c * POOL;
        const T* g = src + c * hw + static_cast<long long>(r) * Wd;
        T* d = s + c * P + r * rowlen;
        for (int v = v0; v < vrow; v += vl) {
          if constexpr (VEC * sizeof(T) == 16) {
            *reinterpret_cast<uint4*>(d + v * VEC) = __ldg(reinterpret_cast<const uint4*>(g + v * VEC));
          } else {
            d[v] = g[v];
          }
        }
      }
    }
  }
  __syncthreads();

  // phase 2: L[p] = max_c z + log(sum_c exp(z - max))
  constexpr float kLog2e = 1.4426950408889634f;
  if ((rowlen & 1) == 0) {
    const int NP = P / 2;
    const int slices = NP >= 256 ? 1 : 256 / NP;
    const int cs = (C + slices - 1) / slices;
    for (int wi = tid; wi < NP * slices; wi += 256) {
      const int slice = wi / NP;
      const int p = 2 * (wi - slice * NP);
      const int c0 = slice * cs, c1 = min(C, c0 + cs);
      const T* col = s + p;
      float m0 = -INFINITY, m1 = -INFINITY;
      if constexpr (sizeof(T) == 2) {
        __nv_bfloat162 mm = __floats2bfloat162_rn(-INFINITY, -INFINITY);
#pragma unroll 8
        for (int c = c0; c < c1; ++c)
          mm = __hmax2(mm, *reinterpret_cast<const __nv_bfloat162*>(col + c * P));
        m0 = __low2float(mm); m1 = __high2float(mm);
      } else {
#pragma unroll 8
        for (int c = c0; c < c1; ++c) {
          float v[2];
          ld_row<2>(col + c * P, v);
          m0 = fmaxf(m0, v[0]); m1 = fmaxf(m1, v[1]);
        }
      }
      // both pixels' exponent arguments in one packed multiply-add, both sums in one packed add
      const uint64_t l2e2 = f32x2_pack(kLog2e, kLog2e), off2 = f32x2_pack(-m0 * kLog2e, -m1 * kLog2e);
      uint64_t sum2 = f32x2_pack(0.0f, 0.0f);
#pragma unroll 8
      for (int c = c0; c < c1; ++c) {
        float v[2];
        ld_row<2>(col + c * P, v);
        float t0, t1;
        f32x2_unpack(f32x2_fma(f32x2_pack(v[0], v[1]), l2e2, off2), t0, t1);
        sum2 = f32x2_add(sum2, f32x2_pack(ex2_approx(t0), ex2_approx(t1)));
      }
      float s0, s1;
      f32x2_unpack(sum2, s0, s1);
      if (slices == 1) {
        lse[p] = m0 + __logf(s0);
        lse[p + 1] = m1 + __logf(s1);
      } else {
        part[slice * P + p] = make_float2(m0, s0);
        part[slice * P + p + 1] = make_float2(m1, s1);
      }
    }
    if (slices > 1) {
      __syncthreads();
      for (int p = tid; p < P; p += 256) {
        float m = -INFINITY;
        for (int k = 0; k < slices; ++k) m = fmaxf(m, part[k * P + p].x);
        float sum = 0.0f;
        for (int k = 0; k < slices; ++k) {
          const float2 q = part[k * P + p];
          sum += q.y * ex2_approx((q.x - m) * kLog2e);     // an empty slice holds (-inf, 0): adds 0
        }
        lse[p] = m + __logf(sum);
      }
    }
  } else {
    for (int p = tid; p < P; p += 256) {
      if (p % rowlen >= cols) continue;
      float m = -INFINITY;
      for (int c = 0; c < C; ++c) m = fmaxf(m, to_f32(s[c * P + p]));
      float sum = 0.0f;
      for (int c = 0; c < C; ++c) sum += ex2_approx((to_f32(s[c * P + p]) - m) * kLog2e);
      lse[p] = m + __logf(sum);
    }
  }
  __syncthreads();

  // phase 3: window maxima of z - L, one exponential per output.  A thread keeps one pooled
  // column (its window's L values stay in registers) and strides over channels; the column
  // extent of the thread grid is the power of two covering twb, so no index needs a division.
  {
    int tl = 1;
    while (tl < twb && tl < 256) tl <<= 1;
    const int cstep = 256 / tl;
    T* yo = y + (n * C * Ho + i) * Wo + j0;
    for (int jo = tid & (tl - 1); jo < twb; jo += tl) {
      float l[POOL][POOL];
#pragma unroll
      for (int r = 0; r < POOL; ++r) ld_row<POOL>(lse + r * rowlen + jo * POOL, l[r]);
      const T* zc = s + jo * POOL;
#pragma unroll 2
      for (int c = tid / tl; c < C; c += cstep) {
        float best = -INFINITY;
#pragma unroll
        for (int r = 0; r < POOL; ++r) {
          float z[POOL];
          ld_row<POOL>(zc + c * P + r * rowlen, z);
#pragma unroll
          for (int q = 0; q < POOL; ++q) best = fmaxf(best, z[q] - l[r][q]);
        }
        yo[static_cast<long long>(c) * Ho * Wo + jo] = from_f32<T>(ex2_approx(best * kLog2e));
      }
    }
  }
}

}  // namespace kf
