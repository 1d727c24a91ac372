// kf_umma.cuh -- the tensor-core mainloop shared by every bf16 chain, with its epilogues.
//
// One persistent CTA per SM walks output tiles of 128 rows x BN columns.  Warp roles:
//   warp 0 (one lane)  TMA producer: fills a ring of shared-memory stages (A 128x64, B BNx64
//                      bf16, 128-byte swizzle) and signals `full[s]` by transaction bytes.
//   warp 1 (one lane)  UMMA issuer: four tcgen05.mma (K=16 each) per stage into one of two
//                      TMEM accumulators, tcgen05.commit to `empty[s]` (stage free) and, after
//                      the last K block, to `tmem_full[a]`.
//   warps 2..5         epilogue: tcgen05.ld the accumulator (thread = one row of the tile),
//                      apply the chain's epilogue in fp32 registers, store, then release the
//                      accumulator through `tmem_empty[a]` so the next tile's MMAs overlap.
// Every wait is bounded (mbar_wait); a wait that runs out raises the CTA's abort flag, all
// roles leave their loops, in-flight copies are given time to land, TMEM is freed.
#pragma once

#include "kf_act.cuh"
#include "kf_ptx.cuh"

namespace kf {

enum : int { EPI_ELEMENTWISE = 0, EPI_SOFTMAX = 1, EPI_ROWSUM = 2, EPI_CONV = 3 };

constexpr int kBM = 128;         // tile rows = UMMA M = TMEM lanes
constexpr int kBK = 64;          // K per stage: 64 bf16 = one 128-byte swizzled row
constexpr int kUmmaK = 16;       // K per tcgen05.mma for 16-bit inputs
constexpr int kNumThreads = 192; // 6 warps
constexpr int kEpiThreads = 128; // warps 2..5

struct UmmaParams {
  int M, N, K;                 // GEMM view (conv: M = Nb*H*W pixels, N = Cout, K = 9*Cin)
  int tiles_m, tiles_n, num_tiles, k_blocks;
  const __nv_bfloat16* bias;   // [N] or null
  const __nv_bfloat16* R;      // residual [M,N] or null
  long long ldr;
  void* out;                   // Y / softmax numerators / conv activations
  long long ldo;
  float* partial;              // row-reduce partial statistics
  float scale;
  int vec_ok;                  // rows of out (and R) are 16-byte aligned
  uint32_t* status;            // device status word
  // conv only
  int H, Wd, Cin, rows_per_tile, tiles_per_image, kb_per_tap;
};

template <int BN>
struct UmmaSmem {
  static constexpr int kStageA = kBM * kBK * 2;
  static constexpr int kStageB = BN * kBK * 2;
  static constexpr int kStage = kStageA + kStageB;
  static constexpr int kStages = (BN == 256) ? 4 : (BN == 128 ? 6 : 8);
  static constexpr int kRing = kStage * kStages;
  static constexpr int kBiasBytes = 2 * BN * 4;
  static constexpr int kBarBytes = 8 * (2 * kStages + 4) + 16;
  static constexpr int kTotal = 1024 /*alignment slack*/ + kRing + kBiasBytes + kBarBytes;
};

template <int BN, int EPI, int ACT, typename OutT>
__global__ void __launch_bounds__(kNumThreads, 1)
umma_chain_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const UmmaParams p) {
  using S = UmmaSmem<BN>;
  constexpr int kStages = S::kStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* ring = smem;
  float* sbias = reinterpret_cast<float*>(smem + S::kRing);              // [2][BN]
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + S::kRing + S::kBiasBytes);
  uint64_t* empty = full + kStages;
  uint64_t* tmem_full = empty + kStages;
  uint64_t* tmem_empty = tmem_full + 2;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(tmem_empty + 2);
  volatile uint32_t* abort_flag = tmem_holder + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tmem_full[a], 1); mbar_init(&tmem_empty[a], kEpiThreads); }
    *abort_flag = 0;
    mbar_init_fence();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
  }
  if (warp == 1) {          // TMEM: two accumulators of BN fp32 columns
    tmem_alloc(tmem_holder, 2 * BN);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int s = 0; uint32_t ph = 0;
      for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
        int tm, tn, img = 0, h0 = 0;
        if constexpr (EPI == EPI_CONV) {
          tm = tile; tn = 0;
          img = tile / p.tiles_per_image;
          h0 = (tile % p.tiles_per_image) * p.rows_per_tile;
        } else {
          tm = tile / p.tiles_n; tn = tile % p.tiles_n;
        }
        bool ok = true;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          ok = mbar_wait(&empty[s], ph ^ 1u, abort_flag, p.status, KF_DEV_TIMEOUT_PRODUCER);
          if (!ok) break;
          uint8_t* sa = ring + s * S::kStage;
          uint8_t* sb = sa + S::kStageA;
          mbar_expect_tx(&full[s], S::kStage);
          if constexpr (EPI == EPI_CONV) {
            const int tap = kb / p.kb_per_tap, cb = kb % p.kb_per_tap;
            const int r = tap / 3, sx = tap % 3;
            // A: 128 pixels x 64 channels of the shifted window; out-of-image taps read zeros.
            tma_load_4d(sa, &tmA, &full[s], cb * kBK, sx - 1, h0 + r - 1, img);
            tma_load_2d(sb, &tmB, &full[s], cb * kBK, tap * p.N);
          } else {
            tma_load_2d(sa, &tmA, &full[s], kb * kBK, tm * kBM);
            tma_load_2d(sb, &tmB, &full[s], kb * kBK, tn * BN);
          }
          if (++s == kStages) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ UMMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16_f32(kBM, BN);
      int s = 0; uint32_t ph = 0; int a = 0; uint32_t aph = 0;
      for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
        bool ok = mbar_wait(&tmem_empty[a], aph ^ 1u, abort_flag, p.status, KF_DEV_TIMEOUT_MMA);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(a * BN);
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          ok = mbar_wait(&full[s], ph, abort_flag, p.status, KF_DEV_TIMEOUT_MMA);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t sa = smem_u32(ring + s * S::kStage);
          const uint64_t adesc = smem_desc_kmajor_sw128(sa);
          const uint64_t bdesc = smem_desc_kmajor_sw128(sa + S::kStageA);
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) {
            // +32 bytes per K step inside the 128-byte swizzled row = +2 in the address field
            umma_f16_ss(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(&empty[s]);
          if (++s == kStages) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        umma_commit(&tmem_full[a]);
        if (++a == 2) { a = 0; aph ^= 1u; }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int quad = warp & 3;                 // TMEM lane quarter this warp may read
    const int row = quad * 32 + lane;          // row of the tile = TMEM lane
    const int et = threadIdx.x - 64;           // 0..127 among epilogue threads
    const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
    int a = 0; uint32_t aph = 0;
    for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
      int tm, tn;
      if constexpr (EPI == EPI_CONV) { tm = tile; tn = 0; }
      else { tm = tile / p.tiles_n; tn = tile % p.tiles_n; }
      // stage this tile's bias slice as fp32 (zeros past N or without a bias)
      float* sb = sbias + a * BN;
      for (int j = et; j < BN; j += kEpiThreads) {
        const int n = tn * BN + j;
        sb[j] = (p.bias != nullptr && n < p.N) ? __bfloat162float(p.bias[n]) : 0.0f;
      }
      bool ok = mbar_wait(&tmem_full[a], aph, abort_flag, p.status, KF_DEV_TIMEOUT_EPILOGUE);
      // one uniform go/no-go for all four epilogue warps; also publishes the bias slice
      ok = named_barrier_and(1, kEpiThreads, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t t_acc = tmem_base + static_cast<uint32_t>(a * BN) + lane_off;
      const long long m = static_cast<long long>(tm) * kBM + row;
      const bool row_ok = m < p.M;
      const int n_tile = tn * BN;
      const int n_valid = min(BN, p.N - n_tile);          // valid columns in this tile (>0)

      if constexpr (EPI == EPI_ELEMENTWISE) {
        __nv_bfloat16* Y = reinterpret_cast<__nv_bfloat16*>(p.out);
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          if (c * 32 >= n_valid) break;
          uint32_t v[32];
          tmem_ld_32x32(t_acc + c * 32, v);
          tmem_ld_wait();
          float f[32];
#pragma unroll
          for (int j = 0; j < 32; ++j)
            f[j] = p.scale * act_f<ACT, true>(__uint_as_float(v[j]) + sb[c * 32 + j]);
          if (row_ok) {
            const int n0 = n_tile + c * 32;
            if (p.vec_ok && c * 32 + 32 <= n_valid) {
              if (p.R != nullptr) {
                const uint4* rp = reinterpret_cast<const uint4*>(p.R + m * p.ldr + n0);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  const uint4 r4 = __ldg(rp + q);
                  f[8 * q + 0] += bf16_lo(r4.x); f[8 * q + 1] += bf16_hi(r4.x);
                  f[8 * q + 2] += bf16_lo(r4.y); f[8 * q + 3] += bf16_hi(r4.y);
                  f[8 * q + 4] += bf16_lo(r4.z); f[8 * q + 5] += bf16_hi(r4.z);
                  f[8 * q + 6] += bf16_lo(r4.w); f[8 * q + 7] += bf16_hi(r4.w);
                }
              }
              uint4* yp = reinterpret_cast<uint4*>(Y + m * p.ldo + n0);
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                yp[q] = make_uint4(pack_bf16x2(f[8 * q + 0], f[8 * q + 1]),
                                   pack_bf16x2(f[8 * q + 2], f[8 * q + 3]),
                                   pack_bf16x2(f[8 * q + 4], f[8 * q + 5]),
                                   pack_bf16x2(f[8 * q + 6], f[8 * q + 7]));
              }
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                if (c * 32 + j < n_valid) {
                  float y = f[j];
                  if (p.R != nullptr) y += __bfloat162float(p.R[m * p.ldr + n0 + j]);
                  Y[m * p.ldo + n0 + j] = __float2bfloat16_rn(y);
                }
              }
            }
          }
        }
      } else if constexpr (EPI == EPI_SOFTMAX) {
        // pass 1: tile maximum of a = pre_act(z + b) over the valid columns of this row
        float mx = -INFINITY;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          if (c * 32 >= n_valid) break;
          uint32_t v[32];
          tmem_ld_32x32(t_acc + c * 32, v);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float z = act_f<ACT, true>(__uint_as_float(v[j]) + sb[c * 32 + j]);
            if (c * 32 + j < n_valid) mx = fmaxf(mx, z);
          }
        }
        // pass 2: numerators e = exp(a - mx), their fp32 sum, store e in the output dtype
        OutT* P = reinterpret_cast<OutT*>(p.out);
        float sum = 0.0f;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          if (c * 32 >= n_valid) break;
          uint32_t v[32];
          tmem_ld_32x32(t_acc + c * 32, v);
          tmem_ld_wait();
          float f[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float z = act_f<ACT, true>(__uint_as_float(v[j]) + sb[c * 32 + j]);
            f[j] = __expf(z - mx);
            if (c * 32 + j < n_valid) sum += f[j];
          }
          if (row_ok) {
            const int n0 = n_tile + c * 32;
            if (p.vec_ok && c * 32 + 32 <= n_valid) {
              if constexpr (sizeof(OutT) == 2) {
                uint4* yp = reinterpret_cast<uint4*>(P + m * p.ldo + n0);
#pragma unroll
                for (int q = 0; q < 4; ++q)
                  yp[q] = make_uint4(pack_bf16x2(f[8 * q + 0], f[8 * q + 1]),
                                     pack_bf16x2(f[8 * q + 2], f[8 * q + 3]),
                                     pack_bf16x2(f[8 * q + 4], f[8 * q + 5]),
                                     pack_bf16x2(f[8 * q + 6], f[8 * q + 7]));
              } else {
                float4* yp = reinterpret_cast<float4*>(P + m * p.ldo + n0);
#pragma unroll
                for (int q = 0; q < 8; ++q)
                  yp[q] = make_float4(f[4 * q], f[4 * q + 1], f[4 * q + 2], f[4 * q + 3]);
              }
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (c * 32 + j < n_valid) P[m * p.ldo + n0 + j] = from_f32<OutT>(f[j]);
            }
          }
        }
        if (row_ok) {
          float2* part = reinterpret_cast<float2*>(p.partial);
          part[m * p.tiles_n + tn] = make_float2(mx, sum);
        }
      } else if constexpr (EPI == EPI_ROWSUM) {
        float sum = 0.0f;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          if (c * 32 >= n_valid) break;
          uint32_t v[32];
          tmem_ld_32x32(t_acc + c * 32, v);
          tmem_ld_wait();
          float part = 0.0f;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float z = act_f<ACT, true>(__uint_as_float(v[j]) + sb[c * 32 + j]);
            if (c * 32 + j < n_valid) part += z;
          }
          sum += part;
        }
        if (row_ok) p.partial[m * p.tiles_n + tn] = sum;
      } else {  // EPI_CONV: a = act(z + b) stored NCHW; thread = pixel, column = output channel
        OutT* Yc = reinterpret_cast<OutT*>(p.out);
        const long long hw = static_cast<long long>(p.H) * p.Wd;
        const long long img = m / hw;
        const long long pix = m - img * hw;
        OutT* base = Yc + img * p.N * hw + pix;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          if (c * 32 >= n_valid) break;
          uint32_t v[32];
          tmem_ld_32x32(t_acc + c * 32, v);
          tmem_ld_wait();
          if (row_ok) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (c * 32 + j < n_valid) {
                const float y = act_f<ACT, true>(__uint_as_float(v[j]) + sb[c * 32 + j]);
                base[static_cast<long long>(c * 32 + j) * hw] = from_f32<OutT>(y);
              }
            }
          }
        }
      }
      // accumulator drained: hand it back to the UMMA issuer
      tc_fence_before_sync();
      mbar_arrive(&tmem_empty[a]);
      if (++a == 2) { a = 0; aph ^= 1u; }
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before_sync();
  __syncthreads();
  if (*abort_flag) {
    // give copies that may still be in flight time to land before the CTA's memory is reused
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 2 * BN);
  }
}

}  // namespace kf
