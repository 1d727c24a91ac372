// fp32 3x3 convolution (pad 1) + bias + activation on the tensor cores, as an implicit GEMM
// with split fp32 operands ("3xTF32", see kf_tf32.cuh): A = one tap's weights (rows = output
// channels), B = the tap-shifted window of tile_px pixels x 16 input channels fetched by a 4-D
// TMA box from NHWC copies of the activations (out-of-image pixels read zeros: the padding).
// A prepass writes hi / lo NHWC copies of x (channels padded to a multiple of 16) and hi / lo
// weights [tap][o][c] into the workspace.  Tiles, chunked accumulation into an fp32 running sum
// in TMEM and the roles are those of tf32x3_chain_kernel; the epilogue thread is an output
// channel, whose 32 pixels of a piece are 128 contiguous bytes of the NCHW output.
#pragma once

#include "kf_tf32.cuh"

namespace kf {

// x NCHW fp32 -> xh, xl NHWC [Nb][H*W][Cp] and w OIHW -> wh, wl [9][Cout][Cp], Cp a multiple of 16,
// padding channels zero.  One thread per pixel and group of four channels (pixels fastest).
__global__ void __launch_bounds__(256)
conv_prep_tf32_kernel(int Nb, int Cin, int Cp, long long hw, int Cout, const float* __restrict__ x,
                      const float* __restrict__ w, float* __restrict__ xh, float* __restrict__ xl,
                      float* __restrict__ wh, float* __restrict__ wl, long long x_items) {
  const long long gid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  const int cg = Cp / 4;
  if (gid < x_items) {
    const long long px = gid % hw;
    long long t = gid / hw;
    const int g = static_cast<int>(t % cg);
    const long long n = t / cg;
    float h[4], l[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int c = g * 4 + i;
      const float v = c < Cin ? __ldg(x + (n * Cin + c) * hw + px) : 0.0f;
      tf32_split(v, h[i], l[i]);
    }
    const long long o = (n * hw + px) * Cp + g * 4;
    *reinterpret_cast<float4*>(xh + o) = make_float4(h[0], h[1], h[2], h[3]);
    *reinterpret_cast<float4*>(xl + o) = make_float4(l[0], l[1], l[2], l[3]);
  } else {
    const long long i = gid - x_items;                   // index into w?[tap][o][Cp]
    const long long total = 9ll * Cout * Cp;
    if (i < total) {
      const int c = static_cast<int>(i % Cp);
      const int o = static_cast<int>((i / Cp) % Cout);
      const int tap = static_cast<int>(i / (static_cast<long long>(Cp) * Cout));
      float h = 0.0f, l = 0.0f;
      if (c < Cin) tf32_split(w[(static_cast<long long>(o) * Cin + c) * 9 + tap], h, l);
      wh[i] = h;
      wl[i] = l;
    }
  }
}

template <int BN>
__global__ void __launch_bounds__(kNumThreads, 1)
tf32x3_conv_kernel(const __grid_constant__ CUtensorMap tmAh, const __grid_constant__ CUtensorMap tmAl,
                   const __grid_constant__ CUtensorMap tmBh, const __grid_constant__ CUtensorMap tmBl,
                   const Tf32ConvParams p) {
  using C = Tf32Cfg<BN>;
  constexpr int kStages = C::kStages;
  const int cta = static_cast<int>(blockIdx.x), ncta = static_cast<int>(gridDim.x);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* ring = smem;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kStages * C::kStage + C::kStaging);
  uint64_t* empty = full + kStages;
  uint64_t* tmem_full = empty + kStages;
  uint64_t* tmem_empty = tmem_full + 2;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(tmem_empty + 2);
  volatile uint32_t* abort_flag = tmem_holder + 1;

  // warp index from a shuffle: provably warp-uniform, so the loops below keep their TMA / MMA
  // operands in uniform registers
  const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(&tmem_full[0], 1);
    mbar_init(&tmem_empty[0], kEpiThreads / 32);
    *abort_flag = 0;
    mbar_init_fence();
    tma_prefetch_desc(&tmAh); tma_prefetch_desc(&tmAl);
    tma_prefetch_desc(&tmBh); tma_prefetch_desc(&tmBl);
  }
  __syncwarp();
  if (warp == 1) { tmem_alloc(tmem_holder, 2 * BN); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;
  const uint32_t b_bytes = static_cast<uint32_t>(p.tile_px) * kTfBK * 4;   // one B operand per stage

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    // every lane waits (warp-uniform loop), one elected lane issues
    {
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      for (int tile = cta; tile < p.num_tiles && ok; tile += ncta) {
        const int tm = tile % p.tiles_m, tn = tile / p.tiles_m;
        const int img = tn / p.tiles_per_image;
        const int pt = tn % p.tiles_per_image;
        const int h0 = (pt / p.w_segs) * p.rows_per_tile;
        const int x0 = (pt % p.w_segs) * (p.Wd / p.w_segs);
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          ok = mbar_wait(&empty[s], ph ^ 1u, abort_flag, p.status, KF_DEV_TIMEOUT_PRODUCER);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          const int tap = kb / p.kb_per_tap, cb = kb % p.kb_per_tap;
          const int r = tap / 3, sx = tap % 3;
          uint8_t* st = ring + s * C::kStage;
          if (elect_one()) {
            mbar_expect_tx(&full[s], 2 * C::kTileA + 2 * b_bytes);
            tma_load_2d(st, &tmAh, &full[s], cb * kTfBK, tap * p.Cout + tm * kBM);
            tma_load_2d(st + C::kTileA, &tmAl, &full[s], cb * kTfBK, tap * p.Cout + tm * kBM);
            tma_load_4d(st + 2 * C::kTileA, &tmBh, &full[s], cb * kTfBK, x0 + sx - 1, h0 + r - 1, img);
            tma_load_4d(st + 2 * C::kTileA + C::kTileB, &tmBl, &full[s], cb * kTfBK, x0 + sx - 1,
                        h0 + r - 1, img);
          }
          if (++s == kStages) { s = 0; ph ^= 1u; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    {
      const uint32_t idesc = umma_idesc_tf32_f32(kBM, static_cast<uint32_t>(p.tile_px));
      int s = 0; uint32_t ph = 0; uint32_t cph = 0;
      bool ok = true;
      for (int tile = cta; tile < p.num_tiles && ok; tile += ncta) {
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          const bool chunk_start = kb % kTfChunk == 0;
          if (chunk_start) {
            ok = mbar_wait(&tmem_empty[0], cph ^ 1u, abort_flag, p.status, KF_DEV_TIMEOUT_MMA);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
          }
          ok = mbar_wait(&full[s], ph, abort_flag, p.status, KF_DEV_TIMEOUT_MMA);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t st = smem_u32(ring + s * C::kStage);
          const uint64_t ah = smem_desc_kmajor_sw64(st);
          const uint64_t al = smem_desc_kmajor_sw64(st + C::kTileA);
          const uint64_t bh = smem_desc_kmajor_sw64(st + 2 * C::kTileA);
          const uint64_t bl = smem_desc_kmajor_sw64(st + 2 * C::kTileA + C::kTileB);
          const bool chunk_end = kb % kTfChunk == kTfChunk - 1 || kb == p.k_blocks - 1;
          if (elect_one()) {
#pragma unroll
            for (int k = 0; k < kTfBK / kTfUmmaK; ++k) {
              umma_tf32_ss(tmem_base, ah + 2u * k, bl + 2u * k, idesc, (chunk_start && k == 0) ? 0u : 1u);
              umma_tf32_ss(tmem_base, al + 2u * k, bh + 2u * k, idesc, 1u);
              umma_tf32_ss(tmem_base, ah + 2u * k, bh + 2u * k, idesc, 1u);
            }
            umma_commit(&empty[s]);
            if (chunk_end) umma_commit(&tmem_full[0]);
          }
          if (++s == kStages) { s = 0; ph ^= 1u; }
          if (chunk_end) cph ^= 1u;
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int quad = warp & 3;
    const int row = quad * 32 + lane;            // output channel inside the tile
    const int et = threadIdx.x - 64;
    const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
    const long long hw = static_cast<long long>(p.H) * p.Wd;
    const int pieces = p.tile_px / 32;
    const int n_chunks = (p.k_blocks + kTfChunk - 1) / kTfChunk;
    uint32_t cph = 0;
    bool alive = true;
    for (int tile = cta; tile < p.num_tiles && alive; tile += ncta) {
      const int tm = tile % p.tiles_m, tn = tile / p.tiles_m;
      const int img = tn / p.tiles_per_image;
      const int pt = tn % p.tiles_per_image;
      const uint32_t t_acc = tmem_base + lane_off;
      const uint32_t t_sum = tmem_base + static_cast<uint32_t>(BN) + lane_off;
      for (int ch = 0; ch < n_chunks; ++ch) {
        bool ok = true;
        if (et == 0) ok = mbar_wait(&tmem_full[0], cph, abort_flag, p.status, KF_DEV_TIMEOUT_EPILOGUE);
        ok = named_barrier_and(1, kEpiThreads, ok);
        if (!ok) { alive = false; break; }
        cph ^= 1u;
        tc_fence_after_sync();
#pragma unroll 1
        for (int c = 0; c < pieces; ++c) {
          uint32_t v[32];
          tmem_ld_32x32(t_acc + c * 32, v);
          if (ch > 0) {
            uint32_t sv[32];
            tmem_ld_32x32(t_sum + c * 32, sv);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j)
              v[j] = __float_as_uint(__uint_as_float(sv[j]) + __uint_as_float(v[j]));
          } else {
            tmem_ld_wait();
          }
          tmem_st_32x32(t_sum + c * 32, v);
        }
        tmem_st_wait();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tmem_empty[0]);
      }
      if (!alive) break;
      const int cho = tm * kBM + row;
      const bool ch_ok = cho < p.Cout;
      const float bias_v = (p.bias != nullptr && ch_ok) ? __ldg(p.bias + cho) : 0.0f;
      const int px0 = pt * p.tile_px;
      const int px_valid = static_cast<int>(min(static_cast<long long>(p.tile_px), hw - px0));
      float* dst = p.out + (static_cast<long long>(img) * p.Cout + cho) * hw + px0;
#pragma unroll 1
      for (int c = 0; c < pieces; ++c) {
        const int left = px_valid - c * 32;
        if (left <= 0) break;                      // uniform across the CTA
        uint32_t v[32];
        tmem_ld_32x32(t_sum + c * 32, v);
        tmem_ld_wait();
        float f[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) f[j] = __uint_as_float(v[j]) + bias_v;
        apply_act32_precise(p.act, 1.0f, f);
        if (!ch_ok) continue;
        if (p.vec_ok && left >= 32) {
#pragma unroll
          for (int q = 0; q < 8; ++q)
            reinterpret_cast<float4*>(dst + c * 32)[q] =
                make_float4(f[4 * q + 0], f[4 * q + 1], f[4 * q + 2], f[4 * q + 3]);
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (j < left) dst[c * 32 + j] = f[j];
        }
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before_sync();
  __syncthreads();
  if (*abort_flag) {
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

template <int BN>
inline cudaError_t launch_tf32_conv_instance(const CUtensorMap& ah, const CUtensorMap& al,
                                             const CUtensorMap& bh, const CUtensorMap& bl,
                                             const Tf32ConvParams& p, int grid, cudaStream_t st) {
  using C = Tf32Cfg<BN>;
  auto kern = tf32x3_conv_kernel<BN>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kTotal);
  if (e != cudaSuccess) return e;
  kern<<<grid, kNumThreads, C::kTotal, st>>>(ah, al, bh, bl, p);
  return cudaGetLastError();
}

}  // namespace kf
