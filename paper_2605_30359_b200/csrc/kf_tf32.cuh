// fp32 elementwise chain Y = scale*act(XW^T + b) + R on the tensor cores with fp32-level
// accuracy ("3xTF32"): every fp32 operand is split into hi = its leading 11 significand bits
// (exactly a TF32 number) and lo = the next 11 bits of the remainder, and
//     x*w ~= hi(x)*lo(w) + lo(x)*hi(w) + hi(x)*hi(w)
// (the dropped lo*lo term and the truncation of lo are below 2^-21 |x*w|), accumulated in fp32
// in TMEM by three tcgen05.mma kind::tf32 per K step.  A prepass writes the four split operands
// (dense, rows padded to 16 bytes) into the workspace, so the GEMM kernel's loads are plain
// TMA tiles and X / W may have any pitch and alignment.
//
// A stage holds 16 fp32 columns (64-byte rows, 64-byte TMA swizzle) of all four split operands:
// 48 KB at BN = 256, so four stages fit; with 128-byte rows only two did and the loads' latency
// showed (2.5-3 us per K block of 32 instead of the 1 us its 12 MMAs take).  A K step is 8
// elements = 32 bytes.  Roles: warp 0
// TMA producer, warp 1 MMA issuer, warps 2..5 epilogue (thread = accumulator row).
//
// Accumulation: the tensor core adds into its fp32 accumulator with truncation, an error of
// up to 2^-24 per MMA that always points the same way (measured: 9.6e-5 absolute on outputs of
// magnitude 1 after the 1536 MMAs of K = 4096, eleven times the error of an fp32 FMA loop).
// So K is cut into chunks of kTfChunk K blocks: the MMAs of a chunk start a fresh accumulator
// (TMEM columns [0, BN)), and the epilogue warps add each finished chunk, rounding to nearest,
// into a running sum kept in TMEM columns [BN, 2*BN) with tcgen05.ld / tcgen05.st.  The MMAs of
// the next chunk wait only for that short drain; the tile's real epilogue then reads the sum
// while the next tile's first chunk is already running.  The epilogue moves 32-column pieces
// through shared memory so that global reads (R) and writes (Y) run along rows.
#pragma once

#include "kf_internal.h"

namespace kf {

constexpr int kTfBK = 16;          // fp32 elements per stage row (64 bytes)
constexpr int kTfUmmaK = 8;        // K per tcgen05.mma kind::tf32
constexpr int kTfChunk = 32;       // K blocks (of 16) per accumulation chunk: K = 512, 192 MMAs

template <int BN>
struct Tf32Cfg {
  static constexpr int kTileA = kBM * kTfBK * 4;                  // 8 KB
  static constexpr int kTileB = BN * kTfBK * 4;
  static constexpr int kStage = 2 * kTileA + 2 * kTileB;          // hi and lo of both operands
  static constexpr int kPiece = kBM * 32 * 4;                     // one fp32 piece: 16 KB
  static constexpr int kStaging = 2 * kPiece;                     // two alternating output pieces
  static constexpr int kBarBytes = 256;
  static constexpr int kStages = (kMaxDynSmem - 1024 - kStaging - kBarBytes) / kStage;
  static_assert(kStages >= 2, "at least two stages");
  static constexpr int kTotal = 1024 + kStages * kStage + kStaging + kBarBytes;
};

// Instruction descriptor for kind::tf32: A and B formats 2 (tf32), fp32 accumulate, K-major.
__host__ __device__ constexpr uint32_t umma_idesc_tf32_f32(uint32_t M, uint32_t N) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((N >> 3) << 17) | ((M >> 4) << 24);
}

__device__ __forceinline__ void umma_tf32_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                             uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n"
      "}\n"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// 32 consecutive TMEM columns of this warp's 32 lanes <- registers.
__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]),
        "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]),
        "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),
        "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
        "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() {
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor for a K-major operand tile whose rows are 64 bytes written by
// TMA with SWIZZLE_64B: 8-row groups 512 bytes apart, swizzle mode 4 (64 B); other fields as in
// smem_desc_kmajor_sw128.  The tile base is 1024-byte aligned; a K step adds 32 bytes.
__device__ __forceinline__ uint64_t smem_desc_kmajor_sw64(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>(512 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(4) << 61;
  return d;
}

// hi = x with the low 13 mantissa bits cleared; lo = (x - hi) with its low 13 bits cleared.
// x - hi is exact in fp32.  Non-finite x gives hi = x, lo = 0.
__device__ __forceinline__ void tf32_split(float x, float& hi, float& lo) {
  hi = __uint_as_float(__float_as_uint(x) & 0xFFFFE000u);
  const float r = x - hi;
  lo = (r == r && fabsf(r) <= 3.0e38f) ? __uint_as_float(__float_as_uint(r) & 0xFFFFE000u) : 0.0f;
}

// in [rows, ld] fp32 (any alignment) -> hi, lo dense [rows, kp] (kp = K rounded up to 4;
// the padding columns are written as zeros).  One thread per group of four columns.
__global__ void __launch_bounds__(256)
tf32_split_kernel(long long rows, int K, int kp, const float* __restrict__ in, long long ld,
                  int vec_in, float* __restrict__ hi, float* __restrict__ lo) {
  const int gpr = kp / 4;                                  // groups per row
  const long long total = rows * gpr;
  for (long long g = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; g < total;
       g += static_cast<long long>(gridDim.x) * blockDim.x) {
    const long long r = g / gpr;
    const int k = static_cast<int>(g - r * gpr) * 4;
    const float* src = in + r * ld + k;
    float x[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    if (vec_in && k + 4 <= K) {
      const float4 t = __ldg(reinterpret_cast<const float4*>(src));
      x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) if (k + j < K) x[j] = __ldg(src + j);
    }
    float h[4], l[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) tf32_split(x[j], h[j], l[j]);
    reinterpret_cast<float4*>(hi)[g] = make_float4(h[0], h[1], h[2], h[3]);
    reinterpret_cast<float4*>(lo)[g] = make_float4(l[0], l[1], l[2], l[3]);
  }
}

// f[j] = scale * act(f[j]) with the library-accurate activations (fp32 chains).
template <int ACT>
__device__ __forceinline__ void act32_precise(float scale, float (&f)[32]) {
#pragma unroll
  for (int j = 0; j < 32; ++j) f[j] = scale * act_f<ACT, false>(f[j]);
}
__device__ __forceinline__ void apply_act32_precise(int act, float scale, float (&f)[32]) {
  switch (act) {
    case ACT_RELU: act32_precise<ACT_RELU>(scale, f); break;
    case ACT_GELU_TANH: act32_precise<ACT_GELU_TANH>(scale, f); break;
    case ACT_SIGMOID: act32_precise<ACT_SIGMOID>(scale, f); break;
    case ACT_GELU_ERF: act32_precise<ACT_GELU_ERF>(scale, f); break;
    case ACT_SWISH: act32_precise<ACT_SWISH>(scale, f); break;
    case ACT_TANH: act32_precise<ACT_TANH>(scale, f); break;
    case ACT_HARDTANH: act32_precise<ACT_HARDTANH>(scale, f); break;
    case ACT_CHAIN95: act32_precise<ACT_CHAIN95>(scale, f); break;
    case ACT_NONE: act32_precise<ACT_NONE>(scale, f); break;
    default:                                   // the run-time selected activations
#pragma unroll
      for (int j = 0; j < 32; ++j) f[j] = scale * act_rt<false>(act, f[j]);
      break;
  }
}

// Byte offset of 16-byte chunk j (0..7) of row r in a 128-row x 128-byte piece, chunk position
// xor-ed with the row: conflict-free for lanes = consecutive rows and for lanes = consecutive
// columns of one row alike.
__device__ __forceinline__ uint32_t piece32_off(int r, int j) {
  return static_cast<uint32_t>(r * 128 + ((j ^ (r & 7)) << 4));
}

template <int BN>
__global__ void __launch_bounds__(kNumThreads, 1)
tf32x3_chain_kernel(const __grid_constant__ CUtensorMap tmAh, const __grid_constant__ CUtensorMap tmAl,
                    const __grid_constant__ CUtensorMap tmBh, const __grid_constant__ CUtensorMap tmBl,
                    const Tf32Params p) {
  using C = Tf32Cfg<BN>;
  constexpr int kStages = C::kStages;
  const int cta = static_cast<int>(blockIdx.x), ncta = static_cast<int>(gridDim.x);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* ring = smem;
  uint8_t* ybuf = smem + kStages * C::kStage;
  uint64_t* full = reinterpret_cast<uint64_t*>(ybuf + 2 * C::kPiece);   // ybuf: two pieces
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

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    // every lane waits (warp-uniform loop), one elected lane issues
    {
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      for (int tile = cta; tile < p.num_tiles && ok; tile += ncta) {
        const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          ok = mbar_wait(&empty[s], ph ^ 1u, abort_flag, p.status, KF_DEV_TIMEOUT_PRODUCER);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          uint8_t* st = ring + s * C::kStage;
          if (elect_one()) {
            mbar_expect_tx(&full[s], C::kStage);
            tma_load_2d(st, &tmAh, &full[s], kb * kTfBK, tm * kBM);
            tma_load_2d(st + C::kTileA, &tmAl, &full[s], kb * kTfBK, tm * kBM);
            tma_load_2d(st + 2 * C::kTileA, &tmBh, &full[s], kb * kTfBK, tn * BN);
            tma_load_2d(st + 2 * C::kTileA + C::kTileB, &tmBl, &full[s], kb * kTfBK, tn * BN);
          }
          if (++s == kStages) { s = 0; ph ^= 1u; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    {
      constexpr uint32_t idesc = umma_idesc_tf32_f32(kBM, BN);
      int s = 0; uint32_t ph = 0; uint32_t cph = 0;      // cph: parity of the chunk handshake
      bool ok = true;
      for (int tile = cta; tile < p.num_tiles && ok; tile += ncta) {
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          const bool chunk_start = kb % kTfChunk == 0;
          if (chunk_start) {                       // the epilogue has drained the previous chunk
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
              // +32 bytes per K step inside the 64-byte swizzled row = +2 in the address field;
              // the two correction terms first, the leading term last
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
    constexpr int PIECES = BN / 32;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int et = threadIdx.x - 64;
    const int er = et >> 5;                      // row group of this warp in the copy loops
    const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
    const bool has_r = p.R != nullptr;
    uint32_t cph = 0;
    const int n_chunks = (p.k_blocks + kTfChunk - 1) / kTfChunk;
    bool alive = true;
    for (int tile = cta; tile < p.num_tiles && alive; tile += ncta) {
      const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
      const long long m0 = static_cast<long long>(tm) * kBM;
      const int n_tile = tn * BN;
      const int n_valid = min(BN, p.N - n_tile);
      const uint32_t t_acc = tmem_base + lane_off;                                 // chunk accumulator
      const uint32_t t_sum = tmem_base + static_cast<uint32_t>(BN) + lane_off;     // running sum
      // fold every chunk into the running sum (round to nearest), then release the accumulator
      for (int ch = 0; ch < n_chunks; ++ch) {
        bool ok = true;
        if (et == 0) ok = mbar_wait(&tmem_full[0], cph, abort_flag, p.status, KF_DEV_TIMEOUT_EPILOGUE);
        ok = named_barrier_and(1, kEpiThreads, ok);
        if (!ok) { alive = false; break; }
        cph ^= 1u;
        tc_fence_after_sync();
#pragma unroll 1
        for (int c = 0; c < PIECES; ++c) {
          if (c * 32 >= n_valid) break;
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
      // The tile's epilogue, from the running sum.  Per 32-column piece: the residual is
      // fetched in the row-contiguous layout of the final store (registers), the activation
      // is computed one row per thread into a swizzled shared-memory piece, and after one
      // barrier the piece leaves along rows with the residual added on the way out.  Two
      // pieces of shared memory alternate, so one barrier per piece is enough.
#pragma unroll 1
      for (int c = 0; c < PIECES; ++c) {
        if (c * 32 >= n_valid) break;            // uniform across the CTA
        const int n0 = n_tile + c * 32;
        uint8_t* yb = ybuf + (c & 1) * C::kPiece;
        const bool vec = p.vec_ok && n0 + 32 <= p.N;
        float4 rr4[8];
        float rr1[32];
        if (has_r) {
          if (vec) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const long long mr = m0 + i * 16 + (et >> 3);
              rr4[i] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
              if (mr < p.M) rr4[i] = __ldg(reinterpret_cast<const float4*>(p.R + mr * p.ldr + n0) + (et & 7));
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const long long mr = m0 + i * 4 + er;
              rr1[i] = (n0 + lane < p.N && mr < p.M) ? __ldg(p.R + mr * p.ldr + n0 + lane) : 0.0f;
            }
          }
        }
        uint32_t v[32];
        tmem_ld_32x32(t_sum + c * 32, v);
        float f[32];
#pragma unroll
        for (int j = 0; j < 32; ++j)
          f[j] = (p.bias != nullptr && n0 + j < p.N) ? __ldg(p.bias + n0 + j) : 0.0f;
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) f[j] += __uint_as_float(v[j]);
        apply_act32_precise(p.act, p.scale, f);
#pragma unroll
        for (int q = 0; q < 8; ++q)
          *reinterpret_cast<float4*>(yb + piece32_off(row, q)) =
              make_float4(f[4 * q + 0], f[4 * q + 1], f[4 * q + 2], f[4 * q + 3]);
        named_barrier_sync(2, kEpiThreads);
        if (vec) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int r = i * 16 + (et >> 3);
            if (m0 + r < p.M) {
              float4 y = *reinterpret_cast<const float4*>(yb + piece32_off(r, et & 7));
              if (has_r) { y.x += rr4[i].x; y.y += rr4[i].y; y.z += rr4[i].z; y.w += rr4[i].w; }
              reinterpret_cast<float4*>(p.out + (m0 + r) * p.ldo + n0)[et & 7] = y;
            }
          }
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int r = i * 4 + er;
            if (n0 + lane < p.N && m0 + r < p.M) {
              float y = *reinterpret_cast<const float*>(yb + piece32_off(r, lane >> 2) + (lane & 3) * 4);
              if (has_r) y += rr1[i];
              p.out[(m0 + r) * p.ldo + n0 + lane] = y;
            }
          }
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
inline cudaError_t launch_tf32_instance(const CUtensorMap& ah, const CUtensorMap& al,
                                        const CUtensorMap& bh, const CUtensorMap& bl,
                                        const Tf32Params& p, int grid, cudaStream_t st) {
  using C = Tf32Cfg<BN>;
  auto kern = tf32x3_chain_kernel<BN>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kTotal);
  if (e != cudaSuccess) return e;
  kern<<<grid, kNumThreads, C::kTotal, st>>>(ah, al, bh, bl, p);
  return cudaGetLastError();
}

}  // namespace kf
