// Split-K form of the elementwise chain Y = scale*act(XW^T + b) + R for problems too small to
// fill the GPU with whole tiles: a cluster of S CTAs owns ONE 128 x BN output tile, CTA r
// contracts the r-th share of K into its own TMEM accumulator, and the S partial tiles are
// combined through distributed shared memory as a reduce-scatter: CTA r receives from every peer
// the BN/S columns it owns, adds the S partials in rank order (the same order whichever CTA
// adds, so results do not depend on the schedule), applies the epilogue to those columns and
// stores them.  No workspace, no atomics, one launch.
//
// Why: one tcgen05.mma on 128 rows costs about the same for 32 as for 256 columns, so narrow
// tiles cannot speed a small problem up; splitting K can.
//
// Synchronisation: every thread of every CTA executes the same two cluster barriers, whatever
// happened before (a wait that ran out only skips work), so no CTA can be left waiting.
#pragma once
#include <cstdlib>

#include "kf_umma.cuh"

namespace kf {

// STAGES = 3 with 128-column tiles keeps a CTA under half of the SM's shared memory, so that two
// CTAs share an SM: one streams its K share while the other exchanges and finishes its slice.
template <int BN, int S, int STAGES = 4>
struct SplitKCfg {
  static constexpr int kSlice = BN / S;                          // columns a CTA finishes
  static_assert(kSlice == 32 || kSlice == 64, "a CTA finishes one or two 32-column chunks");
  static constexpr int kStage = kBM * kBK * 2 + BN * kBK * 2;
  static constexpr int kStages = STAGES;
  static constexpr int kRing = kStage * kStages;
  static constexpr int kChunk = kBM * 32 * 4;                    // 128 rows x 32 fp32 = 16 KB
  static constexpr int kSlot = (kSlice / 32) * kChunk;           // one peer's partial slice
  static constexpr int kSlots = (S - 1) * kSlot;
  // Outgoing slices are staged locally and moved by bulk copies into the peers' incoming slots;
  // both areas reuse the operand ring: they are written only after every CTA's MMAs are done.
  static constexpr int kData = kRing > 2 * kSlots ? kRing : 2 * kSlots;
  static constexpr int kBarBytes = 128;
  static constexpr int kTotal = 1024 + kData + kBarBytes;
  static_assert(kTotal <= kMaxDynSmem, "shared-memory plan exceeds the per-CTA limit");
};

// (Remote st.shared::cluster stores moved the 96 KB of one exchange in 5 us; bulk_copy_to_peer,
// i.e. the copy engine, does it in a fraction of that.)

// f[j] = scale * act(f[j]) for a run-time activation code (this kernel is latency-bound; one
// instantiation per tile shape keeps the library small).
template <int ACT>
__device__ __forceinline__ void act32(float scale, float (&f)[32]) {
#pragma unroll
  for (int j = 0; j < 32; ++j) f[j] = scale * act_f<ACT, true>(f[j]);
}
__device__ __forceinline__ void apply_act32(int act, float scale, float (&f)[32]) {
  switch (act) {
    case ACT_RELU: act32<ACT_RELU>(scale, f); break;
    case ACT_GELU_TANH: act32<ACT_GELU_TANH>(scale, f); break;
    case ACT_SIGMOID: act32<ACT_SIGMOID>(scale, f); break;
    case ACT_GELU_ERF: act32<ACT_GELU_ERF>(scale, f); break;
    case ACT_SWISH: act32<ACT_SWISH>(scale, f); break;
    case ACT_TANH: act32<ACT_TANH>(scale, f); break;
    case ACT_HARDTANH: act32<ACT_HARDTANH>(scale, f); break;
    case ACT_CHAIN95: act32<ACT_CHAIN95>(scale, f); break;
    case ACT_NONE: act32<ACT_NONE>(scale, f); break;
    default:                                   // the run-time selected activations
#pragma unroll
      for (int j = 0; j < 32; ++j) f[j] = scale * act_rt<true>(act, f[j]);
      break;
  }
}

template <int BN, int S, int STAGES = 4>
__global__ void __launch_bounds__(kNumThreads, 1)
umma_splitk_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                   const UmmaParams p, const int act) {
  using C = SplitKCfg<BN, S, STAGES>;
  constexpr int kStages = C::kStages;
  const uint32_t rank = cluster_ctarank();
  const int tile = static_cast<int>(blockIdx.x) / S;
  const int tm = tile / p.tiles_n, tn = tile % p.tiles_n;
  const int kb0 = static_cast<int>(static_cast<long long>(rank) * p.k_blocks / S);
  const int kb1 = static_cast<int>(static_cast<long long>(rank + 1) * p.k_blocks / S);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* ring = smem;                 // operand stages, later the peers' partial slices
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + C::kData);
  uint64_t* empty = full + kStages;
  uint64_t* tmem_full = empty + kStages;
  uint64_t* recv_bar = tmem_full + 1;   // completes when every peer's slice has arrived
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(recv_bar + 1);
  volatile uint32_t* abort_flag = tmem_holder + 1;

  // warp index from a shuffle: provably warp-uniform, so the loops below keep their TMA / MMA
  // operands in uniform registers
  const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(tmem_full, 1);
    mbar_init(recv_bar, 1);
    *abort_flag = 0;
    mbar_init_fence();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
  }
  __syncwarp();
  if (warp == 1) { tmem_alloc(tmem_holder, BN); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;
  // a launch that was allowed to start early waits here for the kernel before it; the next
  // launch of the stream may start its prologue
  griddep_wait();
  griddep_launch_dependents();

  bool have_acc = false;       // epilogue threads: this CTA's accumulator is complete
  // Rows of the tile that exist (few for skinny problems), rounded up to whole warps: only they
  // are exchanged, added and stored; the epilogue warps above them only attend the barriers.
  const int rows32 = (min(kBM, p.M - tm * kBM) + 31) & ~31;
  if (warp == 0) {
    // every lane waits (warp-uniform loop), one elected lane issues
    int s = 0; uint32_t ph = 0;
    for (int kb = kb0; kb < kb1; ++kb) {
      bool ok = mbar_wait(&empty[s], ph ^ 1u, abort_flag, p.status, KF_DEV_TIMEOUT_PRODUCER);
      if (!__all_sync(0xffffffffu, ok)) break;
      uint8_t* sa = ring + s * C::kStage;
      if (elect_one()) {
        mbar_expect_tx(&full[s], C::kStage);
        tma_load_2d(sa, &tmA, &full[s], kb * kBK, tm * kBM);
        tma_load_2d(sa + kBM * kBK * 2, &tmB, &full[s], kb * kBK, tn * BN);
      }
      if (++s == kStages) { s = 0; ph ^= 1u; }
    }
    __syncwarp();
  } else if (warp == 1) {
    constexpr uint32_t idesc = umma_idesc_bf16_f32(kBM, BN);
    int s = 0; uint32_t ph = 0;
    bool ok = true;
    for (int kb = kb0; kb < kb1; ++kb) {
      ok = mbar_wait(&full[s], ph, abort_flag, p.status, KF_DEV_TIMEOUT_MMA);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t sa = smem_u32(ring + s * C::kStage);
      const uint64_t adesc = smem_desc_kmajor_sw128(sa);
      const uint64_t bdesc = smem_desc_kmajor_sw128(sa + kBM * kBK * 2);
      if (elect_one()) {
#pragma unroll
        for (int k = 0; k < kBK / kUmmaK; ++k)
          umma_f16_ss(tmem_base, adesc + 2u * k, bdesc + 2u * k, idesc, (kb > kb0 || k != 0) ? 1u : 0u);
        umma_commit(&empty[s]);
      }
      if (++s == kStages) { s = 0; ph ^= 1u; }
    }
    if (ok && elect_one()) umma_commit(tmem_full);
    __syncwarp();
  } else {
    bool ok = true;
    if (threadIdx.x == 64) {
      // armed before barrier A, i.e. before any peer sends: per peer and chunk, the live rows
      mbar_expect_tx(recv_bar, static_cast<uint32_t>((S - 1) * (C::kSlice / 32) * rows32 * 128));
      ok = mbar_wait(tmem_full, 0, abort_flag, p.status, KF_DEV_TIMEOUT_EPILOGUE);
    }
    have_acc = named_barrier_and(1, kEpiThreads, ok);
    tc_fence_after_sync();
  }

  // ---- barrier A: every CTA of the cluster has finished reading its operand ring and has
  // armed its receive barrier
  cluster_sync_all();

  const int quad = warp & 3;
  const int row = quad * 32 + lane;                       // tile row = TMEM lane (epilogue warps)
  const bool warp_live = quad * 32 < rows32;              // this warp's rows exist
  const uint32_t t_acc = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
  // Partial slices live as [slot][chunk of 32 columns][row][8 x 16 bytes], the 16-byte position
  // xor-ed with the row so that a quarter warp covers all banks.  Outgoing slots first, then
  // incoming ones.
  auto slot_off = [&](int slot, int chunk, int q) -> uint32_t {
    return static_cast<uint32_t>(slot * C::kSlot + chunk * C::kChunk + row * 128 + ((q ^ (row & 7)) << 4));
  };
  uint8_t* incoming = ring + C::kSlots;
  bool have_all = false;
  constexpr int kChunks = C::kSlice / 32;
  const long long m_row = static_cast<long long>(tm) * kBM + row;
  float bs[kChunks][32];
  uint4 rres[kChunks][4];
  bool r_vec[kChunks];
  if (warp >= 2) {
    if (have_acc) {
      // send: the columns peer d owns are staged locally, then one bulk copy carries them into
      // d's incoming slot for this rank
#pragma unroll 1
      for (int i = 1; i < S; ++i) {
        const uint32_t d = (rank + i) % S;
#pragma unroll 1
        for (int ch = 0; ch < C::kSlice / 32 && warp_live; ++ch) {
          uint32_t v[32];
          tmem_ld_32x32(t_acc + d * C::kSlice + ch * 32, v);
          tmem_ld_wait();
#pragma unroll
          for (int q = 0; q < 8; ++q)
            *reinterpret_cast<uint4*>(ring + slot_off(i - 1, ch, q)) =
                make_uint4(v[4 * q + 0], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        }
        fence_proxy_async_smem();
        named_barrier_sync(2, kEpiThreads);
        if (threadIdx.x == 64) {
          const int slot = static_cast<int>(rank < d ? rank : rank - 1);
          for (int ch = 0; ch < C::kSlice / 32; ++ch)      // a chunk's rows are contiguous: the live prefix
            bulk_copy_to_peer(mapa_shared(smem_u32(incoming + slot * C::kSlot + ch * C::kChunk), d),
                              smem_u32(ring + (i - 1) * C::kSlot + ch * C::kChunk),
                              static_cast<uint32_t>(rows32 * 128), mapa_shared(smem_u32(recv_bar), d));
        }
      }
    }
    // bias and residual of the columns this CTA finishes: loaded while the slices travel
#pragma unroll
    for (int ch = 0; ch < kChunks; ++ch) {
      const int n0 = tn * BN + static_cast<int>(rank) * C::kSlice + ch * 32;
      load_bias32(p, n0, bs[ch]);
      r_vec[ch] = p.vec_ok && n0 + 32 <= p.N;
      if (r_vec[ch] && p.R != nullptr && m_row < p.M) {
        const uint4* rp = reinterpret_cast<const uint4*>(p.R + m_row * p.ldr + n0);
#pragma unroll
        for (int q = 0; q < 4; ++q) rres[ch][q] = __ldg(rp + q);
      }
    }
    bool ok = have_acc;
    if (threadIdx.x == 64 && ok)
      ok = mbar_wait(recv_bar, 0, abort_flag, p.status, KF_DEV_TIMEOUT_EPILOGUE);
    have_all = named_barrier_and(1, kEpiThreads, ok);
  }

  if (warp >= 2 && have_all && warp_live) {
    __nv_bfloat16* Y = reinterpret_cast<__nv_bfloat16*>(p.out);
    const long long m = m_row;
    const bool row_ok = m < p.M;
#pragma unroll
    for (int ch = 0; ch < kChunks; ++ch) {
      const int col0 = static_cast<int>(rank) * C::kSlice + ch * 32;
      const int n0 = tn * BN + col0;
      if (n0 < p.N) {
        uint32_t own[32];
        tmem_ld_32x32(t_acc + col0, own);
        tmem_ld_wait();
        float f[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) f[j] = 0.0f;
#pragma unroll 1
        for (int src = 0; src < S; ++src) {          // rank order: the sum does not depend on who adds
          if (src == static_cast<int>(rank)) {
#pragma unroll
            for (int j = 0; j < 32; ++j) f[j] += __uint_as_float(own[j]);
          } else {
            const int slot = src < static_cast<int>(rank) ? src : src - 1;
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const float4 t = *reinterpret_cast<const float4*>(incoming + slot_off(slot, ch, q));
              f[4 * q + 0] += t.x; f[4 * q + 1] += t.y; f[4 * q + 2] += t.z; f[4 * q + 3] += t.w;
            }
          }
        }
#pragma unroll
        for (int j = 0; j < 32; ++j) f[j] += bs[ch][j];
        apply_act32(act, p.scale, f);
        if (row_ok) {
          if (r_vec[ch]) {
            if (p.R != nullptr) {
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const uint4 r4 = rres[ch][q];
                f[8 * q + 0] += bf16_lo(r4.x); f[8 * q + 1] += bf16_hi(r4.x);
                f[8 * q + 2] += bf16_lo(r4.y); f[8 * q + 3] += bf16_hi(r4.y);
                f[8 * q + 4] += bf16_lo(r4.z); f[8 * q + 5] += bf16_hi(r4.z);
                f[8 * q + 6] += bf16_lo(r4.w); f[8 * q + 7] += bf16_hi(r4.w);
              }
            }
            uint4* yp = reinterpret_cast<uint4*>(Y + m * p.ldo + n0);
#pragma unroll
            for (int q = 0; q < 4; ++q)
              yp[q] = make_uint4(pack_bf16x2(f[8 * q + 0], f[8 * q + 1]),
                                 pack_bf16x2(f[8 * q + 2], f[8 * q + 3]),
                                 pack_bf16x2(f[8 * q + 4], f[8 * q + 5]),
                                 pack_bf16x2(f[8 * q + 6], f[8 * q + 7]));
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (n0 + j < p.N) {
                float y = f[j];
                if (p.R != nullptr) y += __bfloat162float(p.R[m * p.ldr + n0 + j]);
                Y[m * p.ldo + n0 + j] = __float2bfloat16_rn(y);
              }
            }
          }
        }
      }
    }
  }

  // ---- barrier B: no CTA leaves while a peer may still copy to or from its shared memory (a
  // CTA arrives here only after all its incoming slices have landed, or after giving up)
  cluster_sync_all();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, BN);
  }
}

template <int BN, int S, int STAGES = 4>
inline cudaError_t launch_splitk_instance(const CUtensorMap& tmA, const CUtensorMap& tmB,
                                          const UmmaParams& p, int act, cudaStream_t st) {
  using C = SplitKCfg<BN, S, STAGES>;
  auto kern = umma_splitk_kernel<BN, S, STAGES>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kTotal);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(p.num_tiles) * S, 1, 1);
  cfg.blockDim = dim3(kNumThreads, 1, 1);
  cfg.dynamicSmemBytes = C::kTotal;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = S;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  static const bool pdl = getenv("KF_NO_PDL") == nullptr;
  cfg.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, kern, tmA, tmB, p, act);
}

}  // namespace kf
