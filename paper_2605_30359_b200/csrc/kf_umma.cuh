// kf_umma.cuh -- the tensor-core mainloop shared by every bf16 chain, with its epilogues.
//
// One persistent CTA per SM walks output tiles of 128 rows x BN columns.  Warp roles:
//   warp 0             TMA producer: fills a ring of shared-memory stages (A 128x64, B BNx64
//                      bf16, 128-byte swizzle) and signals `full[s]` by transaction bytes.  For
//                      the convolution A is the weight tile of one tap (rows = output channels)
//                      and B the shifted window of BN pixels, so that the accumulator comes out
//                      channel-major like the NCHW output.
//   warp 1             UMMA issuer: four tcgen05.mma (K=16 each) per stage into one of two
//                      TMEM accumulators, tcgen05.commit to `empty[s]` (stage free) and, after
//                      the last K block, to `tmem_full[a]`.
//                      In both warps every lane runs the loop and waits, a vote makes the outcome
//                      warp-uniform and one elected lane issues (operands in uniform registers).
//   warps 2..5 (and 6..9 where a second epilogue group runs: see epi_groups)
//                      epilogue: tcgen05.ld the accumulator (thread = one row of the tile; a
//                      group owns BN / groups columns), apply the chain's epilogue in fp32
//                      registers and release the accumulator through `tmem_empty[a]` so the next
//                      tile's MMAs overlap.  Results leave through shared-memory staging and TMA
//                      stores (the residual arrives the same way): a row-per-lane global access
//                      touches 32 cache lines per instruction and was measured to cost the
//                      mainloop 10-15 % of its speed; a direct path remains for operands whose
//                      alignment TMA cannot take.
// Every wait is bounded (mbar_wait); a wait that runs out raises the CTA's abort flag, all
// roles leave their loops, in-flight copies are given time to land, TMEM is freed.
#pragma once

#include "kf_act.cuh"
#include "kf_ptx.cuh"

namespace kf {

// EPI_CONV_GN: the convolution with GroupNorm finished inside the epilogue; the CTAs that hold
// the tiles of one image form a cluster and exchange the group statistics through distributed
// shared memory (two epilogue groups).
// EPI_SOFTMAX_CL: the softmax of a row whose column tiles are held by the CTAs of one cluster: the
// per-row (maximum, sum) pairs travel through distributed shared memory and every CTA stores
// final probabilities (one kernel, no second pass).
// EPI_CONV_GNX: the same chain on all SMs without clusters: the tiles of an image are held by
// neighbouring CTAs of one co-resident (cooperative) grid, which exchange the group statistics
// through global memory; the epilogue is software-pipelined so that the exchange is not waited for.
// EPI_SOFTMAX_GX: the row softmax of a wide row (several 256-column tiles) in ONE kernel without
// clusters: the tiles of a row block sit on neighbouring CTAs of a co-resident (cooperative) grid,
// which exchange per-row (maximum, sum) through global memory; the numerators wait in registers.
enum : int { EPI_ELEMENTWISE = 0, EPI_SOFTMAX = 1, EPI_ROWSUM = 2, EPI_CONV = 3, EPI_CONV_GN = 4,
             EPI_SOFTMAX_CL = 5, EPI_CONV_GNX = 6, EPI_SOFTMAX_GX = 7 };
constexpr bool is_conv(int epi) { return epi == 3 || epi == 4 || epi == 6; }
constexpr bool is_softmax(int epi) { return epi == 1 || epi == 5; }
constexpr bool is_cluster_epi(int epi) { return epi == 4 || epi == 5; }

constexpr int kBM = 128;          // tile rows = UMMA M = TMEM lanes
constexpr int kBK = 64;           // K per stage: 64 bf16 = one 128-byte swizzled row
constexpr int kUmmaK = 16;        // K per tcgen05.mma for 16-bit inputs
constexpr int kEpiThreads = 128;  // threads of one epilogue group: four warps, one per TMEM lane quarter
constexpr int kNumThreads = 192;  // 6 warps: producer, UMMA issuer, epilogue
// The softmax epilogue is the longest (two TMEM passes, an exponential per element) and with
// one warp per scheduler it is latency-bound, so it runs as TWO groups of four warps, each
// owning half of the tile's columns as a slice of its own: own statistics, own staging, own
// named barriers, own TMA stores.  The second pass combines slices, so the groups never talk.
// Epilogue groups of four warps, each owning BN / groups columns of every tile: two for the softmax
// first pass and for the elementwise chain (one warp per scheduler left the epilogue latency-bound:
// a 128x256 tile took 7 us to drain, more than its MMAs take up to K = 1536), one where a group
// would be narrower than a 32-column piece and for the other epilogues.
// The CTA-pair form (large K only: its epilogue hides behind the MMAs anyway, and the extra warps
// cost it 2 %) keeps one group.
constexpr int epi_groups(int epi, int bn, bool cta2) {
  return epi == 1 /* EPI_SOFTMAX */ || epi == 4 /* EPI_CONV_GN */ || epi == 5 /* EPI_SOFTMAX_CL */ ||
                 epi == 6 /* EPI_CONV_GNX */ || epi == 7 /* EPI_SOFTMAX_GX */ ||
                 (epi == 0 /* EPI_ELEMENTWISE */ && bn >= 64 && !cta2)
             ? 2 : 1;
}
// (EPI_CONV_GNX carries one more warp, which does the epilogue's global-memory work: see conv_gnx_helper)
constexpr int num_threads(int epi, int bn, bool cta2) {
  return 64 + kEpiThreads * epi_groups(epi, bn, cta2) + (epi == 6 /* EPI_CONV_GNX */ ? 32 : 0);
}
constexpr int kPieceCols = 32;    // epilogue piece: 128 rows x 32 columns
constexpr int kPieceBytes = kBM * kPieceCols * 2;   // 8 KB of bf16
constexpr int kMaxDynSmem = 232448;                 // 227 KB opt-in limit per CTA

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
  int act_rt;                  // activation code, read by the ACT_RUNTIME instantiations
  // GroupNorm over groups of gn_pieces * 32 consecutive columns in the elementwise epilogue
  // (0 = off): y = scale * act((z - mu) * rstd * gamma + beta) with mu, rstd per row and group
  int gn_pieces;
  // 1: also write this row's (sum, sum of squares) of z = XW^T + b over the tile's columns to
  // partial[m * tiles_n + tn] (float2) - the first pass of a GroupNorm whose groups span tiles
  int gn_tile_stats;
  float gn_eps;
  const __nv_bfloat16* gn_gamma;   // [N] or null (1)
  const __nv_bfloat16* gn_beta;    // [N] or null (0)
  int stats_only;              // softmax first pass without numerators: 1 = (max, sum of exp)
                               // for the log-sum-exp, 2 = maximum only
  int vec_ok;                  // rows of out (and R) are 16-byte aligned (direct path vectors)
  int staged;                  // out (and R) go through shared memory and TMA
  int bias_vec;                // bias is 16-byte aligned
  uint32_t* status;            // device status word
  // Tile schedule: CTA (or pair) c takes units c, c+ncta, ...; a unit is `tiles_per_unit`
  // consecutive tiles.  1 = plain round-robin; tiles_n = one CTA owns whole row blocks (row sum
  // without a second pass).
  int tiles_per_unit;
  // conv only
  int H, Wd, Cin, rows_per_tile, tiles_per_image, kb_per_tap;
  int tile_px;                 // pixels per tile = UMMA N (a multiple of 32, <= BN): rows_per_tile
                               // whole rows, or one of w_segs equal segments of a row
  int w_segs;                  // 1, or segments per row when Wd > 256 (then rows_per_tile = 1)
  int softmax_fused;           // EPI_SOFTMAX: the row lies in one tile (tiles_n == 1): finish it in the epilogue
  int gn_cluster;              // EPI_CONV_GN: CTAs per cluster = pixel tiles per image (1..8 or 16);
                               // EPI_SOFTMAX_CL: CTAs per cluster = column tiles per row (2..16)
  int gn_groups;               // EPI_CONV_GN: GroupNorm groups (channels per group a power of two, 4..32)
  int slab;                    // convolution: 1 = the producer loads, per column shift, ONE copy of the tile's
                               // pixel window with its two halo rows ((rows_per_tile + 2) x box_w pixels,
                               // through tmR) and the three row taps read it at offsets of whole rows
  int slab_bytes;              // bytes of one such copy (<= 48 KB)
  int slab_row_bytes;          // bytes of one image row of the copy: box_w * 128, a multiple of 1024
  // EPI_CONV_GNX: per (image, channel tile) unit u: gx_part[(u * tiles_per_image + t) * 32 + g] =
  // (sum, sum of squares) of GroupNorm group g over pixel tile t; all bits set where no pair has
  // been stored yet (the state the kernel starts from)
  // EPI_SOFTMAX_GX: gx_part[(row block * tiles_n + t) * 128 + row] = (maximum, sum) of a row over
  // column tile t, the same convention
  float2* gx_part;
  int y_wide;                  // EPI_CONV_GNX in slab mode: tmB is a store map of 64 pixels x 32 channels (128-byte swizzle)
  int pool2;                   // convolution: 0, or 2x2 pooling in the epilogue (1 = max, 2 = mean);
                               // needs w_segs == 1, Wd % 32 == 0, rows_per_tile and H even
};

// The it-th tile of scheduling slot `cta` out of `ncta`, or -1 when the slot has no more work.
// Convolution: the i-th scheduled pixel tile.  Images are taken last to first, so that the images
// written last, which are the ones still in L2 when the kernel ends, are the first ones the pass
// that follows (normalisation, pooling: increasing image order) reads.
__device__ __forceinline__ int conv_pixel_tile(const UmmaParams& p, int i) {
  const int img = p.tiles_n / p.tiles_per_image - 1 - i / p.tiles_per_image;
  return img * p.tiles_per_image + i % p.tiles_per_image;
}

__device__ __forceinline__ int sched_tile(const UmmaParams& p, int cta, int ncta, int it) {
  const int tpu = p.tiles_per_unit;
  const int unit = cta + (it / tpu) * ncta;
  if (unit >= p.num_tiles / tpu) return -1;
  return unit * tpu + it % tpu;
}

// CTA2: two CTAs of a cluster share one 256-row x BN tile (tcgen05 cta_group::2): each loads its
// own 128 rows of A and HALF of the B tile, so a stage costs a CTA a third less shared memory
// and L2 traffic for the same number of flops.
template <int BN, int EPI, bool CTA2 = false>
struct UmmaCfg {
  static constexpr int kStageA = kBM * kBK * 2;
  static constexpr int kStageB = (CTA2 ? BN / 2 : BN) * kBK * 2;
  static constexpr int kStage1 = kStageA + kStageB;          // one 64-wide K block of A and B
  // staging: elementwise = 2 output + 2 residual pieces; softmax = 2 output pieces per epilogue
  // group; conv = 2 output pieces
  static constexpr int kStaging =
      EPI == EPI_ELEMENTWISE || is_softmax(EPI) || EPI == EPI_CONV_GNX || EPI == EPI_CONV ? 4 * kPieceBytes      // (EPI_SOFTMAX_GX: one piece per group, below; EPI_CONV_GNX: a 4 KB slab per epilogue warp; EPI_CONV: two)
                                                    : (EPI == EPI_ROWSUM ? 0 : 2 * kPieceBytes);     // EPI_CONV_GN: one piece per epilogue group
  static constexpr int kBarBytes = 256;
  // GEMM epilogues: the tile's BN bias values as fp32, staged once per tile
  // (EPI_CONV_GNX: partial sums [2][2 groups][32] and group statistics [2][32], float2;
  //  EPI_SOFTMAX_GX: the bias, then the groups' per-row (maximum, sum) [2 groups][128 rows] float2)
  static constexpr int kBiasBytes = EPI == EPI_CONV ? 0 : (EPI == EPI_CONV_GNX ? 1536 : (EPI == EPI_SOFTMAX_GX ? BN * 4 + 2048 : BN * 4));   // EPI_CONV_GN: the statistics it sends
  // EPI_CONV_GN: statistics arriving from the cluster, [2 buffers][16 CTAs x 2 groups][32 x float2]
  // EPI_SOFTMAX_CL: [2 buffers][16 CTAs x 2 groups][128 rows x float2] arriving, then the
  // [2 buffers][2 groups][128 x float2] it sends
  // (EPI_SOFTMAX_CL: clusters of up to 16 CTAs with 64-column tiles, up to 8 with wider ones)
  static constexpr int kClMax = BN <= 64 ? 16 : 8;
  static constexpr int kInboxBytes = EPI == EPI_CONV_GN ? 2 * 32 * 256 : (EPI == EPI_SOFTMAX_CL ? 2 * 2 * kClMax * 1024 + 4 * 1024 : 0);
  // GEMMs: a stage holds two K blocks behind one barrier where three such stages fit.  The UMMA
  // issuer pays a barrier wait, an election and a commit per stage, each of which waits its turn
  // behind the operand reads of the MMAs in flight (150 cycles and more): with one block per
  // stage it needed about 600 cycles per block against the tensor pipe's 512 (256 at 128-column
  // tiles), and the pipe's short queue ran dry.
  static constexpr int kBudget = kMaxDynSmem - 1024 - kStaging - kBarBytes - kBiasBytes - kInboxBytes;
  static constexpr int kKB = (!is_conv(EPI) && !CTA2 && kBudget / (2 * kStage1) >= 3) ? 2 : 1;
  static constexpr int kStage = kKB * kStage1;
  static constexpr int kFit = kBudget / kStage;
  static constexpr int kStages = kFit > 8 ? 8 : kFit;
  static constexpr int kRing = kStage * kStages;
  static constexpr int kTotal = 1024 /*alignment slack*/ + kRing + kStaging + kBarBytes + kBiasBytes + kInboxBytes;
};

// 32 consecutive bias values as fp32 (zeros past N or without a bias).  All lanes read the same
// addresses, so each load is one broadcast transaction.
__device__ __forceinline__ void load_bias32(const UmmaParams& p, int n0, float (&b)[32]) {
  if (p.bias == nullptr) {
#pragma unroll
    for (int j = 0; j < 32; ++j) b[j] = 0.0f;
  } else if (p.bias_vec && n0 + 32 <= p.N) {
    const uint4* bp = reinterpret_cast<const uint4*>(p.bias + n0);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint4 w = __ldg(bp + q);
      b[8 * q + 0] = bf16_lo(w.x); b[8 * q + 1] = bf16_hi(w.x);
      b[8 * q + 2] = bf16_lo(w.y); b[8 * q + 3] = bf16_hi(w.y);
      b[8 * q + 4] = bf16_lo(w.z); b[8 * q + 5] = bf16_hi(w.z);
      b[8 * q + 6] = bf16_lo(w.w); b[8 * q + 7] = bf16_hi(w.w);
    }
  } else {
#pragma unroll
    for (int j = 0; j < 32; ++j)
      b[j] = (n0 + j < p.N) ? __bfloat162float(p.bias[n0 + j]) : 0.0f;
  }
}

// 32 consecutive values of a bf16 vector of length N as fp32 (`dflt` past N or for a null
// pointer); 16-byte loads when the vector is 16-byte aligned.
__device__ __forceinline__ void load_vec32(const __nv_bfloat16* ptr, int N, int n0, float dflt,
                                           float (&o)[32]) {
  if (ptr == nullptr) {
#pragma unroll
    for (int j = 0; j < 32; ++j) o[j] = dflt;
  } else if ((reinterpret_cast<uintptr_t>(ptr) & 15u) == 0 && n0 + 32 <= N) {
    const uint4* bp = reinterpret_cast<const uint4*>(ptr + n0);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint4 w = __ldg(bp + q);
      o[8 * q + 0] = bf16_lo(w.x); o[8 * q + 1] = bf16_hi(w.x);
      o[8 * q + 2] = bf16_lo(w.y); o[8 * q + 3] = bf16_hi(w.y);
      o[8 * q + 4] = bf16_lo(w.z); o[8 * q + 5] = bf16_hi(w.z);
      o[8 * q + 6] = bf16_lo(w.w); o[8 * q + 7] = bf16_hi(w.w);
    }
  } else {
#pragma unroll
    for (int j = 0; j < 32; ++j) o[j] = (n0 + j < N) ? __bfloat162float(ptr[n0 + j]) : dflt;
  }
}

// Byte offset of 16-byte chunk j (0..3) of row r in a 128-row x 64-byte piece laid out the way
// TMA's SWIZZLE_64B expects it (address bits 4..5 xor bits 7..8): conflict-free for a warp
// whose lanes are consecutive rows.
__device__ __forceinline__ uint32_t piece_off(int r, int j) {
  return static_cast<uint32_t>(r * 64 + ((j ^ ((r >> 1) & 3)) << 4));
}

// 32 consecutive staged bias values (shared memory, same address in every lane: broadcast).
__device__ __forceinline__ void load_sbias32(const float* sb, float (&b)[32]) {
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    const float4 t = *reinterpret_cast<const float4*>(sb + 4 * q);
    b[4 * q + 0] = t.x; b[4 * q + 1] = t.y; b[4 * q + 2] = t.z; b[4 * q + 3] = t.w;
  }
}

// ---------------------------------------------------------------------------------------------
// Epilogue of EPI_CONV_GNX: conv3x3 -> activation -> GroupNorm in one kernel on every SM.
//
// Tiles are dealt round-robin, tile t to CTA t mod grid, so the pixel tiles of one image are held
// by neighbouring CTAs at (almost) the same time; the grid is launched cooperatively, i.e. all of
// its CTAs are resident together.  Two epilogue groups of four warps, each owning half of the
// tile's pixels; a thread is one output channel.  Per tile:
//   A  the thread reads its share of the accumulator ONCE (the warp hands the accumulator back to
//      the UMMA issuer as soon as its last load has landed), applies bias and activation, adds up
//      sum and sum of squares in fp32 and keeps the activations in registers as bf16; shuffles
//      reduce the sums over the channels of a GroupNorm group; the helper warp adds the two
//      groups' partial sums and stores the tile's 32 (sum, sum of squares) pairs to global memory.
//   B  the helper warp has read the pairs of all of the image's tiles (each 64-bit pair is its own
//      "present" flag: no counter, no fence), added them up in tile order and left (mean, 1/std)
//      per group in shared memory; every thread normalises its activations from the registers
//      and stores them through the warp's 2 KB slab (32 channels x 32 pixels) with TMA.
// The loop is software-pipelined: A of this CTA's next tile runs BEFORE B of the current one (two
// register buffers of activations), so by the time B asks, the other CTAs have long published and
// the exchange's latency is hidden behind an accumulator pass.  A only ever waits for this CTA's
// own MMAs, so the waits cannot form a cycle.  No thread leaves the loop inside a tile: a wait
// that runs out is reported at the next go/no-go, which all eight warps take together.
// ---------------------------------------------------------------------------------------------
template <int BN, int ACT, typename TileAt>
__device__ __forceinline__ void conv_gnx_epilogue(const UmmaParams& p, const CUtensorMap* tmY,
                                                  const CUtensorMap* tmYw, uint8_t* stg,
                                                  float2* aux, uint64_t* tmem_full, uint64_t* tmem_empty,
                                                  uint64_t* gx_parts, uint64_t* gx_stats,
                                                  volatile uint32_t* abort_flag, uint32_t tmem_base,
                                                  int warp, int lane, int my_tiles, TileAt tile_at) {
  constexpr int kGroups = 2;
  constexpr int kGroupCols = BN / kGroups;
  constexpr int kGP = kGroupCols / 32;                  // pieces per thread: 4 (BN = 256) or 2
  const int grp = (warp - 2) >> 2;
  const int quad = warp & 3;                            // TMEM lane quarter this warp may read
  const int row = quad * 32 + lane;                     // output channel inside the 128-channel tile
  const bool leader = threadIdx.x == 64;                // polls for all
  const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
  const int cpg = p.N / p.gn_groups;                    // channels per group: 4, 8, 16 or 32
  const int gidx = row / cpg;                           // this channel's group inside the tile: 0..31
  const long long hw = static_cast<long long>(p.H) * p.Wd;
  const float inv_cnt = 1.0f / static_cast<float>(static_cast<long long>(cpg) * hw);
  const int pieces = p.tile_px / 32;
  const int piece0 = grp * kGP;
  const int my_pieces = max(0, min(kGP, pieces - piece0));
  const int tpi = p.tiles_per_image;
  uint8_t* wslab = stg + (grp * 4 + quad) * 4096;       // this warp's staging slab (4 KB; the 32-pixel form uses half)
  bool failed = false;                                  // one of this thread's waits ran out

  struct Tile { int tm, img, pt, unit, px0, px_valid; float bias_v, ga, be; };
  auto locate = [&](int it) {
    const int tile = tile_at(it);
    Tile t;
    t.tm = tile % p.tiles_m;
    const int tn = conv_pixel_tile(p, tile / p.tiles_m);
    t.img = tn / tpi;
    t.pt = tn % tpi;
    t.unit = t.img * p.tiles_m + t.tm;
    t.px0 = t.pt * p.tile_px;
    t.px_valid = static_cast<int>(min(static_cast<long long>(p.tile_px), hw - t.px0));
    const int ch = t.tm * kBM + row;
    const bool ch_ok = ch < p.N;
    t.bias_v = (p.bias != nullptr && ch_ok) ? __bfloat162float(p.bias[ch]) : 0.0f;
    t.ga = (p.gn_gamma != nullptr && ch_ok) ? __bfloat162float(p.gn_gamma[ch]) : 1.0f;
    t.be = (p.gn_beta != nullptr && ch_ok) ? __bfloat162float(p.gn_beta[ch]) : 0.0f;
    return t;
  };

  // A: accumulator -> activations in `st` (bf16 pairs); this tile's statistics published.
  // Returns false when the go/no-go said stop (then every epilogue thread got false).
  auto phase_a = [&](int it, uint32_t (&st)[kGP * 16]) -> bool {
    const Tile t = locate(it);
    const int a = it & 1;
    bool ok = true;
    if (leader)
      ok = mbar_wait(&tmem_full[a], static_cast<uint32_t>((it >> 1) & 1), abort_flag, p.status,
                     KF_DEV_TIMEOUT_EPILOGUE);
    ok = named_barrier_and(9u, kGroups * kEpiThreads, ok && !failed);
    if (!ok) return false;
    tc_fence_after_sync();
    const uint32_t t_acc = tmem_base + static_cast<uint32_t>(a * BN + grp * kGroupCols) + lane_off;
    const uint64_t bias2 = f32x2_pack(t.bias_v, t.bias_v);
    float s1 = 0.0f, s2 = 0.0f;
    uint64_t s1p = f32x2_pack(0.0f, 0.0f), s2p = s1p;   // (even, odd) pixel partial sums
    // (the whole-tile case and the ragged case are two separate unrolled loops: the hot one stays
    // contiguous in the instruction stream)
    const bool whole = t.px_valid >= (piece0 + my_pieces) * 32 && my_pieces == kGP;
    if (whole) {
#pragma unroll
      for (int c = 0; c < kGP; ++c) {
        uint32_t v[32];
        tmem_ld_32x32(t_acc + c * 32, v);
        tmem_ld_wait();
        if (c == kGP - 1) {
          // the last of this warp's loads has landed: hand the accumulator back (one arrival per warp)
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tmem_empty[a]);
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          float y0, y1;
          f32x2_unpack(f32x2_add(f32x2_pack(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])), bias2), y0, y1);
          y0 = act_f<ACT, true>(y0, p.act_rt);
          y1 = act_f<ACT, true>(y1, p.act_rt);
          const uint64_t y = f32x2_pack(y0, y1);
          s1p = f32x2_add(s1p, y);
          s2p = f32x2_fma(y, y, s2p);
          st[c * 16 + j] = pack_bf16x2(y0, y1);
        }
      }
    } else {
      // a tile that hangs over the end of its image (those pixels were read as zeros, are left out
      // of the statistics and are not stored), or a group with fewer pieces than it has room for
#pragma unroll
      for (int c = 0; c < kGP; ++c) {
        uint32_t v[32];
        if (c < my_pieces) {
          tmem_ld_32x32(t_acc + c * 32, v);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = 0u;
        }
        if (c == kGP - 1) {
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tmem_empty[a]);
        }
        const int left = t.px_valid - (piece0 + c) * 32;  // valid pixels from this piece on
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          float y0 = act_f<ACT, true>(__uint_as_float(v[2 * j]) + t.bias_v, p.act_rt);
          float y1 = act_f<ACT, true>(__uint_as_float(v[2 * j + 1]) + t.bias_v, p.act_rt);
          if (2 * j >= left) y0 = 0.0f;
          if (2 * j + 1 >= left) y1 = 0.0f;
          s1 += y0 + y1;
          s2 = fmaf(y0, y0, fmaf(y1, y1, s2));
          st[c * 16 + j] = pack_bf16x2(y0, y1);
        }
      }
    }
    {
      float e, o;
      f32x2_unpack(s1p, e, o); s1 += e + o;
      f32x2_unpack(s2p, e, o); s2 += e + o;
    }
    for (int o = cpg >> 1; o > 0; o >>= 1) {            // the group's channels: adjacent lanes
      s1 += __shfl_xor_sync(0xffffffffu, s1, o);
      s2 += __shfl_xor_sync(0xffffffffu, s2, o);
    }
    // the partial sums go to the helper warp, which publishes them (see conv_gnx_helper)
    float2* part = aux + (it & 1) * 64;                 // [2 tiles in flight][2 groups][32]
    if ((row & (cpg - 1)) == 0) part[grp * 32 + gidx] = make_float2(s1, s2);
    __syncwarp();
    if (lane == 0) mbar_arrive(&gx_parts[it & 1]);      // (release: the warp's writes above are ordered before it)
    return true;
  };

  // B: the image's statistics -> normalised activations -> global memory.
  auto phase_b = [&](int it, const uint32_t (&st)[kGP * 16]) {
    const Tile t = locate(it);
    // the helper warp has added the image's tiles up and left (mean, 1/std) per group
    if (!mbar_wait(&gx_stats[it & 1], static_cast<uint32_t>((it >> 1) & 1), abort_flag, p.status, KF_DEV_TIMEOUT_EPILOGUE))
      failed = true;                      // the status word has it; finish the tile with the others
    const float2 ms = aux[128 + (it & 1) * 32 + gidx];  // [2][32] after the partial sums
    const float sc = ms.y * t.ga;
    const float sh = fmaf(-ms.x, sc, t.be);
    const uint64_t sc2 = f32x2_pack(sc, sc), sh2 = f32x2_pack(sh, sh);
    if (p.y_wide && my_pieces == kGP && t.px_valid >= (piece0 + kGP) * 32) {
      // whole shares leave in slabs of 64 pixels x 32 channels (128-byte rows, 128-byte swizzle):
      // half as many waits for the slab, fences and store issues as with 32-pixel slabs
#pragma unroll
      for (int c2 = 0; c2 < kGP / 2; ++c2) {
        uint32_t w[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const uint32_t u = st[c2 * 32 + j];
          float y0, y1;
          f32x2_unpack(f32x2_fma(f32x2_pack(bf16_lo(u), bf16_hi(u)), sc2, sh2), y0, y1);
          w[j] = pack_bf16x2(y0, y1);
        }
        bulk_wait_group_read<0>();       // this warp's previous store has let go of the slab
        __syncwarp();
#pragma unroll
        for (int q = 0; q < 8; ++q)
          *reinterpret_cast<uint4*>(wslab + lane * 128 + ((q ^ (lane & 7)) << 4)) =
              make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
        fence_proxy_async_smem();
        __syncwarp();
        if (elect_one()) {
          if (t.tm * kBM + quad * 32 < p.N)
            tma_store_3d(tmYw, wslab, t.px0 + (piece0 + 2 * c2) * 32, t.tm * kBM + quad * 32, t.img);
          bulk_commit_group();
        }
      }
      return;
    }
#pragma unroll
    for (int c = 0; c < kGP; ++c) {
      if (c < my_pieces) {
        uint32_t w[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const uint32_t u = st[c * 16 + j];
          float y0, y1;
          f32x2_unpack(f32x2_fma(f32x2_pack(bf16_lo(u), bf16_hi(u)), sc2, sh2), y0, y1);
          w[j] = pack_bf16x2(y0, y1);
        }
        bulk_wait_group_read<0>();       // this warp's previous store has let go of the slab
        __syncwarp();
#pragma unroll
        for (int q = 0; q < 4; ++q)
          *reinterpret_cast<uint4*>(wslab + piece_off(lane, q)) =
              make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
        fence_proxy_async_smem();
        __syncwarp();
        if (elect_one()) {
          const int px = (piece0 + c) * 32;               // first pixel of the piece inside the tile
          if (t.px_valid - px > 0 && t.tm * kBM + quad * 32 < p.N)
            tma_store_3d(tmY, wslab, t.px0 + px, t.tm * kBM + quad * 32, t.img);
          bulk_commit_group();
        }
      }
    }
  };

  // One copy of each phase's code (the unrolled per-piece loops are long, and instruction fetch was
  // a visible stall with two): the new tile's activations are moved over to `st_old` after B.
  uint32_t st_new[kGP * 16], st_old[kGP * 16];
  bool alive = true;
  for (int it = 0; it <= my_tiles && alive; ++it) {
    if (it < my_tiles) alive = phase_a(it, st_new);
    if (alive && it >= 1) phase_b(it - 1, st_old);
#pragma unroll
    for (int j = 0; j < kGP * 16; ++j) st_old[j] = st_new[j];
  }
  bulk_wait_group_read<0>();
}

// The helper warp of EPI_CONV_GNX: everything in the GroupNorm exchange that touches global memory.
// A small state machine over this CTA's tiles, never blocking on one thing while another is due:
//   publish(k)  once the epilogue warps have left tile k's partial sums (tested, not waited for: a
//               try_wait may suspend the warp while statistics are due): the two groups' sums in
//               a fixed order to global memory as one 256-byte row of 64-bit pairs;
//   stats(k)    lane g loads group g's pair of every tile of tile k's image; once none of them is
//               the "empty" pattern any more it adds them in tile order and leaves (mean, 1/std)
//               for the epilogue warps.  (With a counter per image, a release after the stores
//               and an acquire before the loads, the two fences cost this warp about 3000 cycles
//               per tile beside the mainloop, and the image's statistics arrived 4000 cycles
//               after the epilogue asked for them.)
// Every wait is bounded; a wait that runs out raises the abort flag, and the outstanding hand-overs
// are still completed so that no epilogue warp is left waiting on a barrier.
constexpr uint64_t kGxEmpty = ~0ull;   // what the exchange buffer holds before a tile's pair arrives

template <typename TileAt>
__device__ __forceinline__ void conv_gnx_helper(const UmmaParams& p, float2* aux, uint64_t* gx_parts,
                                                uint64_t* gx_stats, volatile uint32_t* abort_flag,
                                                int lane, int my_tiles, TileAt tile_at) {
  const int tpi = p.tiles_per_image;
  const int cpg = p.N / p.gn_groups;
  const long long hw = static_cast<long long>(p.H) * p.Wd;
  const float inv_cnt = 1.0f / static_cast<float>(static_cast<long long>(cpg) * hw);
  auto unit_of = [&](int it, int* pt) {
    const int tile = tile_at(it);
    const int tn = conv_pixel_tile(p, tile / p.tiles_m);
    *pt = tn % tpi;
    return (tn / tpi) * p.tiles_m + tile % p.tiles_m;
  };
  int pub = 0, stt = 0;
  bool dead = false;
  uint64_t t0 = globaltimer_ns();
  uint32_t spins = 0;
  uint64_t* gx = reinterpret_cast<uint64_t*>(p.gx_part);
  while (stt < my_tiles) {
    bool progressed = false;
    if (pub < my_tiles && (dead || mbar_test_wait(&gx_parts[pub & 1], static_cast<uint32_t>((pub >> 1) & 1)))) {
      int pt;
      const int unit = unit_of(pub, &pt);
      const float2* part = aux + (pub & 1) * 64;
      float2 m = make_float2(0.0f, 0.0f);
      if (lane < kBM / cpg) {
        const float2 a0 = part[lane], a1 = part[32 + lane];
        m = make_float2(a0.x + a1.x, a0.y + a1.y);
      }
      // the pair is its own flag (see st_relaxed_gpu_b64); the one pattern that means "not yet"
      // (two NaNs of all ones, which no addition produces) is stored as the canonical NaN pair
      uint64_t bits = (static_cast<uint64_t>(__float_as_uint(m.y)) << 32) | __float_as_uint(m.x);
      if (bits == kGxEmpty) bits = 0x7fffffff7fffffffull;
      st_relaxed_gpu_b64(gx + (static_cast<long long>(unit) * tpi + pt) * 32 + lane, bits);
      ++pub;
      progressed = true;
    }
    if (stt < pub) {
      int pt;
      const int unit = unit_of(stt, &pt);
      const uint64_t* gp = gx + static_cast<long long>(unit) * tpi * 32 + lane;
      float g1 = 0.0f, g2 = 0.0f;
      bool all = true;
      for (int r0 = 0; r0 < tpi; r0 += 16) {             // all loads in flight, the additions in tile order
        uint64_t qv[16];
#pragma unroll
        for (int r = 0; r < 16; ++r) qv[r] = (r0 + r < tpi) ? ld_relaxed_gpu_b64(gp + (r0 + r) * 32) : 0ull;
#pragma unroll
        for (int r = 0; r < 16; ++r) {
          all = all && qv[r] != kGxEmpty;
          g1 += __uint_as_float(static_cast<uint32_t>(qv[r]));
          g2 += __uint_as_float(static_cast<uint32_t>(qv[r] >> 32));
        }
      }
      all = __all_sync(0xffffffffu, all);
      if (dead || all) {
        const float mu = g1 * inv_cnt;
        aux[128 + (stt & 1) * 32 + lane] = make_float2(mu, rsqrtf(fmaxf(g2 * inv_cnt - mu * mu, 0.0f) + p.gn_eps));
        __syncwarp();
        if (lane == 0) mbar_arrive(&gx_stats[stt & 1]);
        ++stt;
        progressed = true;
      }
    }
    if (progressed) { t0 = globaltimer_ns(); spins = 0; continue; }
    __nanosleep(200);                                    // nothing due: do not compete with the mainloop for shared memory
    if ((++spins & 15u) == 0u && !dead) {
      if (*abort_flag) dead = true;                      // another role gave up: hand over what is owed and leave
      else if (globaltimer_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1u;
        atomicOr(p.status, KF_DEV_TIMEOUT_EPILOGUE);
        dead = true;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Epilogue of EPI_SOFTMAX_GX: GEMM + bias (+ activation) + softmax over rows of several 256-column
// tiles in one kernel, probabilities written once (no numerators in memory, no second pass).
//
// Tiles are dealt round-robin with the column tile fastest, so the tiles of a block of 128 rows
// are held by neighbouring CTAs (CTA pairs) of one cooperative grid at (almost) the same time.  Two
// epilogue groups of four warps, each owning 128 of the tile's columns; a thread is one row.
//   A  maximum of the row's 128 values (first pass over the accumulator), then numerators
//      e = exp(a - maximum) and their fp32 sum (second pass); the numerators stay in registers as
//      bf16, the accumulator goes back to the UMMA issuer; one warp merges the two groups' (maximum,
//      sum) per row and stores the tile's 128 pairs to global memory, each 64-bit pair being its
//      own "present" flag in a buffer that starts out as all ones (no counter, no fence);
//   B  a thread loads its row's pairs of all column tiles (again, bounded, while one of them is
//      still the empty pattern), forms the row's maximum M and denominator S = sum s_t exp(m_t - M)
//      in tile order, scales its numerators by exp(m - M) / S and stores them through shared
//      memory and TMA.
// The loop is software-pipelined: A of this CTA's next tile runs before B of the current one, so
// the other CTAs have published by the time B asks.  A only waits for this CTA's own MMAs: the
// waits cannot form a cycle.  A wait that runs out is reported at the next go/no-go, which all
// eight warps take together.  Whole 256-column tiles only (N a multiple of 256).
// ---------------------------------------------------------------------------------------------
template <int BN, int ACT, bool CTA2, typename TileAt>
__device__ __forceinline__ void softmax_gx_epilogue(const UmmaParams& p, const CUtensorMap* tmY,
                                                    const CUtensorMap* tmYw, uint8_t* stg,
                                                    float* sbias_all, float2* part, uint64_t* tmem_full,
                                                    uint64_t* tmem_empty, volatile uint32_t* abort_flag,
                                                    uint32_t tmem_base, uint32_t rank, int warp, int lane,
                                                    int my_tiles, TileAt tile_at) {
  constexpr int kGroups = 2;
  constexpr int kGroupCols = BN / kGroups;              // 128
  constexpr int PIECES = kGroupCols / 32;               // 4
  constexpr int kTileM = CTA2 ? 2 * kBM : kBM;
  constexpr float kLog2e = 1.4426950408889634f;
  const int grp = (warp - 2) >> 2;
  const int quad = warp & 3;
  const int row = quad * 32 + lane;
  const int et = static_cast<int>(threadIdx.x) - 64 - grp * kEpiThreads;
  const bool leader = threadIdx.x == 64;
  const bool grp_leader = et == 0;
  const uint32_t bar_b = 2u + 2u * grp;
  const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
  float* sbias = sbias_all + grp * kGroupCols;
  uint8_t* ybuf = stg + grp * kPieceBytes;              // the group's staging piece
  const int tiles_n = p.tiles_n;
  bool failed = false;

  struct Tile { int tm, tn, m_cta, rb; };
  auto locate = [&](int it) {
    const int tile = tile_at(it);
    Tile t;
    t.tm = tile / tiles_n; t.tn = tile % tiles_n;
    t.m_cta = t.tm * kTileM + static_cast<int>(rank) * kBM;
    t.rb = t.m_cta / kBM;
    return t;
  };

  auto phase_a = [&](int it, uint32_t (&st)[PIECES * 16], float& mx_out) -> bool {
    const Tile t = locate(it);
    const int a = it & 1;
    const int n_tile = t.tn * BN + grp * kGroupCols;
    // this thread's two of the group's bias values, fetched before the wait for the accumulator
    float2 bpre = make_float2(0.0f, 0.0f);
    if (p.bias != nullptr && 2 * et < kGroupCols) {
      bpre.x = __bfloat162float(p.bias[n_tile + 2 * et]);
      bpre.y = __bfloat162float(p.bias[n_tile + 2 * et + 1]);
    }
    bool ok = true;
    if (leader)
      ok = mbar_wait(&tmem_full[a], static_cast<uint32_t>((it >> 1) & 1), abort_flag, p.status,
                     KF_DEV_TIMEOUT_EPILOGUE);
    ok = named_barrier_and(9u, kGroups * kEpiThreads, ok && !failed);
    if (!ok) return false;
    tc_fence_after_sync();
    if (2 * et < kGroupCols) *reinterpret_cast<float2*>(sbias + 2 * et) = bpre;
    named_barrier_sync(bar_b, kEpiThreads);
    const uint32_t t_acc = tmem_base + static_cast<uint32_t>(a * BN + grp * kGroupCols) + lane_off;
    float mx = -INFINITY;
#pragma unroll 1
    for (int c = 0; c < PIECES; ++c) {
      uint32_t v[32];
      tmem_ld_32x32(t_acc + c * 32, v);
      float bs[32];
      load_sbias32(sbias + c * 32, bs);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        float z0, z1;
        f32x2_unpack(f32x2_add(f32x2_pack(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])),
                               f32x2_pack(bs[2 * j], bs[2 * j + 1])), z0, z1);
        mx = fmaxf(mx, fmaxf(act_f<ACT, true>(z0, p.act_rt), act_f<ACT, true>(z1, p.act_rt)));
      }
    }
    const uint64_t l2e2 = f32x2_pack(kLog2e, kLog2e);
    const uint64_t off2 = f32x2_pack(-mx * kLog2e, -mx * kLog2e);
    uint64_t sum2 = f32x2_pack(0.0f, 0.0f);
#pragma unroll
    for (int c = 0; c < PIECES; ++c) {
      uint32_t v[32];
      tmem_ld_32x32(t_acc + c * 32, v);
      float bs[32];
      load_sbias32(sbias + c * 32, bs);
      tmem_ld_wait();
      if (c == PIECES - 1) {
        // the last load has landed: hand the accumulator back (one arrival per warp)
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
          if constexpr (CTA2) mbar_arrive_cluster(mapa_shared(smem_u32(&tmem_empty[a]), 0));
          else mbar_arrive(&tmem_empty[a]);
        }
      }
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        float z0, z1;
        f32x2_unpack(f32x2_add(f32x2_pack(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])),
                               f32x2_pack(bs[2 * j], bs[2 * j + 1])), z0, z1);
        f32x2_unpack(f32x2_fma(f32x2_pack(act_f<ACT, true>(z0, p.act_rt), act_f<ACT, true>(z1, p.act_rt)), l2e2, off2),
                     z0, z1);
        const float e0 = exp2_approx(z0), e1 = exp2_approx(z1);
        sum2 = f32x2_add(sum2, f32x2_pack(e0, e1));
        st[c * 16 + j] = pack_bf16x2(e0, e1);
      }
    }
    float se, so;
    f32x2_unpack(sum2, se, so);
    mx_out = mx;
    part[grp * kBM + row] = make_float2(mx, se + so);
    if (warp == 2) {
      // the combiner: once all eight warps have arrived, the two groups' pairs merged per row go to
      // global memory as 128 pairs (four coalesced stores per lane)
      named_barrier_sync(10u, kGroups * kEpiThreads);
      uint64_t* dst = reinterpret_cast<uint64_t*>(p.gx_part) + (static_cast<long long>(t.rb) * tiles_n + t.tn) * kBM;
#pragma unroll
      for (int i = 0; i < kBM / 32; ++i) {
        const int r = i * 32 + lane;
        const float2 q0 = part[r], q1 = part[kBM + r];
        const float m = fmaxf(q0.x, q1.x);
        const float sm = q0.y * exp2_approx((q0.x - m) * kLog2e) + q1.y * exp2_approx((q1.x - m) * kLog2e);
        // the pair is its own "present" flag (see st_relaxed_gpu_b64): no counter and no fence
        uint64_t bits = (static_cast<uint64_t>(__float_as_uint(sm)) << 32) | __float_as_uint(m);
        if (bits == kGxEmpty) bits = 0x7fffffff7fffffffull;
        st_relaxed_gpu_b64(dst + r, bits);
      }
    } else {
      __threadfence_block();
      named_barrier_arrive(10u, kGroups * kEpiThreads);
    }
    return true;
  };

  auto phase_b = [&](int it, const uint32_t (&st)[PIECES * 16], float mx) {
    const Tile t = locate(it);
    // the row's maximum and denominator from the tiles' pairs, in tile order (sixteen loads in
    // flight); a pair that is still the "empty" pattern sends the thread round again (bounded)
    float M = -INFINITY, S = 0.0f;
    {
      const uint64_t* gp = reinterpret_cast<const uint64_t*>(p.gx_part) + static_cast<long long>(t.rb) * tiles_n * kBM + row;
      uint64_t t_start = 0;
      uint32_t spins = 0;
      int t0 = 0;
      while (t0 < tiles_n) {
        uint64_t q[16];
#pragma unroll
        for (int i = 0; i < 16; ++i)
          q[i] = (t0 + i < tiles_n) ? ld_relaxed_gpu_b64(gp + static_cast<long long>(t0 + i) * kBM) : 0xff800000ull;   // (-inf, 0)
        bool all = true;
#pragma unroll
        for (int i = 0; i < 16; ++i) all = all && q[i] != kGxEmpty;
        if (!all && !failed) {
          __nanosleep(100);
          if ((++spins & 15u) == 0u) {
            if (t_start == 0) t_start = globaltimer_ns();
            if (*abort_flag) failed = true;
            else if (globaltimer_ns() - t_start > kWaitLimitNs) {
              *abort_flag = 1u;
              atomicOr(p.status, KF_DEV_TIMEOUT_EPILOGUE);
              failed = true;              // the status word has it; finish the tile with the others
            }
          }
          continue;
        }
        float bm = M;
#pragma unroll
        for (int i = 0; i < 16; ++i) bm = fmaxf(bm, __uint_as_float(static_cast<uint32_t>(q[i])));
        if (bm > -INFINITY) {
          S *= exp2_approx((M - bm) * kLog2e);
#pragma unroll
          for (int i = 0; i < 16; ++i)
            S += __uint_as_float(static_cast<uint32_t>(q[i] >> 32)) *
                 exp2_approx((__uint_as_float(static_cast<uint32_t>(q[i])) - bm) * kLog2e);
          M = bm;
        }
        t0 += 16;
      }
    }
    const float scale = exp2_approx((mx - M) * kLog2e) / S;
    const uint64_t sc2 = f32x2_pack(scale, scale);
    if (p.y_wide) {
      // every warp stages and stores its own 32 rows of a piece (2 KB slab, the store map in tmR):
      // no barrier between the warps of a group
      uint8_t* wslab = stg + (grp * 4 + quad) * 2048;
#pragma unroll
      for (int c = 0; c < PIECES; ++c) {
        uint32_t w[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const uint32_t u = st[c * 16 + j];
          float y0, y1;
          f32x2_unpack(f32x2_mul(f32x2_pack(bf16_lo(u), bf16_hi(u)), sc2), y0, y1);
          w[j] = pack_bf16x2(y0, y1);
        }
        bulk_wait_group_read<0>();       // this warp's previous store has let go of the slab
        __syncwarp();
#pragma unroll
        for (int q = 0; q < 4; ++q)
          *reinterpret_cast<uint4*>(wslab + piece_off(lane, q)) =
              make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
        fence_proxy_async_smem();
        __syncwarp();
        if (elect_one()) {
          if (t.m_cta + quad * 32 < p.M)
            tma_store_2d(tmYw, wslab, t.tn * BN + grp * kGroupCols + c * kPieceCols, t.m_cta + quad * 32);   // clipped at M
          bulk_commit_group();
        }
      }
      return;
    }
#pragma unroll
    for (int c = 0; c < PIECES; ++c) {
      uint32_t w[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        const uint32_t u = st[c * 16 + j];
        float y0, y1;
        f32x2_unpack(f32x2_mul(f32x2_pack(bf16_lo(u), bf16_hi(u)), sc2), y0, y1);
        w[j] = pack_bf16x2(y0, y1);
      }
      if (grp_leader) bulk_wait_group_read<0>();     // the previous piece's store has let go of the buffer
      named_barrier_sync(bar_b, kEpiThreads);
#pragma unroll
      for (int q = 0; q < 4; ++q)
        *reinterpret_cast<uint4*>(ybuf + piece_off(row, q)) =
            make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
      fence_proxy_async_smem();
      named_barrier_sync(bar_b, kEpiThreads);
      if (grp_leader) {
        tma_store_2d(tmY, ybuf, t.tn * BN + grp * kGroupCols + c * kPieceCols, t.m_cta);   // clipped at M
        bulk_commit_group();
      }
    }
  };

  uint32_t st_new[PIECES * 16], st_old[PIECES * 16];
  float mx_new = 0.0f, mx_old = 0.0f;
  bool alive = true;
  for (int it = 0; it <= my_tiles && alive; ++it) {
    if (it < my_tiles) alive = phase_a(it, st_new, mx_new);
    if (alive && it >= 1) phase_b(it - 1, st_old, mx_old);
#pragma unroll
    for (int j = 0; j < PIECES * 16; ++j) st_old[j] = st_new[j];
    mx_old = mx_new;
  }
  bulk_wait_group_read<0>();
}

template <int BN, int EPI, int ACT, typename OutT, bool CTA2>
__global__ void __launch_bounds__(num_threads(EPI, BN, CTA2), 1)
umma_chain_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmR, const __grid_constant__ CUtensorMap tmY,
                  const UmmaParams p) {
  using C = UmmaCfg<BN, EPI, CTA2>;
  static_assert(!CTA2 || !is_conv(EPI), "the convolution runs one CTA per tile");
  constexpr int kTileM = CTA2 ? 2 * kBM : kBM;            // rows of one scheduled tile
  // In a pair, rank 0 issues the MMAs; both ranks load, and both run the epilogue on their own
  // 128 accumulator rows.  `cta` / `ncta` index the tile schedule (pairs count once).
  uint32_t rank = 0;
  if constexpr (CTA2) rank = cluster_ctarank();
  int cta = CTA2 ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
  int ncta = CTA2 ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);
  // EPI_CONV_GN: a cluster takes whole (image, channel tile) units (the schedule counts clusters
  // and units), its CTA of rank r the r-th pixel tile of each
  [[maybe_unused]] uint32_t crank = 0;
  if constexpr (is_cluster_epi(EPI)) {
    crank = cluster_ctarank();
    cta = static_cast<int>(blockIdx.x) / p.gn_cluster;
    ncta = static_cast<int>(gridDim.x) / p.gn_cluster;
  }
  auto tile_at = [&](int it) -> int {
    const int t = sched_tile(p, cta, ncta, it);
    if constexpr (EPI == EPI_CONV_GN) {
      // unit t = (image, channel tile); this CTA takes the pixel tile of its rank
      if (t < 0) return t;
      return ((t / p.tiles_m) * p.gn_cluster + static_cast<int>(crank)) * p.tiles_m + t % p.tiles_m;
    } else if constexpr (EPI == EPI_SOFTMAX_CL) {
      // unit t = row block; this CTA takes the column tile of its rank (tiles_n == cluster size)
      return t < 0 ? t : t * p.gn_cluster + static_cast<int>(crank);
    } else {
      return t;
    }
  };
  constexpr int kStages = C::kStages;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~static_cast<uintptr_t>(1023));
  uint8_t* ring = smem;
  uint8_t* stg = smem + C::kRing;                                    // epilogue staging
  uint64_t* full = reinterpret_cast<uint64_t*>(stg + C::kStaging);
  uint64_t* empty = full + kStages;
  uint64_t* tmem_full = empty + kStages;
  uint64_t* tmem_empty = tmem_full + 2;
  uint64_t* r_full = tmem_empty + 2;
  uint64_t* rbar = r_full + 8;             // EPI_CONV_GN: [2] statistics from the cluster have arrived
  // EPI_CONV_GNX: gx_parts[2] = the epilogue warps have left a tile's partial sums for the helper
  // warp; gx_stats[2] = the helper warp has left the image's (mean, 1/std) per group
  constexpr int kGxBars = EPI == EPI_CONV_GNX ? 4 : 0;
  [[maybe_unused]] uint64_t* gx_parts = rbar + 2;
  [[maybe_unused]] uint64_t* gx_stats = rbar + 4;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(rbar + 2 + kGxBars);   // r_full: [epilogue warp][2]
  static_assert((2 * kStages + 4 + 8 + 2 + kGxBars) * 8 + 8 <= C::kBarBytes, "barrier block overflows");
  volatile uint32_t* abort_flag = tmem_holder + 1;
  // Convolution in slab mode: the ring holds two pixel copies of up to 48 KB and six weight slots
  // of 16 KB; its barriers are the stage barriers followed by r_full's (which only the
  // elementwise chain uses).
  [[maybe_unused]] constexpr int kSlabPx = 49152;
  [[maybe_unused]] constexpr int kSlabBufs = 2;     // pixel copies in flight
  [[maybe_unused]] constexpr int kSlabW = 6;        // weight slots: the three taps of two column shifts
  // barriers: "this column shift's copy and its three weight blocks have landed" [0,2); weight slot
  // free [2,8); copy buffer free [8,10)
  [[maybe_unused]] constexpr int kGFull = 0, kWEmpty = 2, kCEmpty = 8;
  static_assert(!is_conv(EPI) || (C::kRing >= kSlabBufs * kSlabPx + kSlabW * C::kStageA && kStages >= 4), "slab layout");
  [[maybe_unused]] auto slab_bar = [&](int i) -> uint64_t* {
    return i < 2 * kStages ? full + i : r_full + (i - 2 * kStages);
  };

  // The warp index comes out of a shuffle so that the compiler knows it is the same in every
  // lane: the producer and issuer loops below then run with warp-uniform control flow, and the
  // operands of the TMA and tcgen05 instructions (descriptors, coordinates, barrier addresses)
  // stay in uniform registers.  With the loops inside an `if (lane == 0)` every such operand was
  // moved over from a vector register at each use: about 130 cycles per tcgen05.mma instead of 45
  // at 32-column tiles.
  const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;

  // the 30 barriers are initialised by the lanes of warp 0 side by side (one thread doing all of
  // them was 0.2 us of every launch)
  if (warp == 0) {
    if (lane < kStages) { mbar_init(&full[lane], 1); mbar_init(&empty[lane], 1); }
    if (lane >= 8 && lane < 10) {
      const int a = lane - 8;
      mbar_init(&tmem_full[a], 1);
      mbar_init(&tmem_empty[a], (kEpiThreads / 32) * epi_groups(EPI, BN, CTA2) * (CTA2 ? 2 : 1));
      mbar_init(&rbar[a], 1);
      if constexpr (EPI == EPI_CONV_GNX) {
        mbar_init(&gx_parts[a], 2 * kEpiThreads / 32);      // one arrival per epilogue warp
        mbar_init(&gx_stats[a], 1);
      }
    }
    if (lane >= 16 && lane < 24) mbar_init(&r_full[lane - 16], 1);       // one per epilogue warp and buffer
    if (lane == 31) {
      *abort_flag = 0;
      tma_prefetch_desc(&tmA);
      tma_prefetch_desc(&tmB);
    }
    mbar_init_fence();
  }
  __syncwarp();
  if (warp == 1) {          // TMEM: two accumulators of BN fp32 columns (in both CTAs of a pair)
    if constexpr (CTA2) { tmem_alloc_pair(tmem_holder, 2 * BN); tmem_relinquish_pair(); }
    else { tmem_alloc(tmem_holder, 2 * BN); tmem_relinquish(); }
  }
  tc_fence_before_sync();
  if constexpr (CTA2 || is_cluster_epi(EPI)) cluster_sync_all();   // the peers' barriers exist before anyone signals them
  else __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_holder;
  // Everything above touched only this CTA's shared memory, TMEM and parameters.  A launch that
  // was allowed to start early waits here for the kernel before it; the kernel after this one
  // may start its own prologue now.
  griddep_wait();
  griddep_launch_dependents();

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    // every lane waits for the stage (so the loop stays warp-uniform); one elected lane issues
    {
      int s = 0; uint32_t ph = 0;
      [[maybe_unused]] int pb = 0; [[maybe_unused]] uint32_t pph = 0;   // slab mode: pixel-copy buffer and its phase
      for (int it = 0;; ++it) {
        const int tile = tile_at(it);
        if (tile < 0) break;
        int tm, tn, img = 0, h0 = 0, x0 = 0;
        if constexpr (is_conv(EPI)) {
          tm = tile % p.tiles_m; tn = conv_pixel_tile(p, tile / p.tiles_m);   // output-channel tile, pixel tile
          img = tn / p.tiles_per_image;
          const int pt = tn % p.tiles_per_image;
          h0 = (pt / p.w_segs) * p.rows_per_tile;
          x0 = (pt % p.w_segs) * (p.Wd / p.w_segs);
        } else {
          tm = tile / p.tiles_n; tn = tile % p.tiles_n;
        }
        bool ok = true;
        if constexpr (is_conv(EPI)) {
          if (p.slab) {
            // Per 64-channel block and column shift: one copy of the window with its halo rows
            // (out-of-image pixels read zeros: the padding), then the three row taps' weights.
            for (int cs = 0; cs < 3 * p.kb_per_tap && ok; ++cs) {
              const int cb = cs / 3, sx = cs % 3;
              ok = mbar_wait(slab_bar(kCEmpty + pb), pph ^ 1u, abort_flag, p.status, KF_DEV_TIMEOUT_PRODUCER);
              ok = __all_sync(0xffffffffu, ok);
              if (!ok) break;
              // (one barrier per column shift takes the copy's bytes and the three weight blocks')
              uint64_t* gfull = slab_bar(kGFull + pb);
              if (elect_one()) {
                mbar_expect_tx(gfull, static_cast<uint32_t>(p.slab_bytes) + 3u * C::kStageA);
                tma_load_4d(ring + pb * kSlabPx, &tmR, gfull, cb * kBK, x0 + sx - 1, h0 - 1, img);
              }
              if (++pb == kSlabBufs) { pb = 0; pph ^= 1u; }
              for (int r = 0; r < 3; ++r) {
                ok = mbar_wait(slab_bar(kWEmpty + s), ph ^ 1u, abort_flag, p.status, KF_DEV_TIMEOUT_PRODUCER);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (elect_one()) {
                  tma_load_2d(ring + kSlabBufs * kSlabPx + s * C::kStageA, &tmA, gfull, cb * kBK,
                              (r * 3 + sx) * p.N + tm * kBM);
                }
                if (++s == kSlabW) { s = 0; ph ^= 1u; }
              }
            }
            if (!ok) break;
            continue;
          }
        }
        for (int kb = 0; kb < p.k_blocks; kb += C::kKB) {
          ok = mbar_wait(&empty[s], ph ^ 1u, abort_flag, p.status, KF_DEV_TIMEOUT_PRODUCER);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          uint8_t* sa = ring + s * C::kStage;
          uint8_t* sb = sa + C::kStageA;
          [[maybe_unused]] const int kbs = min(C::kKB, p.k_blocks - kb);   // K blocks in this stage
          if constexpr (CTA2) {
            if (elect_one()) {
              // both CTAs' bytes complete on rank 0's barrier, which rank 0 arms for the pair
              if (rank == 0) mbar_expect_tx(&full[s], static_cast<uint32_t>(2 * kbs * C::kStage1));
              for (int j = 0; j < kbs; ++j) {
                tma_load_2d_pair(sa + j * C::kStage1, &tmA, &full[s], (kb + j) * kBK,
                                 tm * kTileM + static_cast<int>(rank) * kBM);
                tma_load_2d_pair(sb + j * C::kStage1, &tmB, &full[s], (kb + j) * kBK,
                                 tn * BN + static_cast<int>(rank) * (BN / 2));
              }
            }
          } else if constexpr (is_conv(EPI)) {
            const int tap = kb / p.kb_per_tap, cb = kb % p.kb_per_tap;
            const int r = tap / 3, sx = tap % 3;
            if (elect_one()) {
              // a convolution tile fetches tile_px <= BN pixel rows of 128 bytes
              mbar_expect_tx(&full[s], C::kStageA + p.tile_px * kBK * 2);
              // A: this tap's weights for 128 output channels.  B: BN pixels x 64 input channels
              // of the window shifted by the tap; out-of-image pixels read zeros (the padding).
              tma_load_2d(sa, &tmA, &full[s], cb * kBK, tap * p.N + tm * kBM);
              tma_load_4d(sb, &tmB, &full[s], cb * kBK, x0 + sx - 1, h0 + r - 1, img);
            }
          } else {
            if (elect_one()) {
              mbar_expect_tx(&full[s], static_cast<uint32_t>(kbs * C::kStage1));
              for (int j = 0; j < kbs; ++j) {
                tma_load_2d(sa + j * C::kStage1, &tmA, &full[s], (kb + j) * kBK, tm * kBM);
                tma_load_2d(sb + j * C::kStage1, &tmB, &full[s], (kb + j) * kBK, tn * BN);
              }
            }
          }
          if (++s == kStages) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ UMMA issuer
    // every lane waits (warp-uniform loop), one elected lane issues the MMAs and the commits
    if (rank == 0) {
      const uint32_t idesc =
          umma_idesc_bf16_f32(kTileM, is_conv(EPI) ? static_cast<uint32_t>(p.tile_px) : BN);
      int s = 0; uint32_t ph = 0; int a = 0; uint32_t aph = 0;
      [[maybe_unused]] int pb = 0; [[maybe_unused]] uint32_t pph = 0;   // slab mode: pixel-copy buffer and its phase
      bool ok = true;
      bool slab_done = false;
      if constexpr (is_conv(EPI)) {
        if (p.slab) {
          // Slab mode, all of this CTA's tiles as one sequence of column shifts (three per 64-channel
          // block of a tile).  Per shift ONE barrier says that its copy and its weight blocks have
          // landed; one elected lane then issues its twelve MMAs and the commits.  (A barrier
          // operation waits its turn behind the MMAs' operand reads, 150 cycles and more: with a
          // wait, an election and a branch per weight block the issuer needed about 600 cycles
          // per block against the tensor pipe's 512.)
          int my_tiles = 0;
          while (tile_at(my_tiles) >= 0) ++my_tiles;
          const int ncs = 3 * p.kb_per_tap;
          const int total = my_tiles * ncs;
          int cs = 0;
          for (int g = 0; g < total && ok; ++g) {
            if (cs == 0) ok = mbar_wait(&tmem_empty[a], aph ^ 1u, abort_flag, p.status, KF_DEV_TIMEOUT_MMA);
            ok = ok && mbar_wait(slab_bar(kGFull + pb), pph, abort_flag, p.status, KF_DEV_TIMEOUT_MMA);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(a * BN);
            const uint32_t px = smem_u32(ring + pb * kSlabPx);
            const uint32_t wbase = smem_u32(ring + kSlabBufs * kSlabPx);
            const bool tile_end = cs == ncs - 1;
            if (elect_one()) {
#pragma unroll
              for (int r = 0; r < 3; ++r) {
                const int slot = s + r;                                // the shift's three blocks: slots s..s+2
                const uint64_t adesc = smem_desc_kmajor_sw128(wbase + static_cast<uint32_t>(slot * C::kStageA));
                // the window of tap row r starts r image rows (whole 1024-byte groups) into the copy
                const uint64_t bdesc = smem_desc_kmajor_sw128(px + static_cast<uint32_t>(r * p.slab_row_bytes));
#pragma unroll
                for (int k = 0; k < kBK / kUmmaK; ++k)
                  umma_f16_ss(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (cs | r | k) != 0 ? 1u : 0u);
                umma_commit(slab_bar(kWEmpty + slot));                  // frees the weight slot
              }
              umma_commit(slab_bar(kCEmpty + pb));                  // after the third tap, the copy
              if (tile_end) umma_commit(&tmem_full[a]);
            }
            __syncwarp();
            s = s == 0 ? 3 : 0;                                     // (slots 0..2 and 3..5 in turn)
            if (++pb == kSlabBufs) { pb = 0; pph ^= 1u; }
            if (tile_end) { cs = 0; if (++a == 2) { a = 0; aph ^= 1u; } } else { ++cs; }
          }
          slab_done = true;
        }
      }
      for (int it = 0; ok && !slab_done; ++it) {
        if (tile_at(it) < 0) break;
        ok = mbar_wait(&tmem_empty[a], aph ^ 1u, abort_flag, p.status, KF_DEV_TIMEOUT_MMA);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(a * BN);
        for (int kb = 0; kb < p.k_blocks; kb += C::kKB) {
          ok = mbar_wait(&full[s], ph, abort_flag, p.status, KF_DEV_TIMEOUT_MMA);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          tc_fence_after_sync();
          const uint32_t sa = smem_u32(ring + s * C::kStage);
          const int kbs = min(C::kKB, p.k_blocks - kb);              // K blocks in this stage
          if (elect_one()) {
#pragma unroll
            for (int j = 0; j < C::kKB; ++j) {
              if (j < kbs) {
                const uint64_t adesc = smem_desc_kmajor_sw128(sa + static_cast<uint32_t>(j * C::kStage1));
                const uint64_t bdesc = smem_desc_kmajor_sw128(sa + static_cast<uint32_t>(j * C::kStage1 + C::kStageA));
#pragma unroll
                for (int k = 0; k < kBK / kUmmaK; ++k) {
                  // +32 bytes per K step inside the 128-byte swizzled row = +2 in the address field
                  if constexpr (CTA2)
                    umma_f16_ss_pair(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (kb | j | k) != 0 ? 1u : 0u);
                  else
                    umma_f16_ss(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (kb | j | k) != 0 ? 1u : 0u);
                }
              }
            }
            if constexpr (CTA2) umma_commit_pair(&empty[s], 3);      // frees the stage in both CTAs
            else umma_commit(&empty[s]);
          }
          if (++s == kStages) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        if (elect_one()) {
          if constexpr (CTA2) umma_commit_pair(&tmem_full[a], 3);    // wakes both epilogues
          else umma_commit(&tmem_full[a]);
        }
        if (++a == 2) { a = 0; aph ^= 1u; }
      }
    }
    __syncwarp();
  } else if (EPI == EPI_CONV_GNX && warp == 2 + 4 * epi_groups(EPI, BN, CTA2)) {
    // ------------------------------------------------------------ helper warp (EPI_CONV_GNX)
    if constexpr (EPI == EPI_CONV_GNX) {
      const int my_tiles = cta < p.num_tiles ? (p.num_tiles - cta + ncta - 1) / ncta : 0;
      conv_gnx_helper(p, reinterpret_cast<float2*>(stg + C::kStaging + C::kBarBytes), gx_parts, gx_stats, abort_flag,
                      lane, my_tiles, tile_at);
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5, and 6..9 with two groups)
    if constexpr (EPI == EPI_SOFTMAX_GX) {
      const int my_tiles = cta < p.num_tiles ? (p.num_tiles - cta + ncta - 1) / ncta : 0;
      float* sb = reinterpret_cast<float*>(stg + C::kStaging + C::kBarBytes);
      softmax_gx_epilogue<BN, ACT, CTA2>(p, &tmY, &tmR, stg, sb, reinterpret_cast<float2*>(sb + BN), tmem_full, tmem_empty,
                                         abort_flag, tmem_base, rank, warp, lane, my_tiles, tile_at);
    } else if constexpr (EPI == EPI_CONV_GNX) {
      const int my_tiles = cta < p.num_tiles ? (p.num_tiles - cta + ncta - 1) / ncta : 0;
      conv_gnx_epilogue<BN, ACT>(p, &tmY, &tmB, stg, reinterpret_cast<float2*>(stg + C::kStaging + C::kBarBytes),
                                 tmem_full, tmem_empty, gx_parts, gx_stats, abort_flag, tmem_base, warp, lane,
                                 my_tiles, tile_at);
    } else {
    constexpr int kGroups = epi_groups(EPI, BN, CTA2);
    constexpr int NB = 2 / kGroups;            // elementwise: staging buffers per group (4 pieces in all)
    constexpr int kGroupCols = BN / kGroups;   // columns of the tile one epilogue group owns
    constexpr int PIECES = kGroupCols / kPieceCols;
    const int grp = kGroups > 1 ? (warp - 2) >> 2 : 0;
    const uint32_t bar_a = 1u + 2u * grp, bar_b = 2u + 2u * grp;   // the group's named barriers
    const int quad = warp & 3;                 // TMEM lane quarter this warp may read
    const int row = quad * 32 + lane;          // row of the tile = TMEM lane
    const int et = threadIdx.x - 64 - grp * kEpiThreads;   // 0..127 inside the group
    const bool leader = et == 0;               // polls for the group; issues the whole-piece TMA stores where those are used
    [[maybe_unused]] const bool lead_warp = warp == 2 + 4 * grp;   // its warp (a warp-uniform predicate)
    const uint32_t lane_off = static_cast<uint32_t>(quad * 32) << 16;
    [[maybe_unused]] uint8_t* ybuf = stg + grp * 2 * kPieceBytes;   // [2][kPieceBytes] output pieces
    // elementwise: per group NB output pieces, then NB residual pieces (each warp owns a 2 KB slab of each)
    [[maybe_unused]] uint8_t* rbuf = ybuf + NB * kPieceBytes;
    [[maybe_unused]] uint64_t* my_r_full = &r_full[(warp - 2) * NB];   // [NB]
    const bool staged = p.staged != 0;
    [[maybe_unused]] float* sbias = reinterpret_cast<float*>(stg + C::kStaging + C::kBarBytes) + grp * kGroupCols;   // the group's [kGroupCols] of [BN]
    [[maybe_unused]] const bool has_r = EPI == EPI_ELEMENTWISE && p.R != nullptr;
    const int num_units = p.num_tiles / p.tiles_per_unit;
    const int my_tiles = cta < num_units ? (num_units - cta + ncta - 1) / ncta * p.tiles_per_unit : 0;
    const int row0 = static_cast<int>(rank) * kBM;      // this CTA's first row inside the tile
    [[maybe_unused]] const long long total_pieces = static_cast<long long>(my_tiles) * PIECES;
    [[maybe_unused]] long long g = 0;          // running piece index of this CTA

    // residual piece gi -> rbuf[gi & 1] (leader only)
    [[maybe_unused]] auto issue_r = [&](long long gi) {
      const int ti = static_cast<int>(gi / PIECES), c = static_cast<int>(gi % PIECES);
      const int tile = sched_tile(p, cta, ncta, ti);
      const int b = static_cast<int>(gi % NB);
      // this warp's 32 rows of the group's piece (2 KB of the 8 KB buffer)
      mbar_expect_tx(&my_r_full[b], kPieceBytes / 4);
      tma_load_2d(rbuf + b * kPieceBytes + quad * (kPieceBytes / 4), &tmR, &my_r_full[b],
                  (tile % p.tiles_n) * BN + grp * kGroupCols + c * kPieceCols,
                  (tile / p.tiles_n) * kTileM + row0 + quad * 32);
    };
    if constexpr (EPI == EPI_ELEMENTWISE) {
      if (staged && has_r) {
        if (elect_one()) {
          for (int i = 0; i < NB; ++i)
            if (total_pieces > i) issue_r(i);
        }
      }
    }

    int a = 0; uint32_t aph = 0;
    bool alive = true;
    bool warp_failed = false;    // this warp gave up on one of its own waits inside a tile
    [[maybe_unused]] uint64_t keep_policy = 0;
    if constexpr (is_softmax(EPI)) keep_policy = l2_policy_evict_last();
    [[maybe_unused]] float unit_sum = 0.0f;    // row sum carried across the tiles of a unit
    for (int it = 0; alive; ++it) {
      const int tile = tile_at(it);
      if (tile < 0) break;
      int tm, tn;
      if constexpr (is_conv(EPI)) { tm = tile % p.tiles_m; tn = conv_pixel_tile(p, tile / p.tiles_m); }
      else { tm = tile / p.tiles_n; tn = tile % p.tiles_n; }
      const int m_cta = tm * kTileM + row0;               // first row of this CTA's 128 rows
      const long long m = static_cast<long long>(m_cta) + row;
      [[maybe_unused]] const bool row_ok = m < p.M;
      [[maybe_unused]] const int n_tile = tn * BN + grp * kGroupCols;   // the group's first column
      [[maybe_unused]] const int n_valid = min(kGroupCols, p.N - n_tile);   // its valid columns (may be <= 0)

      // GEMM epilogues: this thread's two of the group's bias values, fetched before the wait for
      // the accumulator so that the L2 latency is hidden, and staged in shared memory after it
      // (per piece every lane then reads the same 32 values: broadcast loads).
      [[maybe_unused]] float2 bpre = make_float2(0.0f, 0.0f);
      if constexpr (!is_conv(EPI)) {
        const int n = n_tile + 2 * et;
        if (p.bias != nullptr && 2 * et < kGroupCols) {
          if (n < p.N) bpre.x = __bfloat162float(p.bias[n]);
          if (n + 1 < p.N) bpre.y = __bfloat162float(p.bias[n + 1]);
        }
      }
      // One thread polls the accumulator barrier; the rest block in hardware at the named
      // barrier, which hands every epilogue warp the same go/no-go.
      bool ok = true;
      if (leader)
        ok = mbar_wait(&tmem_full[a], aph, abort_flag, p.status, KF_DEV_TIMEOUT_EPILOGUE);
      ok = named_barrier_and(bar_a, kEpiThreads, ok && !warp_failed);
      if (!ok) break;
      tc_fence_after_sync();
      if constexpr (!is_conv(EPI)) {
        // every thread is past its last read of the previous tile's values (barrier above)
        if (2 * et < kGroupCols) *reinterpret_cast<float2*>(sbias + 2 * et) = bpre;
        named_barrier_sync(bar_b, kEpiThreads);
      }
      const uint32_t t_acc = tmem_base + static_cast<uint32_t>(a * BN + grp * kGroupCols) + lane_off;
      // hand the accumulator back to the UMMA issuer (one arrival per warp)
      auto release_acc = [&]() {
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
          if constexpr (CTA2) mbar_arrive_cluster(mapa_shared(smem_u32(&tmem_empty[a]), 0));
          else mbar_arrive(&tmem_empty[a]);
        }
      };

      if constexpr (EPI == EPI_ELEMENTWISE) {
        __nv_bfloat16* Y = reinterpret_cast<__nv_bfloat16*>(p.out);
        if (staged) {
          [[maybe_unused]] float gn_mu = 0.0f, gn_rstd = 1.0f;
          float ts1 = 0.0f, ts2 = 0.0f;
#pragma unroll 1
          for (int c = 0; c < PIECES; ++c, ++g) {
            const int b = static_cast<int>(g % NB);
            uint4 rv[4];
            if (has_r) {
              // this warp's slab of the residual piece, then at once the request for the piece
              // that will use the same buffer
              bool rok = mbar_wait(&my_r_full[b], static_cast<uint32_t>((g / NB) & 1), abort_flag, p.status,
                                   KF_DEV_TIMEOUT_EPILOGUE);
              // a slab that never arrived: the status word has the time-out; keep going (every
              // warp of the group must reach the group's barriers) and leave with the others
              if (!rok) warp_failed = true;
#pragma unroll
              for (int q = 0; q < 4; ++q)
                rv[q] = *reinterpret_cast<const uint4*>(rbuf + b * kPieceBytes + piece_off(row, q));
              __syncwarp();
              if (elect_one()) {
                if (g + NB < total_pieces) issue_r(g + NB);
              }
            }
            if (p.gn_pieces > 0 && c % p.gn_pieces == 0) {
              // statistics of the group that starts here: its columns are all in this tile
              float s1 = 0.0f, s2 = 0.0f;
#pragma unroll 1
              for (int q = 0; q < p.gn_pieces; ++q) {
                uint32_t u[32];
                tmem_ld_32x32(t_acc + (c + q) * kPieceCols, u);
                float bq[32];
                load_sbias32(sbias + (c + q) * kPieceCols, bq);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  const float z = __uint_as_float(u[j]) + bq[j];
                  s1 += z;
                  s2 = fmaf(z, z, s2);
                }
              }
              const float inv_n = 1.0f / static_cast<float>(p.gn_pieces * kPieceCols);
              gn_mu = s1 * inv_n;
              gn_rstd = rsqrtf(fmaxf(s2 * inv_n - gn_mu * gn_mu, 0.0f) + p.gn_eps);
            }
            uint32_t v[32];
            tmem_ld_32x32(t_acc + c * kPieceCols, v);
            float bs[32];
            load_sbias32(sbias + c * kPieceCols, bs);
            tmem_ld_wait();
            if (c == PIECES - 1) release_acc();
            float f[32];
            if (p.gn_pieces > 0) {
              float ga[32], be[32];
              load_vec32(p.gn_gamma, p.N, n_tile + c * kPieceCols, 1.0f, ga);
              load_vec32(p.gn_beta, p.N, n_tile + c * kPieceCols, 0.0f, be);
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                const float u = (__uint_as_float(v[j]) + bs[j] - gn_mu) * gn_rstd;
                f[j] = p.scale * act_f<ACT, true>(fmaf(u, ga[j], be[j]), p.act_rt);
              }
            } else if (CTA2 || p.gn_tile_stats) {
              // (the CTA-pair kernel's epilogue hides behind its MMAs: it keeps the scalar form)
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                const float z = __uint_as_float(v[j]) + bs[j];
                if (p.gn_tile_stats) { ts1 += z; ts2 = fmaf(z, z, ts2); }   // columns past N hold 0
                f[j] = p.scale * act_f<ACT, true>(z, p.act_rt);
              }
            } else {
              // the plain chain on packed pairs: bias, then scale (and residual) in one
              // instruction per two columns
              const uint64_t scale2 = f32x2_pack(p.scale, p.scale);
              const uint32_t* rw = reinterpret_cast<const uint32_t*>(rv);   // 16 bf16 pairs
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                float z0, z1;
                f32x2_unpack(f32x2_add(f32x2_pack(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])),
                                       f32x2_pack(bs[2 * j], bs[2 * j + 1])), z0, z1);
                const uint64_t a2 = f32x2_pack(act_f<ACT, true>(z0, p.act_rt), act_f<ACT, true>(z1, p.act_rt));
                if (has_r) f32x2_unpack(f32x2_fma(a2, scale2, f32x2_pack(bf16_lo(rw[j]), bf16_hi(rw[j]))), f[2 * j], f[2 * j + 1]);
                else f32x2_unpack(f32x2_mul(a2, scale2), f[2 * j], f[2 * j + 1]);
              }
            }
            if (has_r && (CTA2 || p.gn_pieces > 0 || p.gn_tile_stats)) {
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                f[8 * q + 0] += bf16_lo(rv[q].x); f[8 * q + 1] += bf16_hi(rv[q].x);
                f[8 * q + 2] += bf16_lo(rv[q].y); f[8 * q + 3] += bf16_hi(rv[q].y);
                f[8 * q + 4] += bf16_lo(rv[q].z); f[8 * q + 5] += bf16_hi(rv[q].z);
                f[8 * q + 6] += bf16_lo(rv[q].w); f[8 * q + 7] += bf16_hi(rv[q].w);
              }
            }
            // Every warp stages and stores its own 32 rows of the piece (a 2 KB slab of the 8 KB
            // buffer, TMA box of 32 rows): no barrier between the warps anywhere in this loop.
            // First the store issued from this slab NB pieces ago must have finished reading it.
            bulk_wait_group_read<NB - 1>();     // a no-op in the lanes that issue no stores
            __syncwarp();
            uint8_t* yb = ybuf + b * kPieceBytes;
#pragma unroll
            for (int q = 0; q < 4; ++q)
              *reinterpret_cast<uint4*>(yb + piece_off(row, q)) =
                  make_uint4(pack_bf16x2(f[8 * q + 0], f[8 * q + 1]),
                             pack_bf16x2(f[8 * q + 2], f[8 * q + 3]),
                             pack_bf16x2(f[8 * q + 4], f[8 * q + 5]),
                             pack_bf16x2(f[8 * q + 6], f[8 * q + 7]));
            fence_proxy_async_smem();
            __syncwarp();
            if (elect_one()) {
              if (m_cta + quad * 32 < p.M && n_tile + c * kPieceCols < p.N)
                tma_store_2d(&tmY, yb + quad * (kPieceBytes / 4), n_tile + c * kPieceCols,
                             m_cta + quad * 32);                     // clipped at M, N
              bulk_commit_group();
            }
          }
          if (p.gn_tile_stats && alive && row_ok)
            reinterpret_cast<float2*>(p.partial)[(m * p.tiles_n + tn) * kGroups + grp] = make_float2(ts1, ts2);
        } else {
          // Output (or residual) rows that do not start on 16 bytes: no TMA.  Pieces still go
          // through shared memory so that global accesses run along rows: a warp moves 32 rows,
          // its lanes one bf16 column each (64 contiguous bytes per row and instruction).
          const int er = et >> 5;                      // this warp's row group in the copy loops
#pragma unroll 1
          for (int c = 0; c < PIECES; ++c) {
            if (c * 32 >= n_valid) break;
            const int n0 = n_tile + c * 32;
            const bool col_ok = n0 + lane < p.N;
            uint8_t* rb = rbuf;
            uint8_t* yb = ybuf;
            if (has_r) {
#pragma unroll 4
              for (int i = 0; i < 32; ++i) {
                const int r = i * 4 + er;
                const long long mr = static_cast<long long>(m_cta) + r;
                __nv_bfloat16 rv = __float2bfloat16_rn(0.0f);
                if (col_ok && mr < p.M) rv = p.R[mr * p.ldr + n0 + lane];
                *reinterpret_cast<__nv_bfloat16*>(rb + piece_off(r, lane >> 3) + (lane & 7) * 2) = rv;
              }
              named_barrier_sync(bar_b, kEpiThreads);
            }
            uint32_t v[32];
            tmem_ld_32x32(t_acc + c * 32, v);
            float bs[32];
            load_sbias32(sbias + c * 32, bs);
            tmem_ld_wait();
            float f[32];
#pragma unroll
            for (int j = 0; j < 32; ++j)
              f[j] = p.scale * act_f<ACT, true>(__uint_as_float(v[j]) + bs[j], p.act_rt);
            if (has_r) {
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const uint4 r4 = *reinterpret_cast<const uint4*>(rb + piece_off(row, q));
                f[8 * q + 0] += bf16_lo(r4.x); f[8 * q + 1] += bf16_hi(r4.x);
                f[8 * q + 2] += bf16_lo(r4.y); f[8 * q + 3] += bf16_hi(r4.y);
                f[8 * q + 4] += bf16_lo(r4.z); f[8 * q + 5] += bf16_hi(r4.z);
                f[8 * q + 6] += bf16_lo(r4.w); f[8 * q + 7] += bf16_hi(r4.w);
              }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q)
              *reinterpret_cast<uint4*>(yb + piece_off(row, q)) =
                  make_uint4(pack_bf16x2(f[8 * q + 0], f[8 * q + 1]),
                             pack_bf16x2(f[8 * q + 2], f[8 * q + 3]),
                             pack_bf16x2(f[8 * q + 4], f[8 * q + 5]),
                             pack_bf16x2(f[8 * q + 6], f[8 * q + 7]));
            named_barrier_sync(bar_b, kEpiThreads);
#pragma unroll 4
            for (int i = 0; i < 32; ++i) {
              const int r = i * 4 + er;
              const long long mr = static_cast<long long>(m_cta) + r;
              if (col_ok && mr < p.M)
                Y[mr * p.ldo + n0 + lane] =
                    *reinterpret_cast<const __nv_bfloat16*>(yb + piece_off(r, lane >> 3) + (lane & 7) * 2);
            }
            named_barrier_sync(bar_b, kEpiThreads);        // buffers free for the next piece
          }
          release_acc();
        }
      } else if constexpr (is_softmax(EPI)) {
        // pass 1: tile maximum of a = pre_act(z + b) over the valid columns of this row
        float mx = -INFINITY;
#pragma unroll 1
        for (int c = 0; c < PIECES; ++c) {
          if (c * 32 >= n_valid) break;
          uint32_t v[32];
          tmem_ld_32x32(t_acc + c * 32, v);
          float bs[32];
          load_sbias32(sbias + c * 32, bs);
          tmem_ld_wait();
          if (c * 32 + 32 <= n_valid) {          // whole piece: bias on packed pairs, no masks
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              float z0, z1;
              f32x2_unpack(f32x2_add(f32x2_pack(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])),
                                     f32x2_pack(bs[2 * j], bs[2 * j + 1])), z0, z1);
              mx = fmaxf(mx, fmaxf(act_f<ACT, true>(z0, p.act_rt), act_f<ACT, true>(z1, p.act_rt)));
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float z = act_f<ACT, true>(__uint_as_float(v[j]) + bs[j], p.act_rt);
              if (c * 32 + j < n_valid) mx = fmaxf(mx, z);
            }
          }
        }
        // A row that lies in this one tile (tiles_n == 1) is finished here: the two groups
        // exchange their maxima and their sums through shared memory (five barriers over both
        // groups per tile), a third pass over the accumulator stores the probabilities, and no
        // second kernel runs.  phase 0: the two-kernel form; 1: sum only; 2: scaled stores.
        constexpr bool kCl = EPI == EPI_SOFTMAX_CL;
        const bool whole_row = kCl || p.softmax_fused != 0;
        float* xch = reinterpret_cast<float*>(stg);                   // [2 groups][128 rows], in staging
        if (whole_row && !kCl) {
          bulk_wait_group_read<0>();               // the previous tile's stores have let go of staging ...
          named_barrier_sync(5u, kGroups * kEpiThreads);         // ... in both groups
          xch[grp * kEpiThreads + et] = mx;
          named_barrier_sync(5u, kGroups * kEpiThreads);
          mx = fmaxf(mx, xch[(grp ^ 1) * kEpiThreads + et]);
          named_barrier_sync(5u, kGroups * kEpiThreads);         // both maxima read: the slots are reused
        }
        // pass 2: numerators e = exp(a - mx), their fp32 sum, e stored in the output dtype
        // (statistics-only runs skip the stores; a maximum-only run skips the pass)
        OutT* P = reinterpret_cast<OutT*>(p.out);
        float sum = 0.0f;
        float inv = 1.0f;
        for (int phase = whole_row ? 1 : 0; phase <= (whole_row ? 2 : 0); ++phase) {
        if (phase == 2 && !kCl) {
          xch[grp * kEpiThreads + et] = sum;
          named_barrier_sync(5u, kGroups * kEpiThreads);
          inv = 1.0f / (xch[et] + xch[kEpiThreads + et]);           // group 0 + group 1: fixed order
          named_barrier_sync(5u, kGroups * kEpiThreads);         // read before staging is written again
        }
        if constexpr (kCl) {
          if (phase == 2) {
            // This group's (maximum, sum of exp(a - maximum)) per row goes to every CTA of the
            // cluster (bulk copies through distributed shared memory, completing on the
            // receiver's mbarrier); from the 2 x cluster-size pairs that arrive here every
            // thread forms its row's maximum M and denominator S = sum s_i * exp(m_i - M) in a
            // fixed order.  Buffers alternate per tile (see EPI_CONV_GN for why two suffice).
            const int buf = it & 1;
            const int csize = p.gn_cluster;
            float2* inbox = reinterpret_cast<float2*>(stg + C::kStaging + C::kBarBytes + C::kBiasBytes);
            constexpr int kClMax = C::kClMax;             // inbox slots per buffer: 2 groups x kClMax ranks
            float2* sbuf = inbox + 2 * 2 * kClMax * 128 + (buf * 2 + grp) * 128;
            sbuf[et] = make_float2(mx, sum);
            fence_proxy_async_smem();
            named_barrier_sync(bar_b, kEpiThreads);
            if (lead_warp) {
              if (elect_one()) {
                if (grp == 0) mbar_expect_tx(&rbar[buf], static_cast<uint32_t>(csize) * 2u * 1024u);
                const uint32_t dst = smem_u32(inbox + ((buf * kClMax + static_cast<int>(crank)) * 2 + grp) * 128);
                for (int r = 0; r < csize; ++r)
                  bulk_copy_to_peer(mapa_shared(dst, r), smem_u32(sbuf), 1024u, mapa_shared(smem_u32(&rbar[buf]), r));
              }
            }
            bool all_in = mbar_wait(&rbar[buf], static_cast<uint32_t>((it >> 1) & 1), abort_flag, p.status,
                                    KF_DEV_TIMEOUT_EPILOGUE);
            all_in = named_barrier_and(bar_a, kEpiThreads, all_in);
            if (!all_in) { alive = false; break; }
            const float2* ib = inbox + buf * 2 * kClMax * 128 + et;
            float big = -INFINITY;
            for (int r = 0; r < 2 * csize; ++r) big = fmaxf(big, ib[r * 128].x);
            float den = 0.0f;
            for (int r = 0; r < 2 * csize; ++r) { const float2 q = ib[r * 128]; den += q.y * __expf(q.x - big); }
            mx = big;
            inv = 1.0f / den;
          }
        }
#pragma unroll 1
        for (int c = 0; c < PIECES && p.stats_only != 2; ++c, ++g) {
          if (!staged && c * 32 >= n_valid) break;
          uint32_t v[32];
          tmem_ld_32x32(t_acc + c * 32, v);
          float bs[32];
          load_sbias32(sbias + c * 32, bs);
          tmem_ld_wait();
          if (staged && c == PIECES - 1 && phase != 1) release_acc();
          float f[32];
          if (c * 32 + 32 <= n_valid) {
            // whole piece on packed pairs: exp(z - mx) = 2^(z log2(e) - mx log2(e)), one fused
            // multiply-add per two columns; even and odd columns add up separately
            constexpr float kLog2e = 1.4426950408889634f;
            const uint64_t l2e2 = f32x2_pack(kLog2e, kLog2e);
            const uint64_t off2 = f32x2_pack(-mx * kLog2e, -mx * kLog2e);
            const uint64_t inv2 = f32x2_pack(inv, inv);
            uint64_t sum2 = f32x2_pack(0.0f, 0.0f);
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              float z0, z1;
              f32x2_unpack(f32x2_add(f32x2_pack(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])),
                                     f32x2_pack(bs[2 * j], bs[2 * j + 1])), z0, z1);
              f32x2_unpack(f32x2_fma(f32x2_pack(act_f<ACT, true>(z0, p.act_rt), act_f<ACT, true>(z1, p.act_rt)), l2e2, off2),
                           z0, z1);
              uint64_t e2 = f32x2_pack(exp2_approx(z0), exp2_approx(z1));
              if (whole_row) e2 = f32x2_mul(e2, inv2);
              f32x2_unpack(e2, f[2 * j], f[2 * j + 1]);
              if (phase != 2) sum2 = f32x2_add(sum2, e2);
            }
            float se, so;
            f32x2_unpack(sum2, se, so);
            sum += se + so;
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float z = act_f<ACT, true>(__uint_as_float(v[j]) + bs[j], p.act_rt);
              f[j] = __expf(z - mx) * inv;
              if (phase != 2 && c * 32 + j < n_valid) sum += f[j];
            }
          }
          if (p.stats_only != 0 || phase == 1) continue;
          if constexpr (sizeof(OutT) == 2) {
            if (staged) {
              const int b = static_cast<int>(g & 1);
              uint8_t* yb = ybuf + b * kPieceBytes;
#pragma unroll
              for (int q = 0; q < 4; ++q)
                *reinterpret_cast<uint4*>(yb + piece_off(row, q)) =
                    make_uint4(pack_bf16x2(f[8 * q + 0], f[8 * q + 1]),
                               pack_bf16x2(f[8 * q + 2], f[8 * q + 3]),
                               pack_bf16x2(f[8 * q + 4], f[8 * q + 5]),
                               pack_bf16x2(f[8 * q + 6], f[8 * q + 7]));
              fence_proxy_async_smem();
              if (leader) bulk_wait_group_read<0>();   // the other buffer's store has let go
              named_barrier_sync(bar_b, kEpiThreads);
              if (leader) {
                // the second pass reads these numerators back: ask L2 to keep them
                tma_store_2d_hint(&tmY, yb, n_tile + c * kPieceCols, m_cta, keep_policy);
                bulk_commit_group();
              }
              continue;
            }
          }
          if constexpr (sizeof(OutT) == 2) {
            // bf16 rows that do not start on 16 bytes: through shared memory, then along rows
            // (a warp moves 32 rows, its lanes one column each)
            uint8_t* yb = ybuf;
#pragma unroll
            for (int q = 0; q < 4; ++q)
              *reinterpret_cast<uint4*>(yb + piece_off(row, q)) =
                  make_uint4(pack_bf16x2(f[8 * q + 0], f[8 * q + 1]),
                             pack_bf16x2(f[8 * q + 2], f[8 * q + 3]),
                             pack_bf16x2(f[8 * q + 4], f[8 * q + 5]),
                             pack_bf16x2(f[8 * q + 6], f[8 * q + 7]));
            named_barrier_sync(bar_b, kEpiThreads);
            const int er = et >> 5;
            if (c * 32 + lane < n_valid) {
#pragma unroll 4
              for (int i = 0; i < 32; ++i) {
                const int r = i * 4 + er;
                const long long mr = static_cast<long long>(m_cta) + r;
                if (mr < p.M)
                  P[mr * p.ldo + n_tile + c * 32 + lane] =
                      *reinterpret_cast<const OutT*>(yb + piece_off(r, lane >> 3) + (lane & 7) * 2);
              }
            }
            named_barrier_sync(bar_b, kEpiThreads);    // the buffer is free for the next piece
            continue;
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
        }   // phase
        if (!alive) break;
        if (!staged) release_acc();
        if (row_ok && !whole_row) {
          float2* part = reinterpret_cast<float2*>(p.partial);
          part[(m * p.tiles_n + tn) * kGroups + grp] = make_float2(mx, sum);
        }
      } else if constexpr (EPI == EPI_ROWSUM) {
        float sum = 0.0f;
#pragma unroll 1
        for (int c = 0; c < PIECES; ++c) {
          if (c * 32 >= n_valid) break;
          uint32_t v[32];
          tmem_ld_32x32(t_acc + c * 32, v);
          float bs[32];
          load_sbias32(sbias + c * 32, bs);
          tmem_ld_wait();
          float part = 0.0f;
          if (c * 32 + 32 <= n_valid) {          // whole piece: packed pairs, no masks
            uint64_t part2 = f32x2_pack(0.0f, 0.0f);
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              float z0, z1;
              f32x2_unpack(f32x2_add(f32x2_pack(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])),
                                     f32x2_pack(bs[2 * j], bs[2 * j + 1])), z0, z1);
              part2 = f32x2_add(part2, f32x2_pack(act_f<ACT, true>(z0, p.act_rt), act_f<ACT, true>(z1, p.act_rt)));
            }
            float pe, po;
            f32x2_unpack(part2, pe, po);
            part = pe + po;
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float z = act_f<ACT, true>(__uint_as_float(v[j]) + bs[j], p.act_rt);
              if (c * 32 + j < n_valid) part += z;
            }
          }
          sum += part;
        }
        release_acc();
        if (p.partial != nullptr) {
          if (row_ok) p.partial[m * p.tiles_n + tn] = sum;
        } else {
          // this CTA owns the whole row block: add the tiles in order, write the row sum once
          unit_sum = (tn == 0) ? sum : unit_sum + sum;
          if (tn == p.tiles_n - 1 && row_ok) reinterpret_cast<float*>(p.out)[m] = unit_sum * p.scale;
        }
      } else {
        // EPI_CONV: rows = output channels, columns = BN consecutive pixels of one image, so a
        // thread's 32-column chunk is 64 contiguous bytes of the NCHW output.  a = act(z + b) is
        // rounded to bf16 and stored; the per-channel sum and sum of squares of a (in fp32,
        // before rounding) over this tile go to `partial` for the GroupNorm that follows.
        const int ch = tm * kBM + row;                      // output channel of this thread
        const bool ch_ok = ch < p.N;
        const int img = tn / p.tiles_per_image;
        const int pt = tn % p.tiles_per_image;              // pixel tile inside the image
        const float bias_v = (p.bias != nullptr && ch_ok) ? __bfloat162float(p.bias[ch]) : 0.0f;
        const long long hw = static_cast<long long>(p.H) * p.Wd;
        const int pieces = p.tile_px / 32;                  // <= PIECES
        const int px0 = pt * p.tile_px;                     // first pixel of the tile in its image
        // the last tile of an image may hang over its end: those pixels were read as zeros, are
        // left out of the statistics and are not stored
        const int px_valid = static_cast<int>(min(static_cast<long long>(p.tile_px), hw - px0));
        float s1 = 0.0f, s2 = 0.0f;
        const uint64_t bias2 = f32x2_pack(bias_v, bias_v);
        uint64_t s1p = f32x2_pack(0.0f, 0.0f), s2p = s1p;   // (even, odd) pixel partial sums
        const bool want_stats = p.partial != nullptr;
        if constexpr (EPI == EPI_CONV_GN) {
          // GroupNorm without a second kernel.  The CTAs of this cluster hold the tiles of one
          // image, one each.  The accumulator stays in TMEM while (1) each epilogue group adds
          // up its half of the tile per channel and, by shuffles, per GroupNorm group (sum, sum
          // of squares), (2) sends those 32 pairs to every CTA of the cluster with bulk copies
          // through distributed shared memory, which complete on the receiver's mbarrier, (3)
          // waits (bounded) for the 2 x cluster-size contributions to its own inbox, adds them
          // in a fixed order, and (4) reads the accumulator again, normalises and stores.
          // Meanwhile the MMA warp fills the other accumulator.  Buffers alternate per tile; a
          // CTA sends tile k+2 only after every peer has sent tile k+1, i.e. after every peer
          // has finished reading tile k's buffers.
          constexpr int kGP = kGroupCols / 32;                    // pieces per epilogue group
          const int my_pieces = max(0, min(kGP, pieces - grp * kGP));
          const int piece0 = grp * kGP;
          const int buf = it & 1;
          const int csize = p.gn_cluster;
          const int cpg = p.N / p.gn_groups;                      // channels per group: 4, 8, 16 or 32
          float2* sbuf = reinterpret_cast<float2*>(stg + C::kStaging + C::kBarBytes) + (buf * 2 + grp) * 32;
          float2* inbox = reinterpret_cast<float2*>(stg + C::kStaging + C::kBarBytes + C::kBiasBytes);
          uint8_t* yslab = stg + grp * kPieceBytes;               // the group's staging piece
#pragma unroll 1
          for (int c = 0; c < my_pieces; ++c) {
            uint32_t v[32];
            tmem_ld_32x32(t_acc + c * 32, v);
            tmem_ld_wait();
            const int left = px_valid - (piece0 + c) * 32;
            if (left >= 32) {
              // whole piece: bias, sum and sum of squares on packed pairs (even and odd pixels
              // accumulate separately and are added after the loop)
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                float y0, y1;
                f32x2_unpack(f32x2_add(f32x2_pack(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])), bias2), y0, y1);
                const uint64_t y = f32x2_pack(act_f<ACT, true>(y0, p.act_rt), act_f<ACT, true>(y1, p.act_rt));
                s1p = f32x2_add(s1p, y);
                s2p = f32x2_fma(y, y, s2p);
              }
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                float y0 = act_f<ACT, true>(__uint_as_float(v[2 * j]) + bias_v, p.act_rt);
                float y1 = act_f<ACT, true>(__uint_as_float(v[2 * j + 1]) + bias_v, p.act_rt);
                if (2 * j >= left) y0 = 0.0f;
                if (2 * j + 1 >= left) y1 = 0.0f;
                s1 += y0 + y1;
                s2 = fmaf(y0, y0, fmaf(y1, y1, s2));
              }
            }
          }
          {
            float e, o;
            f32x2_unpack(s1p, e, o); s1 += e + o;
            f32x2_unpack(s2p, e, o); s2 += e + o;
          }
          for (int o = cpg >> 1; o > 0; o >>= 1) {                // the group's channels: adjacent lanes
            s1 += __shfl_xor_sync(0xffffffffu, s1, o);
            s2 += __shfl_xor_sync(0xffffffffu, s2, o);
          }
          if ((row & (cpg - 1)) == 0) sbuf[row / cpg] = make_float2(s1, s2);
          fence_proxy_async_smem();
          named_barrier_sync(bar_b, kEpiThreads);
          if (lead_warp) {
            if (elect_one()) {
              if (grp == 0) mbar_expect_tx(&rbar[buf], static_cast<uint32_t>(csize) * 2u * 256u);
              const uint32_t dst = smem_u32(inbox + ((buf * 16 + static_cast<int>(crank)) * 2 + grp) * 32);
              for (int r = 0; r < csize; ++r)
                bulk_copy_to_peer(mapa_shared(dst, r), smem_u32(sbuf), 256u, mapa_shared(smem_u32(&rbar[buf]), r));
            }
          }
          // every thread waits itself (it reads what the copies wrote), then one decision for all
          bool all_in = mbar_wait(&rbar[buf], static_cast<uint32_t>((it >> 1) & 1), abort_flag, p.status,
                                  KF_DEV_TIMEOUT_EPILOGUE);
          all_in = named_barrier_and(bar_a, kEpiThreads, all_in);
          if (!all_in) break;
          float sc = 0.0f, sh = 0.0f;
          {
            const float2* ib = inbox + buf * 16 * 2 * 32 + row / cpg;
            float g1 = 0.0f, g2 = 0.0f;
#pragma unroll 4      // loads in flight together; the additions keep their order
            for (int r = 0; r < 2 * csize; ++r) { const float2 q = ib[r * 32]; g1 += q.x; g2 += q.y; }
            const float cnt = static_cast<float>(static_cast<long long>(cpg) * hw);
            const float mu = g1 / cnt;
            const float rstd = rsqrtf(fmaxf(g2 / cnt - mu * mu, 0.0f) + p.gn_eps);
            const float ga = (p.gn_gamma != nullptr && ch_ok) ? __bfloat162float(p.gn_gamma[ch]) : 1.0f;
            const float be = (p.gn_beta != nullptr && ch_ok) ? __bfloat162float(p.gn_beta[ch]) : 0.0f;
            sc = rstd * ga;
            sh = fmaf(-mu, sc, be);
          }
          if (my_pieces == 0) release_acc();
          const uint64_t sc2 = f32x2_pack(sc, sc), sh2 = f32x2_pack(sh, sh);
#pragma unroll 1
          for (int c = 0; c < my_pieces; ++c) {
            uint32_t v[32];
            tmem_ld_32x32(t_acc + c * 32, v);
            tmem_ld_wait();
            if (c == my_pieces - 1) release_acc();
            uint32_t w[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              float y0, y1;
              f32x2_unpack(f32x2_add(f32x2_pack(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])), bias2), y0, y1);
              const uint64_t y = f32x2_pack(act_f<ACT, true>(y0, p.act_rt), act_f<ACT, true>(y1, p.act_rt));
              f32x2_unpack(f32x2_fma(y, sc2, sh2), y0, y1);
              w[j] = pack_bf16x2(y0, y1);
            }
            bulk_wait_group_read<0>();       // this warp's previous store has let go of the slab
            __syncwarp();
#pragma unroll
            for (int q = 0; q < 4; ++q)
              *reinterpret_cast<uint4*>(yslab + piece_off(row, q)) =
                  make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
            fence_proxy_async_smem();
            __syncwarp();
            if (elect_one()) {
              if (px_valid - (piece0 + c) * 32 > 0 && tm * kBM + quad * 32 < p.N)
                tma_store_3d(&tmY, yslab + quad * (kPieceBytes / 4), px0 + (piece0 + c) * 32,
                             tm * kBM + quad * 32, img);
              bulk_commit_group();
            }
          }
          if (++a == 2) { a = 0; aph ^= 1u; }
          continue;
        }
        if (p.pool2 != 0) {
          // 2x2 pooling of a = act(z + b): the tile holds whole pairs of image rows, a 32-pixel
          // piece is a stretch of one row, so the thread combines the pieces at the same place
          // of an even and the following odd row into 16 pooled pixels (32 contiguous bytes of
          // the pooled NCHW plane).  The activations themselves are never stored.
          const int wp = p.Wd / 32;                          // pieces per image row
          const int Wo = p.Wd / 2;
          const int h0 = pt * p.rows_per_tile;               // first image row of the tile
          const int pairs = min(p.rows_per_tile, p.H - h0) / 2;
          __nv_bfloat16* plane = reinterpret_cast<__nv_bfloat16*>(p.out) +
                                 (static_cast<long long>(img) * p.N + ch) * (hw / 4) +
                                 static_cast<long long>(h0 / 2) * Wo;
#pragma unroll 1
          for (int c = 0; c < pairs * wp; ++c) {
            const int pr = c / wp, hh = c - pr * wp;
            uint32_t v0[32], v1[32];
            tmem_ld_32x32(t_acc + (2 * pr * wp + hh) * 32, v0);
            tmem_ld_32x32(t_acc + ((2 * pr + 1) * wp + hh) * 32, v1);
            tmem_ld_wait();
            if (c == pairs * wp - 1) release_acc();
            uint32_t w[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              float o[2];
#pragma unroll
              for (int t = 0; t < 2; ++t) {
                const int i = 4 * j + 2 * t;
                float a00, a01, a10, a11;
                f32x2_unpack(f32x2_add(f32x2_pack(__uint_as_float(v0[i]), __uint_as_float(v0[i + 1])), bias2), a00, a01);
                f32x2_unpack(f32x2_add(f32x2_pack(__uint_as_float(v1[i]), __uint_as_float(v1[i + 1])), bias2), a10, a11);
                a00 = act_f<ACT, true>(a00, p.act_rt);
                a01 = act_f<ACT, true>(a01, p.act_rt);
                a10 = act_f<ACT, true>(a10, p.act_rt);
                a11 = act_f<ACT, true>(a11, p.act_rt);
                o[t] = p.pool2 == 1 ? fmaxf(fmaxf(a00, a01), fmaxf(a10, a11))
                                    : 0.25f * ((a00 + a01) + (a10 + a11));
              }
              w[j] = pack_bf16x2(o[0], o[1]);
            }
            if (ch_ok) {
              __nv_bfloat16* dst = plane + static_cast<long long>(pr) * Wo + hh * 16;
              if (p.vec_ok) {
                *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
                *reinterpret_cast<uint4*>(dst + 8) = make_uint4(w[4], w[5], w[6], w[7]);
              } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) {      // the plane may start on any 2-byte boundary
                  dst[2 * j] = __ushort_as_bfloat16(static_cast<unsigned short>(w[j] & 0xffffu));
                  dst[2 * j + 1] = __ushort_as_bfloat16(static_cast<unsigned short>(w[j] >> 16));
                }
              }
            }
          }
          if (++a == 2) { a = 0; aph ^= 1u; }
          continue;
        }
        int c = 0;
        if constexpr (EPI == EPI_CONV) {
          // whole pairs of pieces leave as slabs of 64 pixels x 32 channels (128-byte rows,
          // 128-byte swizzle, the store map in tmB, which slab mode does not use): half as many
          // waits for the slab, fences and store issues
          if (staged && p.y_wide && p.stats_only == 0) {
#pragma unroll 1
            for (; c + 2 <= pieces && px_valid - c * 32 >= 64; c += 2, ++g) {
              uint32_t w[32];
#pragma unroll
              for (int h = 0; h < 2; ++h) {
                uint32_t v[32];
                tmem_ld_32x32(t_acc + (c + h) * 32, v);
                tmem_ld_wait();
                if (h == 1 && c + 2 == pieces) release_acc();
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                  float y0, y1;
                  f32x2_unpack(f32x2_add(f32x2_pack(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])), bias2), y0, y1);
                  y0 = act_f<ACT, true>(y0, p.act_rt);
                  y1 = act_f<ACT, true>(y1, p.act_rt);
                  w[h * 16 + j] = pack_bf16x2(y0, y1);
                  if (want_stats) {
                    const uint64_t y = f32x2_pack(y0, y1);
                    s1p = f32x2_add(s1p, y);
                    s2p = f32x2_fma(y, y, s2p);
                  }
                }
              }
              uint8_t* yw = stg + ((static_cast<int>(g & 1)) * 4 + quad) * 4096;
              bulk_wait_group_read<1>();     // the store from this buffer two slabs ago has let go
              __syncwarp();
#pragma unroll
              for (int q = 0; q < 8; ++q)
                *reinterpret_cast<uint4*>(yw + lane * 128 + ((q ^ (lane & 7)) << 4)) =
                    make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
              fence_proxy_async_smem();
              __syncwarp();
              if (elect_one()) {
                if (tm * kBM + quad * 32 < p.N)
                  tma_store_3d(&tmB, yw, px0 + c * 32, tm * kBM + quad * 32, img);
                bulk_commit_group();
              }
            }
          }
        }
#pragma unroll 1
        for (; c < pieces; ++c, ++g) {
          uint32_t v[32];
          tmem_ld_32x32(t_acc + c * 32, v);
          tmem_ld_wait();
          if (c == pieces - 1) release_acc();
          uint32_t w[16];
          const int left = px_valid - c * 32;               // valid pixels from this piece on
          if (left >= 32) {
            // whole piece: bias (and the statistics, where a later pass wants them) on packed
            // pairs; even and odd pixels accumulate separately and are added after the loop
            if (want_stats) {
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                float y0, y1;
                f32x2_unpack(f32x2_add(f32x2_pack(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])), bias2), y0, y1);
                y0 = act_f<ACT, true>(y0, p.act_rt);
                y1 = act_f<ACT, true>(y1, p.act_rt);
                w[j] = pack_bf16x2(y0, y1);
                const uint64_t y = f32x2_pack(y0, y1);
                s1p = f32x2_add(s1p, y);
                s2p = f32x2_fma(y, y, s2p);
              }
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                float y0, y1;
                f32x2_unpack(f32x2_add(f32x2_pack(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])), bias2), y0, y1);
                w[j] = pack_bf16x2(act_f<ACT, true>(y0, p.act_rt), act_f<ACT, true>(y1, p.act_rt));
              }
            }
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              float y0 = act_f<ACT, true>(__uint_as_float(v[2 * j]) + bias_v, p.act_rt);
              float y1 = act_f<ACT, true>(__uint_as_float(v[2 * j + 1]) + bias_v, p.act_rt);
              w[j] = pack_bf16x2(y0, y1);
              if (2 * j >= left) y0 = 0.0f;
              if (2 * j + 1 >= left) y1 = 0.0f;
              s1 += y0 + y1;
              s2 = fmaf(y0, y0, fmaf(y1, y1, s2));
            }
          }
          if (p.stats_only != 0) continue;     // only the per-channel statistics are wanted
          if (staged) {
            // every warp stages and stores its own 32 channels of the piece (2 KB slab, TMA box
            // of 32 pixels x 32 channels): no barrier between the warps
            // (two buffers of a 4 KB slab per warp, shared with the 64-pixel form above, which
            // uses all of a slab: the 32-pixel form uses its first half)
            constexpr int kWarpSlab = EPI == EPI_CONV ? 4096 : 2048;   // (only EPI_CONV has room for the wide form)
            uint8_t* yb = stg + ((static_cast<int>(g & 1)) * 4 + quad) * kWarpSlab;
            bulk_wait_group_read<1>();       // the store from this buffer two pieces ago has let go
            __syncwarp();
#pragma unroll
            for (int q = 0; q < 4; ++q)
              *reinterpret_cast<uint4*>(yb + piece_off(lane, q)) =
                  make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
            fence_proxy_async_smem();
            __syncwarp();
            if (elect_one()) {
              // channels past Cout and pixels past the image are clipped
              if (left > 0 && tm * kBM + quad * 32 < p.N)
                tma_store_3d(&tmY, yb, px0 + c * 32, tm * kBM + quad * 32, img);
              bulk_commit_group();
            }
          } else {
            // Image planes that do not start on 16 bytes: no TMA store.  The piece still goes
            // through shared memory so that the global writes run along pixels: a warp moves
            // 32 channel rows, its lanes one pixel each (64 contiguous bytes per instruction).
            uint8_t* yb = ybuf;
#pragma unroll
            for (int q = 0; q < 4; ++q)
              *reinterpret_cast<uint4*>(yb + piece_off(row, q)) =
                  make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
            named_barrier_sync(bar_b, kEpiThreads);
            const int er = et >> 5;
            __nv_bfloat16* plane = reinterpret_cast<__nv_bfloat16*>(p.out) +
                                   static_cast<long long>(img) * p.N * hw + px0 + c * 32 + lane;
#pragma unroll 4
            for (int i = 0; i < 32; ++i) {
              const int r = i * 4 + er;
              const int cho = tm * kBM + r;
              if (lane < left && cho < p.N)
                plane[static_cast<long long>(cho) * hw] =
                    *reinterpret_cast<const __nv_bfloat16*>(yb + piece_off(r, lane >> 3) + (lane & 7) * 2);
            }
            named_barrier_sync(bar_b, kEpiThreads);    // the buffer is free for the next piece
          }
        }
        if (want_stats && ch_ok) {                // one entry per pixel tile and channel
          float e, o;
          f32x2_unpack(s1p, e, o); s1 += e + o;
          f32x2_unpack(s2p, e, o); s2 += e + o;
          float2* part = reinterpret_cast<float2*>(p.partial);
          part[static_cast<long long>(tn) * p.N + ch] = make_float2(s1, s2);
        }
      }
      if (++a == 2) { a = 0; aph ^= 1u; }
    }
    // every output store has finished reading shared memory (a no-op in lanes that issued none);
    // the writes themselves complete with the kernel, like any store in flight at exit
    bulk_wait_group_read<0>();
    }   // the epilogues other than EPI_CONV_GNX
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
  // a pair leaves together: the peer's MMAs read this CTA's shared memory and signal its barriers
  if constexpr (CTA2 || is_cluster_epi(EPI)) cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after_sync();
    if constexpr (CTA2) tmem_dealloc_pair(tmem_base, 2 * BN);
    else tmem_dealloc(tmem_base, 2 * BN);
  }
}

}  // namespace kf
