/* kf.h -- C ABI of the fused-operator-chain library for NVIDIA B200 (sm_100a).
 *
 * The library executes, as one hand-written CUDA kernel per chain (plus a streaming second
 * pass where a reduction spans tiles), the operator chains the Kernel Foundry paper's search
 * targets: a dense contraction followed by its elementwise and reduction epilogue.  The
 * problem statement mirrored here is the paper's own (Section 3.1 and Appendix A, output
 * requirement 1): a given PyTorch operator chain in, a kernel that computes the same function
 * out, with every operator computed inside the kernel rather than by an external library
 * call (Section 3.2.2, anti-cheating rule).
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers on the current CUDA device.  The caller owns
 *     every buffer, including the workspace; the library allocates no device memory.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Calls only enqueue work on that stream and return; nothing synchronises.
 *   - Matrices are row-major with a leading dimension in ELEMENTS (ld >= row length).
 *   - dtype KF_F32 = IEEE fp32, KF_BF16 = bfloat16.  bf16 chains accumulate in fp32 on the
 *     tensor cores, apply the epilogue in fp32 and round once (nearest-even) on store.
 *     fp32 chains never use single-pass TF32: small ones run on fp32 FMA, large ones on the
 *     tensor cores with every operand split into two TF32 parts (three products per term,
 *     fp32 running sum), which stays inside the fp32 tolerance.
 *   - bias / gamma / beta vectors have the chain's io dtype.
 *   - Errors are return codes; nothing throws, aborts or prints.  On any code other than
 *     KF_OK no kernel was launched by that call.  Inputs must be finite.
 *   - The workspace must be 256-byte aligned and at least the size the matching
 *     *_workspace_bytes() query returns (which may be 0, in which case NULL is accepted).
 *     Its contents need not be initialised and are undefined afterwards.  Two calls that
 *     share a workspace must be ordered on one stream.
 *   - There is no CPU fallback: without a CUDA device the calls return KF_ERR_CUDA.
 */
#ifndef KF_H_
#define KF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  KF_OK = 0,
  KF_ERR_INVALID_ARG = 1, /* null/misaligned pointer, non-positive size, ld too small, bad enum */
  KF_ERR_UNSUPPORTED = 2, /* a valid request this build has no kernel for */
  KF_ERR_WORKSPACE = 3,   /* workspace null, misaligned or too small */
  KF_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed (no device, launch error) */
  KF_ERR_TIMEOUT = 5      /* a device-side bounded wait ran out (reported by kf_device_status) */
} kf_status;

typedef enum { KF_F32 = 0, KF_BF16 = 1 } kf_dtype;

/* Activations.  0..3 are the benchmark chains' (the paper's "matmul + relu" class,
 * Appendix A strategy 2); 4..8 are the operators of the paper's worked chain (Appendix C.2):
 * erf-form GELU t*0.5*(1+erf(t/sqrt 2)), swish sigmoid(x)*x, tanh, hardtanh clamp[-1,1], and
 * KF_ACT_CHAIN95 = hardtanh(gelu_erf(tanh(swish(z)))) applied to z = XW^T + bias.  9..15 are
 * further elementwise operators of operator chains like the paper's (its Table 2 names chain
 * categories, not formulas): PyTorch's definitions with default parameters - leaky ReLU (slope
 * 0.01), ELU (alpha 1), Mish z*tanh(softplus z), hardswish z*relu6(z+3)/6, softplus log(1+e^z),
 * ReLU6, hardsigmoid relu6(z+3)/6.  They share one kernel instantiation and are selected by a
 * switch inside the epilogue. */
typedef enum {
  KF_ACT_NONE = 0,
  KF_ACT_RELU = 1,
  KF_ACT_GELU_TANH = 2,
  KF_ACT_SIGMOID = 3,
  KF_ACT_GELU_ERF = 4,
  KF_ACT_SWISH = 5,
  KF_ACT_TANH = 6,
  KF_ACT_HARDTANH = 7,
  KF_ACT_CHAIN95 = 8,
  KF_ACT_LEAKY_RELU = 9,
  KF_ACT_ELU = 10,
  KF_ACT_MISH = 11,
  KF_ACT_HARDSWISH = 12,
  KF_ACT_SOFTPLUS = 13,
  KF_ACT_RELU6 = 14,
  KF_ACT_HARDSIGMOID = 15
} kf_act;

typedef enum {
  KF_RED_SOFTMAX = 0,
  KF_RED_SUM = 1,
  KF_RED_MAX = 2,
  KF_RED_MEAN = 3,
  KF_RED_LOGSUMEXP = 4
} kf_rowred;

/* GEMM + elementwise epilogue (Appendix A, "Operator Fusion": matmul + activation class;
 * Table 2 "Matmul-centered").
 *   Y[m,n] = scale * act( sum_k X[m,k]*W[n,k] + bias[n] ) + residual[m,n]
 * in that order: bias, activation, scale, residual.  X is [M,K] (ldx), W is [N,K] (ldw) as in
 * torch.nn.Linear, residual and Y are [M,N] (ldr, ldy).  bias and residual may be NULL.
 * Y must not alias X or W; Y may alias residual only if ldr == ldy (same element, same place).
 * Shapes: any M,N,K >= 1.  bf16 problems with K % 8 == 0, ldx % 8 == 0, ldw % 8 == 0 and
 * 16-byte aligned X, W take the bf16 tensor-core kernels (whole tiles, or a split-K cluster when
 * there are few tiles and K is long).  fp32 problems with M*N*K >= 2^29 take the tensor cores
 * too: each operand is split into two TF32 numbers (22 significant bits together), three
 * products per element pair are accumulated, and partial sums are folded into an fp32 running
 * sum every 512 elements of K; absolute error about 1e-5 on outputs of magnitude 1, like an
 * fp32 FMA loop, for any K.  That path needs the workspace kf_gemm_epilogue_workspace_bytes()
 * returns (the split operands: 8*(M+N)*ceil4(K) bytes) and fails with KF_ERR_WORKSPACE
 * without it.  bf16 operands that TMA cannot load as they are (K, ldx or ldw not a multiple of
 * 8, X or W off 16 bytes) are copied into zero-padded dense rows and take the tensor cores too
 * when M*N*K >= 2^24 and the workspace holds the copies (2*(M+N)*ceil8(K) bytes, rounded up
 * to 256 per operand; the query returns that size when K % 8 != 0); otherwise they, and
 * everything else, take a scalar kernel. */
kf_status kf_gemm_epilogue(int64_t M, int64_t N, int64_t K, kf_dtype io_dtype,
                           const void* X, int64_t ldx, const void* W, int64_t ldw,
                           const void* bias, kf_act act, float scale,
                           const void* residual, int64_t ldr, void* Y, int64_t ldy,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/* GEMM + bias + GroupNorm over groups of consecutive columns + activation (a "mixed reduction"
 * chain in the sense of the paper's Table 2; the normalisation is torch.nn.GroupNorm applied to
 * a [M,N] matrix, N being the channel axis).  With Z[m,n] = sum_k X[m,k]*W[n,k] + bias[n] and
 * gs = N / groups, per row m and group g (columns [g*gs, (g+1)*gs)):
 *   mu = mean Z, var = mean (Z-mu)^2 (biased), Y = post_act((Z-mu)/sqrt(var+eps)*gamma[n]+beta[n]).
 * gamma, beta [N] of io_dtype, may be NULL (1, 0); groups must divide N (groups = 1 normalises
 * the whole row, as a LayerNorm does).  bf16 problems whose group size is 32, 64 or
 * 128, with TMA-loadable operands (see kf_gemm_epilogue) and a 16-byte aligned Y with
 * ldy % 8 == 0, run in ONE tensor-core kernel: the half tile an epilogue group owns holds whole
 * groups, so the epilogue takes the statistics from the accumulator and normalises before
 * storing.  Group sizes that are multiples of 256 take the same GEMM kernel storing Z plus
 * per-slice statistics (workspace: 16 bytes per row and 256 columns) and a row kernel that
 * normalises in place.
 * Everything else computes Z in fp32 into the workspace (M*N*4 bytes, plus the split operands for large fp32
 * problems) and normalises with a second kernel. */
kf_status kf_gemm_groupnorm(int64_t M, int64_t N, int64_t K, kf_dtype io_dtype,
                            const void* X, int64_t ldx, const void* W, int64_t ldw,
                            const void* bias, int groups, float eps, const void* gamma,
                            const void* beta, kf_act post_act, void* Y, int64_t ldy,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);
size_t kf_gemm_groupnorm_workspace_bytes(int64_t M, int64_t N, int64_t K, kf_dtype io_dtype,
                                         int groups);

/* GEMM + row reduction over N (Appendix A, "Algorithmic Optimization": online softmax;
 * Appendix C.1 prints the three-pass softmax definition; Table 2 "Mixed reduction" and
 * "Reduction-dominated").  With A[m,n] = pre_act( sum_k X[m,k]*W[n,k] + bias[n] ):
 *   KF_RED_SOFTMAX: out[m,n] = exp(A[m,n]-max_n A[m,:]) / sum_n exp(A[m,n]-max_n A[m,:]),
 *                   out is [M,N] with leading dimension ldo, dtype out_dtype.
 *   KF_RED_SUM:     out[m] = sum_n A[m,n], out is [M] fp32 (out_dtype must be KF_F32, ldo
 *                   ignored).
 *   KF_RED_MAX, KF_RED_MEAN, KF_RED_LOGSUMEXP: out[m] = max_n A[m,n], (sum_n A[m,n]) / N,
 *                   log sum_n exp A[m,n] (computed as max + log sum exp(A - max)); out as for
 *                   KF_RED_SUM.  Further reductions of chains like the paper's (Table 2,
 *                   "Mixed reduction" / "Reduction-dominated"); PyTorch's definitions.
 * The reduction is deterministic (no floating-point atomics): repeated calls give identical
 * bits.  The workspace holds per-tile partial statistics.  bf16 softmax: a GEMM kernel that
 * leaves numerators and per-tile (max, sum), then a rescaling kernel; rows that lie in one tile,
 * or in up to 16 tiles of 64 columns or up to 8 tiles of 128 columns (small problems; their CTAs
 * form a cluster and exchange the pairs through distributed shared memory), are finished by the
 * GEMM kernel alone.  So are rows of 2..64 whole 256-column tiles on problems of at least two waves
 * with K >= 2048 (bf16 out, TMA-storable out): the tiles of a row block sit on neighbouring CTAs of
 * one cooperative launch, which exchange the per-row (max, sum) pairs through the workspace and
 * write final probabilities; no numerators reach memory.  A device that cannot hold that grid at
 * once takes the two-kernel route. */
kf_status kf_gemm_rowreduce(int64_t M, int64_t N, int64_t K, kf_dtype in_dtype,
                            const void* X, int64_t ldx, const void* W, int64_t ldw,
                            const void* bias, kf_act pre_act, kf_rowred red,
                            void* out, int64_t ldo, kf_dtype out_dtype,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Row reduction for callers that cannot allocate device memory (no counterpart in the paper:
 * this is a packaging variant of kf_gemm_rowreduce, not another chain).
 *
 * Who needs it: anything that calls from a place where cudaMalloc is forbidden or bound to
 * fail -- inside an inference runtime's enqueue hook, in a process whose own allocator
 * already owns all device memory, or in a serving loop that must not allocate after
 * start-up -- and that therefore has no workspace to pass.
 *
 * Same arguments, results and error codes as kf_gemm_rowreduce, minus the workspace: the
 * per-tile partial statistics go to a fixed KF_STATIC_SCRATCH_BYTES array that is part of the
 * library image (each GPU that loads the library holds those bytes until the process exits).
 * The call allocates nothing: no cudaMalloc/cudaFree, no allocating library routine.
 *   - Limit: a problem whose kf_gemm_rowreduce_workspace_bytes() exceeds
 *     KF_STATIC_SCRATCH_BYTES is refused with KF_ERR_WORKSPACE and nothing is launched
 *     (bf16, K % 8 == 0: M * ceil(N/256) * 16 bytes for softmax, * 4 for sum; otherwise M*N*4).
 *   - The first call on each device looks up the array's device address (a one-time host-side
 *     query, made with that device current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the last call wrote.
 *     No entry has to start at zero (every entry read was written earlier in the same call),
 *     but two calls that may overlap on the GPU -- different streams without an ordering
 *     between them -- race on it.  Keep calls to this function ordered on one stream. */
#define KF_STATIC_SCRATCH_BYTES (2u << 20)
kf_status kf_gemm_rowreduce_static(int64_t M, int64_t N, int64_t K, kf_dtype in_dtype,
                                   const void* X, int64_t ldx, const void* W, int64_t ldw,
                                   const void* bias, kf_act pre_act, kf_rowred red,
                                   void* out, int64_t ldo, kf_dtype out_dtype,
                                   void* cuda_stream);

/* 3x3 convolution (pad 1, stride 1, cross-correlation as in torch.nn.Conv2d) + activation +
 * optional GroupNorm (Table 2 "Conv-centered" chains).
 *   c[n,o,h,w] = bias[o] + sum_{c,r,s} x[n,c,h+r-1,w+s-1] * w[o,c,r,s]      (zero padding)
 *   a = act(c)
 *   groups > 0: per image n and group g (channels [g*Cout/groups,(g+1)*Cout/groups)):
 *       mu = mean(a), var = mean((a-mu)^2) (biased), y = (a-mu)/sqrt(var+eps)*gamma[o]+beta[o]
 *   groups == 0: y = a.
 * x is NCHW [Nb,Cin,H,Wd], w is OIHW [Cout,Cin,3,3], y is NCHW [Nb,Cout,H,Wd], all dense, of
 * io_dtype.  bias, gamma, beta may be NULL (0, 1, 0).  y must not alias x.
 * bf16 problems take the implicit-GEMM tensor-core kernel whenever some number of image rows
 * r makes r*Wd a multiple of 32 that is at most 256 (every Wd <= 256 that is a multiple of 8,
 * also Wd = 7, 14, 28, 56; Wd = 30 is not); Cin is padded to a multiple of 64 in the
 * workspace copy, H may leave a partial last tile, and rows wider than 256 pixels are cut into
 * equal segments that are multiples of 32 (Wd = 320, 384, 512, ...).  fp32 problems with the
 * same tiling and Nb*H*Wd*Cout*Cin >= 2^24 take the tensor cores as well (operands split into
 * two TF32 numbers each, as in kf_gemm_epilogue; GroupNorm by a two-pass kernel afterwards).
 * Everything else takes a scalar kernel.
 * GroupNorm: the tensor-core convolution leaves per-tile channel statistics and a second kernel
 * normalises in place; with 1..8 or 16 tiles per image and 4, 8, 16 or 32 channels per group
 * (bf16, 16-byte aligned y, H*Wd % 8 == 0) the CTAs of an image (and channel tile) form a
 * cluster, exchange the statistics through distributed shared memory and normalise inside the
 * convolution kernel: one kernel after the NHWC copy, the activations are written once.
 * Images of 9..64 whole tiles on problems of at least two waves (same conditions otherwise) run
 * the same chain on every SM: one cooperative launch whose neighbouring CTAs hold an image's
 * tiles and exchange the group statistics through the workspace.
 * groups must divide Cout. */
kf_status kf_conv3x3_epilogue(int64_t Nb, int64_t Cin, int64_t H, int64_t Wd, int64_t Cout,
                              kf_dtype io_dtype, const void* x, const void* w, const void* bias,
                              kf_act act, int groups, float eps, const void* gamma,
                              const void* beta, void* y,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);

/* 3x3 convolution -> softmax over the channel dimension -> max-pool: the 2-D form of the chain in
 * the paper's Appendix C.1 case study (3-D there: conv, softmax, max-pool, max-pool; two pools of size k in a row equal
 * one of size k*k), with the softmax as printed there (per position: max over channels, sum of
 * exp, quotient).
 *   c[n,o,h,w] = bias[o] + sum_{c,r,s} x[n,c,h+r-1,w+s-1] * w[o,c,r,s]
 *   s[n,o,h,w] = exp(c[n,o,h,w] - max_o c[n,:,h,w]) / sum_o exp(c[n,o,h,w] - max_o c[n,:,h,w])
 *   y[n,o,i,j] = max of s over the pool x pool window at (i*pool, j*pool)
 * x NCHW [Nb,Cin,H,Wd], w OIHW, y NCHW [Nb,Cout,H/pool,Wd/pool] (floor; a ragged rim is dropped),
 * all dense, of io_dtype; bias may be NULL.  1 <= pool <= 4 (larger: KF_ERR_UNSUPPORTED); pool
 * above H or Wd gives an empty y and the call returns KF_OK without work.  The
 * convolution takes the same kernels as kf_conv3x3_epilogue; its output is staged in the
 * workspace (io_dtype), whose size kf_conv3x3_softmax_pool_workspace_bytes() returns. */
kf_status kf_conv3x3_softmax_pool(int64_t Nb, int64_t Cin, int64_t H, int64_t Wd, int64_t Cout,
                                  kf_dtype io_dtype, const void* x, const void* w, const void* bias,
                                  int pool, void* y,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream);
size_t kf_conv3x3_softmax_pool_workspace_bytes(int64_t Nb, int64_t Cin, int64_t H, int64_t Wd,
                                               int64_t Cout, kf_dtype io_dtype);

/* 3x3 convolution (pad 1) + bias + activation + global average pooling: one number per image and
 * output channel.  A reduction-dominated conv chain in the sense of the paper's Table 2; the
 * pooling is PyTorch's AdaptiveAvgPool2d(1).
 *   out[n,o] = (1 / (H*Wd)) * sum_{h,w} act( bias[o] + sum_{c,r,s} x[n,c,h+r-1,w+s-1]*w[o,c,r,s] )
 * x NCHW, w OIHW of io_dtype; out is [Nb,Cout] fp32, dense.  On the bf16 tensor-core path (same
 * shapes as kf_conv3x3_epilogue) the per-channel sums are taken in the convolution's epilogue
 * from the fp32 values and the activation tensor is never written; on the other paths it is
 * written to the workspace in io_dtype and averaged by a second kernel. */
kf_status kf_conv3x3_act_gap(int64_t Nb, int64_t Cin, int64_t H, int64_t Wd, int64_t Cout,
                             kf_dtype io_dtype, const void* x, const void* w, const void* bias,
                             kf_act act, float* out,
                             void* workspace, size_t workspace_bytes, void* cuda_stream);
size_t kf_conv3x3_act_gap_workspace_bytes(int64_t Nb, int64_t Cin, int64_t H, int64_t Wd, int64_t Cout,
                                          kf_dtype io_dtype);

/* 3x3 convolution (pad 1) + bias + activation + max or average pooling (kernel = stride = pool,
 * no padding; PyTorch's MaxPool2d(pool) / AvgPool2d(pool)): the conv + activation + pooling
 * chains among the reduction-dominated operator sequences of the paper's Table 2.
 *   a[n,o,h,w] = act( bias[o] + sum_{c,r,s} x[n,c,h+r-1,w+s-1] * w[o,c,r,s] )
 *   y[n,o,i,j] = max (pool_kind 0) or mean (pool_kind 1) of a over the pool x pool window at
 *                (i*pool, j*pool)
 * x NCHW [Nb,Cin,H,Wd], w OIHW, y NCHW [Nb,Cout,H/pool,Wd/pool] (floor; a ragged rim is dropped),
 * all dense, of io_dtype; bias may be NULL; pool >= 1.  pool above H or Wd gives an empty y and
 * the call returns KF_OK without work.  bf16 with pool 2, Wd a multiple of 32 (at most 128) and
 * even H pools inside the tensor-core convolution's epilogue from the fp32 activations, which are
 * then never written; every other case writes a (io_dtype) to the workspace with the kernels of
 * kf_conv3x3_epilogue and pools it with a second kernel.  Other pool_kind: KF_ERR_INVALID_ARG. */
kf_status kf_conv3x3_act_pool(int64_t Nb, int64_t Cin, int64_t H, int64_t Wd, int64_t Cout,
                              kf_dtype io_dtype, const void* x, const void* w, const void* bias,
                              kf_act act, int pool_kind, int pool, void* y,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);
size_t kf_conv3x3_act_pool_workspace_bytes(int64_t Nb, int64_t Cin, int64_t H, int64_t Wd, int64_t Cout,
                                           kf_dtype io_dtype, int pool);

/* Workspace sizes in bytes for the calls above with the same arguments (0 = none needed).
 * Pure host arithmetic; no CUDA call is made.  The short forms assume operands the TMA engine can
 * load as they are: 16-byte aligned bases and, for bf16, leading dimensions that are multiples
 * of 8 elements (for kf_gemm_groupnorm also a 16-byte aligned Y with ldy % 8 == 0).  For any
 * other operands ask the *_for forms, which take the pointers and leading dimensions of the call
 * and return what the route the call will take for them needs (repacked copies of X and W, or the
 * scalar kernels' M*N floats). */
size_t kf_gemm_epilogue_workspace_bytes(int64_t M, int64_t N, int64_t K, kf_dtype io_dtype);
size_t kf_gemm_epilogue_workspace_bytes_for(int64_t M, int64_t N, int64_t K, kf_dtype io_dtype,
                                            const void* X, int64_t ldx, const void* W, int64_t ldw);
size_t kf_gemm_rowreduce_workspace_bytes_for(int64_t M, int64_t N, int64_t K, kf_dtype in_dtype,
                                             kf_rowred red, const void* X, int64_t ldx,
                                             const void* W, int64_t ldw);
size_t kf_gemm_groupnorm_workspace_bytes_for(int64_t M, int64_t N, int64_t K, kf_dtype io_dtype,
                                             int groups, const void* X, int64_t ldx, const void* W,
                                             int64_t ldw, const void* Y, int64_t ldy);
size_t kf_gemm_rowreduce_workspace_bytes(int64_t M, int64_t N, int64_t K, kf_dtype in_dtype,
                                         kf_rowred red);
size_t kf_conv3x3_workspace_bytes(int64_t Nb, int64_t Cin, int64_t H, int64_t Wd, int64_t Cout,
                                  kf_dtype io_dtype, int groups);

/* Every wait inside the kernels (on an mbarrier) is bounded; a wait that runs out sets a
 * device-side status word and the kernel drains and returns.  This call synchronises the
 * current device, reads that word, clears it, and returns KF_OK, KF_ERR_TIMEOUT or
 * KF_ERR_CUDA.  It is not needed for correct runs; tests call it after each launch. */
kf_status kf_device_status(void);

/* Self-test of that mechanism (no counterpart in the paper): launches one warp that waits, with
 * the same bounded wait the kernels use, on an mbarrier nothing will ever complete, with a limit
 * of limit_ns (1e3 .. 1e9) instead of the kernels' 4 s.  Synchronises the stream.  Returns KF_OK
 * when the wait gave up after at least limit_ns (*waited_ns, a host pointer or NULL, receives
 * the time it waited), KF_ERR_UNSUPPORTED when it did not behave so.  As after a real timeout,
 * the device status word is left set: the next kf_device_status() returns KF_ERR_TIMEOUT and
 * clears it.  Nothing traps, faults or loops without bound. */
kf_status kf_selftest_bounded_wait(uint64_t limit_ns, uint64_t* waited_ns, void* cuda_stream);

/* kf_gemm_epilogue for HOST buffers (the chain of kf_gemm_epilogue, same formula; the paper has
 * no counterpart: this is the end-to-end form of the call for a caller whose tensors live in host
 * memory).  X, W, bias, residual and Y are HOST pointers -- page-locked memory if the copies are
 * to run asynchronously -- with leading dimensions in elements; `staging` is a DEVICE buffer, 256-
 * byte aligned, of at least kf_gemm_epilogue_host_staging_bytes() bytes (dense copies of X, W, Y,
 * bias, residual, then the chain's own workspace), owned by the caller.  The batch is cut into
 * `row_blocks` blocks of rows (1..32; rows are independent): block i is computed on `cuda_stream`
 * while block i+1 is still arriving and block i-1 is already leaving, on two copy streams the
 * library creates once per device (host objects; no device memory).  Everything is enqueued when
 * the call returns; the downloads are joined into `cuda_stream`, so synchronising that stream
 * makes Y readable.  A later call's uploads start as soon as this call's kernels are done.
 * Calls are serialised per process.  Errors as for kf_gemm_epilogue; KF_ERR_WORKSPACE when the
 * staging buffer is null, misaligned or too small. */
size_t kf_gemm_epilogue_host_staging_bytes(int64_t M, int64_t N, int64_t K, kf_dtype io_dtype,
                                           int has_bias, int has_residual);
kf_status kf_gemm_epilogue_host(int64_t M, int64_t N, int64_t K, kf_dtype io_dtype, const void* X,
                                int64_t ldx, const void* W, int64_t ldw, const void* bias, kf_act act,
                                float scale, const void* residual, int64_t ldr, void* Y, int64_t ldy,
                                void* staging, size_t staging_bytes, int row_blocks, void* cuda_stream);

/* Launches an empty kernel (one warp that does nothing) on the stream: the launch-latency
 * reference the benchmark prints beside the smallest chain (no counterpart in the paper). */
kf_status kf_launch_noop(void* cuda_stream);

/* Number of kernels the library has launched from this process since load (all streams). */
int64_t kf_launch_count(void);

/* Host-side state of the call path (no counterpart in the paper: library plumbing).
 * The dispatch switches (KF_NO_PAIR, KF_NO_SPLITK, KF_NO_FUSED_GN, KF_NO_FUSED_SOFTMAX,
 * KF_NO_CLUSTER_SOFTMAX, KF_NO_FUSED_POOL, KF_NO_TF32X3, KF_NO_CONV_SLAB, KF_NO_GNX, KF_NO_SOFTMAX_GX,
 * KF_NO_WIDE_STORE) and thresholds
 * (KF_PAIR_MIN_K, KF_PAIR_MIN_KB_PER_CTA, KF_SPLITK_MIN_KB, KF_SPLITK_TWO_PER_SM, KF_CL128_MAX_CTAS,
 * KF_GNX_MIN_TILES, KF_GNX_MIN_TPI, KF_GNX_MAX_TPI, KF_SOFTMAX_GX_MIN_TILES) are read
 * from the environment once, at the first call; kf_reload_tuning() reads them again (tests
 * and A/B measurements that force a route).  Encoded TMA tensor maps are cached by (base
 * pointer, extents, pitches, box, swizzle); kf_tensor_map_cache_stats reports how many
 * lookups hit and how many had to ask the driver (either pointer may be NULL). */
void kf_reload_tuning(void);
void kf_tensor_map_cache_stats(int64_t* hits, int64_t* misses);

const char* kf_status_string(kf_status s);
int kf_version(void);

#ifdef __cplusplus
}
#endif
#endif /* KF_H_ */
