/* fp4root.h -- C ABI of the NVFP4 Root Newton-Schulz library for B200 (sm_100a).
 *
 * One hot path of the paper "Full-Stack FP4": the NVFP4 Root step (Section 3.4),
 * i.e. outlier clip, Frobenius normalisation and k Newton-Schulz iterations whose
 * three matrix products per iteration run on NVFP4 operands (Section 2, "NVFP4
 * format": E2M1 values, one E4M3 scale per 16 contiguous elements of the
 * contraction axis, one FP32 scale per tensor) with FP32 accumulation.
 *
 * General rules
 *   - Every pointer named "device" is a CUDA device pointer on the current device;
 *     every other pointer is host memory that is read before the call returns.
 *   - The caller owns all buffers.  The library allocates no device memory.  Between calls it
 *     keeps, on the host, the driver entry point it resolves on first use and a bounded cache of
 *     the TMA descriptors and workspace plans of recent (buffers, shape, parameters)
 *     combinations, so that a call with the same buffers as an earlier one skips their set-up.
 *   - All work is enqueued on `stream`; no call synchronises the host except
 *     fp4_last_device_status.
 *   - Shapes: for fp4_root_ns, fp4_root_ns_batched and fp4_root_ns_static every matrix
 *     dimension must be a positive multiple of 16 (the block length; the work matrices
 *     are zero-padded to multiples of 128 inside the workspace, which changes no result);
 *     for fp4_quantize and fp4_gemm_nt a positive multiple of 128.  Else FP4_ERR_SHAPE.
 *     Device pointers must be 16-byte aligned (the workspace 256), else FP4_ERR_ALIGNMENT.
 *   - Errors are return codes.  A kernel that gives up on a bounded wait records
 *     FP4_ERR_DEVICE_TIMEOUT in the workspace header and ends normally; it never
 *     traps.  Read it with fp4_last_device_status.
 *   - Non-finite inputs give unspecified values but no fault (conversions saturate).
 *   - There is no CPU fallback: on a device that is not compute capability 10.x
 *     every compute entry point returns FP4_ERR_ARCH.
 */
#ifndef FP4ROOT_H_
#define FP4ROOT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* cudaStream_t;

typedef enum {
  FP4_OK = 0,
  FP4_ERR_INVALID_ARG = 1,
  FP4_ERR_SHAPE = 2,
  FP4_ERR_ALIGNMENT = 3,
  FP4_ERR_WORKSPACE = 4,
  FP4_ERR_ARCH = 5,
  FP4_ERR_CUDA = 6,
  FP4_ERR_DEVICE_TIMEOUT = 7,
  FP4_ERR_UNIMPLEMENTED = 8,
  FP4_ERR_STATIC_LIMIT = 9
} fp4_status;

/* flags of fp4_ns_params */
#define FP4_FLAG_KEEP_OPERANDS 1u /* the last iteration also writes the NVFP4 copies of
                                     its result (otherwise skipped as dead work); for
                                     inspection through fp4_root_ns_workspace_layout */
/* Paper-faithful quantiser options (Section 3.4: operands are rotated by a random Hadamard
 * transform along the contraction axis, and every quantisation uses adaptive 4/6 scaling).
 * Off by default; each costs epilogue arithmetic.
 *   FP4_FLAG_RHT: every 16-block b along the contraction axis becomes b diag(r) H_16 / 4
 *     before it is quantised, r = 16 random signs and H_16 the Sylvester Hadamard matrix.
 *     Both operands of a product share r, so the transform cancels in exact arithmetic.
 *     Tensor scales are derived from 4 amax (|b H| <= 4 amax(b)).
 *   FP4_FLAG_FOUR_SIX: a block is encoded twice, with its maximum mapped to 6 (block scale
 *     E4M3(amax/(6 s_g))) and to 4 (E4M3(amax/(4 s_g))); the encoding with the smaller sum
 *     of squared errors (FP32, summed in element order) is kept, a tie keeps 6.
 * fp4_root_ns draws the signs of product j of a call (j = 2k: X_k, B_k; j = 2k+1: A_k) from
 * splitmix64: z = seed + 0x9E3779B97F4A7C15 (j+1), the generator's output mix of z, low 16
 * bits; bit i set means element i is negated.  fp4_quantize takes the 16 sign bits in the
 * upper half of its flags word: FP4_FLAG_RHT | FP4_QUANT_SIGNS(mask). */
#define FP4_FLAG_RHT 2u
#define FP4_FLAG_FOUR_SIX 4u
/* BF16 storage of the high-precision copies between the stages (the paper does not state their
 * precision; FP32 is the default): A_k and X_k (k >= 1) are kept in BF16, round to nearest
 * even, which halves the FP32 traffic of the fused epilogues.  The NVFP4 operand copies and the
 * running maxima are still derived from the FP32 values in the epilogue, X_0 stays FP32 and
 * the result is FP32.  When every dimension of the work shape is a multiple of 256 the copies
 * really are 2-byte tensors; otherwise they stay FP32 tensors that hold BF16-rounded values
 * (same results, no traffic saved). */
#define FP4_FLAG_STORE_BF16 8u
/* With fp4_ns_params.weights: the FP32 result is not written (the parameter update is all the caller
 * wants).  `out` is still required - it is the working copy of X during the iterations of a wide matrix -
 * and its contents are unspecified afterwards. */
#define FP4_FLAG_NO_OUT 16u
/* fp4_root_ns_batched only: groups of equal shapes, which do not depend on one another, alternate between
 * the caller's stream and a second stream of the library's own (one per host thread and device, created on
 * first use).  The second stream waits for everything enqueued on the caller's stream before the call, and
 * the caller's stream waits for it before the call returns, so callers see ordinary stream order and the
 * call can still be captured in a CUDA graph.  Off by default: with two large groups (the decoder-stack
 * benchmark) the gain or loss of about 1.5 % depends on the order in which the two groups' launches meet
 * on the device; the option is for batches of many small groups. */
#define FP4_FLAG_OVERLAP_GROUPS 32u
#define FP4_QUANT_SIGNS(mask) ((uint32_t)(mask) << 16)

/* Parameters of the step.  Pass NULL for the defaults noted on each field. */
typedef struct {
  float a, b, c;       /* quintic coefficients of X+ = aX + (bA + cA^2)X (Section 2, "Root
                          optimizer").  a = NaN (default): fp4_root_coeffs(m, n, steps).   */
  float clip_quantile; /* outlier clip (Section 3.4, "p99 outlier clipping"): entries are
                          clamped to the nearest-rank quantile of |G|, resolved to parts
                          per million.  Default 0.99; <= 0 or >= 1 disables the clip.      */
  float eps;           /* X0 = G_c / (||G_c||_F + eps).  Default 1e-7.                     */
  uint32_t flags;      /* FP4_FLAG_*; default 0; unknown bits: FP4_ERR_INVALID_ARG             */
  uint32_t max_group;  /* fp4_root_ns_batched: at most this many equal-shape matrices run their
                          stages in lockstep as single launches; 0 or more than 16 = 16        */
  uint64_t seed;       /* FP4_FLAG_RHT: seed of the sign draws; default 0                    */
  uint32_t* const* top_hist; /* NULL (default), or a host array with one entry per matrix of the call
                          (one entry for fp4_root_ns and fp4_root_ns_static): NULL, or a device
                          array of 8192 counters that already holds, for that matrix, the number
                          of elements whose |g| has each value of its top 13 magnitude bits
                          (bits >> 18), as fp4_momentum_update writes for its M_t.  The clip then
                          skips its first pass over the matrix.  The counters must describe
                          exactly the matrix passed as G; they are consumed: zero when the step
                          has run.  Ignored when the clip is disabled.                        */
  uint16_t* const* weights;  /* NULL (default), or a host array with one entry per matrix of the call:
                          NULL, or the device address of that matrix's parameter, m x n BF16
                          row-major (16-byte aligned), which receives Root's update in the same
                          call (Section 3.4: the orthogonalised matrix is applied to the
                          projection; Section 3.3: BF16 weights, no FP32 master copy):
                            W <- BF16( fl(W * fl(1 - fl(lr * weight_decay)))
                                       - fl(fl(lr * update_scale) * X_steps) ),  nearest even,
                          fused into the epilogue of the last product (into the final transpose for
                          a tall matrix), so X_steps is not read back from memory.             */
  float lr;            /* with weights: learning rate                                        */
  float weight_decay;  /* with weights: decoupled decay                                      */
  float update_scale;  /* with weights: the shape factor Root-style optimisers put on the
                          orthogonalised step (e.g. sqrt(max(1, m/n))); the caller's choice     */
} fp4_ns_params;

const char* fp4_status_string(fp4_status s);

/* ---- NVFP4 block quantiser (Section 2, "NVFP4 format"; Q_1x16 of Section 3.4) ----------
 *
 * x: device, row-major rows x cols FP32 (leading dimension = cols).
 * codes: device, out, rows x cols/2 bytes row-major; byte j of a row holds element 2j in
 *   bits 3:0 and element 2j+1 in bits 7:4; a nibble is sign<<3 | index into
 *   {0, 0.5, 1, 1.5, 2, 3, 4, 6}.
 * scales: device, out, fp4_scale_bytes(rows, cols) bytes of unsigned E4M3 block scales in
 *   the layout the tcgen05 block-scaled MMA reads: 512-byte atoms that hold 128 rows x 4
 *   consecutive blocks; the scale of (row r, block kb) is at
 *     ((r/128) * (cols/64) + kb/4) * 512 + (r%32)*16 + ((r%128)/32)*4 + kb%4.
 * tensor_scale: device, out, one FP32: s_g = amax(x)/2688 (1 if x is all zero).  It is
 *   also used as scratch while the call runs.
 * Decoded value of an element = E2M1 value * E4M3 scale * s_g.  Rounding is to nearest,
 * ties to even, saturating.  Block scale = E4M3(amax_block / (6 s_g)); elements are
 * multiplied by the FP32 reciprocal of (scale * s_g) before conversion.
 * flags: 0, or FP4_FLAG_RHT | FP4_QUANT_SIGNS(mask) and / or FP4_FLAG_FOUR_SIX (see above);
 *   with FP4_FLAG_RHT, s_g = 4 amax(x)/2688.
 */
size_t fp4_scale_bytes(int64_t rows, int64_t cols);
fp4_status fp4_quantize(const float* x, int64_t rows, int64_t cols, uint8_t* codes,
                        uint8_t* scales, float* tensor_scale, uint32_t flags,
                        cudaStream_t stream);

/* ---- shape-dependent coefficients (Section 3.4: "Root's shape-dependent coefficients") --
 * Host function, pure.  The paper does not print the values; this provider returns a
 * quintic with p(1) = 1, p'(1) = 0 whose slope at zero grows with max(m,n)/min(m,n)
 * (15/8, -10/8, 3/8 for square matrices).  abc: host, out, 3 floats.
 */
fp4_status fp4_root_coeffs(int64_t m, int64_t n, int steps, float abc[3]);

/* ---- the Root Newton-Schulz step on one matrix (Section 3.4, display equations) --------
 *
 * G: device, m x n FP32 row-major.  out: device, m x n FP32 row-major; may equal G exactly
 *   (no partial overlap).  steps >= 0 iterations (0: clip and normalise only).
 * ws: device workspace of at least fp4_root_ns_workspace_bytes(m, n, steps, flags) bytes,
 *   256-byte aligned; its contents need not be initialised and are overwritten.
 * m, n: positive multiples of 16.
 * Computes, with s = min(m,n), l = max(m,n) and X = G or G^T so that X is s x l:
 *   tau = quantile of |G|, G_c = clamp(G, -tau, tau), X0 = G_c/(||G_c||_F + eps), then
 *   per iteration A = qX qX^T, B = bA + c qA qA^T, X+ = aX + qB qX^{16x1}, every q*
 *   an NVFP4 quantisation with 16-element blocks along the contraction axis; the
 *   result is X_steps (transposed back when m > n).
 * Two calls that share a workspace must not overlap in time.
 * Launches: 6 kernels for clip, normalisation and the first quantisation plus 3 per iteration
 *   (and a transpose pass for a tall matrix on the routes that cannot write the result
 *   transposed from the last product).  Calls on small matrices (up to 8 M elements per group
 *   of equal shapes) chain their kernels with programmatic dependent launch; the environment
 *   variable FP4ROOT_NO_PDL (any value) switches that off.  Kernels launched before or after
 *   the call on the same stream see ordinary stream order either way.
 */
size_t fp4_root_ns_workspace_bytes(int64_t m, int64_t n, int steps, uint32_t flags);
fp4_status fp4_root_ns(const float* G, float* out, int64_t m, int64_t n, int steps,
                       const fp4_ns_params* p, void* ws, size_t ws_bytes, cudaStream_t stream);

/* ---- many matrices of different shapes in one call (the matrices of a layer stack) ------
 * count matrices; G, out, m, n: host arrays of length count (G[i], out[i] device pointers).
 * One parameter block applies to all (coefficients per matrix when p->a is NaN).
 * ws: device, at least fp4_root_ns_batched_workspace_bytes(...) bytes, 256-byte aligned: one
 *   single-matrix workspace per matrix plus the tables of the grouped launches.
 * Matrices of equal shape (after orientation) are grouped: each Newton-Schulz stage of a
 * group is one launch whose tile list spans all its matrices.  Results are bit-identical to
 * calling fp4_root_ns on each matrix.
 * All launches go to `stream` unless FP4_FLAG_OVERLAP_GROUPS is set (see there).
 */
size_t fp4_root_ns_batched_workspace_bytes(int count, const int64_t* m, const int64_t* n,
                                           int steps, uint32_t flags);
fp4_status fp4_root_ns_batched(int count, const float* const* G, float* const* out,
                               const int64_t* m, const int64_t* n, int steps,
                               const fp4_ns_params* p, void* ws, size_t ws_bytes,
                               cudaStream_t stream);

/* ---- the same step for callers that cannot allocate device memory --------------------------
 * (The paper has no counterpart; this is a packaging variant of fp4_root_ns.)
 *
 * Some callers have nowhere to get a workspace from: code that runs inside another
 * framework's callback or a real-time loop where cudaMalloc is forbidden because it may
 * synchronise the device, plug-ins that are handed input and output buffers and nothing
 * else, and programs whose memory pool is already fully committed.  For them this entry
 * point keeps the workspace inside the library: a fixed array of
 * FP4_STATIC_SCRATCH_BYTES (16 MiB) in the device's global memory, part of the loaded
 * module, held by every GPU that uses the library until the process exits.
 *
 * Arguments as for fp4_root_ns, without ws.  Works for every (m, n, steps, flags) with
 * fp4_root_ns_workspace_bytes(m, n, steps, flags) <= FP4_STATIC_SCRATCH_BYTES -- for example
 * 1024 x 1024 and 1024 x 2048; a tall 2048 x 1024 needs more -- and returns
 * FP4_ERR_STATIC_LIMIT for anything larger, before any work is enqueued.
 * device_status: device, optional (may be NULL): one uint32 that receives, in stream order,
 *   the status word of this call (FP4_OK or FP4_ERR_DEVICE_TIMEOUT).
 *
 * It calls no cudaMalloc, cudaFree or other allocating routine (as long as fp4_profile_enable is
 * off: the profiling brackets create events).  The first call on each device loads the module
 * and resolves the array's device address, with that device current; make that first call
 * outside any stream capture.  The address is looked up again on every call (a cheap table read),
 * so a context that was destroyed and rebuilt between calls is handled; kernel attributes set
 * during the library's per-device set-up are not re-applied after a cudaDeviceReset, which the
 * library does not support while it is loaded.  All calls on a device
 * share the one array, which keeps whatever the previous call left in it; the call itself
 * clears the parts that must start from zero.  Two calls whose kernels could overlap on the
 * GPU (different streams without an ordering between them) race on the array: order them.
 * Results are identical to fp4_root_ns on the same input.
 */
#define FP4_STATIC_SCRATCH_BYTES ((size_t)16 << 20)
fp4_status fp4_root_ns_static(const float* G, float* out, int64_t m, int64_t n, int steps,
                              const fp4_ns_params* p, uint32_t* device_status,
                              cudaStream_t stream);

/* Synchronises `stream`, then returns the status word that the kernels of the last call
 * on workspace `ws` left in its header: FP4_OK or FP4_ERR_DEVICE_TIMEOUT. */
fp4_status fp4_last_device_status(const void* ws, cudaStream_t stream);

/* ---- inspection (tests) -----------------------------------------------------------------
 * Byte offsets, inside the workspace of fp4_root_ns(m, n, ...), of the intermediates the
 * last executed iteration leaves behind.  All are in the work orientation (s x l).
 * Operands are NVFP4 tensors: codes as in fp4_quantize, scales in the atom layout, tensor
 * scale in the FP32 array `scalars` at the given index.
 */
typedef struct {
  size_t header;      /* uint32 status word first                                  */
  size_t scalars;     /* float array, see the idx_* fields                          */
  size_t X;           /* FP32 s x l: X (only when m > n; otherwise X lives in out)  */
  size_t A;           /* FP32 s x s: A of the last iteration, upper-triangle tiles  */
  size_t qX_codes, qX_scales;       /* Q_1x16(X): G1 operand, s x l                 */
  size_t qXt_codes[2], qXt_scales[2]; /* Q_1x16(X^T): G3 operand, l x s, ping-pong  */
  size_t qA_codes, qA_scales;       /* s x s                                        */
  size_t qB_codes, qB_scales;       /* s x s                                        */
  int32_t idx_tau, idx_nu, idx_inv; /* scalars[idx]                                 */
  int32_t idx_amax_X0;              /* scalars[idx + k] = amax of X_k               */
  int32_t idx_amax_A0;              /* scalars[idx + k] = amax of A_k               */
  int32_t idx_sg_X0;                /* scalars[idx + k] = tensor scale of qX_k      */
  int32_t idx_sg_A0, idx_sg_B0;     /* likewise for qA_k, qB_k                      */
  size_t total;
  size_t Xh;          /* FP4_FLAG_STORE_BF16 with 2-byte storage: BF16 s x l, X_k (k >= 1); the A
                         region then holds A as BF16 s x s.  0 otherwise.                  */
} fp4_ws_layout;
fp4_status fp4_root_ns_workspace_layout(int64_t m, int64_t n, int steps, uint32_t flags,
                                        fp4_ws_layout* layout);

/* One block-scaled product on the tcgen05 path, for testing the GEMM alone:
 * D = (deq(A) deq(B)^T) as FP32, A: M x K, B: N x K NVFP4 tensors (device; codes, scales in
 * the atom layout, host tensor scales).  D: device, M x N FP32 row-major.  M, N, K
 * multiples of 128. */
fp4_status fp4_gemm_nt(const uint8_t* a_codes, const uint8_t* a_scales, float a_tensor_scale,
                       const uint8_t* b_codes, const uint8_t* b_scales, float b_tensor_scale,
                       int64_t M, int64_t N, int64_t K, float* D,
                       uint32_t* device_status /* device, may be NULL: receives
                       FP4_ERR_DEVICE_TIMEOUT if a bounded wait gives up */,
                       cudaStream_t stream);

/* Measurement helper: the same launch as fp4_gemm_nt (same kernel, tiles, instruction stream and epilogue)
 * in which every pair of SMs fetches only the first operand stages of its first tile and runs all
 * later MMAs on those resident stages.  Times the tensor-core side of the product without any operand
 * traffic: the ceiling the benchmark reports beside the nominal peak.  D receives meaningless values.
 * M, N, K multiples of 256 (else FP4_ERR_SHAPE). */
fp4_status fp4_gemm_nt_resident(const uint8_t* a_codes, const uint8_t* a_scales, float a_tensor_scale,
                                const uint8_t* b_codes, const uint8_t* b_scales, float b_tensor_scale,
                                int64_t M, int64_t N, int64_t K, float* D, uint32_t* device_status,
                                cudaStream_t stream);

/* ---- first-moment momentum in a 5-bit NVFP4 state ---------------------------------------------
 * Section 3.3 (first-moment recipe: Hadamard mixing, then stochastic rounding and adaptive 4/6
 * quantisation; 5 bits per element in the appendix's memory accounting) and Section 3.4 (Root's
 * momentum is stored with that recipe).  The step that precedes fp4_root_ns in the optimiser:
 *     M_t = mu * M_{t-1} + g_scale * G_t,
 * with M_{t-1} read from the state, M_t written in FP32 (the Newton-Schulz input) and the state
 * replaced by the encoding of M_t, all in one pass over the matrix.
 *
 * State of a rows x cols matrix (row-major; rows > 0, cols a positive multiple of 16, else
 * FP4_ERR_SHAPE), blocks of 1x16 along the rows:
 *   codes   device, rows*cols/2 bytes: E2M1 codes of each block multiplied by H_16 / 4 (the
 *           Sylvester Hadamard matrix, no signs; its own inverse), element 2j of the transformed
 *           block in the low nibble of byte j
 *   scales  device, rows*cols/16 uint16: the block scales as BF16 bit patterns; no tensor scale
 * An all-zero state is zero momentum.  Encoding a block h: the two candidate scales are
 * BF16(amax/6) and BF16(amax/4); each is tried with round-to-nearest-even codes of h/scale, the
 * one with the smaller sum of squared FP32 errors (element order) is kept, a tie keeps 6.
 * FP4_MOM_FLAG_SR then encodes the block again with the chosen scale by stochastic rounding:
 * with lo <= |y| < hi the neighbouring grid values and f = floor(65536 (|y| - lo) / (hi - lo)),
 * y becomes hi when f + r >= 65536 (probability f / 65536).  The 16 random bits r: elements
 * 8q .. 8q+7 of the matrix (row-major index) share output q of splitmix64 (z = seed +
 * 0x9E3779B97F4A7C15 (q+1), then the generator's output mix), its low 32 bits for the first
 * four; of a 32-bit word, the low half is r of element 0, the same 16 bits in reverse order
 * r of element 1, the high half r of element 2, reversed r of element 3.
 * Arithmetic: m_prev = (code * scale) H_16 / 4 (natural-order butterfly, FP32), then
 * M = fl(fl(mu m_prev) + fl(g_scale G)).
 *
 * G       device, in : rows x cols FP32, 32-byte aligned (the kernel moves 256 bits per access)
 * codes, scales  device, in/out: the state, updated in place; 16-byte aligned
 * M_out   device, out: rows x cols FP32 or NULL, 32-byte aligned; must not overlap G
 * hist    device, in/out or NULL: 8192 uint32 counters; counter ((bits of |M|) >> 18) is
 *         incremented for every element of M_t (the top 13 magnitude bits: the first pass of the
 *         outlier clip's quantile selection); the caller zeroes it
 * Errors: FP4_ERR_INVALID_ARG (null pointer, unknown flag), FP4_ERR_SHAPE, FP4_ERR_ALIGNMENT,
 * FP4_ERR_ARCH, FP4_ERR_CUDA.
 */
#define FP4_MOM_FLAG_SR 1u
typedef struct fp4_momentum_params {
  float mu;        /* momentum coefficient                                   */
  float g_scale;   /* factor on the gradient: 1 (heavy ball) or 1 - mu (EMA) */
  uint32_t flags;  /* FP4_MOM_FLAG_*                                         */
  uint32_t reserved;
  uint64_t seed;   /* FP4_MOM_FLAG_SR: a different seed every step           */
} fp4_momentum_params;
fp4_status fp4_momentum_update(const float* G, int64_t rows, int64_t cols, uint8_t* codes, uint16_t* scales,
                               float* M_out, uint32_t* hist, const fp4_momentum_params* params,
                               cudaStream_t stream);
/* M_out = the decoded state (device, rows x cols FP32, 32-byte aligned); the state is not changed. */
fp4_status fp4_momentum_decode(const uint8_t* codes, const uint16_t* scales, int64_t rows, int64_t cols,
                               float* M_out, cudaStream_t stream);

/* ---- packed AdamW step on NVFP4 moment states --------------------------------------------------
 * Section 3.3 ("Quantized-State AdamW") and the appendix's accounting: BF16 weight and gradient,
 * a 5-bit first moment and a 5.0625-bit second moment, 42.0625 bits per parameter, no FP32
 * master weight; decay and parameter update fused into the pass that reconstructs and re-packs
 * the states.  Section 2 gives the moment recursions.
 *
 * A tensor is a flat array of n elements, n a positive multiple of 256 (else FP4_ERR_SHAPE).
 *   W         device, in/out: n BF16 weights, 32-byte aligned
 *   G         device, in    : n BF16 gradients, 32-byte aligned; must not overlap W
 *   m_codes, m_scales       : the first moment in the state format of fp4_momentum_update
 *                             (n/2 bytes, n/16 uint16), in/out
 *   v_codes, v_scales, v_means: the second moment, in/out: with s = sqrt(v) and a tile = 256
 *       consecutive elements, v_means (n/256 uint16) holds BF16(sum(s) / 256) per tile (FP32 sums:
 *       each block of 16 in element order, then a pairwise tree over the 16 block sums);
 *       v_codes / v_scales hold the blocks of s - mean times H_16 / 4, encoded like the first
 *       moment with round to nearest (two candidate BF16 scales amax/6, amax/4).  Decoding:
 *       ((code * scale) H_16 / 4 + mean)^2.  All-zero states are zero moments.
 *   All state arrays 16-byte aligned.
 * Arithmetic, FP32, one rounded operation per step, t = params->step >= 1:
 *   m = b1 m' + (1-b1) g,  v = b2 v' + (1-b2) (g g),  s = sqrt(v),  den = s * rsb2 + eps,
 *   w2 = w (1 - lr wd) - (lr / bc1) (m / den),  W = BF16(w2) to nearest even;
 *   bc1 = 1 - b1^t and rsb2 = 1 / sqrt(1 - b2^t) are evaluated in double and rounded to FP32.
 * FP4_MOM_FLAG_SR: stochastic rounding of the first moment as in fp4_momentum_update, the
 * random stream numbered by element index and seeded by params->seed.
 * Errors: FP4_ERR_INVALID_ARG (null pointer, unknown flag, step < 1), FP4_ERR_SHAPE,
 * FP4_ERR_ALIGNMENT, FP4_ERR_ARCH, FP4_ERR_CUDA.
 */
typedef struct fp4_adamw_params {
  float lr, beta1, beta2, eps, weight_decay;
  int32_t step;    /* t, from 1 */
  uint32_t flags;  /* FP4_MOM_FLAG_SR */
  uint32_t reserved;
  uint64_t seed;
} fp4_adamw_params;
fp4_status fp4_adamw_update(uint16_t* W, const uint16_t* G, int64_t n, uint8_t* m_codes, uint16_t* m_scales,
                            uint8_t* v_codes, uint16_t* v_scales, uint16_t* v_means,
                            const fp4_adamw_params* params, cudaStream_t stream);

/* ---- measurement support (the paper has no counterpart) -----------------------------------
 * While profiling is enabled, every group of launches of the step is bracketed by a pair of
 * CUDA events on the caller's stream; fp4_profile_collect waits for them, adds the elapsed
 * times per class into ms[class] and the number of bracketed groups into groups[class]
 * (both host arrays of FP4_PROF_CLASSES entries), then forgets them.  Off by default; the
 * events add stream operations, so time whole calls with profiling off.
 * fp4_kernel_launches returns how many kernels this library has launched in this process.
 */
enum { FP4_PROF_CLIP = 0, FP4_PROF_STATS = 1, FP4_PROF_PREP = 2, FP4_PROF_G1 = 3, FP4_PROF_G2 = 4,
       FP4_PROF_G3 = 5, FP4_PROF_TRANSPOSE = 6, FP4_PROF_QUANTIZE = 7, FP4_PROF_MOMENTUM = 8,
       FP4_PROF_ADAMW = 9, FP4_PROF_CLASSES = 10 };
void fp4_profile_enable(int on);
fp4_status fp4_profile_collect(float* ms, int* groups);
uint64_t fp4_kernel_launches(void);

/* ---- self-test of the bounded device-side waits (the paper has no counterpart) -------------
 * Every wait of the GEMM kernels on a shared-memory barrier gives up after a time limit,
 * raises the CTA's abort flag and ends normally, leaving FP4_ERR_DEVICE_TIMEOUT in the status
 * word.  This entry point runs that same wait routine in a one-warp kernel on a barrier that
 * nothing ever arrives on, with a limit of limit_us microseconds (1 .. 100000), after a
 * second barrier whose arrival it does see.
 * device_status: device, one uint32, out: FP4_ERR_DEVICE_TIMEOUT if the first wait was seen
 *   to succeed and the second to time out (what must happen), FP4_ERR_INVALID_ARG otherwise.
 * The kernel neither traps nor spins past the limit; the context stays usable.
 */
fp4_status fp4_selftest_bounded_wait(uint32_t* device_status, uint32_t limit_us, cudaStream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* FP4ROOT_H_ */
