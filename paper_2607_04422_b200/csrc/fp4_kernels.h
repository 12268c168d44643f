// Internal interfaces between the translation units of the library.
#pragma once

#include <utility>

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "fp4_common.cuh"

namespace fp4 {

constexpr int kMaxSteps = 64;

// First 128 bytes of a workspace.
struct NsHeader {
  uint32_t status;       // fp4_status left by the kernels (0 or FP4_ERR_DEVICE_TIMEOUT)
  uint32_t reserved[3];
  uint32_t sel_prefix;   // radix select: magnitude bits fixed so far
  uint32_t sel_rank;     // radix select: rank still to find inside the prefix
  uint32_t maxabs_bits;  // max |g| below the clip bin (or of everything without a clip), bit pattern
  uint32_t bin_count;    // elements in the bin picked by the first radix pass
  uint32_t count_below;  // elements in the bins below it
  uint32_t cand_count;   // candidates appended by the second pass (may exceed the list's capacity)
  uint32_t overflow;     // 1: the candidate list overflowed, the fallback passes run
  uint32_t pad[21];
};

// Indices into the FP32 `scalars` array of a workspace.
struct NsScalarIdx {
  int tau, nu, inv;
  int amax_X0, amax_A0;        // + k
  int sg_X0, sg_A0, sg_B0;     // + k
};

struct NsPlan {
  fp4_ws_layout lay;
  NsScalarIdx ix;
  int64_t m, n;      // the caller's matrix
  int64_t s0, l0;    // its short and long side
  int64_t s, l;      // work shape: s0, l0 rounded up to multiples of 128 (zero padding)
  int tall;
  int clip;
  int bf16_mode;     // 0: FP32 storage of X_k / A_k; 1: BF16 tensors; 2: FP32 tensors holding BF16-rounded values
  size_t off_Xh;     // bf16_mode 1: BF16 X in the workspace
  int64_t clip_rank;
  float eps;
  int sms;
  int stat_blocks;
  size_t off_hist, off_partial;
  size_t zero_bytes;  // header + scalars + histogram, cleared at the start of a call
};

// Epilogue variants of the GEMM kernel.
enum GemmMode : int {
  kPlain = 0,  // D = acc * sgA*sgB                                  (fp4_gemm_nt)
  kG1 = 1,     // A = qX qX^T; store A, emit qA (both triangles), track amax(A)
  kG2 = 2,     // S = qA qA^T; B = bA + cS; emit qB (both triangles)
  kG3 = 3      // P = qB qXt^T; X+ = aX + P; store X+, emit qX+, qXt+, track amax(X+)
};

// One matrix product of a launch.  A launch runs the same stage for a group of matrices
// of one shape; the problems of a group sit in an array in device memory (or, for a single
// problem, in the kernel's parameter space).
struct alignas(64) GemmProblem {
  CUtensorMap tmA, tmB;      // NVFP4 codes of the row and the column operand
  CUtensorMap tmAux, tmOut;  // FP32 tile combined in the epilogue / FP32 result (box: 16 columns x 128 rows in
                             // the single-CTA kernel, 16 x 32 - one epilogue warp's block - in the CTA-pair kernel)
  CUtensorMap tmSfa, tmSfb;  // scale atoms of the two operands as 2-D maps (CTA-pair kernel)
  CUtensorMap tmH;           // BF16 storage: the 2-byte tensor this stage reads its tile from and / or stores its
                             // result to (A for G1 / G2, X for G3); box 16 columns x 32 rows, no swizzle
  CUtensorMap tmRq, tmCq;    // CTA-pair kernel: byte maps over rq_codes (box 32 bytes x 32 rows: one warp's part of a
                             // tile) and cq_codes (box 64 bytes x 128 rows, 64-byte swizzle: a CTA's 128 rows of
                             // 128 tile columns) for the stores of the quantised outputs
  const uint8_t* sfa;        // scale atoms of the row operand
  const uint8_t* sfb;        // scale atoms of the column operand
  float* scalars;            // workspace scalars of this matrix (device)
  uint8_t* rq_codes; uint8_t* rq_sf;  // quantised output, blocks along the tile's columns
  uint8_t* cq_codes; uint8_t* cq_sf;  // quantised output, blocks along the tile's rows
  float ca, cb, cc;          // coefficients
  float sg_a, sg_b;          // kPlain: tensor scales from the host
  int aux_raw;               // kG3: tmAux maps the raw input G; X0 = clamp(G, tau) * inv is formed on the fly
  int aux_tr;                // kG3, CTA-pair kernel: tmAux maps a matrix stored as the transpose of the tile grid (box = 32 x 16)
  int out_tr;                // kG3, CTA-pair kernel: so does tmOut (the caller's result of a tall input)
  int out_rows, out_cols;    // extent of the matrix behind tmOut (chunks that start outside it are not stored)
  void* out_direct;          // out_h == 2: the FP32 tensor the epilogue warps store the rounded result to
  int64_t out_direct_ld;     //   (row-major, leading dimension in elements)
  uint16_t* W;               // kG3 with launch.update: the BF16 parameter (same shape and orientation as the
  int64_t W_ld;              //   result, row-major, leading dimension in elements) updated with the result; or null
};

// The problems of one launch travel as a kernel parameter (descriptors in parameter space need no
// proxy fence before TMA uses them, and nothing has to be written to device memory first).
constexpr int kPackMax = 16;
struct ProblemPack { GemmProblem p[kPackMax]; };
static_assert(sizeof(ProblemPack) + 256 <= 32764, "kernel parameter space");

// What all problems of a launch share.
struct GemmLaunch {
  int num_problems;
  int K;               // contraction length in elements (multiple of 128)
  int tiles_m, tiles_n;
  int symmetric;       // only tiles with tile_n >= tile_m; mirrored quantised output
  int iter;            // Newton-Schulz iteration index k
  int write_q;         // emit the quantised outputs
  int rq_K, cq_K;      // row lengths (elements) of the two quantised outputs
  float l_cols;        // (float) l, for the bound on amax(A)
  QuantOpts q;         // how this stage's output is quantised (q.widen = 1 in the base mode)
  int clip;            // kG3 on a problem with aux_raw: whether tau applies
  int aux_h;           // the combined tile is read from tmH (BF16)
  int out_h;           // 0: FP32 result by TMA store; 1: rounded to BF16, staged and stored through tmH (CTA-pair
                       // kernel); 2: rounded to BF16, stored as FP32 by the epilogue warps (single-CTA kernel)
  int update;          // kG3, CTA-pair kernel, last iteration: Root's parameter update W <- BF16(W * upd_decay -
  float upd_decay;     //   upd_step * X+) on every problem whose W is set, in the epilogue
  float upd_step;
  int no_out;          // with update: the FP32 result is not stored
  int dry_operands;    // kPlain, CTA-pair kernel: measurement of the tensor-pipe ceiling - no operand is fetched
  NsScalarIdx ix;
  uint32_t* status;
};

// Measurement support: counts kernel launches and, when profiling is on, brackets a group of
// launches with events.
void count_launches(int n);

// Launch of a kernel of the Newton-Schulz chain: with the programmatic-stream-serialisation attribute (the
// kernel's blocks may become resident before the previous launch has completed; the kernel itself waits,
// see pdl_wait) for the groups of a call that are bound by launch latency (pdl_select, called per group),
// unless the environment variable FP4ROOT_NO_PDL is set.
bool pdl_enabled();
void pdl_select(int64_t group_elements);
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = pdl_enabled() ? 1 : 0;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// First-moment momentum state (fp4_momentum.cu): one step in place on codes/scales; M_out and
// hist may be null.
cudaError_t launch_momentum_update(const float* G, int64_t rows, int64_t cols, float mu, float g_scale, bool sr,
                                   uint64_t seed, uint8_t* codes, uint16_t* scales, float* M_out, uint32_t* hist,
                                   int sms, cudaStream_t st);
// Packed AdamW step on NVFP4 moment states (fp4_adamw.cu).  The constants are derived on the host
// in a fixed way (adamw_consts) and passed by value.
struct AdamwConsts {
  float b1, b2, omb1, omb2, eps, rsb2, step_size, decay;
  uint64_t seed;
};
AdamwConsts adamw_consts(float lr, float beta1, float beta2, float eps, float weight_decay, int step, uint64_t seed);
cudaError_t launch_adamw_update(uint16_t* W, const uint16_t* G, int64_t n, const AdamwConsts& k, bool sr,
                                uint8_t* m_codes, uint16_t* m_scales, uint8_t* v_codes, uint16_t* v_scales,
                                uint16_t* v_means, cudaStream_t st);
cudaError_t launch_momentum_decode(const uint8_t* codes, const uint16_t* scales, int64_t rows, int64_t cols,
                                   float* M_out, int sms, cudaStream_t st);
struct ProfScope {
  int cls; cudaStream_t st; cudaEvent_t e0; bool on;
  ProfScope(int cls, cudaStream_t st);
  ~ProfScope();
};

cudaError_t launch_quantize(const float* x, int64_t rows, int64_t cols, uint8_t* codes, uint8_t* scales,
                            float* tensor_scale, const QuantOpts& q, int sms, cudaStream_t st);
struct PrologueItem {
  const float* G;
  float* X;
  uint8_t* ws;
  const NsPlan* pl;
  bool clear_status;
  bool store_x;   // write X0 in FP32 (not needed when the first G3 stage reads G itself)
  int64_t x_rows, x_cols;  // extent and row pitch of X: the work shape in the workspace, the caller's shape in `out`
  uint32_t* hist_top;      // the caller's histogram of the top 13 magnitude bits of G, or null
  const CUtensorMap* tmG;  // G as an FP32 tensor: box = 32 columns x 128 rows, 128-byte swizzle
};
// count matrices that share the shape (s, l) and the clip / eps parameters
cudaError_t launch_prologue_group(const PrologueItem* items, int count, int write_q, const QuantOpts& q,
                                  uint32_t* status, cudaStream_t st);
// Root's parameter update on BF16 weights: decay = fl(1 - fl(lr * wd)), step = fl(lr * scale),
// w <- BF16(fl(fl(w * decay) - fl(step * o))).
struct ParamUpdate {
  uint16_t* W;     // null: no update
  float decay, step;
  int no_out;      // where the update is fused with the store of the FP32 result: skip that store
};
__device__ __forceinline__ float param_update_value(float w, float o, float decay, float step) {
  return __fsub_rn(__fmul_rn(w, decay), __fmul_rn(step, o));
}
// out (l0 x s0, row-major) = the leading s0 x l0 part of X^T, X being s x l with row pitch l; with
// upd.W set, W (l0 x s0 like out) takes the update from the same values
cudaError_t launch_transpose_out(const float* X, int64_t s, int64_t l, float* out, int64_t s0, int64_t l0,
                                 const ParamUpdate& upd, cudaStream_t st);
// W (n elements) updated from the FP32 matrix O of the same layout
cudaError_t launch_param_update(const float* O, int64_t n, const ParamUpdate& upd, int sms, cudaStream_t st);
cudaError_t prologue_set_attributes();

cudaError_t gemm_set_attributes();
cudaError_t gemm_pair_set_attributes();
// pack: the launch.num_problems (<= kPackMax) problems of the launch
cudaError_t launch_gemm_pair(GemmMode mode, const ProblemPack& pack, const GemmLaunch& launch, int sms,
                             cudaStream_t st);
int gemm_stage_k();  // elements of K per operand stage (the codes maps' box is this / 2 bytes wide)
int gemm_pair_stage_k(GemmMode mode);  // the same for a mode of the CTA-pair kernel
cudaError_t launch_gemm(GemmMode mode, const ProblemPack& pack, const GemmLaunch& launch, int sms, cudaStream_t st);

}  // namespace fp4
