// Host side of the library: argument checks, workspace layout, TMA descriptors, and the
// sequence of launches of the Root Newton-Schulz step (Section 3.4).  Everything here
// only enqueues work on the caller's stream.
#include <atomic>
#include <cmath>
#include <mutex>
#include <stdlib.h>
#include <unordered_map>
#include <vector>

#include "fp4_gemm_common.cuh"

namespace fp4 {

namespace {
std::atomic<uint64_t> g_launches{0};
std::atomic<int> g_prof_on{0};
struct ProfRec { int cls; cudaEvent_t e0, e1; };
std::vector<ProfRec> g_prof;
std::mutex g_prof_mu;
}  // namespace

void count_launches(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

// Programmatic dependent launch pays where a call is bound by launch latency (a 5-iteration call on one
// 512 x 512 .. 2048 x 2048 matrix: 0.22 -> 0.19, 0.25 -> 0.21, 0.28 -> 0.25 ms) and measured 2 % slower on
// groups that fill the machine for milliseconds, so each group of a call decides by its size.
namespace {
thread_local bool t_pdl_group = false;
}
bool pdl_enabled() {
  static const bool allowed = getenv("FP4ROOT_NO_PDL") == nullptr;
  return allowed && t_pdl_group;
}
void pdl_select(int64_t group_elements) { t_pdl_group = group_elements <= (int64_t)8 << 20; }

ProfScope::ProfScope(int cls_, cudaStream_t st_) : cls(cls_), st(st_), e0(nullptr), on(g_prof_on.load() != 0) {
  if (on) {
    if (cudaEventCreate(&e0) != cudaSuccess) { on = false; return; }
    cudaEventRecord(e0, st);
  }
}
ProfScope::~ProfScope() {
  if (!on) return;
  cudaEvent_t e1;
  if (cudaEventCreate(&e1) != cudaSuccess) { cudaEventDestroy(e0); return; }
  cudaEventRecord(e1, st);
  std::lock_guard<std::mutex> lock(g_prof_mu);
  g_prof.push_back({cls, e0, e1});
}

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DeviceInfo {
  bool ready = false;
  fp4_status status = FP4_OK;
  int sms = 0;
  EncodeTiledFn encode = nullptr;
};
DeviceInfo g_dev[64];
std::mutex g_mu;

// Per-device set-up on first use: architecture check, driver entry point, kernel attributes.
const DeviceInfo* device_info() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(g_mu);
  DeviceInfo& d = g_dev[dev];
  if (d.ready) return &d;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) { d.status = FP4_ERR_CUDA; d.ready = true; return &d; }
  if (prop.major != 10) { d.status = FP4_ERR_ARCH; d.ready = true; return &d; }
  d.sms = prop.multiProcessorCount;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || fn == nullptr) {
    d.status = FP4_ERR_CUDA; d.ready = true; return &d;
  }
  d.encode = reinterpret_cast<EncodeTiledFn>(fn);
  if (gemm_set_attributes() != cudaSuccess || gemm_pair_set_attributes() != cudaSuccess ||
      prologue_set_attributes() != cudaSuccess)
    d.status = FP4_ERR_CUDA;
  d.ready = true;
  return &d;
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline bool shape_ok(int64_t v) { return v >= 128 && v % 128 == 0 && v <= (1 << 20); }
// The Newton-Schulz entry points pad internally: any positive multiple of the block length.
inline bool ns_shape_ok(int64_t v) { return v >= 16 && v % 16 == 0 && v <= (1 << 20); }
inline int64_t pad128(int64_t v) { return (v + 127) / 128 * 128; }
// flag bits the Newton-Schulz entry points know
constexpr uint32_t kNsFlags =
    FP4_FLAG_KEEP_OPERANDS | FP4_FLAG_RHT | FP4_FLAG_FOUR_SIX | FP4_FLAG_STORE_BF16 | FP4_FLAG_NO_OUT |
    FP4_FLAG_OVERLAP_GROUPS;

// 2-D map over a row-major byte matrix (NVFP4 codes): box = one operand stage of `stage_k` elements of K
// (64 or 128 bytes x 128 rows), swizzled over the box width.
bool make_codes_map(const DeviceInfo* d, CUtensorMap* tm, const void* base, int64_t rows, int64_t row_bytes, int stage_k) {
  const cuuint32_t bw = (cuuint32_t)(stage_k / 2);
  cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
  cuuint32_t box[2] = {bw, 128};
  cuuint32_t estr[2] = {1, 1};
  return d->encode(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, bw == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// 2-D map over a row-major FP32 matrix: box = 16 columns x box_rows rows (128: a chunk of the single-CTA
// kernel; 32: one epilogue warp's block in the CTA-pair kernel), 64-byte swizzle.
bool make_f32_map(const DeviceInfo* d, CUtensorMap* tm, const void* base, int64_t rows, int64_t cols, int box_rows) {
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
  cuuint32_t box[2] = {16, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return d->encode(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 2-D map over a row-major FP32 matrix for the operand preparation: box = 32 columns x 128 rows (a quarter
// of a 128 x 128 tile), 128-byte swizzle.
bool make_f32_tile_map(const DeviceInfo* d, CUtensorMap* tm, const void* base, int64_t rows, int64_t cols) {
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
  cuuint32_t box[2] = {32, 128};
  cuuint32_t estr[2] = {1, 1};
  return d->encode(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 2-D map over a row-major FP32 matrix whose transpose the CTA-pair kernel works on: box = 32 columns x 16 rows
// (one epilogue warp's 32 x 16 block, transposed), no swizzle.
bool make_f32_tr_map(const DeviceInfo* d, CUtensorMap* tm, const void* base, int64_t rows, int64_t cols) {
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
  cuuint32_t box[2] = {32, 16};
  cuuint32_t estr[2] = {1, 1};
  return d->encode(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 2-D map over a row-major BF16 matrix: box = 16 columns x 32 rows (32-byte rows), no swizzle: the block of
// one epilogue warp of the CTA-pair kernel.
bool make_bf16_map(const DeviceInfo* d, CUtensorMap* tm, const void* base, int64_t rows, int64_t cols) {
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {16, 32};
  cuuint32_t estr[2] = {1, 1};
  return d->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 2-D map over a row-major byte matrix (NVFP4 codes) for the stores of the CTA-pair kernel's epilogue
// warps: box = box_bytes x box_rows, no swizzle.
bool make_code_store_map(const DeviceInfo* d, CUtensorMap* tm, const void* base, int64_t rows, int64_t row_bytes,
                         int box_bytes, int box_rows, bool swizzle64 = false) {
  cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
  cuuint32_t box[2] = {(cuuint32_t)box_bytes, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return d->encode(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kDefaultMaxGroup = kPackMax;

// 2-D map over the scale atoms of a rows x K operand: one map row per 128-row block, 64-bit
// elements, box = the atoms of one operand stage (`stage_k` elements of 8 bytes: 1 or 2 KB), no swizzle.
bool make_sf_map(const DeviceInfo* d, CUtensorMap* tm, const void* base, int64_t rows, int64_t K, int stage_k) {
  if (K < 256) { memset(tm, 0, sizeof(*tm)); return true; }   // never used by the CTA-pair kernel
  cuuint64_t dims[2] = {(cuuint64_t)(K / 64) * 64, (cuuint64_t)(rows / 128)};
  cuuint64_t strides[1] = {(cuuint64_t)(K / 64) * 512};
  cuuint32_t box[2] = {(cuuint32_t)stage_k, 1};
  cuuint32_t estr[2] = {1, 1};
  return d->encode(tm, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The CTA-pair kernel takes every product whose dimensions are all multiples of 256 (tile counts in 128-blocks).
// The descriptors of a problem are built for the kernel that runs it (pair_kernel decides both).
bool pair_kernel(int64_t tiles_m, int64_t tiles_n, int64_t K, int sms, bool force_single = false) {
#ifndef FP4_DISABLE_PAIR
  return !force_single && !(tiles_m & 1) && !(tiles_n & 1) && K % 256 == 0 && sms >= 2;
#else
  (void)tiles_m; (void)tiles_n; (void)K; (void)sms; (void)force_single;
  return false;
#endif
}
cudaError_t launch_gemm_auto(GemmMode mode, const ProblemPack& pack, const GemmLaunch& L, int sms, cudaStream_t st,
                             bool force_single = false) {
  if (pair_kernel(L.tiles_m, L.tiles_n, L.K, sms, force_single)) return launch_gemm_pair(mode, pack, L, sms, st);
  return launch_gemm(mode, pack, L, sms, st);
}

void default_params(fp4_ns_params* p) {
  p->a = p->b = p->c = NAN;
  p->clip_quantile = 0.99f;
  p->eps = 1e-7f;
  p->flags = 0;
  p->max_group = 0;
  p->seed = 0;
  p->top_hist = nullptr;
  p->weights = nullptr;
  p->lr = p->weight_decay = 0.0f;
  p->update_scale = 1.0f;
}

// The 16 signs of the j-th random Hadamard matrix of a call: splitmix64 on seed + j.
uint32_t rht_signs(uint64_t seed, uint64_t j) {
  uint64_t z = seed + 0x9E3779B97F4A7C15ull * (j + 1);
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  z ^= z >> 31;
  return (uint32_t)(z & 0xFFFFu);
}

// Quantiser options of the j-th product of a call.
QuantOpts quant_opts(const fp4_ns_params* p, uint64_t j) {
  QuantOpts q;
  q.rht = (p->flags & FP4_FLAG_RHT) ? 1u : 0u;
  q.four_six = (p->flags & FP4_FLAG_FOUR_SIX) ? 1u : 0u;
  q.mask = q.rht ? rht_signs(p->seed, j) : 0u;
  q.widen = q.rht ? 4.0f : 1.0f;
  return q;
}

int64_t quantile_rank(int64_t n, float q) {
  // resolved to parts per million so that 0.99f means 99/100
  int64_t ppm = (int64_t)llround((double)q * 1e6);
  int64_t k = (ppm * n + 999999) / 1000000;
  if (k < 1) k = 1;
  if (k > n) k = n;
  return k;
}

void coeffs(int64_t m, int64_t n, float abc[3]) {
  // quintic with p(1) = 1, p'(1) = 0: b = 2.5 - 2a, c = a - 1.5; a from the aspect ratio
  double s = (double)(m < n ? m : n), l = (double)(m < n ? n : m);
  double delta = (std::sqrt(7.0 / 3.0) - 1.0) / 2.0;
  double rr = 1.0 + delta * (1.0 + std::sqrt(s / l));
  double R = rr * rr;
  double a = (1.5 * R - 1.0) / (R - 1.0);
  abc[0] = (float)a;
  abc[1] = (float)(2.5 - 2.0 * a);
  abc[2] = (float)(a - 1.5);
}

// Workspace layout of one matrix.
fp4_status make_plan(int64_t m, int64_t n, int steps, const fp4_ns_params* p, int sms, NsPlan* pl) {
  if (!ns_shape_ok(m) || !ns_shape_ok(n)) return FP4_ERR_SHAPE;
  if (steps < 0 || steps > kMaxSteps) return FP4_ERR_INVALID_ARG;
  memset(pl, 0, sizeof(*pl));
  pl->m = m; pl->n = n;
  pl->tall = m > n;
  pl->s0 = m < n ? m : n;
  pl->l0 = m < n ? n : m;
  // Zero rows and columns stay zero through the iteration and add nothing to any product or
  // maximum; since the dimensions are multiples of 16 no block mixes data and padding.
  pl->s = pad128(pl->s0);
  pl->l = pad128(pl->l0);
  // BF16 storage: 2-byte tensors when all three stages run in the CTA-pair kernel, else FP32
  // tensors that hold rounded values (and all stages in the single-CTA kernel)
  if (p->flags & FP4_FLAG_STORE_BF16) pl->bf16_mode = (pl->s % 256 == 0 && pl->l % 256 == 0) ? 1 : 2;
#ifdef FP4_DISABLE_PAIR
  if (pl->bf16_mode == 1) pl->bf16_mode = 2;
#endif
  const int64_t s = pl->s, l = pl->l;
  pl->clip = p->clip_quantile > 0.0f && p->clip_quantile < 1.0f;
  pl->clip_rank = pl->clip ? quantile_rank(m * n, p->clip_quantile) : 0;
  pl->eps = p->eps;
  pl->sms = sms;
  int64_t blocks = (m * n / 4 + 1023) / 1024;
  pl->stat_blocks = (int)(blocks < 1024 ? blocks : 1024);

  NsScalarIdx& ix = pl->ix;
  ix.tau = 0; ix.nu = 1; ix.inv = 2;
  const int span = kMaxSteps + 2;
  ix.amax_X0 = 8; ix.amax_A0 = 8 + span; ix.sg_X0 = 8 + 2 * span; ix.sg_A0 = 8 + 3 * span; ix.sg_B0 = 8 + 4 * span;
  const size_t scalar_bytes = align_up((size_t)(8 + 5 * span) * 4, 1024);

  fp4_ws_layout& L = pl->lay;
  size_t off = 0;
  L.header = off; off += 1024;
  L.scalars = off; off += scalar_bytes;
  pl->off_hist = off; off += 8192 * 4;
  pl->zero_bytes = off;
  pl->off_partial = off; off += 1024 * 8;
  off = align_up(off, 1024);
  L.X = off; if (pl->tall) off += align_up((size_t)s * l * 4, 1024);
  L.A = off; off += align_up((size_t)s * s * 4, 1024);
  L.qX_codes = off; off += align_up((size_t)s * l / 2, 1024);
  L.qX_scales = off; off += align_up((size_t)s * l / 16, 1024);
  for (int i = 0; i < 2; ++i) {
    L.qXt_codes[i] = off; off += align_up((size_t)s * l / 2, 1024);
    L.qXt_scales[i] = off; off += align_up((size_t)s * l / 16, 1024);
  }
  L.qA_codes = off; off += align_up((size_t)s * s / 2, 1024);
  L.qA_scales = off; off += align_up((size_t)s * s / 16, 1024);
  L.qB_codes = off; off += align_up((size_t)s * s / 2, 1024);
  L.qB_scales = off; off += align_up((size_t)s * s / 16, 1024);
  L.Xh = 0;
  if (pl->bf16_mode == 1) { pl->off_Xh = off; L.Xh = off; off += align_up((size_t)s * l * 2, 1024); }
  L.idx_tau = ix.tau; L.idx_nu = ix.nu; L.idx_inv = ix.inv;
  L.idx_amax_X0 = ix.amax_X0; L.idx_amax_A0 = ix.amax_A0;
  L.idx_sg_X0 = ix.sg_X0; L.idx_sg_A0 = ix.sg_A0; L.idx_sg_B0 = ix.sg_B0;
  L.total = off;
  return FP4_OK;
}

// Everything the launches need to know about one matrix of a call.
struct MatrixCtx {
  NsPlan pl;
  const float* G;
  float* out;
  float* X;        // FP32 X in the work orientation: `out` itself, or the workspace when tall
  uint8_t* ws;     // this matrix's workspace
  GemmProblem g1, g2, g3[2];  // g3[cur]: reads qXt[cur], writes qXt[cur ^ 1]
  GemmProblem g3_first;       // iteration 0: as g3[0], but a wide input's FP32 tile is G itself (no X0 copy)
  bool store_x0;              // the prologue writes X0 in FP32
  int64_t x_rows, x_cols;     // extent (and row pitch) of X
  uint32_t* hist_top;         // the caller's first-pass histogram of G, or null
  uint16_t* W;                // the BF16 parameter that takes Root's update in this call, or null
  CUtensorMap tm_G;           // the caller's matrix for the operand preparation (tiles of 128 x 128)
  // A tall input in the CTA-pair kernel: the first G3 stage reads the caller's matrix and the last one
  // writes the caller's result through transposing boxes.
  bool native_tall;
  CUtensorMap tm_outT;
};

fp4_status build_matrix(const DeviceInfo* d, const float* G, float* out, int64_t m, int64_t n, int steps,
                        const fp4_ns_params* p, uint8_t* ws, MatrixCtx* c) {
  fp4_status rc = make_plan(m, n, steps, p, d->sms, &c->pl);
  if (rc != FP4_OK) return rc;
  const fp4_ws_layout& L = c->pl.lay;
  const int64_t s = c->pl.s, l = c->pl.l;
  c->G = G; c->out = out; c->ws = ws;
  c->hist_top = nullptr;
  c->W = nullptr;
  c->X = c->pl.tall ? reinterpret_cast<float*>(ws + L.X) : out;
  // extent of X: the padded work shape in the workspace, the caller's shape in `out` (TMA fills what
  // lies outside with zeros on loads and drops it on stores)
  const int64_t xr = c->pl.tall ? s : c->pl.s0, xc = c->pl.tall ? l : c->pl.l0;
  c->x_rows = xr; c->x_cols = xc;
  c->store_x0 = c->pl.tall || steps == 0;
  c->native_tall = false;
  if (!make_f32_tile_map(d, &c->tm_G, G, m, n)) return FP4_ERR_CUDA;
  if (steps == 0) return FP4_OK;
  float abc[3] = {p->a, p->b, p->c};
  if (std::isnan(p->a)) coeffs(m, n, abc);
  // which kernel runs each stage (rounded-FP32 storage is implemented by the single-CTA kernel only)
  const bool fs = c->pl.bf16_mode == 2;
  const bool pair1 = pair_kernel(s / 128, s / 128, l, d->sms, fs), pair2 = pair_kernel(s / 128, s / 128, s, d->sms, fs),
             pair3 = pair_kernel(s / 128, l / 128, s, d->sms, fs);
  CUtensorMap tm_qX, tm_qXt[2], tm_qA, tm_qB, tm_A1, tm_A2, tm_X;
  CUtensorMap sf_qX, sf_qXt[2], sf_qA, sf_qB;
  // every operand is read by exactly one stage: its descriptors take that stage's depth in K
  const int k1 = pair1 ? gemm_pair_stage_k(kG1) : gemm_stage_k(), k2 = pair2 ? gemm_pair_stage_k(kG2) : gemm_stage_k(),
            k3 = pair3 ? gemm_pair_stage_k(kG3) : gemm_stage_k();
  bool ok = make_sf_map(d, &sf_qX, ws + L.qX_scales, s, l, k1) && make_sf_map(d, &sf_qXt[0], ws + L.qXt_scales[0], l, s, k3) &&
            make_sf_map(d, &sf_qXt[1], ws + L.qXt_scales[1], l, s, k3) && make_sf_map(d, &sf_qA, ws + L.qA_scales, s, s, k2) &&
            make_sf_map(d, &sf_qB, ws + L.qB_scales, s, s, k3) &&
            make_codes_map(d, &tm_qX, ws + L.qX_codes, s, l / 2, k1) &&
            make_codes_map(d, &tm_qXt[0], ws + L.qXt_codes[0], l, s / 2, k3) &&
            make_codes_map(d, &tm_qXt[1], ws + L.qXt_codes[1], l, s / 2, k3) &&
            make_codes_map(d, &tm_qA, ws + L.qA_codes, s, s / 2, k2) &&
            make_codes_map(d, &tm_qB, ws + L.qB_codes, s, s / 2, k3) &&
            make_f32_map(d, &tm_A1, ws + L.A, s, s, pair1 ? 32 : 128) &&
            make_f32_map(d, &tm_A2, ws + L.A, s, s, pair2 ? 32 : 128) &&
            make_f32_map(d, &tm_X, c->X, xr, xc, pair3 ? 32 : 128);
  if (!ok) return FP4_ERR_CUDA;
  // stores of the quantised outputs by the CTA-pair kernel's epilogue warps
  CUtensorMap st_qA_r, st_qA_c, st_qB_r, st_qB_c, st_qX_r, st_qXt_c[2];
  ok = make_code_store_map(d, &st_qA_r, ws + L.qA_codes, s, s / 2, 32, 32) &&
       make_code_store_map(d, &st_qA_c, ws + L.qA_codes, s, s / 2, 64, 128, true) &&
       make_code_store_map(d, &st_qB_r, ws + L.qB_codes, s, s / 2, 32, 32) &&
       make_code_store_map(d, &st_qB_c, ws + L.qB_codes, s, s / 2, 64, 128, true) &&
       make_code_store_map(d, &st_qX_r, ws + L.qX_codes, s, l / 2, 32, 32) &&
       make_code_store_map(d, &st_qXt_c[0], ws + L.qXt_codes[0], l, s / 2, 64, 128, true) &&
       make_code_store_map(d, &st_qXt_c[1], ws + L.qXt_codes[1], l, s / 2, 64, 128, true);
  if (!ok) return FP4_ERR_CUDA;
  GemmProblem base;
  memset(&base, 0, sizeof(base));
  base.scalars = reinterpret_cast<float*>(ws + L.scalars);
  base.ca = abc[0]; base.cb = abc[1]; base.cc = abc[2];
  base.out_rows = (int)s; base.out_cols = (int)s;
  const int bmode = c->pl.bf16_mode;
  CUtensorMap tm_Ah, tm_Xh;
  uint8_t* Xh = bmode == 1 ? ws + c->pl.off_Xh : nullptr;
  if (bmode == 1 && (!make_bf16_map(d, &tm_Ah, ws + L.A, s, s) || !make_bf16_map(d, &tm_Xh, Xh, s, l))) return FP4_ERR_CUDA;
  // G1: A = qX qX^T (upper-triangle tiles), qA in both triangles
  c->g1 = base;
  c->g1.tmA = c->g1.tmB = tm_qX; c->g1.tmAux = c->g1.tmOut = tm_A1;
  c->g1.tmRq = st_qA_r; c->g1.tmCq = st_qA_c;
  c->g1.tmSfa = c->g1.tmSfb = sf_qX;
  c->g1.sfa = c->g1.sfb = ws + L.qX_scales;
  c->g1.rq_codes = c->g1.cq_codes = ws + L.qA_codes; c->g1.rq_sf = c->g1.cq_sf = ws + L.qA_scales;
  if (bmode == 1) c->g1.tmH = tm_Ah;                                           // A as a BF16 tensor
  if (bmode == 2) { c->g1.out_direct = ws + L.A; c->g1.out_direct_ld = s; }   // A as rounded FP32
  // G2: B = bA + c qA qA^T, qB in both triangles
  c->g2 = base;
  c->g2.tmA = c->g2.tmB = tm_qA; c->g2.tmAux = c->g2.tmOut = tm_A2;
  c->g2.tmRq = st_qB_r; c->g2.tmCq = st_qB_c;
  c->g2.tmSfa = c->g2.tmSfb = sf_qA;
  c->g2.sfa = c->g2.sfb = ws + L.qA_scales;
  if (bmode == 1) c->g2.tmH = tm_Ah;
  c->g2.rq_codes = c->g2.cq_codes = ws + L.qB_codes; c->g2.rq_sf = c->g2.cq_sf = ws + L.qB_scales;
  // G3: X+ = aX + qB qXt^T in place on X; new operand copies
  for (int cur = 0; cur < 2; ++cur) {
    GemmProblem& g = c->g3[cur];
    g = base;
    g.tmA = tm_qB; g.tmB = tm_qXt[cur]; g.tmAux = g.tmOut = tm_X;
    g.out_rows = (int)xr; g.out_cols = (int)xc;
    if (bmode == 1) g.tmH = tm_Xh;
    if (bmode == 2) { g.out_direct = c->X; g.out_direct_ld = xc; }
    g.tmSfa = sf_qB; g.tmSfb = sf_qXt[cur];
    g.sfa = ws + L.qB_scales; g.sfb = ws + L.qXt_scales[cur];
    g.rq_codes = ws + L.qX_codes; g.rq_sf = ws + L.qX_scales;
    g.cq_codes = ws + L.qXt_codes[cur ^ 1]; g.cq_sf = ws + L.qXt_scales[cur ^ 1];
    g.tmRq = st_qX_r; g.tmCq = st_qXt_c[cur ^ 1];
  }
  c->g3_first = c->g3[0];
  c->native_tall = c->pl.tall && pair3;   // (rounded-FP32 storage, bmode 2, never runs in the CTA-pair kernel)
  if (c->native_tall) {
    // the caller's matrices are l0 x s0
    CUtensorMap tm_Gt;
    if (!make_f32_tr_map(d, &tm_Gt, G, c->pl.l0, c->pl.s0) || !make_f32_tr_map(d, &c->tm_outT, out, c->pl.l0, c->pl.s0))
      return FP4_ERR_CUDA;
    c->store_x0 = false;
    c->g3_first.tmAux = tm_Gt;
    c->g3_first.aux_raw = 1;
    c->g3_first.aux_tr = 1;
  } else if (!c->store_x0) {
    CUtensorMap tm_G;
    if (!make_f32_map(d, &tm_G, G, c->pl.s0, c->pl.l0, pair3 ? 32 : 128)) return FP4_ERR_CUDA;
    c->g3_first.tmAux = tm_G;
    c->g3_first.aux_raw = 1;
  }
  return FP4_OK;
}

// Everything build_matrix derives (workspace plan, a dozen and a half TMA descriptors, the problem
// descriptions) depends only on the pointers, the shape and a few parameters: an optimiser calls with
// the same buffers every step, so the results are kept, keyed by exactly those inputs.  The library
// keeps no other state between calls; a hit costs one hash lookup instead of ~20 driver calls.
struct CtxKey {
  int dev; int steps; uint32_t flags;
  const void* G; const void* out; const void* ws;
  int64_t m, n;
  uint32_t a, b, c, q, eps;   // bit patterns of the float parameters
  bool operator==(const CtxKey& o) const {
    return dev == o.dev && steps == o.steps && flags == o.flags && G == o.G && out == o.out && ws == o.ws && m == o.m &&
           n == o.n && a == o.a && b == o.b && c == o.c && q == o.q && eps == o.eps;
  }
};
struct CtxKeyHash {
  size_t operator()(const CtxKey& k) const {
    uint64_t h = 1469598103934665603ull;
    auto mix = [&](uint64_t v) { h = (h ^ v) * 1099511628211ull; };
    mix((uint64_t)k.dev); mix((uint64_t)k.steps); mix(k.flags);
    mix((uint64_t)(uintptr_t)k.G); mix((uint64_t)(uintptr_t)k.out); mix((uint64_t)(uintptr_t)k.ws);
    mix((uint64_t)k.m); mix((uint64_t)k.n); mix(k.a); mix(k.b); mix(k.c); mix(k.q); mix(k.eps);
    return (size_t)h;
  }
};
std::unordered_map<CtxKey, MatrixCtx, CtxKeyHash> g_ctx_cache;
std::mutex g_ctx_mu;
constexpr size_t kCtxCacheMax = 1024;   // entries (about 8 KB each); the cache is emptied when it is full

inline uint32_t fbits(float v) { uint32_t u; memcpy(&u, &v, 4); return u; }

fp4_status prepare_matrix(const DeviceInfo* d, const float* G, float* out, int64_t m, int64_t n, int steps,
                          const fp4_ns_params* p, uint8_t* ws, MatrixCtx* c) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return FP4_ERR_CUDA;
  // NO_OUT only matters to the launch sequence, not to what is prepared here
  const CtxKey key{dev, steps, p->flags & ~FP4_FLAG_NO_OUT, G, out, ws, m, n,
                   fbits(p->a), fbits(p->b), fbits(p->c), fbits(p->clip_quantile), fbits(p->eps)};
  {
    std::lock_guard<std::mutex> lock(g_ctx_mu);
    auto it = g_ctx_cache.find(key);
    if (it != g_ctx_cache.end()) { *c = it->second; return FP4_OK; }
  }
  fp4_status rc = build_matrix(d, G, out, m, n, steps, p, ws, c);
  if (rc != FP4_OK) return rc;
  std::lock_guard<std::mutex> lock(g_ctx_mu);
  if (g_ctx_cache.size() >= kCtxCacheMax) g_ctx_cache.clear();
  g_ctx_cache.emplace(key, *c);
  return FP4_OK;
}

// Enqueue the whole step for a group of matrices of one shape (s, l): the prologue per matrix,
// then every Newton-Schulz stage as one launch over all matrices of the group.
// count <= kPackMax: the problems of a launch travel as its parameter.
fp4_status run_group(const DeviceInfo* d, MatrixCtx* mats, int count, int steps, const fp4_ns_params* p,
                     uint32_t* status, bool clear_first_status, cudaStream_t st) {
  if (count < 1 || count > kPackMax) return FP4_ERR_INVALID_ARG;
  const bool keep = (p->flags & FP4_FLAG_KEEP_OPERANDS) != 0;
  ParamUpdate upd;
  upd.W = nullptr;
  {
    // every operation rounded to FP32 on its own (volatile keeps the host compiler from fusing them)
    volatile float t = p->lr * p->weight_decay;
    volatile float dec = 1.0f - t;
    volatile float stp = p->lr * p->update_scale;
    upd.decay = dec;
    upd.step = stp;
  }
  upd.no_out = (p->flags & FP4_FLAG_NO_OUT) ? 1 : 0;
  bool any_update = false;
  for (int i = 0; i < count; ++i) any_update = any_update || mats[i].W != nullptr;
  std::vector<char> fused_update((size_t)count, 0);
  // a tall input's result leaves the last G3 stage transposed (no transpose pass) unless that stage also has to
  // write operand copies, or the call updates parameters (the update of a tall matrix rides on the transpose)
  std::vector<char> direct_out((size_t)count, 0);
  bool any_direct = false;
  for (int i = 0; i < count; ++i)
    if (steps > 0 && mats[i].native_tall && !keep && !any_update) { direct_out[(size_t)i] = 1; any_direct = true; }
  const NsPlan& pl0 = mats[0].pl;
  const int64_t s = pl0.s, l = pl0.l;
  pdl_select(s * l * count);
  {
    std::vector<PrologueItem> items((size_t)count);
    for (int i = 0; i < count; ++i) {
      MatrixCtx& c = mats[i];
      items[(size_t)i] = PrologueItem{c.G, c.X, c.ws, &c.pl, clear_first_status && i == 0, c.store_x0, c.x_rows, c.x_cols,
                                      c.hist_top, &c.tm_G};
    }
    if (launch_prologue_group(items.data(), count, steps > 0 || keep, quant_opts(p, 0), status, st) != cudaSuccess)
      return FP4_ERR_CUDA;
  }
  if (steps > 0) {
    // the problems of the five kinds of launches: G1, G2, G3 reading qXt[0] / qXt[1], the first G3
    std::vector<ProblemPack> packs(5);
    for (int kind = 0; kind < 5; ++kind) {
      for (int j = 0; j < kPackMax; ++j) {
        const MatrixCtx& c = mats[j < count ? j : 0];
        packs[(size_t)kind].p[j] = kind == 0 ? c.g1 : kind == 1 ? c.g2 : kind == 4 ? c.g3_first : c.g3[kind - 2];
      }
    }
    // Root's parameter update: fused into the last G3 stage where the CTA-pair kernel runs it on a
    // matrix in the caller's orientation and no operand copies are wanted from that stage; into the
    // final transpose for a tall matrix; a separate elementwise pass otherwise (below).
    const bool g3_pair = pair_kernel(s / 128, l / 128, s, d->sms, pl0.bf16_mode == 2);
    if (g3_pair && !keep) {
      for (int kind = 2; kind < 5; ++kind)
        for (int j = 0; j < count; ++j)
          if (mats[j].W && !mats[j].pl.tall) {
            packs[(size_t)kind].p[j].W = mats[j].W;
            packs[(size_t)kind].p[j].W_ld = mats[j].pl.n;
            fused_update[(size_t)j] = 1;
          }
    }
    GemmLaunch base;
    memset(&base, 0, sizeof(base));
    base.num_problems = count;
    base.ix = pl0.ix;
    base.l_cols = (float)l;
    base.status = status;
    base.clip = pl0.clip;
    const int bmode = pl0.bf16_mode;
    const bool fs = bmode == 2;  // rounded-FP32 storage is implemented by the single-CTA kernel only
    for (int k = 0; k < steps; ++k) {
      const int cur = k & 1;
      const bool last = (k == steps - 1);
      GemmLaunch L1 = base;
      L1.iter = k; L1.K = (int)l; L1.tiles_m = L1.tiles_n = (int)(s / 128); L1.symmetric = 1;
      L1.rq_K = L1.cq_K = (int)s; L1.write_q = 1;
      L1.q = quant_opts(p, 2 * (uint64_t)k + 1);  // qA_k
      L1.out_h = bmode;
      {
        ProfScope ps(FP4_PROF_G1, st);
        if (launch_gemm_auto(kG1, packs[0], L1, d->sms, st, fs) != cudaSuccess)
          return FP4_ERR_CUDA;
      }
      GemmLaunch L2 = L1;
      L2.K = (int)s;
      L2.q = quant_opts(p, 2 * (uint64_t)k);      // qB_k meets qX_k^{16x1}
      L2.out_h = 0; L2.aux_h = bmode == 1;
      {
        ProfScope ps(FP4_PROF_G2, st);
        if (launch_gemm_auto(kG2, packs[1], L2, d->sms, st, fs) != cudaSuccess)
          return FP4_ERR_CUDA;
      }
      GemmLaunch L3 = base;
      L3.iter = k; L3.K = (int)s; L3.tiles_m = (int)(s / 128); L3.tiles_n = (int)(l / 128); L3.symmetric = 0;
      L3.rq_K = (int)l; L3.cq_K = (int)s;
      L3.write_q = (!last || keep) ? 1 : 0;
      L3.q = quant_opts(p, 2 * (uint64_t)k + 2);  // both copies of X_{k+1}
      L3.aux_h = (bmode == 1 && k > 0) ? 1 : 0;   // X_0 is FP32 (or the raw input)
      L3.out_h = last ? 0 : bmode;                 // the result itself is FP32
      if (last && g3_pair && !keep && any_update) {
        L3.update = 1;
        L3.upd_decay = upd.decay; L3.upd_step = upd.step;
        L3.no_out = upd.no_out;
      }
      const ProblemPack* pk = &packs[k == 0 ? 4 : 2 + cur];
      ProblemPack last_pack;
      if (last && any_direct) {
        // tall inputs whose result goes straight to the caller's matrix, transposed on the way out
        last_pack = *pk;
        for (int j = 0; j < count; ++j)
          if (direct_out[(size_t)j]) {
            GemmProblem& g = last_pack.p[j];
            g.tmOut = mats[j].tm_outT;
            g.out_tr = 1;
            g.out_rows = (int)pl0.s0; g.out_cols = (int)pl0.l0;
          }
        pk = &last_pack;
      }
      {
        ProfScope ps(FP4_PROF_G3, st);
        if (launch_gemm_auto(kG3, *pk, L3, d->sms, st, fs) != cudaSuccess)
          return FP4_ERR_CUDA;
      }
    }
  }
  for (int i = 0; i < count; ++i) {
    ParamUpdate u = upd;
    u.W = mats[i].W;
    if (direct_out[(size_t)i]) continue;
    if (mats[i].pl.tall) {
      ProfScope ps(FP4_PROF_TRANSPOSE, st);
      if (launch_transpose_out(mats[i].X, s, l, mats[i].out, pl0.s0, pl0.l0, u, st) != cudaSuccess) return FP4_ERR_CUDA;
    } else if (u.W && !fused_update[(size_t)i]) {
      ProfScope ps(FP4_PROF_TRANSPOSE, st);
      if (launch_param_update(mats[i].out, mats[i].pl.m * mats[i].pl.n, u, d->sms, st) != cudaSuccess) return FP4_ERR_CUDA;
    }
  }
  return FP4_OK;
}

// Enqueue the whole step for one matrix.
fp4_status run_one(const DeviceInfo* d, const float* G, float* out, int64_t m, int64_t n, int steps,
                   const fp4_ns_params* p, uint8_t* ws, bool clear_status, cudaStream_t st) {
  MatrixCtx c;
  fp4_status rc = prepare_matrix(d, G, out, m, n, steps, p, ws, &c);
  if (rc != FP4_OK) return rc;
  if (p->top_hist) c.hist_top = p->top_hist[0];
  if (p->weights) c.W = p->weights[0];
  return run_group(d, &c, 1, steps, p, reinterpret_cast<uint32_t*>(ws + c.pl.lay.header), clear_status, st);
}

fp4_status check_common(const DeviceInfo** d) {
  *d = device_info();
  if (*d == nullptr) return FP4_ERR_CUDA;
  return (*d)->status;
}

}  // namespace
}  // namespace fp4

using namespace fp4;

extern "C" {

const char* fp4_status_string(fp4_status s) {
  switch (s) {
    case FP4_OK: return "ok";
    case FP4_ERR_INVALID_ARG: return "invalid argument";
    case FP4_ERR_SHAPE: return "unsupported shape (Newton-Schulz entry points: positive multiples of 16; fp4_quantize, fp4_gemm_nt: of 128)";
    case FP4_ERR_ALIGNMENT: return "misaligned pointer";
    case FP4_ERR_WORKSPACE: return "workspace too small";
    case FP4_ERR_ARCH: return "device is not compute capability 10.x (sm_100a kernels only, no fallback)";
    case FP4_ERR_CUDA: return "CUDA runtime or driver call failed";
    case FP4_ERR_DEVICE_TIMEOUT: return "a kernel gave up on a bounded wait";
    case FP4_ERR_UNIMPLEMENTED: return "not implemented";
    case FP4_ERR_STATIC_LIMIT: return "problem needs more scratch than the library's built-in static array holds";
  }
  return "unknown status";
}

size_t fp4_scale_bytes(int64_t rows, int64_t cols) {
  if (rows <= 0 || cols <= 0) return 0;
  return (size_t)((rows + 127) / 128) * (size_t)((cols + 63) / 64) * 512;
}

fp4_status fp4_quantize(const float* x, int64_t rows, int64_t cols, uint8_t* codes, uint8_t* scales,
                        float* tensor_scale, uint32_t flags, cudaStream_t stream) {
  if (!x || !codes || !scales || !tensor_scale) return FP4_ERR_INVALID_ARG;
  if (flags & 0xFFFFu & ~(FP4_FLAG_RHT | FP4_FLAG_FOUR_SIX)) return FP4_ERR_INVALID_ARG;
  if (!(flags & FP4_FLAG_RHT) && (flags >> 16)) return FP4_ERR_INVALID_ARG;
  QuantOpts q;
  q.rht = (flags & FP4_FLAG_RHT) ? 1u : 0u;
  q.four_six = (flags & FP4_FLAG_FOUR_SIX) ? 1u : 0u;
  q.mask = flags >> 16;
  q.widen = q.rht ? 4.0f : 1.0f;
  if (!shape_ok(rows) || !shape_ok(cols)) return FP4_ERR_SHAPE;
  if (!aligned(x, 16) || !aligned(codes, 16) || !aligned(scales, 16) || !aligned(tensor_scale, 4))
    return FP4_ERR_ALIGNMENT;
  const DeviceInfo* d;
  fp4_status rc = check_common(&d);
  if (rc != FP4_OK) return rc;
  ProfScope ps(FP4_PROF_QUANTIZE, stream);
  return launch_quantize(x, rows, cols, codes, scales, tensor_scale, q, d->sms, stream) == cudaSuccess ? FP4_OK
                                                                                                      : FP4_ERR_CUDA;
}

fp4_status fp4_momentum_update(const float* G, int64_t rows, int64_t cols, uint8_t* codes, uint16_t* scales,
                               float* M_out, uint32_t* hist, const fp4_momentum_params* params,
                               cudaStream_t stream) {
  if (!G || !codes || !scales || !params) return FP4_ERR_INVALID_ARG;
  if (params->flags & ~FP4_MOM_FLAG_SR) return FP4_ERR_INVALID_ARG;
  if (rows <= 0 || cols <= 0 || (cols & 15)) return FP4_ERR_SHAPE;
  if (!aligned(G, 32) || !aligned(codes, 16) || !aligned(scales, 16) || (M_out && !aligned(M_out, 32)) ||
      (hist && !aligned(hist, 4)))
    return FP4_ERR_ALIGNMENT;
  const DeviceInfo* d;
  fp4_status rc = check_common(&d);
  if (rc != FP4_OK) return rc;
  ProfScope ps(FP4_PROF_MOMENTUM, stream);
  return launch_momentum_update(G, rows, cols, params->mu, params->g_scale, (params->flags & FP4_MOM_FLAG_SR) != 0,
                                params->seed, codes, scales, M_out, hist, d->sms, stream) == cudaSuccess
             ? FP4_OK
             : FP4_ERR_CUDA;
}

fp4_status fp4_adamw_update(uint16_t* W, const uint16_t* G, int64_t n, uint8_t* m_codes, uint16_t* m_scales,
                            uint8_t* v_codes, uint16_t* v_scales, uint16_t* v_means,
                            const fp4_adamw_params* params, cudaStream_t stream) {
  if (!W || !G || !m_codes || !m_scales || !v_codes || !v_scales || !v_means || !params) return FP4_ERR_INVALID_ARG;
  if ((params->flags & ~FP4_MOM_FLAG_SR) || params->step < 1) return FP4_ERR_INVALID_ARG;
  if (n <= 0 || (n & 255)) return FP4_ERR_SHAPE;
  if (!aligned(W, 32) || !aligned(G, 32) || !aligned(m_codes, 16) || !aligned(m_scales, 16) ||
      !aligned(v_codes, 16) || !aligned(v_scales, 16) || !aligned(v_means, 16))
    return FP4_ERR_ALIGNMENT;
  const DeviceInfo* d;
  fp4_status rc = check_common(&d);
  if (rc != FP4_OK) return rc;
  ProfScope ps(FP4_PROF_ADAMW, stream);
  const AdamwConsts k = adamw_consts(params->lr, params->beta1, params->beta2, params->eps, params->weight_decay,
                                     params->step, params->seed);
  return launch_adamw_update(W, G, n, k, (params->flags & FP4_MOM_FLAG_SR) != 0, m_codes, m_scales, v_codes, v_scales,
                             v_means, stream) == cudaSuccess
             ? FP4_OK
             : FP4_ERR_CUDA;
}

fp4_status fp4_momentum_decode(const uint8_t* codes, const uint16_t* scales, int64_t rows, int64_t cols,
                               float* M_out, cudaStream_t stream) {
  if (!codes || !scales || !M_out) return FP4_ERR_INVALID_ARG;
  if (rows <= 0 || cols <= 0 || (cols & 15)) return FP4_ERR_SHAPE;
  if (!aligned(codes, 16) || !aligned(scales, 16) || !aligned(M_out, 32)) return FP4_ERR_ALIGNMENT;
  const DeviceInfo* d;
  fp4_status rc = check_common(&d);
  if (rc != FP4_OK) return rc;
  return launch_momentum_decode(codes, scales, rows, cols, M_out, d->sms, stream) == cudaSuccess ? FP4_OK
                                                                                                 : FP4_ERR_CUDA;
}

fp4_status fp4_root_coeffs(int64_t m, int64_t n, int steps, float abc[3]) {
  if (m <= 0 || n <= 0 || steps < 0 || !abc) return FP4_ERR_INVALID_ARG;
  coeffs(m, n, abc);
  return FP4_OK;
}

fp4_status fp4_root_ns_workspace_layout(int64_t m, int64_t n, int steps, uint32_t flags, fp4_ws_layout* layout) {
  if (!layout || (flags & ~kNsFlags)) return FP4_ERR_INVALID_ARG;
  fp4_ns_params p;
  default_params(&p);
  p.flags = flags;
  NsPlan pl;
  fp4_status rc = make_plan(m, n, steps, &p, 1, &pl);
  if (rc != FP4_OK) return rc;
  *layout = pl.lay;
  return FP4_OK;
}

size_t fp4_root_ns_workspace_bytes(int64_t m, int64_t n, int steps, uint32_t flags) {
  fp4_ws_layout L;
  if (fp4_root_ns_workspace_layout(m, n, steps, flags, &L) != FP4_OK) return 0;
  return L.total;
}

fp4_status fp4_root_ns(const float* G, float* out, int64_t m, int64_t n, int steps, const fp4_ns_params* p,
                       void* ws, size_t ws_bytes, cudaStream_t stream) {
  fp4_ns_params dp;
  if (!p) { default_params(&dp); p = &dp; }
  if (!G || !out || !ws || (p->flags & ~kNsFlags)) return FP4_ERR_INVALID_ARG;
  if (!ns_shape_ok(m) || !ns_shape_ok(n)) return FP4_ERR_SHAPE;
  if (steps < 0 || steps > kMaxSteps) return FP4_ERR_INVALID_ARG;
  if (!aligned(G, 16) || !aligned(out, 16) || !aligned(ws, 256)) return FP4_ERR_ALIGNMENT;
  const size_t need = fp4_root_ns_workspace_bytes(m, n, steps, p->flags);
  if (need == 0 || ws_bytes < need) return FP4_ERR_WORKSPACE;
  const DeviceInfo* d;
  fp4_status rc = check_common(&d);
  if (rc != FP4_OK) return rc;
  return run_one(d, G, out, m, n, steps, p, static_cast<uint8_t*>(ws), true, stream);
}

// The second stream of a batched call with FP4_FLAG_OVERLAP_GROUPS, one per host thread and device,
// created on first use.
struct SideStream {
  int dev = -1;
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr;
};
SideStream* side_stream(int dev) {
  thread_local SideStream t;
  if (t.stream && t.dev == dev) return &t;
  if (t.stream) {   // the thread moved to another device
    cudaEventDestroy(t.fork); cudaEventDestroy(t.join); cudaStreamDestroy(t.stream);
    t = SideStream();
  }
  if (cudaStreamCreateWithFlags(&t.stream, cudaStreamNonBlocking) != cudaSuccess) { t = SideStream(); return nullptr; }
  if (cudaEventCreateWithFlags(&t.fork, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&t.join, cudaEventDisableTiming) != cudaSuccess) {
    cudaStreamDestroy(t.stream);
    t = SideStream();
    return nullptr;
  }
  t.dev = dev;
  return &t;
}

// Batched workspace: one workspace per matrix (the stages of equal-shape matrices run in
// lockstep, so none can be shared).
size_t fp4_root_ns_batched_workspace_bytes(int count, const int64_t* m, const int64_t* n, int steps,
                                           uint32_t flags) {
  if (count <= 0 || !m || !n) return 0;
  size_t need = 0;
  for (int i = 0; i < count; ++i) {
    size_t b = fp4_root_ns_workspace_bytes(m[i], n[i], steps, flags);
    if (b == 0) return 0;
    need += align_up(b, 1024);
  }
  return need;
}

fp4_status fp4_root_ns_batched(int count, const float* const* G, float* const* out, const int64_t* m,
                               const int64_t* n, int steps, const fp4_ns_params* p, void* ws, size_t ws_bytes,
                               cudaStream_t stream) {
  fp4_ns_params dp;
  if (!p) { default_params(&dp); p = &dp; }
  if (count < 0 || (count > 0 && (!G || !out || !m || !n)) || !ws || (p->flags & ~kNsFlags)) return FP4_ERR_INVALID_ARG;
  if (steps < 0 || steps > kMaxSteps) return FP4_ERR_INVALID_ARG;
  if (!aligned(ws, 256)) return FP4_ERR_ALIGNMENT;
  for (int i = 0; i < count; ++i) {
    if (!G[i] || !out[i]) return FP4_ERR_INVALID_ARG;
    if (!ns_shape_ok(m[i]) || !ns_shape_ok(n[i])) return FP4_ERR_SHAPE;
    if (!aligned(G[i], 16) || !aligned(out[i], 16)) return FP4_ERR_ALIGNMENT;
  }
  if (count == 0) return FP4_OK;
  const size_t need = fp4_root_ns_batched_workspace_bytes(count, m, n, steps, p->flags);
  if (need == 0 || ws_bytes < need) return FP4_ERR_WORKSPACE;
  const DeviceInfo* d;
  fp4_status rc = check_common(&d);
  if (rc != FP4_OK) return rc;

  uint8_t* base = static_cast<uint8_t*>(ws);
  std::vector<MatrixCtx> ctx((size_t)count);
  size_t off = 0;
  for (int i = 0; i < count; ++i) {
    rc = prepare_matrix(d, G[i], out[i], m[i], n[i], steps, p, base + off, &ctx[(size_t)i]);
    if (rc != FP4_OK) return rc;
    if (p->top_hist) ctx[(size_t)i].hist_top = p->top_hist[i];
    if (p->weights) ctx[(size_t)i].W = p->weights[i];
    off += align_up(ctx[(size_t)i].pl.lay.total, 1024);
  }
  uint32_t* status = reinterpret_cast<uint32_t*>(base);  // header of the first matrix

  // Matrices of one shape form a group whose stages run as single launches over all of
  // them (many tiles per launch: no idle SMs in a last partial wave, the two CTAs of an SM
  // fall out of step so that main loops and epilogues overlap).  A group is split when it
  // exceeds max_group matrices, which bounds the working set competing for L2.
  const int cap = p->max_group > 0 && (int)p->max_group < kPackMax ? (int)p->max_group : kDefaultMaxGroup;
  std::vector<char> done((size_t)count, 0);
  std::vector<std::vector<MatrixCtx>> groups;
  for (int i = 0; i < count; ++i) {
    if (done[(size_t)i]) continue;
    groups.emplace_back();
    std::vector<MatrixCtx>& group = groups.back();
    for (int j = i; j < count && (int)group.size() < cap; ++j) {
      if (done[(size_t)j]) continue;
      if (ctx[(size_t)j].pl.s0 == ctx[(size_t)i].pl.s0 && ctx[(size_t)j].pl.l0 == ctx[(size_t)i].pl.l0) {
        group.push_back(ctx[(size_t)j]);
        done[(size_t)j] = 1;
      }
    }
  }
  // Groups do not depend on one another.  On request (FP4_FLAG_OVERLAP_GROUPS) they alternate between the
  // caller's stream and a second one that forks from it and joins it again before the call returns: every
  // launch is a persistent grid that ends in a partial wave of tiles, and the next launch of the same
  // group cannot start before it has drained - a launch of another group can.  (Not while stage times
  // are being collected: the event pairs of the two streams would overlap.)
  SideStream* side = (p->flags & FP4_FLAG_OVERLAP_GROUPS) && groups.size() >= 2 && g_prof_on.load() == 0
                         ? side_stream((int)(d - g_dev)) : nullptr;
  if (side) {
    // the status word is cleared once, before the fork (a group's own clearing kernel could wipe what
    // a kernel of the other group has just reported)
    if (cudaMemsetAsync(status, 0, 4, stream) != cudaSuccess || cudaEventRecord(side->fork, stream) != cudaSuccess ||
        cudaStreamWaitEvent(side->stream, side->fork, 0) != cudaSuccess)
      return FP4_ERR_CUDA;
  }
  for (size_t gi = 0; gi < groups.size(); ++gi) {
    cudaStream_t st = (side && (gi & 1)) ? side->stream : stream;
    rc = run_group(d, groups[gi].data(), (int)groups[gi].size(), steps, p, status, !side && gi == 0, st);
    if (rc != FP4_OK) break;
  }
  if (side) {
    if (cudaEventRecord(side->join, side->stream) != cudaSuccess || cudaStreamWaitEvent(stream, side->join, 0) != cudaSuccess)
      return FP4_ERR_CUDA;
  }
  return rc;
}

fp4_status fp4_last_device_status(const void* ws, cudaStream_t stream) {
  if (!ws) return FP4_ERR_INVALID_ARG;
  uint32_t word = 0;
  if (cudaMemcpyAsync(&word, ws, 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return FP4_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return FP4_ERR_CUDA;
  return word == 0 ? FP4_OK : (fp4_status)word;
}

static fp4_status gemm_nt_impl(int dry, const uint8_t* a_codes, const uint8_t* a_scales, float a_tensor_scale,
                       const uint8_t* b_codes, const uint8_t* b_scales, float b_tensor_scale, int64_t M, int64_t N,
                       int64_t K, float* D, uint32_t* device_status, cudaStream_t stream) {
  pdl_select(INT64_MAX);  // a single product: plain launch
  if (!a_codes || !a_scales || !b_codes || !b_scales || !D) return FP4_ERR_INVALID_ARG;
  if (!shape_ok(M) || !shape_ok(N) || !shape_ok(K)) return FP4_ERR_SHAPE;
  if (!aligned(a_codes, 16) || !aligned(a_scales, 16) || !aligned(b_codes, 16) || !aligned(b_scales, 16) ||
      !aligned(D, 16))
    return FP4_ERR_ALIGNMENT;
  const DeviceInfo* d;
  fp4_status rc = check_common(&d);
  if (rc != FP4_OK) return rc;
  ProblemPack pack;
  memset(&pack, 0, sizeof(pack));
  GemmProblem& pr = pack.p[0];
  const bool pair = pair_kernel(M / 128, N / 128, K, d->sms);
  const int sk = pair ? gemm_pair_stage_k(kPlain) : gemm_stage_k();
  if (!make_codes_map(d, &pr.tmA, a_codes, M, K / 2, sk) || !make_codes_map(d, &pr.tmB, b_codes, N, K / 2, sk) ||
      !make_f32_map(d, &pr.tmOut, D, M, N, pair ? 32 : 128) || !make_sf_map(d, &pr.tmSfa, a_scales, M, K, sk) ||
      !make_sf_map(d, &pr.tmSfb, b_scales, N, K, sk))
    return FP4_ERR_CUDA;
  pr.tmAux = pr.tmOut;
  pr.sfa = a_scales; pr.sfb = b_scales;
  pr.sg_a = a_tensor_scale; pr.sg_b = b_tensor_scale;
  pr.out_rows = (int)M; pr.out_cols = (int)N;
  GemmLaunch L;
  memset(&L, 0, sizeof(L));
  L.num_problems = 1;
  L.K = (int)K; L.tiles_m = (int)(M / 128); L.tiles_n = (int)(N / 128);
  L.status = device_status;
  L.dry_operands = dry;
  if (dry && !pair_kernel(L.tiles_m, L.tiles_n, L.K, d->sms)) return FP4_ERR_SHAPE;
  return launch_gemm_auto(kPlain, pack, L, d->sms, stream) == cudaSuccess ? FP4_OK : FP4_ERR_CUDA;
}

fp4_status fp4_gemm_nt(const uint8_t* a_codes, const uint8_t* a_scales, float a_tensor_scale,
                       const uint8_t* b_codes, const uint8_t* b_scales, float b_tensor_scale, int64_t M, int64_t N,
                       int64_t K, float* D, uint32_t* device_status, cudaStream_t stream) {
  return gemm_nt_impl(0, a_codes, a_scales, a_tensor_scale, b_codes, b_scales, b_tensor_scale, M, N, K, D, device_status,
                      stream);
}

fp4_status fp4_gemm_nt_resident(const uint8_t* a_codes, const uint8_t* a_scales, float a_tensor_scale,
                                const uint8_t* b_codes, const uint8_t* b_scales, float b_tensor_scale, int64_t M,
                                int64_t N, int64_t K, float* D, uint32_t* device_status, cudaStream_t stream) {
  return gemm_nt_impl(1, a_codes, a_scales, a_tensor_scale, b_codes, b_scales, b_tensor_scale, M, N, K, D, device_status,
                      stream);
}

}  // extern "C"

// ---- fp4_selftest_bounded_wait ----------------------------------------------------------------
namespace fp4 {
static __global__ void __launch_bounds__(32) k_selftest_wait(uint32_t* status, uint64_t limit_ns) {
  __shared__ uint64_t bar_seen, bar_never;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    fp4::mbar_init(&bar_seen, 1);
    fp4::mbar_init(&bar_never, 1);
    abort_flag = 0;
    fp4::mbar_fence_init();
  }
  __syncwarp();
  if (threadIdx.x == 1) fp4::mbar_arrive(&bar_seen);
  if (threadIdx.x == 0) {
    const bool first = fp4::wait_bar(&bar_seen, 0, &abort_flag);                 // lane 1 arrives: must succeed
    const bool second = fp4::wait_limited(&bar_never, 0, &abort_flag, limit_ns);  // nobody arrives: must give up
    *status = (first && !second && abort_flag == 1) ? (uint32_t)FP4_ERR_DEVICE_TIMEOUT : (uint32_t)FP4_ERR_INVALID_ARG;
  }
}
}  // namespace fp4

extern "C" fp4_status fp4_selftest_bounded_wait(uint32_t* device_status, uint32_t limit_us, cudaStream_t stream) {
  if (!device_status || limit_us < 1 || limit_us > 100000) return FP4_ERR_INVALID_ARG;
  const fp4::DeviceInfo* d;
  fp4_status rc = fp4::check_common(&d);
  if (rc != FP4_OK) return rc;
  fp4::count_launches(1);
  fp4::k_selftest_wait<<<1, 32, 0, stream>>>(device_status, (uint64_t)limit_us * 1000ull);
  return cudaGetLastError() == cudaSuccess ? FP4_OK : FP4_ERR_CUDA;
}

// ---- fp4_root_ns_static: the step with the workspace in a static device array ------------
// For callers that cannot allocate device memory (no cudaMalloc allowed where they run, or
// no pool to take a workspace from).  The array is part of the module image: every device
// that loads the library holds these 16 MiB until the process ends.  In host code the
// array's name stands for the symbol, it is not a device address; the address is looked up
// with cudaGetSymbolAddress, with the caller's device current, and handed to the kernels like
// any workspace.
namespace {
static __device__ __align__(256) unsigned char g_static_scratch[FP4_STATIC_SCRATCH_BYTES];

// Device address of the static array on the current device.  Looked up on every call: the lookup is a
// table read once the module is loaded, allocates nothing, and stays right if the context was torn
// down and rebuilt in between (a cached address would not).
fp4_status static_scratch_address(void** ptr) {
  void* p = nullptr;
  if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return FP4_ERR_CUDA;
  *ptr = p;
  return FP4_OK;
}
}  // namespace

extern "C" {

fp4_status fp4_root_ns_static(const float* G, float* out, int64_t m, int64_t n, int steps, const fp4_ns_params* p,
                              uint32_t* device_status, cudaStream_t stream) {
  fp4_ns_params dp;
  if (!p) { default_params(&dp); p = &dp; }
  if (!G || !out || (p->flags & ~kNsFlags)) return FP4_ERR_INVALID_ARG;
  if (!ns_shape_ok(m) || !ns_shape_ok(n)) return FP4_ERR_SHAPE;
  if (steps < 0 || steps > kMaxSteps) return FP4_ERR_INVALID_ARG;
  if (!aligned(G, 16) || !aligned(out, 16) || (device_status && !aligned(device_status, 4))) return FP4_ERR_ALIGNMENT;
  const size_t need = fp4_root_ns_workspace_bytes(m, n, steps, p->flags);
  if (need == 0) return FP4_ERR_SHAPE;
  if (need > FP4_STATIC_SCRATCH_BYTES) return FP4_ERR_STATIC_LIMIT;
  const DeviceInfo* d;
  fp4_status rc = check_common(&d);
  if (rc != FP4_OK) return rc;
  void* scratch = nullptr;
  rc = static_scratch_address(&scratch);
  if (rc != FP4_OK) return rc;
  // run_one clears the header, the scalars and the histogram of the shared array itself
  rc = run_one(d, G, out, m, n, steps, p, static_cast<uint8_t*>(scratch), true, stream);
  if (rc != FP4_OK) return rc;
  if (device_status &&
      cudaMemcpyAsync(device_status, scratch, 4, cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
    return FP4_ERR_CUDA;
  return FP4_OK;
}

void fp4_profile_enable(int on) { g_prof_on.store(on ? 1 : 0); }

fp4_status fp4_profile_collect(float* ms, int* groups) {
  if (!ms || !groups) return FP4_ERR_INVALID_ARG;
  for (int i = 0; i < FP4_PROF_CLASSES; ++i) { ms[i] = 0.0f; groups[i] = 0; }
  std::lock_guard<std::mutex> lock(g_prof_mu);
  fp4_status rc = FP4_OK;
  for (const ProfRec& r : g_prof) {
    float t = 0.0f;
    if (cudaEventSynchronize(r.e1) != cudaSuccess || cudaEventElapsedTime(&t, r.e0, r.e1) != cudaSuccess)
      rc = FP4_ERR_CUDA;
    if (r.cls >= 0 && r.cls < FP4_PROF_CLASSES) { ms[r.cls] += t; groups[r.cls] += 1; }
    cudaEventDestroy(r.e0);
    cudaEventDestroy(r.e1);
  }
  g_prof.clear();
  return rc;
}

uint64_t fp4_kernel_launches(void) { return g_launches.load(); }

}  // extern "C"
