// First-moment momentum kept in a 5-bit NVFP4 state (Section 3.3, first-moment recipe: Hadamard
// mixing, then stochastic or nearest rounding with adaptive 4/6 scaling; Section 3.4: Root's
// momentum uses the same storage).
//
// State of a rows x cols matrix, blocks of 1x16 along the rows:
//   codes   rows x cols/2 bytes   E2M1 codes of the block times H_16 / 4 (element 2j of the
//                                 transformed block in the low nibble of byte j)
//   scales  rows x cols/16 BF16   one block scale each; no tensor scale
// The matrix is row-major with cols a multiple of 16, so block b of the whole matrix starts at
// element 16 b: the kernels are one-dimensional.
//
// One step, one thread per block, everything in registers:
//   decode   h = code * scale, m_prev = h H_16 / 4           (H_16 / 4 is its own inverse)
//   update   m = fl(fl(mu m_prev) + fl(g_scale g))
//   out      m to M_out (the Newton-Schulz input), its top 13 magnitude bits to the histogram
//            that the outlier clip's first pass would otherwise have to read M_out again for
//   encode   h = m H_16 / 4; scale candidates BF16(amax/6), BF16(amax/4); round to nearest with
//            each, keep the smaller squared error (a tie keeps 6); with stochastic rounding the
//            block is encoded again with the chosen scale by cvt.rs.satfinite.e2m1x4.f32, a
//            value going up with probability equal to its position between its two neighbours
//            on the grid (resolved to 2^-16), the random words drawn from splitmix64.
// HBM traffic per element: 4 (G) + 4 (M_out) + 2 x 5/8 (state in and out) = 9.25 bytes.

#include "fp4_common.cuh"
#include "fp4_kernels.h"

namespace fp4 {

namespace {

constexpr int kMomBins = 8192;

__device__ __forceinline__ uint64_t splitmix64_at(uint64_t seed, uint64_t idx) {
  uint64_t z = seed + 0x9E3779B97F4A7C15ull * (idx + 1);
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// Nearest-rounding codes of one transformed block for the block scale d; returns the sum of the
// squared FP32 errors in element order.
__device__ __forceinline__ float mom_encode_rtn(const float (&h)[16], float d, uint32_t& lo, uint32_t& hi) {
  lo = 0; hi = 0;
  float err = 0.0f;
  if (d == 0.0f) {
#pragma unroll
    for (int i = 0; i < 16; ++i) err = __fadd_rn(err, __fmul_rn(h[i], h[i]));
    return err;
  }
  const float rcp = __frcp_rn(d);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const uint32_t byte = cvt_e2m1x2(__fmul_rn(h[2 * i], rcp), __fmul_rn(h[2 * i + 1], rcp));
    const float2 q = e2m1x2_to_float2(byte);
    const float d0 = __fsub_rn(h[2 * i], __fmul_rn(q.x, d));
    err = __fadd_rn(err, __fmul_rn(d0, d0));
    const float d1 = __fsub_rn(h[2 * i + 1], __fmul_rn(q.y, d));
    err = __fadd_rn(err, __fmul_rn(d1, d1));
    if (i < 4) lo |= byte << (8 * i); else hi |= byte << (8 * (i - 4));
  }
  return err;
}

// Stochastic rounding of four values onto the E2M1 grid with the conversion instruction of
// sm_100a; the result holds v0 in bits 3:0 ... v3 in bits 15:12.  Measured behaviour of the
// instruction: with lo <= |v| < hi the neighbouring grid values and f = floor(65536 (|v| - lo) /
// (hi - lo)), v goes to hi when f + r >= 65536, where the 16 random bits r of the four values
// come from the bytes b3 b2 b1 b0 of the random word as
//   v0: b2 b0     v1: the same 16 bits in reverse order     v2: b3 b1     v3: those reversed.
// `w` is the word in the plain form (v0: low half, v2: high half), permuted here.
__device__ __forceinline__ uint32_t cvt_rs_e2m1x4(float v0, float v1, float v2, float v3, uint32_t w) {
  const uint32_t rbits = __byte_perm(w, 0u, 0x3120);  // b0, b2 <- low half; b1, b3 <- high half
  uint32_t r;
  asm("{\n\t.reg .b16 t;\n\tcvt.rs.satfinite.e2m1x4.f32 t, {%1, %2, %3, %4}, %5;\n\tcvt.u32.u16 %0, t;\n\t}"
      : "=r"(r)
      : "f"(v3), "f"(v2), "f"(v1), "f"(v0), "r"(rbits));
  return r;
}

__device__ __forceinline__ void mom_decode(uint2 c, uint32_t scale_bits, float (&v)[16]) {
  const float d = __uint_as_float(scale_bits << 16);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const uint32_t byte = ((i < 4 ? c.x : c.y) >> (8 * (i & 3))) & 0xFFu;
    const float2 q = e2m1x2_to_float2(byte);
    v[2 * i] = __fmul_rn(q.x, d);
    v[2 * i + 1] = __fmul_rn(q.y, d);
  }
  hadamard16(v, 0u);
}

// Encodes m (destroyed); `first` is the matrix index of the block's first element.
template <bool SR>
__device__ __forceinline__ void mom_encode(float (&h)[16], uint64_t seed, uint64_t first, uint2& c,
                                           uint32_t& scale_bits) {
  hadamard16(h, 0u);
  float amax = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(h[i]));
  const uint32_t w = cvt_bf16x2(__fdiv_rn(amax, 6.0f), __fdiv_rn(amax, 4.0f));
  const float d6 = bf16_lo(w), d4 = bf16_hi(w);
  uint32_t lo, hi, lo4, hi4;
  const float err6 = mom_encode_rtn(h, d6, lo, hi);
  const float err4 = mom_encode_rtn(h, d4, lo4, hi4);
  float d = d6;
  scale_bits = w & 0xFFFFu;
  if (err4 < err6) { d = d4; scale_bits = w >> 16; lo = lo4; hi = hi4; }
  if (SR && d != 0.0f) {
    // one generator output per 8 elements of the matrix: its low word for the first four
    const float rcp = __frcp_rn(d);
    const uint64_t z0 = splitmix64_at(seed, first >> 3), z1 = splitmix64_at(seed, (first >> 3) + 1);
    const uint32_t c0 = cvt_rs_e2m1x4(__fmul_rn(h[0], rcp), __fmul_rn(h[1], rcp), __fmul_rn(h[2], rcp),
                                      __fmul_rn(h[3], rcp), (uint32_t)z0);
    const uint32_t c1 = cvt_rs_e2m1x4(__fmul_rn(h[4], rcp), __fmul_rn(h[5], rcp), __fmul_rn(h[6], rcp),
                                      __fmul_rn(h[7], rcp), (uint32_t)(z0 >> 32));
    const uint32_t c2 = cvt_rs_e2m1x4(__fmul_rn(h[8], rcp), __fmul_rn(h[9], rcp), __fmul_rn(h[10], rcp),
                                      __fmul_rn(h[11], rcp), (uint32_t)z1);
    const uint32_t c3 = cvt_rs_e2m1x4(__fmul_rn(h[12], rcp), __fmul_rn(h[13], rcp), __fmul_rn(h[14], rcp),
                                      __fmul_rn(h[15], rcp), (uint32_t)(z1 >> 32));
    lo = c0 | (c1 << 16);
    hi = c2 | (c3 << 16);
  }
  c = make_uint2(lo, hi);
}

// 256-bit global accesses (32-byte aligned): a thread moves its block of 16 floats as two full
// 32-byte sectors, so no sector is touched by two instructions -- with 128-bit pieces at a
// 64-byte lane stride every sector is looked up twice on loads and written as two partial
// sectors on stores.
__device__ __forceinline__ void ldg_f32x8(const float* p, float* v) {
  asm volatile("ld.global.nc.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
               : "l"(p));
}
__device__ __forceinline__ void stg_f32x8(float* p, const float* v) {
  asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(v[0]), "f"(v[1]), "f"(v[2]),
               "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7])
               : "memory");
}

// grid: any number of thread blocks; threads stride over the 16-blocks of the matrix.
template <bool SR, bool HIST>
__global__ void __launch_bounds__(256) k_momentum_update(const float* __restrict__ G, int64_t nblocks, float mu,
                                                         float g_scale, uint64_t seed, uint8_t* codes,
                                                         uint16_t* scales, float* __restrict__ M_out,
                                                         uint32_t* __restrict__ hist) {
  __shared__ uint32_t sh[HIST ? kMomBins : 1];
  if (HIST) {
    for (int i = threadIdx.x; i < kMomBins; i += blockDim.x) sh[i] = 0;
    __syncthreads();
  }
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const uint64_t mu2 = pack2(mu, mu), gs2 = pack2(g_scale, g_scale);
  for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < nblocks; b += stride) {
    const uint2 c_in = *reinterpret_cast<const uint2*>(codes + b * 8);
    const uint32_t s_in = scales[b];
    float g[16], m[16];
    ldg_f32x8(G + b * 16, g);
    ldg_f32x8(G + b * 16 + 8, g + 8);
    mom_decode(c_in, s_in, m);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float a0, a1, b0, b1;
      unpack2(mul2(pack2(m[2 * i], m[2 * i + 1]), mu2), a0, a1);
      unpack2(mul2(pack2(g[2 * i], g[2 * i + 1]), gs2), b0, b1);
      m[2 * i] = __fadd_rn(a0, b0);       // scalar: the sum must not fuse with a product
      m[2 * i + 1] = __fadd_rn(a1, b1);
    }
    if (M_out) {
      stg_f32x8(M_out + b * 16, m);
      stg_f32x8(M_out + b * 16 + 8, m + 8);
    }
    if (HIST) {
#pragma unroll
      for (int i = 0; i < 16; ++i) atomicAdd(&sh[(__float_as_uint(m[i]) & 0x7FFFFFFFu) >> 18], 1u);
    }
    uint2 c_out;
    uint32_t s_out;
    mom_encode<SR>(m, seed, (uint64_t)b * 16, c_out, s_out);
    *reinterpret_cast<uint2*>(codes + b * 8) = c_out;
    scales[b] = (uint16_t)s_out;
  }
  if (HIST) {
    __syncthreads();
    for (int j = threadIdx.x; j < kMomBins; j += blockDim.x)
      if (sh[j]) atomicAdd(&hist[j], sh[j]);
  }
}

__global__ void __launch_bounds__(256) k_momentum_decode(const uint8_t* __restrict__ codes,
                                                         const uint16_t* __restrict__ scales, int64_t nblocks,
                                                         float* __restrict__ M_out) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < nblocks; b += stride) {
    float m[16];
    mom_decode(__ldg(reinterpret_cast<const uint2*>(codes + b * 8)), __ldg(scales + b), m);
    stg_f32x8(M_out + b * 16, m);
    stg_f32x8(M_out + b * 16 + 8, m + 8);
  }
}

// Without the histogram every thread block takes one group of 256 blocks.  With it a thread
// block owns 32 KB of counters that it clears and flushes once, so the grid is what fits on the
// GPU at once, shrunk so that all thread blocks run the same number of iterations.
template <bool SR, bool HIST>
cudaError_t launch_update(const float* G, int64_t nblocks, float mu, float g_scale, uint64_t seed, uint8_t* codes,
                          uint16_t* scales, float* M_out, uint32_t* hist, int sms, cudaStream_t st) {
  const int64_t units = (nblocks + 255) / 256;
  int64_t grid = units;
  if (HIST) {
    int per_sm = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_momentum_update<SR, HIST>, 256, 0);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    if (per_sm > 4) per_sm = 4;  // measured: more resident counters only add clearing and flushing
    const int64_t slots = (int64_t)sms * per_sm;
    const int64_t iters = (units + slots - 1) / slots;
    grid = (units + iters - 1) / iters;
  }
  k_momentum_update<SR, HIST><<<(unsigned)grid, 256, 0, st>>>(G, nblocks, mu, g_scale, seed, codes, scales, M_out,
                                                              hist);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_momentum_update(const float* G, int64_t rows, int64_t cols, float mu, float g_scale, bool sr,
                                   uint64_t seed, uint8_t* codes, uint16_t* scales, float* M_out, uint32_t* hist,
                                   int sms, cudaStream_t st) {
  const int64_t nblocks = rows * (cols / 16);
  if (sr) {
    return hist ? launch_update<true, true>(G, nblocks, mu, g_scale, seed, codes, scales, M_out, hist, sms, st)
                : launch_update<true, false>(G, nblocks, mu, g_scale, seed, codes, scales, M_out, hist, sms, st);
  }
  return hist ? launch_update<false, true>(G, nblocks, mu, g_scale, seed, codes, scales, M_out, hist, sms, st)
              : launch_update<false, false>(G, nblocks, mu, g_scale, seed, codes, scales, M_out, hist, sms, st);
}

cudaError_t launch_momentum_decode(const uint8_t* codes, const uint16_t* scales, int64_t rows, int64_t cols,
                                   float* M_out, int sms, cudaStream_t st) {
  const int64_t nblocks = rows * (cols / 16);
  const int64_t need = (nblocks + 255) / 256;
  const int64_t cap = (int64_t)sms * 8;
  k_momentum_decode<<<(unsigned)(need < cap ? need : cap), 256, 0, st>>>(codes, scales, nblocks, M_out);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace fp4
