// Packed AdamW step with both moments kept in NVFP4 states (Section 3.3): BF16 weights and
// gradients, a 5-bit first moment (Hadamard, adaptive 4/6, BF16 block scales, optional
// stochastic rounding) and a 5.0625-bit second moment (square root, BF16 mean per tile of 256,
// Hadamard, adaptive 4/6, BF16 block scales); no FP32 master weight.  42.0625 bits per parameter
// in memory; one pass reads and writes all of it: 8.516 bytes of HBM traffic per parameter.
//
// A tensor is a flat array whose length is a multiple of 256.  One thread per block of 16
// elements, 16 consecutive threads per tile: the tile mean is the only value that crosses
// threads (four shuffles).  Per element, in FP32, single rounded operations:
//   m = b1 m' + (1-b1) g                 v = b2 v' + (1-b2) g g          s = sqrt(v)
//   den = s * rsb2 + eps                 w1 = w * decay                  w2 = w1 - step_size * (m / den)
// with m', v' decoded from the states, bc1 = 1 - b1^t, rsb2 = 1 / sqrt(1 - b2^t),
// step_size = lr / bc1, decay = 1 - lr * wd; W = BF16(w2), to nearest even.

#include <cmath>

#include "fp4_state.cuh"
#include "fp4_kernels.h"

namespace fp4 {

namespace {

__device__ __forceinline__ void ld_u32x8(const uint16_t* p, uint32_t* v) {
  asm volatile("ld.global.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
               : "l"(p)
               : "memory");
}
__device__ __forceinline__ void ldg_u32x8(const uint16_t* p, uint32_t* v) {
  asm volatile("ld.global.nc.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
               : "l"(p));
}
__device__ __forceinline__ void st_u32x8(uint16_t* p, const uint32_t* v) {
  asm volatile("st.global.v8.u32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(v[0]), "r"(v[1]), "r"(v[2]),
               "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
               : "memory");
}

// The two-candidate nearest-rounding encoding of a transformed block (no stochastic rounding).
__device__ __forceinline__ void state_encode_rtn(const float (&h)[16], uint2& c, uint32_t& scale_bits) {
  float amax = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(h[i]));
  const uint32_t w = cvt_bf16x2(__fdiv_rn(amax, 6.0f), __fdiv_rn(amax, 4.0f));
  uint32_t lo, hi, lo4, hi4;
  const float err6 = mom_encode_rtn(h, bf16_lo(w), lo, hi);
  const float err4 = mom_encode_rtn(h, bf16_hi(w), lo4, hi4);
  scale_bits = w & 0xFFFFu;
  if (err4 < err6) { scale_bits = w >> 16; lo = lo4; hi = hi4; }
  c = make_uint2(lo, hi);
}

// grid: ceil(nblocks / 256) thread blocks of 256 threads; nblocks is a multiple of 16, so the 16
// lanes of a tile are all inside or all outside (outside lanes still take part in the shuffles).
template <bool SR>
__global__ void __launch_bounds__(256) k_adamw_update(uint16_t* W, const uint16_t* __restrict__ G, int64_t nblocks,
                                                      const AdamwConsts k, uint8_t* m_codes, uint16_t* m_scales,
                                                      uint8_t* v_codes, uint16_t* v_scales, uint16_t* v_means) {
  const int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const bool valid = b < nblocks;
  float m[16], s[16];
  uint32_t wq[8];
  float part = 0.0f;
  if (valid) {
    uint32_t gq[8];
    ld_u32x8(W + b * 16, wq);
    ldg_u32x8(G + b * 16, gq);
    const uint2 mc = *reinterpret_cast<const uint2*>(m_codes + b * 8);
    const uint32_t ms = m_scales[b];
    const uint2 vc = *reinterpret_cast<const uint2*>(v_codes + b * 8);
    const uint32_t vs = v_scales[b];
    const float mean_prev = __uint_as_float((uint32_t)v_means[b >> 4] << 16);
    mom_decode(mc, ms, m);   // m'
    mom_decode(vc, vs, s);   // the residual of sqrt(v')
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      float w2[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int i = 2 * j + e;
        const float g = e ? bf16_hi(gq[j]) : bf16_lo(gq[j]);
        const float w = e ? bf16_hi(wq[j]) : bf16_lo(wq[j]);
        const float u = __fadd_rn(s[i], mean_prev);
        const float vprev = __fmul_rn(u, u);
        const float mi = __fadd_rn(__fmul_rn(k.b1, m[i]), __fmul_rn(k.omb1, g));
        const float vi = __fadd_rn(__fmul_rn(k.b2, vprev), __fmul_rn(k.omb2, __fmul_rn(g, g)));
        const float si = __fsqrt_rn(vi);
        const float den = __fadd_rn(__fmul_rn(si, k.rsb2), k.eps);
        const float w1 = __fmul_rn(w, k.decay);
        w2[e] = __fsub_rn(w1, __fmul_rn(k.step_size, __fdiv_rn(mi, den)));
        m[i] = mi;
        s[i] = si;
        part = __fadd_rn(part, si);   // the block's sum of sqrt(v), in element order
      }
      wq[j] = cvt_bf16x2(w2[0], w2[1]);
    }
    st_u32x8(W + b * 16, wq);
  }
  // tile mean: pairwise tree over the 16 block sums of the tile
#pragma unroll
  for (int stride = 1; stride < 16; stride *= 2) part = __fadd_rn(part, __shfl_xor_sync(0xFFFFFFFFu, part, stride));
  if (!valid) return;
  const uint32_t mean_w = cvt_bf16x2(__fmul_rn(part, 0.00390625f), 0.0f) & 0xFFFFu;
  const float mean = __uint_as_float(mean_w << 16);
  if ((b & 15) == 0) v_means[b >> 4] = (uint16_t)mean_w;
  {
    uint2 c;
    uint32_t sc;
    mom_encode<SR>(m, k.seed, (uint64_t)b * 16, c, sc);
    *reinterpret_cast<uint2*>(m_codes + b * 8) = c;
    m_scales[b] = (uint16_t)sc;
  }
  {
#pragma unroll
    for (int i = 0; i < 16; ++i) s[i] = __fsub_rn(s[i], mean);
    hadamard16_pairs(s);
    uint2 c;
    uint32_t sc;
    state_encode_rtn(s, c, sc);
    *reinterpret_cast<uint2*>(v_codes + b * 8) = c;
    v_scales[b] = (uint16_t)sc;
  }
}

}  // namespace

AdamwConsts adamw_consts(float lr, float beta1, float beta2, float eps, float weight_decay, int step, uint64_t seed) {
  AdamwConsts k;
  k.b1 = beta1;
  k.b2 = beta2;
  k.omb1 = 1.0f - beta1;
  k.omb2 = 1.0f - beta2;
  k.eps = eps;
  const float bc1 = (float)(1.0 - std::pow((double)beta1, (double)step));
  k.rsb2 = (float)(1.0 / std::sqrt(1.0 - std::pow((double)beta2, (double)step)));
  k.step_size = lr / bc1;
  const float lrwd = lr * weight_decay;
  k.decay = 1.0f - lrwd;
  k.seed = seed;
  return k;
}

cudaError_t launch_adamw_update(uint16_t* W, const uint16_t* G, int64_t n, const AdamwConsts& k, bool sr,
                                uint8_t* m_codes, uint16_t* m_scales, uint8_t* v_codes, uint16_t* v_scales,
                                uint16_t* v_means, cudaStream_t st) {
  const int64_t nblocks = n / 16;
  const unsigned grid = (unsigned)((nblocks + 255) / 256);
  if (sr) k_adamw_update<true><<<grid, 256, 0, st>>>(W, G, nblocks, k, m_codes, m_scales, v_codes, v_scales, v_means);
  else k_adamw_update<false><<<grid, 256, 0, st>>>(W, G, nblocks, k, m_codes, m_scales, v_codes, v_scales, v_means);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace fp4
