// Shared device helpers of the NVFP4 Root Newton-Schulz library (sm_100a only):
// NVFP4 codecs on the hardware conversion instructions, the scale-factor atom
// layout, and thin wrappers over mbarrier / TMA / tcgen05 PTX.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/fp4root.h"

namespace fp4 {

// ----------------------------------------------------------------------------------
// NVFP4 format (Section 2, "NVFP4 format")
// ----------------------------------------------------------------------------------

// Offset of the E4M3 scale of (row r, block kb) in the 128-row x 4-block atom layout
// read by the block-scaled MMA; kblocks = row length / 16.
__host__ __device__ inline size_t sf_offset(int64_t r, int64_t kb, int64_t kblocks) {
  return (size_t)(((r >> 7) * (kblocks >> 2) + (kb >> 2)) * 512 + (r & 31) * 16 +
                  ((r & 127) >> 5) * 4 + (kb & 3));
}

// Two FP32 -> one byte of two E2M1 codes, `lo` in bits 3:0 and `hi` in bits 7:4,
// round to nearest even, saturating.
__device__ __forceinline__ uint32_t cvt_e2m1x2(float lo, float hi) {
  uint32_t r;
  asm("{\n\t.reg .b8 t;\n\tcvt.rn.satfinite.e2m1x2.f32 t, %1, %2;\n\tcvt.u32.u8 %0, t;\n\t}"
      : "=r"(r)
      : "f"(hi), "f"(lo));
  return r;
}

// FP32 (>= 0) -> unsigned E4M3 byte, round to nearest even, saturating at 448.
__device__ __forceinline__ uint32_t cvt_ue4m3(float t) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(0.0f), "f"(t));
  return (uint32_t)(r & 0xFF);
}

// E4M3 byte (sign bit clear) -> FP32, exact.
__device__ __forceinline__ float ue4m3_to_float(uint32_t b) {
  uint32_t e = (b >> 3) & 0xF, m = b & 7;
  // subnormal: m * 2^-9; normal: (8+m) * 2^(e-10)
  return e == 0 ? (float)m * 0.001953125f : __uint_as_float(((e + 120) << 23) | (m << 20));
}

// Tensor scale rules.  Exact: amax / 2688 (6 * 448).  Predicted: the smallest power of
// two >= bound / 2688.
__device__ __forceinline__ float scale_exact(float amax) {
  return amax == 0.0f ? 1.0f : __fdiv_rn(amax, 2688.0f);
}
__device__ __forceinline__ float scale_predicted(float bound) {
  if (!(bound > 0.0f)) return 1.0f;
  float v = __fdiv_rn(bound, 2688.0f);
  uint32_t u = __float_as_uint(v);
  uint32_t e = u >> 23, mant = u & 0x7FFFFF;
  if (e == 0) return __uint_as_float(1u << 23);      // below the normal range: 2^-126
  if (mant != 0) e += 1;
  return __uint_as_float(e << 23);
}

// Quantise one block of 16 values that share an E4M3 scale.  Returns the scale byte,
// writes the 8 code bytes as two 32-bit words (element 0 in the lowest nibble).
__device__ __forceinline__ uint32_t quantize_block16(const float (&v)[16], float six_sg, float sg,
                                                     uint32_t& lo, uint32_t& hi) {
  float amax = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(v[i]));
  uint32_t sb = cvt_ue4m3(__fdiv_rn(amax, six_sg));
  float d = __fmul_rn(ue4m3_to_float(sb), sg);
  lo = 0; hi = 0;
  if (d != 0.0f) {
    float rcp = __frcp_rn(d);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      lo |= cvt_e2m1x2(__fmul_rn(v[2 * i], rcp), __fmul_rn(v[2 * i + 1], rcp)) << (8 * i);
      hi |= cvt_e2m1x2(__fmul_rn(v[8 + 2 * i], rcp), __fmul_rn(v[9 + 2 * i], rcp)) << (8 * i);
    }
  }
  return sb;
}

// Packed FP32 pairs: sm_100 multiplies two FP32 lanes per instruction, each lane rounded to
// nearest like the scalar operation.  Only used where the product feeds a conversion: a packed
// multiply followed by a packed add was seen to be contracted into a fused multiply-add, which
// changes the rounding the method defines.
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t r, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(r));
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// d = a * b + c per lane, one rounding (what the scalar fused multiply-add gives)
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
// Four FP32 -> two bytes of E2M1 codes (a in bits 3:0, b in 7:4, c in 11:8, d in 15:12).
__device__ __forceinline__ uint32_t cvt_e2m1x4(float a, float b, float c, float d) {
  uint32_t r;
  asm("{\n\t.reg .b8 t0, t1;\n\t.reg .b16 h;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 t0, %2, %1;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 t1, %4, %3;\n\t"
      "mov.b16 h, {t0, t1};\n\t"
      "cvt.u32.u16 %0, h;\n\t}"
      : "=r"(r)
      : "f"(a), "f"(b), "f"(c), "f"(d));
  return r;
}

// Eight FP32 -> four bytes of E2M1 codes (v0 in bits 3:0 ... v7 in bits 31:28).
__device__ __forceinline__ uint32_t cvt_e2m1x8(float v0, float v1, float v2, float v3, float v4, float v5, float v6,
                                               float v7) {
  uint32_t r;
  asm("{\n\t.reg .b8 t0, t1, t2, t3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 t0, %2, %1;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 t1, %4, %3;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 t2, %6, %5;\n\t"
      "cvt.rn.satfinite.e2m1x2.f32 t3, %8, %7;\n\t"
      "mov.b32 %0, {t0, t1, t2, t3};\n\t}"
      : "=r"(r)
      : "f"(v0), "f"(v1), "f"(v2), "f"(v3), "f"(v4), "f"(v5), "f"(v6), "f"(v7));
  return r;
}

// The same quantisation when the tensor scale is a power of two (every tensor produced
// inside the Newton-Schulz loop), with the two IEEE divisions replaced by exact equivalents:
//   amax / (6 sg)  = RN(amax / 6) * (1/sg): the division by the constant 6 is one multiply
//     and two fused multiply-adds (quotient, exact remainder, correction), which gives the
//     correctly rounded quotient; the scaling by a power of two is exact;
//   1 / (s sg): s has 3 mantissa bits, so the correctly rounded reciprocal is one of eight
//     constants with the exponent shifted.
// inv_sg = 1/sg; rcp_base = (7 - log2 sg) << 23.  Also returns the block's amax.
__constant__ uint32_t kRcpMantissa[8] = {0x3F800000u, 0x3F638E39u, 0x3F4CCCCDu, 0x3F3A2E8Cu,
                                         0x3F2AAAABu, 0x3F1D89D9u, 0x3F124925u, 0x3F088889u};
__device__ __forceinline__ uint32_t quantize_block16_pow2(const float (&v)[16], float sg, float inv_sg,
                                                          uint32_t rcp_base, uint32_t& lo, uint32_t& hi,
                                                          float& amax_out) {
  float m8[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) m8[i] = fmaxf(fabsf(v[2 * i]), fabsf(v[2 * i + 1]));
  const float amax = fmaxf(fmaxf(fmaxf(m8[0], m8[1]), fmaxf(m8[2], m8[3])),
                           fmaxf(fmaxf(m8[4], m8[5]), fmaxf(m8[6], m8[7])));
  amax_out = amax;
  const float sixth = 0.16666667163372039794921875f;  // RN(1/6)
  float q = __fmul_rn(amax, sixth);
  const float r = __fmaf_rn(-q, 6.0f, amax);
  q = __fmaf_rn(r, sixth, q);                          // RN(amax / 6)
  const uint32_t sb = cvt_ue4m3(__fmul_rn(q, inv_sg));
  const uint32_t e = sb >> 3;
  // scale bytes below 8 (E4M3 subnormals, zero included) are rare: keep their division out of
  // the common path of the warp
  float rcp = __uint_as_float(kRcpMantissa[sb & 7] + rcp_base - (e << 23));
  if (__any_sync(0xffffffffu, e == 0)) {
    if (e == 0) rcp = sb ? __frcp_rn(__fmul_rn(ue4m3_to_float(sb), sg)) : 0.0f;
  }
  // y = v * rcp, two lanes per instruction; an all-zero block (rcp = 0) gets codes 0 with the
  // sign bits of its elements cleared below
  const uint64_t rcp2 = pack2(rcp, rcp);
  float z[16];
#pragma unroll
  for (int i = 0; i < 8; ++i) unpack2(mul2(pack2(v[2 * i], v[2 * i + 1]), rcp2), z[2 * i], z[2 * i + 1]);
  lo = cvt_e2m1x8(z[0], z[1], z[2], z[3], z[4], z[5], z[6], z[7]);
  hi = cvt_e2m1x8(z[8], z[9], z[10], z[11], z[12], z[13], z[14], z[15]);
  if (sb == 0) { lo = 0; hi = 0; }
  return sb;
}
// rcp_base of a power-of-two tensor scale
__device__ __forceinline__ uint32_t rcp_base_of(float sg) {
  const int esg = (int)(__float_as_uint(sg) >> 23) - 127;
  return (uint32_t)(7 - esg) << 23;
}

// ----------------------------------------------------------------------------------
// Paper-faithful quantiser options (Section 3.4): a random Hadamard transform of every
// 16-block along the contraction axis, and adaptive 4/6 block scaling.
// ----------------------------------------------------------------------------------
struct QuantOpts {
  uint32_t rht;       // 1: multiply each block by diag(signs) H_16 / 4 before quantising
  uint32_t mask;      // bit i set: element i of a block is negated
  uint32_t four_six;  // 1: try the max->4 mapping too, keep the smaller squared error
  float widen;        // factor on the amax bounds of predicted tensor scales: 4 with rht, else 1
};

// One byte of two E2M1 codes -> two FP32 values (x = low nibble), exact.
__device__ __forceinline__ float2 e2m1x2_to_float2(uint32_t byte) {
  uint32_t h2;
  asm("{\n\t.reg .b8 t;\n\tcvt.u8.u32 t, %1;\n\tcvt.rn.f16x2.e2m1x2 %0, t;\n\t}" : "=r"(h2) : "r"(byte));
  float2 f;
  asm("{\n\t.reg .f16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.f32.f16 %0, a;\n\tcvt.f32.f16 %1, b;\n\t}"
      : "=f"(f.x), "=f"(f.y)
      : "r"(h2));
  return f;
}

// v <- v diag(signs) H_16 / 4 in FP32: signs, the natural-order butterfly (strides 1, 2, 4, 8;
// sum to the lower index, difference to the upper), then the factor 1/4.  The stride-1 stage runs on
// scalars, the strides 2, 4, 8 and the factor on packed pairs (v[2k], v[2k+1]): every lane is the same
// single rounded operation as in a scalar butterfly, and no product meets a sum that could absorb it.
__device__ __forceinline__ void hadamard16(float (&v)[16], uint32_t mask) {
  uint64_t p[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const float a = __uint_as_float(__float_as_uint(v[2 * k]) ^ (((mask >> (2 * k)) & 1u) << 31));
    const float b = __uint_as_float(__float_as_uint(v[2 * k + 1]) ^ (((mask >> (2 * k + 1)) & 1u) << 31));
    p[k] = pack2(__fadd_rn(a, b), __fsub_rn(a, b));
  }
#pragma unroll
  for (int h = 1; h < 8; h *= 2) {
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      if ((k & h) == 0) {
        const uint64_t a = p[k], b = p[k + h];
        p[k] = add2(a, b);
        p[k + h] = sub2(a, b);
      }
    }
  }
  const uint64_t q = pack2(0.25f, 0.25f);
#pragma unroll
  for (int k = 0; k < 8; ++k) unpack2(mul2(p[k], q), v[2 * k], v[2 * k + 1]);
}

// Codes of one block for the scale byte sb; returns the sum of the squared FP32 errors,
// accumulated in element order (the 4/6 choice compares two such sums, so the order of the
// roundings is part of the definition).  Products are taken two at a time; every subtraction and
// every addition of the error sum stays a scalar operation, so none can fuse with a product.
__device__ __forceinline__ float encode_block16(const float (&v)[16], uint32_t sb, float sg, uint32_t& lo,
                                                uint32_t& hi) {
  const float d = __fmul_rn(ue4m3_to_float(sb), sg);
  lo = 0; hi = 0;
  float err = 0.0f;
  if (d == 0.0f) {
#pragma unroll
    for (int i = 0; i < 16; ++i) err = __fadd_rn(err, __fmul_rn(v[i], v[i]));
    return err;
  }
  const float rcp = __frcp_rn(d);
  const uint64_t rcp2 = pack2(rcp, rcp), d2 = pack2(d, d);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    float y0, y1, p0, p1, s0, s1;
    unpack2(mul2(pack2(v[2 * i], v[2 * i + 1]), rcp2), y0, y1);
    const uint32_t byte = cvt_e2m1x2(y0, y1);
    const float2 q = e2m1x2_to_float2(byte);
    unpack2(mul2(pack2(q.x, q.y), d2), p0, p1);
    const float d0 = __fsub_rn(v[2 * i], p0), d1 = __fsub_rn(v[2 * i + 1], p1);
    const uint64_t dd = pack2(d0, d1);
    unpack2(mul2(dd, dd), s0, s1);
    err = __fadd_rn(err, s0);
    err = __fadd_rn(err, s1);
    if (i < 4) lo |= byte << (8 * i); else hi |= byte << (8 * (i - 4));
  }
  return err;
}

// The same two functions with scalar operations only (fewer live registers: G3's epilogue, which
// quantises every block twice, is faster with these; the results are the same bit for bit).
// v <- v diag(signs) H_16 / 4 in FP32: signs, the natural-order butterfly (strides 1, 2, 4, 8;
// sum to the lower index, difference to the upper), then the factor 1/4.
__device__ __forceinline__ void hadamard16_scalar(float (&v)[16], uint32_t mask) {
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = (mask >> i) & 1 ? -v[i] : v[i];
#pragma unroll
  for (int h = 1; h < 16; h *= 2) {
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      if ((j & h) == 0) {
        const float a = v[j], b = v[j + h];
        v[j] = __fadd_rn(a, b);
        v[j + h] = __fsub_rn(a, b);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __fmul_rn(v[i], 0.25f);
}

// Codes of one block for the scale byte sb; returns the sum of the squared FP32 errors,
// accumulated in element order (the 4/6 choice compares two such sums, so the order of the
// roundings is part of the definition).
__device__ __forceinline__ float encode_block16_scalar(const float (&v)[16], uint32_t sb, float sg, uint32_t& lo,
                                                uint32_t& hi) {
  const float d = __fmul_rn(ue4m3_to_float(sb), sg);
  lo = 0; hi = 0;
  float err = 0.0f;
  if (d == 0.0f) {
#pragma unroll
    for (int i = 0; i < 16; ++i) err = __fadd_rn(err, __fmul_rn(v[i], v[i]));
    return err;
  }
  const float rcp = __frcp_rn(d);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const uint32_t byte = cvt_e2m1x2(__fmul_rn(v[2 * i], rcp), __fmul_rn(v[2 * i + 1], rcp));
    const float2 q = e2m1x2_to_float2(byte);
    const float d0 = __fsub_rn(v[2 * i], __fmul_rn(q.x, d));
    err = __fadd_rn(err, __fmul_rn(d0, d0));
    const float d1 = __fsub_rn(v[2 * i + 1], __fmul_rn(q.y, d));
    err = __fadd_rn(err, __fmul_rn(d1, d1));
    if (i < 4) lo |= byte << (8 * i); else hi |= byte << (8 * (i - 4));
  }
  return err;
}

// Quantise one block with the options above; any tensor scale.  v is transformed in place.
// Returns the scale byte; amax_in is the block's amax before the transform (what the
// predicted tensor scales of the next stage are derived from).  PACKED selects the form of the
// transform and of the error sums (same results).
template <bool PACKED = true>
__device__ __forceinline__ uint32_t quantize_block16_opts(float (&v)[16], const QuantOpts& q, float sg, uint32_t& lo,
                                                          uint32_t& hi, float& amax_in) {
  float a = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; ++i) a = fmaxf(a, fabsf(v[i]));
  amax_in = a;
  if (q.rht) {
    if (PACKED) hadamard16(v, q.mask); else hadamard16_scalar(v, q.mask);
    a = 0.0f;
#pragma unroll
    for (int i = 0; i < 16; ++i) a = fmaxf(a, fabsf(v[i]));
  }
  uint32_t sb = cvt_ue4m3(__fdiv_rn(a, __fmul_rn(6.0f, sg)));
  const float err6 = PACKED ? encode_block16(v, sb, sg, lo, hi) : encode_block16_scalar(v, sb, sg, lo, hi);
  if (q.four_six) {
    const uint32_t sb4 = cvt_ue4m3(__fdiv_rn(a, __fmul_rn(4.0f, sg)));
    uint32_t lo4, hi4;
    const float err4 = PACKED ? encode_block16(v, sb4, sg, lo4, hi4) : encode_block16_scalar(v, sb4, sg, lo4, hi4);
    if (err4 < err6) { sb = sb4; lo = lo4; hi = hi4; }
  }
  return sb;
}

// ----------------------------------------------------------------------------------
// BF16 storage of the high-precision copies (round to nearest even)
// ----------------------------------------------------------------------------------
// two FP32 -> one word of two BF16 (lo in bits 15:0)
__device__ __forceinline__ uint32_t cvt_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// ----------------------------------------------------------------------------------
// status word
// ----------------------------------------------------------------------------------
__device__ __forceinline__ void report_timeout(uint32_t* status) {
  if (status) atomicMax(status, (uint32_t)FP4_ERR_DEVICE_TIMEOUT);
}

// ----------------------------------------------------------------------------------
// PTX wrappers
// ----------------------------------------------------------------------------------
// Programmatic dependent launch.  Every kernel of a Newton-Schulz call lets the next launch of the stream
// start early (its blocks become resident as soon as this grid's blocks have all started and resources are
// free) and itself waits, after its set-up and before it touches global memory, until the launch before it
// has completed and its writes are visible.  Every kernel waits unconditionally, so completion stays
// transitive along the stream.  Both are no-ops for a kernel launched without the attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait: gives up after `kSpinLimit` polls or when another thread of the CTA has
// raised the abort flag; returns false then.
constexpr uint32_t kSpinLimit = 1u << 26;
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 255u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void tma_prefetch_desc(const void* tmap) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tmap) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const void* tmap, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%2, %3}], [%4];" ::"r"(smem_u32(smem_dst)),
      "l"(tmap), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void bulk_load_1d(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(smem_dst)),
      "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_store_2d(const void* tmap, int x, int y, const void* smem_src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];" ::"l"(
                   tmap),
               "r"(x), "r"(y), "r"(smem_u32(smem_src))
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_all() {
  asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}

// named barrier among `count` threads
__device__ __forceinline__ void bar_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// ---- tcgen05 ------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// smem -> TMEM copy of one 512-byte scale-factor atom (32 rows x 16 bytes, replicated to
// the four 32-lane quadrants)
__device__ __forceinline__ void tc_cp_sf(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, E2M1 operands with one UE4M3 scale per 16 elements
__device__ __forceinline__ void tc_mma_nvf4(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.block16 [%0], %1, %2, %3, [%5], [%6], p;\n\t}" ::"r"(
          d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
      : "memory");
}
// arrive on an mbarrier when all MMAs issued so far by this thread have completed
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                   smem_u32(bar))
               : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns -> 16 registers per thread (lane = row)
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// The same load without the wait: the registers must not be read before tc_wait_ld16 has
// been given them (it names them as operands so that their uses are ordered after it).
__device__ __forceinline__ void tc_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_wait_ld16(uint32_t (&r)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]),
                 "+r"(r[15])
               :
               : "memory");
}

// Shared-memory matrix descriptor of a K-major operand tile whose rows are `row_bytes`
// long (64 or 128) and swizzled by TMA with the matching mode; 8-row groups are
// 8*row_bytes apart.  layout: 2 = 128-byte swizzle, 4 = 64-byte swizzle, 0 = none.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t sbo_bytes, uint32_t layout) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
  d |= (uint64_t)1 << 16;                         // leading byte offset: unused for these layouts
  d |= (uint64_t)(sbo_bytes >> 4) << 32;
  d |= (uint64_t)1 << 46;                         // descriptor version of sm_100
  d |= (uint64_t)layout << 61;
  return d;
}

}  // namespace fp4
