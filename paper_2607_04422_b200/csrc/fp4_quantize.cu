// fp4_quantize: standalone NVFP4 block quantiser (Section 2, "NVFP4 format"), and the
// transposing copy that returns the result of a tall input.
#include "fp4_kernels.h"

namespace fp4 {

// ----------------------------------------------------------------------------------
// amax over a tensor: 128-bit loads (four independent ones in flight per thread), warp
// shuffle reduction, one atomicMax per block on the bit pattern (non-negative floats order
// like unsigned integers).
// ----------------------------------------------------------------------------------
__device__ __forceinline__ float amax4(float4 v) {
  return fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w)));
}

__global__ void __launch_bounds__(256) k_amax(const float4* __restrict__ x, int64_t n4, uint32_t* amax_bits) {
  float m = 0.0f;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  for (; i + 3 * stride < n4; i += 4 * stride) {
    const float4 a = __ldg(x + i), b = __ldg(x + i + stride), c = __ldg(x + i + 2 * stride),
                 d = __ldg(x + i + 3 * stride);
    m = fmaxf(m, fmaxf(fmaxf(amax4(a), amax4(b)), fmaxf(amax4(c), amax4(d))));
  }
  for (; i < n4; i += stride) m = fmaxf(m, amax4(__ldg(x + i)));
#pragma unroll
  for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  __shared__ float wm[8];
  if ((threadIdx.x & 31) == 0) wm[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int w = 1; w < 8; ++w) m = fmaxf(m, wm[w]);
    atomicMax(amax_bits, __float_as_uint(m));
  }
}

// ----------------------------------------------------------------------------------
// Row quantiser: one thread per block of 16 (four 128-bit loads = 64 contiguous bytes, a warp
// covers 512 consecutive elements of a row), so the two IEEE divisions of a block are done
// once; 8-byte code store and 1-byte scale store per thread.  Thread blocks walk the tensor
// from its end: the amax pass has just read it front to back, so the end is what L2 still
// holds.  grid: rows x ceil(cols / 4096) thread blocks.
// amax_bits holds the tensor amax on entry (bit pattern).
// ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_quantize_rows(const float* __restrict__ x, int64_t rows, int64_t cols,
                                                       uint8_t* __restrict__ codes, uint8_t* __restrict__ scales,
                                                       const uint32_t* __restrict__ amax_bits) {
  const float sg = scale_exact(__uint_as_float(*amax_bits));
  const float six_sg = __fmul_rn(6.0f, sg);
  const int64_t groups = ((cols >> 4) + 255) / 256;  // thread blocks per row
  const int64_t bid = (int64_t)gridDim.x - 1 - blockIdx.x;
  const int64_t r = bid / groups;
  const int64_t kb = (bid % groups) * 256 + threadIdx.x;
  if (r >= rows || kb >= (cols >> 4)) return;
  const float4* src = reinterpret_cast<const float4*>(x + r * cols + kb * 16);
  float v[16];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float4 t = __ldg(src + j);
    v[4 * j] = t.x; v[4 * j + 1] = t.y; v[4 * j + 2] = t.z; v[4 * j + 3] = t.w;
  }
  uint32_t lo, hi;
  const uint32_t sb = quantize_block16(v, six_sg, sg, lo, hi);
  *reinterpret_cast<uint2*>(codes + r * (cols / 2) + kb * 8) = make_uint2(lo, hi);
  scales[sf_offset(r, kb, cols >> 4)] = (uint8_t)sb;
}

__global__ void k_finish_tensor_scale(float* ts, float widen) {
  *ts = scale_exact(__fmul_rn(widen, *ts));  // amax (bit pattern of a float) -> s_g
}

// Row quantiser with the paper-faithful options (Section 3.4): one thread per block of 16
// (the transform and the two candidate encodings are local to a block), a warp covers 512
// consecutive elements of a row.  grid: rows x ceil(cols / 4096) thread blocks, row-major.
__global__ void __launch_bounds__(256) k_quantize_rows_opts(const float* __restrict__ x, int64_t rows, int64_t cols,
                                                            uint8_t* __restrict__ codes, uint8_t* __restrict__ scales,
                                                            const uint32_t* __restrict__ amax_bits,
                                                            const QuantOpts q) {
  const float sg = scale_exact(__fmul_rn(q.widen, __uint_as_float(*amax_bits)));
  const int64_t groups = ((cols >> 4) + 255) / 256;  // thread blocks per row
  const int64_t bid = (int64_t)gridDim.x - 1 - blockIdx.x;  // from the end, as k_quantize_rows
  const int64_t r = bid / groups;
  const int64_t kb = (bid % groups) * 256 + threadIdx.x;
  if (r >= rows || kb >= (cols >> 4)) return;
  const float4* src = reinterpret_cast<const float4*>(x + r * cols + kb * 16);
  float v[16];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float4 t = __ldg(src + j);
    v[4 * j] = t.x; v[4 * j + 1] = t.y; v[4 * j + 2] = t.z; v[4 * j + 3] = t.w;
  }
  uint32_t lo, hi;
  float unused;
  const uint32_t sb = quantize_block16_opts(v, q, sg, lo, hi, unused);
  *reinterpret_cast<uint2*>(codes + r * (cols / 2) + kb * 8) = make_uint2(lo, hi);
  scales[sf_offset(r, kb, cols >> 4)] = (uint8_t)sb;
}

// out (l0 x s0) = the leading s0 x l0 part of X^T, X being s x l (row pitch l): 64 x 64 tiles through
// shared memory, 128-bit loads along the rows of X and 128-bit stores along the rows of out
// (s0 and l0 are multiples of 16, so a 16-byte piece is all inside or all outside).
__global__ void __launch_bounds__(256) k_transpose_out(const float* __restrict__ X, int64_t l, float* __restrict__ out,
                                                       int64_t s0, int64_t l0, const ParamUpdate upd) {
  __shared__ float t[64][65];
  pdl_launch_dependents();
  pdl_wait();
  const int64_t r0 = (int64_t)blockIdx.y * 64, c0 = (int64_t)blockIdx.x * 64;  // tile origin in X
  const int q = threadIdx.x & 15, row = threadIdx.x >> 4;                      // 16 pieces per row, 16 rows per sweep
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int r = row + 16 * j;
    const float4 v = __ldg(reinterpret_cast<const float4*>(X + (r0 + r) * l + c0) + q);  // inside the padded work matrix
    t[r][4 * q] = v.x; t[r][4 * q + 1] = v.y; t[r][4 * q + 2] = v.z; t[r][4 * q + 3] = v.w;
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int c = row + 16 * j;  // column of X = row of out
    if (c0 + c < l0 && r0 + 4 * q < s0) {
      const int64_t at = (c0 + c) * s0 + r0 + 4 * q;
      const float4 o = make_float4(t[4 * q][c], t[4 * q + 1][c], t[4 * q + 2][c], t[4 * q + 3][c]);
      if (!(upd.W && upd.no_out)) *reinterpret_cast<float4*>(out + at) = o;
      if (upd.W) {
        // Root's parameter update from the values on their way out (the parameter has the caller's
        // orientation, like `out`)
        uint2* wp = reinterpret_cast<uint2*>(upd.W + at);
        const uint2 w = *wp;
        *wp = make_uint2(cvt_bf16x2(param_update_value(bf16_lo(w.x), o.x, upd.decay, upd.step),
                                    param_update_value(bf16_hi(w.x), o.y, upd.decay, upd.step)),
                         cvt_bf16x2(param_update_value(bf16_lo(w.y), o.z, upd.decay, upd.step),
                                    param_update_value(bf16_hi(w.y), o.w, upd.decay, upd.step)));
      }
    }
  }
}

// W <- update(W, O) elementwise, 8 elements per thread
__global__ void __launch_bounds__(256) k_param_update(const float* __restrict__ O, int64_t n8, const ParamUpdate upd) {
  pdl_launch_dependents();
  pdl_wait();
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n8; i += (int64_t)gridDim.x * blockDim.x) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(O) + 2 * i), b = __ldg(reinterpret_cast<const float4*>(O) + 2 * i + 1);
    uint4* wp = reinterpret_cast<uint4*>(upd.W) + i;
    const uint4 w = *wp;
    *wp = make_uint4(cvt_bf16x2(param_update_value(bf16_lo(w.x), a.x, upd.decay, upd.step),
                                param_update_value(bf16_hi(w.x), a.y, upd.decay, upd.step)),
                     cvt_bf16x2(param_update_value(bf16_lo(w.y), a.z, upd.decay, upd.step),
                                param_update_value(bf16_hi(w.y), a.w, upd.decay, upd.step)),
                     cvt_bf16x2(param_update_value(bf16_lo(w.z), b.x, upd.decay, upd.step),
                                param_update_value(bf16_hi(w.z), b.y, upd.decay, upd.step)),
                     cvt_bf16x2(param_update_value(bf16_lo(w.w), b.z, upd.decay, upd.step),
                                param_update_value(bf16_hi(w.w), b.w, upd.decay, upd.step)));
  }
}

// ----------------------------------------------------------------------------------
// host launchers
// ----------------------------------------------------------------------------------
static int grid_for(int64_t n4, int threads, int sms) {
  int64_t blocks = (n4 + threads - 1) / threads;
  int64_t cap = (int64_t)sms * 8;
  return (int)(blocks < cap ? (blocks < 1 ? 1 : blocks) : cap);
}

cudaError_t launch_quantize(const float* x, int64_t rows, int64_t cols, uint8_t* codes, uint8_t* scales,
                            float* tensor_scale, const QuantOpts& q, int sms, cudaStream_t st) {
  const int64_t n4 = rows * cols / 4;
  cudaError_t e = cudaMemsetAsync(tensor_scale, 0, 4, st);
  if (e != cudaSuccess) return e;
  k_amax<<<grid_for(n4, 256 * 8, sms), 256, 0, st>>>(reinterpret_cast<const float4*>(x), n4,
                                                    reinterpret_cast<uint32_t*>(tensor_scale));
  const unsigned qgrid = (unsigned)(((cols / 16 + 255) / 256) * rows);
  if (q.rht || q.four_six)
    k_quantize_rows_opts<<<qgrid, 256, 0, st>>>(x, rows, cols, codes, scales,
                                                reinterpret_cast<const uint32_t*>(tensor_scale), q);
  else
    k_quantize_rows<<<qgrid, 256, 0, st>>>(x, rows, cols, codes, scales,
                                           reinterpret_cast<const uint32_t*>(tensor_scale));
  k_finish_tensor_scale<<<1, 1, 0, st>>>(tensor_scale, q.widen);
  count_launches(3);
  return cudaGetLastError();
}

cudaError_t launch_transpose_out(const float* X, int64_t s, int64_t l, float* out, int64_t s0, int64_t l0,
                                 const ParamUpdate& upd, cudaStream_t st) {
  dim3 grid((unsigned)((l0 + 63) / 64), (unsigned)((s0 + 63) / 64));
  (void)s;
  count_launches(1);
  launch_chained(k_transpose_out, grid, dim3(256), 0, st, X, l, out, s0, l0, upd);
  return cudaGetLastError();
}

// n is a multiple of 256 (both dimensions are multiples of 16)
cudaError_t launch_param_update(const float* O, int64_t n, const ParamUpdate& upd, int sms, cudaStream_t st) {
  if (!upd.W) return cudaSuccess;
  count_launches(1);
  launch_chained(k_param_update, dim3(grid_for(n / 8, 256, sms)), dim3(256), 0, st, O, n / 8, upd);
  return cudaGetLastError();
}

}  // namespace fp4
