// fp4_quantize: standalone NVFP4 block quantiser (Section 2, "NVFP4 format"), and the
// prologue of the Root step: outlier clip (nearest-rank quantile of |G| by radix
// select), Frobenius normalisation, and the first pair of NVFP4 operand copies
// (Section 3.4: qX = Q_1x16(X), qX^{16x1} = Q_16x1(X)).
#include "fp4_kernels.h"

namespace fp4 {

// ----------------------------------------------------------------------------------
// amax over a tensor: 128-bit loads, warp shuffle reduction, one atomicMax per block on
// the bit pattern (non-negative floats order like unsigned integers).
// ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_amax(const float4* __restrict__ x, int64_t n4, uint32_t* amax_bits) {
  float m = 0.0f;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
    float4 v = __ldg(x + i);
    m = fmaxf(fmaxf(m, fmaxf(fabsf(v.x), fabsf(v.y))), fmaxf(fabsf(v.z), fabsf(v.w)));
  }
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
// Row quantiser.  Four neighbouring lanes own one block of 16 elements (one float4
// each): block amax by two xor-shuffles, the 8 code bytes and the 4 scale bytes of a
// 64-element group are gathered by shuffles so that each store is 8 or 4 bytes wide.
// amax_bits holds the tensor amax on entry (bit pattern).
// ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_quantize_rows(const float4* __restrict__ x, int64_t rows, int64_t cols,
                                                       uint8_t* __restrict__ codes, uint8_t* __restrict__ scales,
                                                       const uint32_t* __restrict__ amax_bits) {
  const float sg = scale_exact(__uint_as_float(*amax_bits));
  const float six_sg = __fmul_rn(6.0f, sg);
  const int64_t n4 = rows * cols / 4;
  const int64_t c4 = cols / 4;
  const int lane = threadIdx.x & 31;
  // n4 is a multiple of 32*... (cols multiple of 128): whole warps stay in range together
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
    float4 v = __ldg(x + i);
    float a = fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w)));
    a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 1));
    a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, 2));
    uint32_t sb = cvt_ue4m3(__fdiv_rn(a, six_sg));
    float d = __fmul_rn(ue4m3_to_float(sb), sg);
    uint32_t w = 0;
    if (d != 0.0f) {
      float rcp = __frcp_rn(d);
      w = cvt_e2m1x2(__fmul_rn(v.x, rcp), __fmul_rn(v.y, rcp)) |
          (cvt_e2m1x2(__fmul_rn(v.z, rcp), __fmul_rn(v.w, rcp)) << 8);
    }
    // codes: 4 lanes x 16 bits -> one 8-byte store by the first lane of the block
    uint32_t w2 = w | (__shfl_down_sync(0xffffffffu, w, 1) << 16);
    uint32_t w3 = __shfl_down_sync(0xffffffffu, w2, 2);
    // scales: 4 blocks (16 lanes) -> one 4-byte store
    uint32_t s2 = sb | (__shfl_down_sync(0xffffffffu, sb, 4) << 8);
    uint32_t s4 = s2 | (__shfl_down_sync(0xffffffffu, s2, 8) << 16);
    int64_t r = i / c4;
    int64_t cb = (i - r * c4) >> 2;  // block index in the row
    if ((lane & 3) == 0) {
      *reinterpret_cast<uint2*>(codes + (i >> 2) * 8) = make_uint2(w2, w3);
    }
    if ((lane & 15) == 0) {
      *reinterpret_cast<uint32_t*>(scales + sf_offset(r, cb, cols >> 4)) = s4;
    }
  }
}

__global__ void k_finish_tensor_scale(float* ts) {
  *ts = scale_exact(*ts);  // amax (bit pattern of a float) -> s_g
}

// ----------------------------------------------------------------------------------
// Outlier clip: nearest-rank quantile of |G| by a three-pass radix select over the 31
// magnitude bits (11 + 11 + 9).  Header words used: sel_prefix, sel_rank.
// ----------------------------------------------------------------------------------
template <int SHIFT, int BITS>
__global__ void __launch_bounds__(512) k_radix_hist(const float4* __restrict__ g, int64_t n4, const NsHeader* hdr,
                                                    uint32_t* __restrict__ hist) {
  constexpr int NB = 1 << BITS;
  __shared__ uint32_t sh[NB];
  for (int i = threadIdx.x; i < NB; i += blockDim.x) sh[i] = 0;
  __syncthreads();
  const uint32_t prefix = hdr->sel_prefix;
  constexpr uint32_t HIGH_MASK = (SHIFT + BITS >= 31) ? 0u : (0x7FFFFFFFu >> (SHIFT + BITS)) << (SHIFT + BITS);
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
    float4 v = __ldg(g + i);
    uint32_t k[4] = {__float_as_uint(v.x) & 0x7FFFFFFFu, __float_as_uint(v.y) & 0x7FFFFFFFu,
                     __float_as_uint(v.z) & 0x7FFFFFFFu, __float_as_uint(v.w) & 0x7FFFFFFFu};
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if ((k[j] & HIGH_MASK) == prefix) atomicAdd(&sh[(k[j] >> SHIFT) & (NB - 1)], 1u);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < NB; i += blockDim.x)
    if (sh[i]) atomicAdd(&hist[i], sh[i]);
}

__global__ void k_select_init(NsHeader* hdr, uint32_t rank) {
  hdr->sel_prefix = 0;
  hdr->sel_rank = rank;
}

// One block: find the bin that holds the element of rank hdr->sel_rank (1-based, counted
// from the smallest), extend the prefix, reduce the rank, clear the histogram.
template <int SHIFT, int BITS>
__global__ void __launch_bounds__(256) k_radix_pick(NsHeader* hdr, uint32_t* __restrict__ hist, float* scalars,
                                                    int idx_tau) {
  constexpr int NB = 1 << BITS;
  constexpr int PER = (NB + 255) / 256;
  __shared__ uint32_t part[256];
  uint32_t local[PER];
  uint32_t sum = 0;
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    int b = threadIdx.x * PER + j;
    local[j] = b < NB ? hist[b] : 0u;
    sum += local[j];
  }
  part[threadIdx.x] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t run = 0;
    for (int i = 0; i < 256; ++i) { uint32_t t = part[i]; part[i] = run; run += t; }
  }
  __syncthreads();
  const uint32_t rank = hdr->sel_rank;
  uint32_t before = part[threadIdx.x];
  __syncthreads();
  if (rank > before && rank <= before + sum) {
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      if (rank > before && rank <= before + local[j]) {
        uint32_t b = threadIdx.x * PER + j;
        uint32_t np = hdr->sel_prefix | (b << SHIFT);
        hdr->sel_prefix = np;
        hdr->sel_rank = rank - before;
        if (SHIFT == 0) scalars[idx_tau] = __uint_as_float(np);
      }
      before += local[j];
    }
  }
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    int b = threadIdx.x * PER + j;
    if (b < NB) hist[b] = 0;
  }
}

// ----------------------------------------------------------------------------------
// Sum of squares of the clamped input (FP64), and max |g|.  One partial per block,
// combined in a fixed order by k_norm_finish so that the result is reproducible.
// ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_clamp_stats(const float4* __restrict__ g, int64_t n4, const float* scalars,
                                                     int idx_tau, int clip, double* __restrict__ partial,
                                                     uint32_t* maxabs_bits) {
  const float tau = clip ? scalars[idx_tau] : __int_as_float(0x7f800000);
  double acc = 0.0;
  float mx = 0.0f;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
    float4 v = __ldg(g + i);
    float c[4] = {fminf(fabsf(v.x), tau), fminf(fabsf(v.y), tau), fminf(fabsf(v.z), tau), fminf(fabsf(v.w), tau)};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      acc += (double)c[j] * (double)c[j];
      mx = fmaxf(mx, c[j]);
    }
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    acc += __shfl_xor_sync(0xffffffffu, acc, o);
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }
  __shared__ double wa[8];
  __shared__ float wm[8];
  if ((threadIdx.x & 31) == 0) { wa[threadIdx.x >> 5] = acc; wm[threadIdx.x >> 5] = mx; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) { acc += wa[w]; mx = fmaxf(mx, wm[w]); }
    partial[blockIdx.x] = acc;
    atomicMax(maxabs_bits, __float_as_uint(mx));
  }
}

__global__ void __launch_bounds__(256) k_norm_finish(const double* __restrict__ partial, int nparts, NsHeader* hdr,
                                                     float* scalars, NsScalarIdx ix, float eps) {
  __shared__ double sh[256];
  double acc = 0.0;
  for (int i = threadIdx.x; i < nparts; i += 256) acc += partial[i];
  sh[threadIdx.x] = acc;
  __syncthreads();
  for (int o = 128; o; o >>= 1) {
    if ((int)threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    float nu = (float)sqrt(sh[0]);
    float inv = __fdiv_rn(1.0f, __fadd_rn(nu, eps));
    float amax0 = __fmul_rn(__uint_as_float(hdr->maxabs_bits), inv);  // max |clamped g| * inv
    scalars[ix.nu] = nu;
    scalars[ix.inv] = inv;
    scalars[ix.amax_X0] = amax0;
    scalars[ix.sg_X0] = scale_exact(amax0);
  }
}

// ----------------------------------------------------------------------------------
// X0 = clamp(G) * inv in the work orientation (s x l; transposed when G is tall), its
// FP32 copy, and both NVFP4 operand copies.  One 128 x 128 tile of X per block.
// ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_prep_operands(const float* __restrict__ G, int64_t ldg, int tall,
                                                       const float* scalars, NsScalarIdx ix, int clip,
                                                       float* __restrict__ X, int64_t s, int64_t l,
                                                       uint8_t* __restrict__ qx_codes, uint8_t* __restrict__ qx_sf,
                                                       uint8_t* __restrict__ qt_codes, uint8_t* __restrict__ qt_sf,
                                                       int write_q) {
  extern __shared__ float xs[];  // [128][129]
  constexpr int P = 129;
  const float tau = clip ? scalars[ix.tau] : __int_as_float(0x7f800000);
  const float inv = scalars[ix.inv];
  const float sg = scalars[ix.sg_X0];
  const float six_sg = __fmul_rn(6.0f, sg);
  const int64_t r0 = (int64_t)blockIdx.y * 128, c0 = (int64_t)blockIdx.x * 128;  // tile origin in X
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  // load: coalesced along G's rows
  for (int rr = warp; rr < 128; rr += 8) {
    // G row: tall -> row (c0+rr), columns r0..; else row (r0+rr), columns c0..
    const float* src = tall ? G + (c0 + rr) * ldg + r0 : G + (r0 + rr) * ldg + c0;
    float4 v = __ldg(reinterpret_cast<const float4*>(src) + lane);
    float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float c = fminf(fmaxf(e[j], -tau), tau);
      float xv = __fmul_rn(c, inv);
      int cc = lane * 4 + j;
      if (tall) xs[cc * P + rr] = xv; else xs[rr * P + cc] = xv;
    }
  }
  __syncthreads();
  // FP32 copy of X0
  for (int rr = warp; rr < 128; rr += 8) {
    float4 v = make_float4(xs[rr * P + lane * 4], xs[rr * P + lane * 4 + 1], xs[rr * P + lane * 4 + 2],
                           xs[rr * P + lane * 4 + 3]);
    *reinterpret_cast<float4*>(X + (r0 + rr) * l + c0 + lane * 4) = v;
  }
  if (!write_q) return;
  if (warp < 4) {
    // blocks along the columns of X (contraction axis of G1): thread = row
    const int rr = warp * 32 + lane;
    uint32_t sfw[2] = {0, 0};
#pragma unroll
    for (int kb = 0; kb < 8; ++kb) {
      float v[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) v[i] = xs[rr * P + kb * 16 + i];
      uint32_t lo, hi;
      uint32_t sb = quantize_block16(v, six_sg, sg, lo, hi);
      *reinterpret_cast<uint2*>(qx_codes + (r0 + rr) * (l / 2) + (c0 + kb * 16) / 2) = make_uint2(lo, hi);
      sfw[kb >> 2] |= sb << (8 * (kb & 3));
    }
    *reinterpret_cast<uint32_t*>(qx_sf + sf_offset(r0 + rr, c0 / 16, l / 16)) = sfw[0];
    *reinterpret_cast<uint32_t*>(qx_sf + sf_offset(r0 + rr, c0 / 16 + 4, l / 16)) = sfw[1];
  } else {
    // blocks along the rows of X (contraction axis of G3): thread = column of X = row of X^T
    const int cc = (warp - 4) * 32 + lane;
    uint32_t sfw[2] = {0, 0};
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      float v[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) v[i] = xs[(g * 16 + i) * P + cc];
      uint32_t lo, hi;
      uint32_t sb = quantize_block16(v, six_sg, sg, lo, hi);
      *reinterpret_cast<uint2*>(qt_codes + (c0 + cc) * (s / 2) + (r0 + g * 16) / 2) = make_uint2(lo, hi);
      sfw[g >> 2] |= sb << (8 * (g & 3));
    }
    *reinterpret_cast<uint32_t*>(qt_sf + sf_offset(c0 + cc, r0 / 16, s / 16)) = sfw[0];
    *reinterpret_cast<uint32_t*>(qt_sf + sf_offset(c0 + cc, r0 / 16 + 4, s / 16)) = sfw[1];
  }
}

// out (m x n, m > n) = X^T where X is n x m: 32 x 32 tiles through shared memory
__global__ void __launch_bounds__(256) k_transpose_out(const float* __restrict__ X, int64_t s, int64_t l,
                                                       float* __restrict__ out) {
  __shared__ float t[32][33];
  const int64_t r0 = (int64_t)blockIdx.y * 32, c0 = (int64_t)blockIdx.x * 32;  // in X (s x l)
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int j = ty; j < 32; j += 8) t[j][tx] = X[(r0 + j) * l + c0 + tx];
  __syncthreads();
  for (int j = ty; j < 32; j += 8) out[(c0 + j) * s + r0 + tx] = t[tx][j];
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
                            float* tensor_scale, int sms, cudaStream_t st) {
  const int64_t n4 = rows * cols / 4;
  cudaError_t e = cudaMemsetAsync(tensor_scale, 0, 4, st);
  if (e != cudaSuccess) return e;
  k_amax<<<grid_for(n4, 256 * 4, sms), 256, 0, st>>>(reinterpret_cast<const float4*>(x), n4,
                                                    reinterpret_cast<uint32_t*>(tensor_scale));
  k_quantize_rows<<<grid_for(n4, 256 * 2, sms), 256, 0, st>>>(reinterpret_cast<const float4*>(x), rows, cols, codes,
                                                            scales, reinterpret_cast<const uint32_t*>(tensor_scale));
  k_finish_tensor_scale<<<1, 1, 0, st>>>(tensor_scale);
  count_launches(3);
  return cudaGetLastError();
}

cudaError_t launch_prologue(const float* G, int64_t m, int64_t n, const NsPlan& pl, uint8_t* ws, float* X,
                            int write_q, bool clear_status, cudaStream_t st) {
  NsHeader* hdr = reinterpret_cast<NsHeader*>(ws + pl.lay.header);
  float* scalars = reinterpret_cast<float*>(ws + pl.lay.scalars);
  uint32_t* hist = reinterpret_cast<uint32_t*>(ws + pl.off_hist);
  double* partial = reinterpret_cast<double*>(ws + pl.off_partial);
  const int64_t N = m * n, n4 = N / 4;
  const float4* g4 = reinterpret_cast<const float4*>(G);
  // header (all of it, or all but the status word), scalars and histogram start from zero
  const size_t skip = clear_status ? 0 : 16;
  cudaError_t e = cudaMemsetAsync(ws + pl.lay.header + skip, 0, pl.zero_bytes - skip, st);
  if (e != cudaSuccess) return e;
  if (pl.clip) {
    ProfScope ps(FP4_PROF_CLIP, st);
    count_launches(7);
    k_select_init<<<1, 1, 0, st>>>(hdr, (uint32_t)pl.clip_rank);
    const int gh = grid_for(n4, 512 * 4, pl.sms);
    k_radix_hist<20, 11><<<gh, 512, 0, st>>>(g4, n4, hdr, hist);
    k_radix_pick<20, 11><<<1, 256, 0, st>>>(hdr, hist, scalars, pl.ix.tau);
    k_radix_hist<9, 11><<<gh, 512, 0, st>>>(g4, n4, hdr, hist);
    k_radix_pick<9, 11><<<1, 256, 0, st>>>(hdr, hist, scalars, pl.ix.tau);
    k_radix_hist<0, 9><<<gh, 512, 0, st>>>(g4, n4, hdr, hist);
    k_radix_pick<0, 9><<<1, 256, 0, st>>>(hdr, hist, scalars, pl.ix.tau);
  }
  {
    ProfScope ps(FP4_PROF_STATS, st);
    count_launches(2);
    k_clamp_stats<<<pl.stat_blocks, 256, 0, st>>>(g4, n4, scalars, pl.ix.tau, pl.clip, partial, &hdr->maxabs_bits);
    k_norm_finish<<<1, 256, 0, st>>>(partial, pl.stat_blocks, hdr, scalars, pl.ix, pl.eps);
  }
  const int tall = m > n;
  dim3 grid((unsigned)(pl.l / 128), (unsigned)(pl.s / 128));
  ProfScope ps(FP4_PROF_PREP, st);
  count_launches(1);
  k_prep_operands<<<grid, 256, 128 * 129 * 4, st>>>(G, n, tall, scalars, pl.ix, pl.clip, X, pl.s, pl.l,
                                                    ws + pl.lay.qX_codes, ws + pl.lay.qX_scales,
                                                    ws + pl.lay.qXt_codes[0], ws + pl.lay.qXt_scales[0], write_q);
  return cudaGetLastError();
}

cudaError_t launch_transpose_out(const float* X, int64_t s, int64_t l, float* out, cudaStream_t st) {
  dim3 grid((unsigned)(l / 32), (unsigned)(s / 32));
  count_launches(1);
  k_transpose_out<<<grid, 256, 0, st>>>(X, s, l, out);
  return cudaGetLastError();
}

cudaError_t prologue_set_attributes() {
  return cudaFuncSetAttribute(k_prep_operands, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 129 * 4);
}

}  // namespace fp4
