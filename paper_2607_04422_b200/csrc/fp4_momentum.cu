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

#include "fp4_state.cuh"
#include "fp4_kernels.h"

namespace fp4 {

namespace {

constexpr int kMomBins = 8192;

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
