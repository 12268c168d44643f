// Prologue of the Root step for a group of equal-size matrices (Section 3.4: "p99 outlier
// clipping"; normalisation; the first operand copies qX = Q_1x16(X), qX^{16x1} = Q_16x1(X)).
// Every kernel covers the whole group (gridDim.y = matrix, or a tile list over all matrices), so a
// group needs six launches instead of six per matrix.
//
// Clip threshold tau = nearest-rank quantile of |g|, found exactly with two passes over
// the data where three were needed before:
//   pass 1  histogram of the top 13 magnitude bits (exponent + 5 mantissa bits);
//   pick    the bin that holds the wanted rank;
//   pass 2  elements of that bin are appended to a candidate list (they are about 1 % of a
//           continuous distribution); in the same pass the squares of all elements below
//           the bin are summed in FP64 (they are certainly not clipped);
//   finish  one block per matrix selects tau among the candidates (two shared-memory radix
//           rounds over the remaining 18 bits), adds the candidates' squares exactly (they
//           share an exponent, so their squares add as integers) and tau^2 for every clipped
//           element, and derives nu, 1/(nu+eps), amax(X0) and the tensor scale of X0.
// If the bin holds more candidates than the list can take (many equal values, e.g. a
// constant matrix) the finishing block itself continues the radix select with two more passes
// over the matrix and a statistics pass (slow, rare, no extra launch).
#include <stddef.h>

#include "fp4_gemm_common.cuh"
#include "fp4_kernels.h"

namespace fp4 {

namespace {

constexpr int kMaxPack = 16;

struct PrepMatrix {
  const float* G;
  float* X;
  NsHeader* hdr;
  float* scalars;
  uint32_t* hist;      // 8192 counters
  uint32_t* hist_top;  // the caller's counters of the first radix pass (then pass 1 is skipped), or null
  double* partial;     // one FP64 partial per statistics block
  uint32_t* cand;      // candidate list (workspace that is unused until the first product)
  uint8_t* qx_codes; uint8_t* qx_sf;
  uint8_t* qt_codes; uint8_t* qt_sf;
  int tall;
  int clear_status;
  int store_x;
  int64_t x_rows, x_cols;  // extent and row pitch of X
};

struct PrepGroup {
  PrepMatrix mat[kMaxPack];
  int count;
  int64_t n4;          // elements of the caller's matrix / 4
  int64_t s, l;        // work shape (multiples of 128)
  int64_t s0, l0;      // the caller's short and long side; the rest of the work shape is zero padding
  int clip;
  uint32_t clip_rank;
  uint32_t cand_cap;
  float eps;
  int stat_blocks;
  int write_q;
  int zero_words;      // 32-bit words of header + scalars + histogram to clear
  QuantOpts q;         // quantiser options of X0's operand copies
  NsScalarIdx ix;
  uint32_t* status;    // the call's status word
  CUtensorMap tmG[kMaxPack];  // the callers' matrices as FP32 tensors, box = 32 columns x 128 rows, 128-byte swizzle
};

__device__ __forceinline__ uint32_t mag_bits(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

// ---- init: clear header (keeping the status word of all but the first matrix of a call),
// scalars and histogram; arm the select
__global__ void __launch_bounds__(256) kp_init(const __grid_constant__ PrepGroup g) {
  pdl_launch_dependents();
  pdl_wait();
  const PrepMatrix& m = g.mat[blockIdx.y];
  uint32_t* w = reinterpret_cast<uint32_t*>(m.hdr);
  const int first = m.clear_status ? 0 : 4;
  // the select starts with an empty prefix and the wanted rank (written instead of the zero)
  const int rank_word = (int)(offsetof(NsHeader, sel_rank) / 4);
  for (int i = first + blockIdx.x * blockDim.x + threadIdx.x; i < g.zero_words; i += gridDim.x * blockDim.x)
    w[i] = (i == rank_word) ? g.clip_rank : 0u;
}

constexpr int kTopBits = 13;                 // bits of the first radix pass
constexpr int kTopShift = 31 - kTopBits;     // 18
constexpr int kTopBins = 1 << kTopBits;      // 8192

// ---- pass 1: histogram of the top 13 magnitude bits
__global__ void __launch_bounds__(512) kp_hist_top(const __grid_constant__ PrepGroup g) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ uint32_t sh[kTopBins];
  const PrepMatrix& m = g.mat[blockIdx.y];
  if (m.hist_top) return;  // the caller counted this matrix already
  for (int i = threadIdx.x; i < kTopBins; i += blockDim.x) sh[i] = 0;
  __syncthreads();
  const float4* src = reinterpret_cast<const float4*>(m.G);
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  for (; i + stride < g.n4; i += 2 * stride) {
    const float4 v = __ldg(src + i), w = __ldg(src + i + stride);
    atomicAdd(&sh[mag_bits(v.x) >> kTopShift], 1u);
    atomicAdd(&sh[mag_bits(v.y) >> kTopShift], 1u);
    atomicAdd(&sh[mag_bits(v.z) >> kTopShift], 1u);
    atomicAdd(&sh[mag_bits(v.w) >> kTopShift], 1u);
    atomicAdd(&sh[mag_bits(w.x) >> kTopShift], 1u);
    atomicAdd(&sh[mag_bits(w.y) >> kTopShift], 1u);
    atomicAdd(&sh[mag_bits(w.z) >> kTopShift], 1u);
    atomicAdd(&sh[mag_bits(w.w) >> kTopShift], 1u);
  }
  for (; i < g.n4; i += stride) {
    const float4 v = __ldg(src + i);
    atomicAdd(&sh[mag_bits(v.x) >> kTopShift], 1u);
    atomicAdd(&sh[mag_bits(v.y) >> kTopShift], 1u);
    atomicAdd(&sh[mag_bits(v.z) >> kTopShift], 1u);
    atomicAdd(&sh[mag_bits(v.w) >> kTopShift], 1u);
  }
  __syncthreads();
  for (int j = threadIdx.x; j < kTopBins; j += blockDim.x)
    if (sh[j]) atomicAdd(&m.hist[j], sh[j]);
}

// ---- pick: the bin (of NB bins of a histogram) that holds rank hdr->sel_rank; extends the
// prefix by bin << SHIFT, reduces the rank, clears the histogram
template <int NB>
__device__ __forceinline__ void pick_bin(NsHeader* hdr, uint32_t* hist, int shift, uint32_t* bin_count_out,
                                         uint32_t* below_out) {
  constexpr int PER = NB / 256;
  static_assert(PER % 4 == 0, "a thread reads its counters as 16-byte pieces");
  __shared__ uint32_t wtot[8];
  uint32_t local[PER];
  uint32_t sum = 0;
  if ((reinterpret_cast<uintptr_t>(hist) & 15) == 0) {
#pragma unroll
    for (int j = 0; j < PER; j += 4) {
      const uint4 v = *reinterpret_cast<const uint4*>(hist + threadIdx.x * PER + j);
      local[j] = v.x; local[j + 1] = v.y; local[j + 2] = v.z; local[j + 3] = v.w;
    }
  } else {   // a caller's histogram need only be 4-byte aligned
#pragma unroll
    for (int j = 0; j < PER; ++j) local[j] = hist[threadIdx.x * PER + j];
  }
#pragma unroll
  for (int j = 0; j < PER; ++j) sum += local[j];
  // exclusive prefix of the 256 chunk sums: scan inside each warp, then add the totals of the warps before
  uint32_t incl = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
    if ((int)(threadIdx.x & 31) >= o) incl += t;
  }
  if ((threadIdx.x & 31) == 31) wtot[threadIdx.x >> 5] = incl;
  __syncthreads();
  uint32_t before = incl - sum;
  for (int w = 0; w < (int)(threadIdx.x >> 5); ++w) before += wtot[w];
  const uint32_t rank = hdr->sel_rank;
  __syncthreads();
  if (rank > before && rank <= before + sum) {
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      if (rank > before && rank <= before + local[j]) {
        hdr->sel_prefix |= (uint32_t)(threadIdx.x * PER + j) << shift;
        hdr->sel_rank = rank - before;
        if (bin_count_out) *bin_count_out = local[j];
        if (below_out) *below_out = before;
      }
      before += local[j];
    }
  }
#pragma unroll
  for (int j = 0; j < PER; ++j) hist[threadIdx.x * PER + j] = 0;
}

__global__ void __launch_bounds__(256) kp_pick_top(const __grid_constant__ PrepGroup g) {
  pdl_launch_dependents();
  pdl_wait();
  const PrepMatrix& m = g.mat[blockIdx.y];
  pick_bin<kTopBins>(m.hdr, m.hist_top ? m.hist_top : m.hist, kTopShift, &m.hdr->bin_count, &m.hdr->count_below);
}

// ---- pass 2: candidates of the picked bin, FP64 sum of squares below the bin, max |g|.
// Candidates are rare: they are collected in a shared-memory buffer per block and copied to
// the global list with one reservation per block (or directly when the buffer is full).
__global__ void __launch_bounds__(256) kp_compact_stats(const __grid_constant__ PrepGroup g) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr uint32_t kBuf = 2048;
  __shared__ uint32_t s_buf[kBuf];
  __shared__ uint32_t s_cnt, s_base;
  const PrepMatrix& m = g.mat[blockIdx.y];
  const uint32_t bin = g.clip ? (m.hdr->sel_prefix >> kTopShift) : 0xFFFFFFFFu;
  const float4* src = reinterpret_cast<const float4*>(m.G);
  const int lane = threadIdx.x & 31;
  if (threadIdx.x == 0) s_cnt = 0;
  __syncthreads();
  double acc = 0.0;
  float mx = 0.0f;
  auto visit = [&](float x) {
    const uint32_t k = mag_bits(x);
    const uint32_t kb = k >> kTopShift;
    if (kb < bin) {
      acc += (double)x * (double)x;
      mx = fmaxf(mx, __uint_as_float(k));
    } else if (kb == bin) {
      const uint32_t pos = atomicAdd(&s_cnt, 1u);
      if (pos < kBuf) {
        s_buf[pos] = k;
      } else {
        const uint32_t gpos = atomicAdd(&m.hdr->cand_count, 1u);
        if (gpos < g.cand_cap) m.cand[gpos] = k;
      }
    }
  };
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  for (; i + stride < g.n4; i += 2 * stride) {
    const float4 v = __ldg(src + i), w = __ldg(src + i + stride);
    visit(v.x); visit(v.y); visit(v.z); visit(v.w);
    visit(w.x); visit(w.y); visit(w.z); visit(w.w);
  }
  for (; i < g.n4; i += stride) {
    const float4 v = __ldg(src + i);
    visit(v.x); visit(v.y); visit(v.z); visit(v.w);
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    acc += __shfl_xor_sync(0xffffffffu, acc, o);
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }
  __shared__ double wa[8];
  __shared__ float wm[8];
  if (lane == 0) { wa[threadIdx.x >> 5] = acc; wm[threadIdx.x >> 5] = mx; }
  __syncthreads();
  const uint32_t nbuf = s_cnt < kBuf ? s_cnt : kBuf;
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) { acc += wa[w]; mx = fmaxf(mx, wm[w]); }
    m.partial[blockIdx.x] = acc;
    atomicMax(&m.hdr->maxabs_bits, __float_as_uint(mx));
    s_base = nbuf ? atomicAdd(&m.hdr->cand_count, nbuf) : 0u;
  }
  __syncthreads();
  for (uint32_t j = threadIdx.x; j < nbuf; j += blockDim.x) {
    const uint32_t gpos = s_base + j;
    if (gpos < g.cand_cap) m.cand[gpos] = s_buf[j];
  }
}

// fixed-order sum of the per-block partials by one block of 1024 threads
__device__ __forceinline__ double sum_partials(const double* partial, int nparts, double* sh) {
  double acc = 0.0;
  for (int i = threadIdx.x; i < nparts; i += blockDim.x) acc += partial[i];
  sh[threadIdx.x] = acc;
  __syncthreads();
  for (int o = blockDim.x / 2; o; o >>= 1) {
    if ((int)threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
    __syncthreads();
  }
  return sh[0];
}

__device__ __forceinline__ void write_norm_scalars(float* scalars, const NsScalarIdx& ix, double sumsq, float maxabs,
                                                   float eps, float widen) {
  const float nu = (float)sqrt(sumsq);
  const float inv = __fdiv_rn(1.0f, __fadd_rn(nu, eps));
  const float amax0 = __fmul_rn(maxabs, inv);
  scalars[ix.nu] = nu;
  scalars[ix.inv] = inv;
  scalars[ix.amax_X0] = amax0;
  scalars[ix.sg_X0] = scale_exact(__fmul_rn(widen, amax0));
}

// ---- fallback when the candidate list overflowed (so many equal magnitudes that the picked bin holds more
// than the list takes: constant matrices and the like).  One block finishes the job alone: two more
// radix rounds over the whole matrix (bits 17..7, then 6..0) and the clamped sum of squares.  Slow
// (three passes by 1024 threads) but rare, and it costs no launch when it is not needed.
// hist: 2048 counters; shd: 1024 doubles.
__device__ void fallback_select_and_stats(const PrepGroup& g, const PrepMatrix& m, uint32_t* hist, double* shd) {
  __shared__ uint32_t s_fb_prefix, s_fb_rank;
  NsHeader* hdr = m.hdr;
  const float4* src = reinterpret_cast<const float4*>(m.G);
  if (threadIdx.x == 0) { s_fb_prefix = hdr->sel_prefix; s_fb_rank = hdr->sel_rank; }
  __syncthreads();
  for (int round = 0; round < 2; ++round) {
    const int shift = round == 0 ? 7 : 0, nbits = round == 0 ? 11 : 7;
    const uint32_t nb = 1u << nbits;
    const uint32_t high_mask = (0x7FFFFFFFu >> (shift + nbits)) << (shift + nbits);
    for (uint32_t i = threadIdx.x; i < nb; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    const uint32_t prefix = s_fb_prefix;
    for (int64_t i = threadIdx.x; i < g.n4; i += blockDim.x) {
      const float4 v = __ldg(src + i);
      const uint32_t k[4] = {mag_bits(v.x), mag_bits(v.y), mag_bits(v.z), mag_bits(v.w)};
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if ((k[j] & high_mask) == prefix) atomicAdd(&hist[(k[j] >> shift) & (nb - 1)], 1u);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      uint32_t run = 0;
      const uint32_t rank = s_fb_rank;
      for (uint32_t b = 0; b < nb; ++b) {
        if (rank <= run + hist[b]) { s_fb_prefix = prefix | (b << shift); s_fb_rank = rank - run; break; }
        run += hist[b];
      }
    }
    __syncthreads();
  }
  const float tau = __uint_as_float(s_fb_prefix);
  double acc = 0.0;
  for (int64_t i = threadIdx.x; i < g.n4; i += blockDim.x) {
    const float4 v = __ldg(src + i);
    const float c[4] = {fminf(fabsf(v.x), tau), fminf(fabsf(v.y), tau), fminf(fabsf(v.z), tau), fminf(fabsf(v.w), tau)};
#pragma unroll
    for (int j = 0; j < 4; ++j) acc += (double)c[j] * (double)c[j];
  }
  shd[threadIdx.x] = acc;
  __syncthreads();
  for (int o = blockDim.x / 2; o; o >>= 1) {
    if ((int)threadIdx.x < o) shd[threadIdx.x] += shd[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    hdr->sel_prefix = s_fb_prefix;
    m.scalars[g.ix.tau] = tau;
    write_norm_scalars(m.scalars, g.ix, shd[0], tau, g.eps, g.q.widen);
  }
}

// ---- finish: select tau among the candidates and derive the normalisation scalars
__global__ void __launch_bounds__(1024) kp_finalize(const __grid_constant__ PrepGroup g) {
  pdl_launch_dependents();
  pdl_wait();
  const PrepMatrix& m = g.mat[blockIdx.y];
  __shared__ double shd[1024];
  __shared__ uint32_t hist[1024];
  __shared__ uint32_t s_prefix, s_rank;
  __shared__ unsigned long long s_lo, s_hi;
  __shared__ uint32_t s_above;
  NsHeader* hdr = m.hdr;
  if (!g.clip) {
    const double total = sum_partials(m.partial, g.stat_blocks, shd);
    if (threadIdx.x == 0) write_norm_scalars(m.scalars, g.ix, total, __uint_as_float(hdr->maxabs_bits), g.eps,
                                               g.q.widen);
    return;
  }
  const uint32_t count = hdr->cand_count;
  if (count > g.cand_cap) {
    if (threadIdx.x == 0) hdr->overflow = 1;
    __shared__ uint32_t fb_hist[2048];
    fallback_select_and_stats(g, m, fb_hist, shd);
    return;
  }
  // two radix rounds over the low 18 bits of the candidates: 9 bits each.  The second round
  // also gathers what the norm needs: squares of the candidates below the sub-bin picked by
  // the first round (certainly not clipped) as exact integers -- all candidates share the
  // exponent field, so x = mant * 2^(e-150) with a 24-bit integer mant -- and the number above it.
  if (threadIdx.x == 0) { s_prefix = hdr->sel_prefix; s_rank = hdr->sel_rank; s_lo = 0; s_hi = 0; s_above = 0; }
  unsigned long long lo = 0, hi = 0;
  uint32_t above = 0;
  const uint32_t efield = hdr->sel_prefix >> 23;
  const uint32_t implicit = efield ? 0x800000u : 0u;
  for (int round = 0; round < 2; ++round) {
    const int shift = round == 0 ? 9 : 0;
    const uint32_t high_mask = ~((1u << (shift + 9)) - 1u) & 0x7FFFFFFFu;
    hist[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    for (uint32_t i0 = threadIdx.x; i0 < count; i0 += 8 * blockDim.x) {
      uint32_t k[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const uint32_t i = i0 + u * blockDim.x;
        k[u] = i < count ? m.cand[i] : 0xFFFFFFFFu;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        if (k[u] == 0xFFFFFFFFu) continue;
        if ((k[u] & high_mask) == (prefix & high_mask)) {
          atomicAdd(&hist[(k[u] >> shift) & 511u], 1u);
        } else if (round == 1) {
          if (k[u] < prefix) {
            const unsigned long long mant = (k[u] & 0x7FFFFFu) | implicit;
            const unsigned long long sq = mant * mant;
            lo += sq & 0xFFFFFFull;
            hi += sq >> 24;
          } else {
            above += 1;
          }
        }
      }
    }
    __syncthreads();
    // the bin that holds the rank: inclusive scan of the 512 counters by the first warps
    if (threadIdx.x < 512) {
      // each of 16 warps scans 32 bins; warp totals are then scanned by thread 0
      uint32_t v = hist[threadIdx.x], incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
        if ((threadIdx.x & 31) >= o) incl += t;
      }
      hist[512 + threadIdx.x] = incl;            // inclusive within the warp's 32 bins
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      uint32_t run = 0;
      const uint32_t rank = s_rank;
      for (int w = 0; w < 16; ++w) {
        const uint32_t wt = hist[512 + w * 32 + 31];
        if (rank <= run + wt) {
          for (int b = 0; b < 32; ++b) {
            const uint32_t incl = run + hist[512 + w * 32 + b];
            if (rank <= incl) {
              s_prefix = prefix | ((uint32_t)(w * 32 + b) << shift);
              s_rank = rank - (incl - hist[w * 32 + b]);
              break;
            }
          }
          break;
        }
        run += wt;
      }
    }
    __syncthreads();
  }
  const uint32_t tau_bits = s_prefix;
  // candidates inside the last sub-bin: a counter of the second round stands for one exact
  // magnitude (all 31 bits known), so its members' squares are count * mant^2
  if (threadIdx.x < 512) {
    const uint32_t cnt = hist[threadIdx.x];
    const uint32_t kk = (tau_bits & ~511u) | threadIdx.x;
    if (cnt) {
      if (kk <= tau_bits) {
        const unsigned long long mant = (kk & 0x7FFFFFu) | implicit;
        const unsigned long long sq = mant * mant;
        lo += (unsigned long long)cnt * (sq & 0xFFFFFFull);
        hi += (unsigned long long)cnt * (sq >> 24);
      } else {
        above += cnt;
      }
    }
  }
  // one shared atomic per warp (64-bit shared atomics from all 1024 threads serialise badly)
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    lo += __shfl_xor_sync(0xffffffffu, lo, o);
    hi += __shfl_xor_sync(0xffffffffu, hi, o);
    above += __shfl_xor_sync(0xffffffffu, above, o);
  }
  if ((threadIdx.x & 31) == 0) {
    atomicAdd(&s_lo, lo);
    atomicAdd(&s_hi, hi);
    atomicAdd(&s_above, above);
  }
  __syncthreads();
  const double below = sum_partials(m.partial, g.stat_blocks, shd);
  if (threadIdx.x == 0) {
    const float tau = __uint_as_float(tau_bits);
    const int e2 = 2 * ((int)(efield ? efield : 1u) - 150);
    const double cand_sq = ldexp((double)s_hi * 16777216.0 + (double)s_lo, e2);
    // clamped to tau: everything in the bins above the picked one, and the candidates above tau
    const double n_total = (double)g.n4 * 4.0;
    const double n_clipped = n_total - (double)hdr->count_below - (double)hdr->bin_count + (double)s_above;
    const double total = below + cand_sq + n_clipped * (double)tau * (double)tau;
    m.scalars[g.ix.tau] = tau;
    write_norm_scalars(m.scalars, g.ix, total, tau, g.eps, g.q.widen);
    hdr->overflow = 0;
  }
}

// ---- X0 = clamp(G) * inv in the work orientation (s x l; transposed when G is tall), its FP32
// copy (unless the first G3 stage will form X0 from G itself), and both NVFP4 operand copies.
//
// A persistent block per SM walks 128 x 128 tiles of G.  Three tiles are kept in flight with TMA
// (64 KB each, four 32-column boxes with the 128-byte swizzle; what lies outside the caller's
// matrix arrives as zeros, which is the padding of the work shape).  Thirty-two warps quantise the
// tiles as they land: sixteen along the rows (a warp takes 8 rows, a thread one 32-column box of a
// row), sixteen along the columns (a warp takes a band of 16 rows and 64 columns, a thread two
// columns).  The tile is never transposed: for a tall G the two passes simply swap destinations
// (blocks along the rows of G are blocks along the columns of X = G^T).  The row pass writes its
// codes itself (the four lanes of a row fill 64 contiguous bytes); the column pass's codes (8 bytes
// per column) and both kinds of scale bytes are staged in shared memory and leave as 64-byte rows
// and whole 512-byte atoms.
// One block-wide barrier per tile: after it the tile's buffer is refilled and the staged bytes go out.
// Tile buffers and staging areas form rings of three.
constexpr int kPrepBufs = 3;
constexpr int kPrepTile = 128 * 128 * 4;       // bytes of a tile
constexpr int kPrepBox = 32 * 128 * 4;         // bytes of one 32-column box
constexpr int kQtSlot = 1024 + 16;             // staged column codes: [band][column][8 B], padded bands
constexpr int kPrepStage = 8 * kQtSlot + 2 * 1024;  // + two scale atoms per pass
constexpr int kPrepWarps = 32;
constexpr int kPrepThreads = kPrepWarps * 32;

struct PrepTileInfo { int mi, gr0, gc0, pad; };  // matrix, origin of the tile in G
struct PrepShared {
  uint64_t full[kPrepBufs];
  uint32_t abort_flag;
  PrepTileInfo info[4];           // tiles it .. it + 3 of this block (ring)
  float rcp_tab[kMaxPack][8];     // per matrix: fl(1 / fl((8 + j) sg))
};
constexpr int kPrepSmem = kPrepBufs * (kPrepTile + kPrepStage) + (int)sizeof(PrepShared) + 1024;
static_assert(kPrepSmem <= 232448, "at most 227 KB of dynamic shared memory");

// address of the 16-byte piece c4 (0..31) of row r in a tile of four swizzled boxes
__device__ __forceinline__ uint32_t prep_piece(uint32_t tile, int r, int c4) {
  return tile + (uint32_t)((c4 >> 3) * kPrepBox + r * 128 + (((c4 & 7) ^ (r & 7)) << 4));
}
__device__ __forceinline__ float4 lds128f(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ float lds32f(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}
// ---- block quantisers of the operand preparation.
// They quantise x0 = clamp(g, +-tau) * inv (quantize_block16 applied to x0) with fewer instructions,
// bit for bit the same result; whatever the short cuts do not cover goes to quantize_block16 itself.
//  * No clamp per element.  With y = fl(g * inv) and tinv = fl(tau * inv), rounding is monotonic, so
//    x0 = clamp(y, +-tinv) exactly and the block's amax is min(max |y|, tinv).  An element beyond the clip
//    level would be quantised from fl(tinv * rcp), which lies near 6 (the block's scale maps its amax = tinv
//    there); every larger product saturates to the same code 6.  Checked per matrix: fl(tinv * rcp) > 5
//    for the scale byte of a block whose amax is tinv.
//  * The scale byte is E4M3(fl(amax / 6sg)).  q = amax * fl(1 / 6sg) with one correction step
//    (r = amax - q * 6sg exactly by FMA, q += r * fl(1 / 6sg)) is within one ulp of the correctly rounded
//    quotient, so both convert to the same byte unless q lies within two ulps of a rounding boundary of
//    E4M3 (mantissa bits 19..0 = 0x80000 in the normal range); those blocks, and scale bytes <= 8
//    (subnormal E4M3, where the boundaries lie elsewhere), take the exact path.
//  * The reciprocal of the decoded scale d = fl(s * sg), s = (8 + m) 2^(E - 10): for sg far from the ends
//    of the exponent range d = fl((8 + m) sg) 2^(E - 10) exactly, so fl(1 / d) is one of eight values per
//    matrix with the exponent shifted; the eight values fl(1 / fl((8 + j) sg)) lie in shared memory.
struct PrepScalars {
  float tau, inv, tinv, six_sg, rcp_six_sg, sg;
  uint32_t rcp_tab;     // shared-memory address of the matrix's eight reciprocals
  uint32_t near_limit;  // 4 when the short cuts hold for this matrix (sg in [2^-60, 2^60], and the clip level
                        // itself is quantised to 6: fl(tinv * rcp) > 5 for the scale of a clipped block), else all ones
};

__device__ __noinline__ uint32_t prep_quant_exact(const float (&gv)[16], float tau, float inv, float six_sg, float sg,
                                                  uint32_t& lo, uint32_t& hi) {
  float v[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __fmul_rn(fminf(fmaxf(gv[i], -tau), tau), inv);
  return quantize_block16(v, six_sg, sg, lo, hi);
}

// amax (of |y|, not yet limited to tinv) -> scale byte and fl(1 / d); `rare` is set when the block must take
// the exact path.
__device__ __forceinline__ uint32_t prep_scale(const PrepScalars& ps, float amax_y, float& rcp, bool& rare) {
  const float amax = fminf(amax_y, ps.tinv);
  float q = __fmul_rn(amax, ps.rcp_six_sg);
  const float r = __fmaf_rn(-q, ps.six_sg, amax);
  q = __fmaf_rn(r, ps.rcp_six_sg, q);
  const uint32_t sb = cvt_ue4m3(q);
  uint32_t tab;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(tab) : "r"(ps.rcp_tab + ((sb & 7u) << 2)));
  rcp = __uint_as_float(tab - (((sb >> 3) - 10u) << 23));
  const uint32_t near = (__float_as_uint(q) + 2u - 0x80000u) & 0xFFFFFu;
  // q < 1.0625 * 2^-6: scale bytes <= 8 (and the boundary to 9)
  rare = near <= ps.near_limit || q < 0.0166015625f;
  return sb;
}

// One block of 16 consecutive elements, given as four 16-byte pieces of two packed pairs each.
// `rare`: the caller must redo the block with prep_quant_exact.
__device__ __forceinline__ uint32_t prep_quant_row(uint64_t (&y2)[8], const PrepScalars& ps, uint32_t& lo,
                                                   uint32_t& hi, bool& rare) {
  const uint64_t inv2 = pack2(ps.inv, ps.inv);
  float m8[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    float a, b;
    y2[i] = mul2(y2[i], inv2);
    unpack2(y2[i], a, b);
    m8[i] = fmaxf(fabsf(a), fabsf(b));
  }
  const float amax_y = fmaxf(fmaxf(fmaxf(m8[0], m8[1]), fmaxf(m8[2], m8[3])),
                             fmaxf(fmaxf(m8[4], m8[5]), fmaxf(m8[6], m8[7])));
  float rcp;
  const uint32_t sb = prep_scale(ps, amax_y, rcp, rare);
  const uint64_t rcp2 = pack2(rcp, rcp);
  float z[16];
#pragma unroll
  for (int i = 0; i < 8; ++i) unpack2(mul2(y2[i], rcp2), z[2 * i], z[2 * i + 1]);
  lo = cvt_e2m1x8(z[0], z[1], z[2], z[3], z[4], z[5], z[6], z[7]);
  hi = cvt_e2m1x8(z[8], z[9], z[10], z[11], z[12], z[13], z[14], z[15]);
  return sb;
}

// Two blocks side by side: g2[i] = the elements of row i in two neighbouring columns; block j runs down
// column j.  The pairs stay together through both multiplications.  Returns the two scale bytes.
__device__ __forceinline__ void prep_quant_col2(uint64_t (&y2)[16], const PrepScalars& ps, uint32_t (&cw)[4],
                                                uint32_t& sb0, uint32_t& sb1, bool& rare) {
  const uint64_t inv2 = pack2(ps.inv, ps.inv);
  float ax = 0.0f, ay = 0.0f;
#pragma unroll
  for (int i = 0; i < 16; i += 2) {
    float a, b, c, d;
    y2[i] = mul2(y2[i], inv2);
    y2[i + 1] = mul2(y2[i + 1], inv2);
    unpack2(y2[i], a, b);
    unpack2(y2[i + 1], c, d);
    ax = fmaxf(ax, fmaxf(fabsf(a), fabsf(c)));
    ay = fmaxf(ay, fmaxf(fabsf(b), fabsf(d)));
  }
  float r0, r1;
  bool rare0, rare1;
  sb0 = prep_scale(ps, ax, r0, rare0);
  sb1 = prep_scale(ps, ay, r1, rare1);
  const uint64_t rcp2 = pack2(r0, r1);
  float zx[16], zy[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) unpack2(mul2(y2[i], rcp2), zx[i], zy[i]);
  cw[0] = cvt_e2m1x8(zx[0], zx[1], zx[2], zx[3], zx[4], zx[5], zx[6], zx[7]);
  cw[1] = cvt_e2m1x8(zx[8], zx[9], zx[10], zx[11], zx[12], zx[13], zx[14], zx[15]);
  cw[2] = cvt_e2m1x8(zy[0], zy[1], zy[2], zy[3], zy[4], zy[5], zy[6], zy[7]);
  cw[3] = cvt_e2m1x8(zy[8], zy[9], zy[10], zy[11], zy[12], zy[13], zy[14], zy[15]);
  rare = rare0 || rare1;
}

template <bool PF>
__global__ void __launch_bounds__(kPrepThreads, 1) kp_prep_operands(const __grid_constant__ PrepGroup g) {
  extern __shared__ uint8_t prep_smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(prep_smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* stage_base = smem + kPrepBufs * kPrepTile;
  PrepShared* sh = reinterpret_cast<PrepShared*>(stage_base + kPrepBufs * kPrepStage);
  volatile uint32_t* abort_flag = &sh->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_per_matrix = (int)((g.s >> 7) * (g.l >> 7));
  const int total = tiles_per_matrix * g.count;
  const int my_tiles = (total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;  // tiles of this block
  pdl_launch_dependents();

  // Tile `it` of this block: work out where it lies, publish that in the ring and start its copy.  Called by
  // one thread, a block-wide barrier before the tile's turn.
  auto fetch = [&](int it_) {
    if (it_ >= my_tiles) return;
    const int t_ = (int)blockIdx.x + it_ * (int)gridDim.x;
    const int b_ = it_ % kPrepBufs;
    PrepTileInfo ti;
    ti.pad = 0;
    ti.mi = t_ / tiles_per_matrix;
    const int r_ = t_ - ti.mi * tiles_per_matrix;
    const int tiles_x = (int)((g.mat[ti.mi].tall ? g.s : g.l) >> 7);  // tiles along a row of G
    const int ty = r_ / tiles_x;
    ti.gr0 = ty * 128;
    ti.gc0 = (r_ - ty * tiles_x) * 128;
    sh->info[it_ & 3] = ti;
    mbar_expect_tx(&sh->full[b_], kPrepTile);
#pragma unroll
    for (int q = 0; q < 4; ++q)
      tma_load_2d(smem + b_ * kPrepTile + q * kPrepBox, &g.tmG[ti.mi], ti.gc0 + 32 * q, ti.gr0, &sh->full[b_]);
  };

  if (threadIdx.x == 0) {
    for (int i = 0; i < kPrepBufs; ++i) mbar_init(&sh->full[i], 1);
    sh->abort_flag = 0;
    mbar_fence_init();
  }
  pdl_wait();   // from here on the kernel reads what the launches before it wrote
  if (threadIdx.x == 0) {
    for (int i = 0; i < kPrepBufs; ++i) fetch(i);
  }
  if (threadIdx.x < g.count * 8) {
    const float sg_ = g.mat[threadIdx.x >> 3].scalars[g.ix.sg_X0];
    sh->rcp_tab[threadIdx.x >> 3][threadIdx.x & 7] = __frcp_rn(__fmul_rn((float)(8 + (threadIdx.x & 7)), sg_));
  }
  __syncthreads();

  // lane-dependent parts of the shared-memory addresses, fixed for the whole kernel
  const bool row_warp = warp < kPrepWarps / 2;
  //   row pass: a warp takes 8 rows, a thread one 32-column box of a row (two blocks)
  const int rr = (warp & 15) * 8 + (lane & 7), box = lane >> 3;
  //   column pass: a warp takes a band of 16 rows and 64 columns, a thread two columns
  const int cwp = warp & 15, band = cwp >> 1, cp = (cwp & 1) * 32 + lane;  // cp: column pair 0..63
  uint32_t base_off, sw;
  if (row_warp) { base_off = (uint32_t)(box * kPrepBox + rr * 128); sw = (uint32_t)(rr & 7) << 4; }
  else { base_off = (uint32_t)((cp >> 4) * kPrepBox + band * 16 * 128 + (cp & 1) * 8); sw = (uint32_t)((cp >> 1) & 7) << 4; }

  int cur = -1;
  PrepScalars ps;
  ps.tau = ps.inv = ps.tinv = ps.six_sg = ps.rcp_six_sg = ps.sg = 0.0f; ps.rcp_tab = 0; ps.near_limit = 0;
  for (int it = 0; it < my_tiles; ++it) {
    const int b = it % kPrepBufs, use = it / kPrepBufs;
    const PrepTileInfo ti = sh->info[it & 3];   // written before an earlier barrier
    wait_or_abort(&sh->full[b], (uint32_t)use & 1u, abort_flag);
    const int mi = ti.mi, gr0 = ti.gr0, gc0 = ti.gc0;
    const PrepMatrix& m = g.mat[mi];
    if (mi != cur) {
      cur = mi;
      ps.tau = g.clip ? m.scalars[g.ix.tau] : __int_as_float(0x7f800000);
      ps.inv = m.scalars[g.ix.inv];
      ps.tinv = __fmul_rn(ps.tau, ps.inv);
      ps.sg = m.scalars[g.ix.sg_X0];
      ps.six_sg = __fmul_rn(6.0f, ps.sg);
      ps.rcp_six_sg = __frcp_rn(ps.six_sg);
      ps.rcp_tab = smem_u32(&sh->rcp_tab[mi][0]);
      const uint32_t esg = (__float_as_uint(ps.sg) >> 23) & 0xFFu;
      bool ok = esg >= 67u && esg <= 187u;   // 2^-60 .. 2^60
      if (ps.tinv < __int_as_float(0x7f800000)) {
        // a block with clipped elements has amax = tinv: is the clip level quantised to 6 there?
        const float dc = __fmul_rn(ue4m3_to_float(cvt_ue4m3(__fdiv_rn(ps.tinv, ps.six_sg))), ps.sg);
        ok = ok && dc != 0.0f && __fmul_rn(ps.tinv, __frcp_rn(dc)) > 5.0f;
      }
      ps.near_limit = ok ? 4u : 0xFFFFFFFFu;
    }
    auto x0 = [&](float gval) { return __fmul_rn(fminf(fmaxf(gval, -ps.tau), ps.tau), ps.inv); };
    const uint32_t tile = smem_u32(smem + b * kPrepTile);
    uint8_t* stage = stage_base + b * kPrepStage;
    const int tall = m.tall;

    if (m.store_x) {
      if (!tall) {
        // X = G: rows of the tile are rows of X
#pragma unroll 4
        for (int r = warp; r < 128; r += kPrepWarps) {
          const float4 v = lds128f(prep_piece(tile, r, lane));
          if ((gr0 + r) < m.x_rows && (gc0 + lane * 4) < m.x_cols)
            *reinterpret_cast<float4*>(m.X + (int64_t)(gr0 + r) * m.x_cols + gc0 + lane * 4) =
                make_float4(x0(v.x), x0(v.y), x0(v.z), x0(v.w));
        }
      } else {
        // X = G^T: a lane group of 8 consecutive tile rows writes one 32-byte sector of a row of X;
        // the 8 rows x 4 columns a warp reads at once lie in 32 different banks
        const int r8 = lane & 7, cq = lane >> 3;
#pragma unroll 4
        for (int k = 0; k < 512 / kPrepWarps; ++k) {
          const int p = warp * (512 / kPrepWarps) + k;
          const int row = (p & 15) * 8 + r8, col = (p >> 4) * 4 + cq;
          const float v = lds32f(prep_piece(tile, row, col >> 2) + (uint32_t)(col & 3) * 4u);
          if ((gc0 + col) < m.x_rows && (gr0 + row) < m.x_cols) m.X[(int64_t)(gc0 + col) * m.x_cols + gr0 + row] = x0(v);
        }
      }
    }

    // destinations of the two passes: blocks along the rows of G are qX for a wide G, qX^T for a tall one
    const int64_t rp_k = tall ? g.s : g.l, cp_k = tall ? g.l : g.s;  // contraction length of each destination
    if (g.write_q) {
      uint8_t* sf_stage = stage + 8 * kQtSlot;
      const uint32_t tb = tile + base_off;
      if (row_warp) {
        uint32_t code[4];
        uint32_t sfw = 0;
        bool redo = false;
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          uint64_t g2[8];
#pragma unroll
          for (int i = 0; i < 4; ++i)
            asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];"
                         : "=l"(g2[2 * i]), "=l"(g2[2 * i + 1])
                         : "r"(tb + (((uint32_t)(q * 4 + i) << 4) ^ sw)));
          uint32_t sb;
          if (PF) {
            float v[16], unused;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              float a, b2;
              unpack2(g2[i], a, b2);
              v[2 * i] = x0(a); v[2 * i + 1] = x0(b2);
            }
            sb = quantize_block16_opts(v, g.q, ps.sg, code[2 * q], code[2 * q + 1], unused);
          } else {
            bool rare;
            sb = prep_quant_row(g2, ps, code[2 * q], code[2 * q + 1], rare);
            redo = redo || rare;
          }
          sfw |= sb << (8 * q);
        }
        if (!PF && redo) {   // rare: both blocks again from the tile, with the plain quantiser
          sfw = 0;
#pragma unroll 1
          for (int q = 0; q < 2; ++q) {
            float gv[16];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float4 f = lds128f(tb + (((uint32_t)(q * 4 + i) << 4) ^ sw));
              gv[4 * i] = f.x; gv[4 * i + 1] = f.y; gv[4 * i + 2] = f.z; gv[4 * i + 3] = f.w;
            }
            sfw |= prep_quant_exact(gv, ps.tau, ps.inv, ps.six_sg, ps.sg, code[2 * q], code[2 * q + 1]) << (8 * q);
          }
        }
        // the four lanes of a row write 64 contiguous bytes
        uint8_t* rp_codes = tall ? m.qt_codes : m.qx_codes;
        *reinterpret_cast<uint4*>(rp_codes + (int64_t)(gr0 + rr) * (rp_k / 2) + gc0 / 2 + box * 16) =
            make_uint4(code[0], code[1], code[2], code[3]);
        *reinterpret_cast<uint16_t*>(sf_stage + (box >> 1) * 512 + (rr & 31) * 16 + (rr >> 5) * 4 + (box & 1) * 2) =
            (uint16_t)sfw;
      } else {
        uint64_t g2[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          // row band * 16 + i of the tile: its low three bits are those of i
          const uint32_t a = tb + (uint32_t)(i * 128) + (sw ^ ((uint32_t)(i & 7) << 4));
          asm volatile("ld.shared.b64 %0, [%1];" : "=l"(g2[i]) : "r"(a));
        }
        uint32_t cw[4], sb0 = 0, sb1 = 0;
        if (PF) {
          float unused;
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            float v[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              float a, b2;
              unpack2(g2[i], a, b2);
              v[i] = x0(j == 0 ? a : b2);
            }
            const uint32_t sb = quantize_block16_opts(v, g.q, ps.sg, cw[2 * j], cw[2 * j + 1], unused);
            if (j == 0) sb0 = sb; else sb1 = sb;
          }
        } else {
          bool rare;
          prep_quant_col2(g2, ps, cw, sb0, sb1, rare);
          if (rare) {   // redo both blocks from the tile with the plain quantiser
#pragma unroll 1
            for (int j = 0; j < 2; ++j) {
              float gv[16];
#pragma unroll
              for (int i = 0; i < 16; ++i)
                gv[i] = lds32f(tb + (uint32_t)(i * 128 + j * 4) + (sw ^ ((uint32_t)(i & 7) << 4)));
              const uint32_t sb = prep_quant_exact(gv, ps.tau, ps.inv, ps.six_sg, ps.sg, cw[2 * j], cw[2 * j + 1]);
              if (j == 0) sb0 = sb; else sb1 = sb;
            }
          }
        }
        uint8_t* sfc = sf_stage + 1024 + (band >> 2) * 512 + (band & 3);
        const int c = cp * 2;
        sfc[(c & 31) * 16 + (c >> 5) * 4] = (uint8_t)sb0;
        sfc[((c + 1) & 31) * 16 + ((c + 1) >> 5) * 4] = (uint8_t)sb1;
        *reinterpret_cast<uint4*>(stage + band * kQtSlot + cp * 16) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
      }
    }

    // Every warp has read the tile and staged its output: the buffer takes the tile three ahead, the
    // staged bytes go out.
    __syncthreads();
    if (threadIdx.x == kPrepThreads - 32) {
      fence_proxy_async_smem();
      fetch(it + kPrepBufs);
    }
    if (g.write_q) {
      const int tid = threadIdx.x;
      if (tid < 512) {
        // column-pass codes: row (gc0 + c) of the destination, 64 bytes from byte gr0 / 2; four lanes per row
        uint8_t* cp_codes = tall ? m.qx_codes : m.qt_codes;
        const int c = tid >> 2, h = tid & 3;
        const uint8_t* src = stage + c * 8;
        const uint2 a = *reinterpret_cast<const uint2*>(src + (2 * h) * kQtSlot);
        const uint2 d = *reinterpret_cast<const uint2*>(src + (2 * h + 1) * kQtSlot);
        *reinterpret_cast<uint4*>(cp_codes + (int64_t)(gc0 + c) * (cp_k / 2) + gr0 / 2 + h * 16) = make_uint4(a.x, a.y, d.x, d.y);
      } else if (tid < 640) {
        // scale atoms: two adjacent 512-byte atoms per pass
        const bool rowpass = tid < 576;
        uint8_t* sf_base = rowpass ? (tall ? m.qt_sf : m.qx_sf) : (tall ? m.qx_sf : m.qt_sf);
        const int64_t row0 = rowpass ? gr0 : gc0, k0 = rowpass ? gc0 : gr0, kk = rowpass ? rp_k : cp_k;
        const int j = tid & 63;
        const uint4 w = *reinterpret_cast<const uint4*>(stage + 8 * kQtSlot + (rowpass ? 0 : 1024) + j * 16);
        *reinterpret_cast<uint4*>(sf_base + sf_offset(row0, k0 / 16, kk / 16) + j * 16) = w;
      }
    }
  }
  if (threadIdx.x == 0 && sh->abort_flag) report_timeout(g.status);
}

}  // namespace

cudaError_t prologue_set_attributes() {
  cudaError_t e = cudaFuncSetAttribute(kp_prep_operands<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPrepSmem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(kp_prep_operands<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPrepSmem);
}

// Enqueue the prologue for `count` matrices of one shape (s, l) and one parameter set.
cudaError_t launch_prologue_group(const PrologueItem* items, int count, int write_q, const QuantOpts& q,
                                  uint32_t* status, cudaStream_t st) {
  for (int i0 = 0; i0 < count; i0 += kMaxPack) {
    const int nn = count - i0 < kMaxPack ? count - i0 : kMaxPack;
    const NsPlan& pl = *items[i0].pl;
    PrepGroup g;
    memset(&g, 0, sizeof(g));
    g.count = nn;
    g.n4 = pl.s0 * pl.l0 / 4;
    g.s = pl.s; g.l = pl.l;
    g.s0 = pl.s0; g.l0 = pl.l0;
    g.clip = pl.clip;
    g.clip_rank = (uint32_t)pl.clip_rank;
    // The candidate list lives in workspace that nothing else uses before the first product: the A buffer
    // (s x s words) or, for a matrix much longer than high, the second set of transposed operand codes
    // (s x l / 8 words).  An eighth of the elements is more than any bin of a spread-out distribution holds.
    const bool cand_in_qxt = pl.s * pl.l / 8 > pl.s * pl.s;
    const int64_t region = cand_in_qxt ? pl.s * pl.l / 8 : pl.s * pl.s;
    const int64_t cap = pl.s0 * pl.l0 / 8 < region ? pl.s0 * pl.l0 / 8 : region;
    g.cand_cap = (uint32_t)cap;
    g.eps = pl.eps;
    g.stat_blocks = pl.stat_blocks;
    g.write_q = write_q;
    g.zero_words = (int)(pl.zero_bytes / 4);
    g.ix = pl.ix;
    g.q = q;
    g.status = status;
    bool all_counted = true;
    for (int j = 0; j < nn; ++j) {
      const PrologueItem& it = items[i0 + j];
      const fp4_ws_layout& L = it.pl->lay;
      PrepMatrix& m = g.mat[j];
      m.G = it.G; m.X = it.X;
      m.hdr = reinterpret_cast<NsHeader*>(it.ws + L.header);
      m.scalars = reinterpret_cast<float*>(it.ws + L.scalars);
      m.hist = reinterpret_cast<uint32_t*>(it.ws + it.pl->off_hist);
      m.partial = reinterpret_cast<double*>(it.ws + it.pl->off_partial);
      m.cand = reinterpret_cast<uint32_t*>(it.ws + (cand_in_qxt ? L.qXt_codes[1] : L.A));
      m.qx_codes = it.ws + L.qX_codes; m.qx_sf = it.ws + L.qX_scales;
      m.qt_codes = it.ws + L.qXt_codes[0]; m.qt_sf = it.ws + L.qXt_scales[0];
      m.tall = it.pl->tall;
      m.clear_status = it.clear_status ? 1 : 0;
      m.store_x = it.store_x ? 1 : 0;
      m.x_rows = it.x_rows; m.x_cols = it.x_cols;
      m.hist_top = it.hist_top;
      if (!it.hist_top) all_counted = false;
      g.tmG[j] = *it.tmG;
    }
    const int sms = pl.sms;
    int64_t hb = (g.n4 + 512 * 4 - 1) / (512 * 4);
    const int hist_blocks = (int)(hb < (int64_t)sms * 4 ? (hb < 1 ? 1 : hb) : (int64_t)sms * 4);
    const dim3 gy1(1, (unsigned)nn), gh((unsigned)hist_blocks, (unsigned)nn), gs((unsigned)g.stat_blocks, (unsigned)nn);
    {
      ProfScope ps(FP4_PROF_CLIP, st);
      launch_chained(kp_init, dim3(4, (unsigned)nn), dim3(256), 0, st, g);
      count_launches(1);
      if (g.clip) {
        if (!all_counted) launch_chained(kp_hist_top, gh, dim3(512), 0, st, g);
        launch_chained(kp_pick_top, gy1, dim3(256), 0, st, g);
        count_launches(all_counted ? 1 : 2);
      }
    }
    {
      ProfScope ps(FP4_PROF_STATS, st);
      launch_chained(kp_compact_stats, gs, dim3(256), 0, st, g);
      launch_chained(kp_finalize, gy1, dim3(1024), 0, st, g);
      count_launches(2);
    }
    {
      ProfScope ps(FP4_PROF_PREP, st);
      const int64_t tiles = (pl.l / 128) * (pl.s / 128) * nn;
      const unsigned gp = (unsigned)(tiles < sms ? tiles : sms);
      if (q.rht || q.four_six) launch_chained(kp_prep_operands<true>, dim3(gp), dim3(kPrepThreads), kPrepSmem, st, g);
      else launch_chained(kp_prep_operands<false>, dim3(gp), dim3(kPrepThreads), kPrepSmem, st, g);
      count_launches(1);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace fp4
