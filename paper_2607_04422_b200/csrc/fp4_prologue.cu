// Prologue of the Root step for a group of equal-size matrices (Section 3.4: "p99 outlier
// clipping"; normalisation; the first operand copies qX = Q_1x16(X), qX^{16x1} = Q_16x1(X)).
// Every kernel covers the whole group (gridDim.y or .z = matrix), so a batch needs a dozen
// launches instead of a dozen per matrix.
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
  uint32_t* cand;      // candidate list (the A buffer of the workspace, unused until G1)
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
};

__device__ __forceinline__ uint32_t mag_bits(float x) { return __float_as_uint(x) & 0x7FFFFFFFu; }

// ---- init: clear header (keeping the status word of all but the first matrix of a call),
// scalars and histogram; arm the select
__global__ void __launch_bounds__(256) kp_init(const __grid_constant__ PrepGroup g) {
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
  __shared__ uint32_t part[256];
  uint32_t local[PER];
  uint32_t sum = 0;
#pragma unroll
  for (int j = 0; j < PER; ++j) { local[j] = hist[threadIdx.x * PER + j]; sum += local[j]; }
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
  const PrepMatrix& m = g.mat[blockIdx.y];
  pick_bin<kTopBins>(m.hdr, m.hist_top ? m.hist_top : m.hist, kTopShift, &m.hdr->bin_count, &m.hdr->count_below);
}

// ---- pass 2: candidates of the picked bin, FP64 sum of squares below the bin, max |g|.
// Candidates are rare: they are collected in a shared-memory buffer per block and copied to
// the global list with one reservation per block (or directly when the buffer is full).
__global__ void __launch_bounds__(256) kp_compact_stats(const __grid_constant__ PrepGroup g) {
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
// copy (unless the first G3 stage will form X0 from G itself), and both NVFP4 operand copies.  One 128 x 128 tile of X per block, gridDim.z = matrix.
// Row pitch of the shared tile in floats: 132 (16-byte aligned rows: 128-bit shared accesses
// along a row, conflict-free per quarter-warp) when the tile is filled row by row; 129 (odd)
// for a tall input, whose tile is filled transposed with 4-byte stores.
constexpr int kPitchWide = 132, kPitchTall = 129;

template <bool PF>
__global__ void __launch_bounds__(512, 3) kp_prep_operands(const __grid_constant__ PrepGroup g) {
  extern __shared__ float xs[];  // [128][pitch]
  const PrepMatrix& m = g.mat[blockIdx.z];
  const int64_t s = g.s, l = g.l;
  const int tall = m.tall;
  const int P = tall ? kPitchTall : kPitchWide;
  const int64_t ldg = tall ? g.s0 : g.l0;  // row length of G: a tall G is l0 x s0
  const float tau = g.clip ? m.scalars[g.ix.tau] : __int_as_float(0x7f800000);
  const float inv = m.scalars[g.ix.inv];
  const float sg = m.scalars[g.ix.sg_X0];
  const float six_sg = __fmul_rn(6.0f, sg);
  const int64_t r0 = (int64_t)blockIdx.y * 128, c0 = (int64_t)blockIdx.x * 128;  // tile origin in X
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  // The tile holds raw G values; clamp and scale are applied where a pass reads them.  A wide
  // input's rows go straight to shared memory with asynchronous 16-byte copies (64 KB in flight
  // per block without holding registers); a tall input's tile is filled transposed from registers.
  auto x0 = [&](float gval) { return __fmul_rn(fminf(fmaxf(gval, -tau), tau), inv); };
  // Rows and columns beyond the caller's matrix are zero padding (source size 0 of the copy
  // fills with zeros); the dimensions are multiples of 16, so a 16-byte piece is all in or all out.
  if (!tall) {
#pragma unroll
    for (int rr = warp; rr < 128; rr += 16) {
      const bool in = (r0 + rr) < g.s0 && (c0 + lane * 4) < g.l0;
      const float* src = in ? m.G + (r0 + rr) * ldg + c0 + lane * 4 : m.G;
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(xs + rr * P + lane * 4)), "l"(src),
                   "r"(in ? 16 : 0)
                   : "memory");
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
  } else {
#pragma unroll 4
    for (int rr = warp; rr < 128; rr += 16) {
      const bool in = (c0 + rr) < g.l0 && (r0 + lane * 4) < g.s0;
      float4 v = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
      if (in) v = __ldg(reinterpret_cast<const float4*>(m.G + (c0 + rr) * ldg + r0) + lane);
      xs[(lane * 4 + 0) * P + rr] = v.x; xs[(lane * 4 + 1) * P + rr] = v.y;
      xs[(lane * 4 + 2) * P + rr] = v.z; xs[(lane * 4 + 3) * P + rr] = v.w;
    }
  }
  __syncthreads();
  if (m.store_x) {
#pragma unroll 4
    for (int rr = warp; rr < 128; rr += 16) {
      const float* row = xs + rr * P + lane * 4;
      if ((r0 + rr) < m.x_rows && (c0 + lane * 4) < m.x_cols)
        *reinterpret_cast<float4*>(m.X + (r0 + rr) * m.x_cols + c0 + lane * 4) =
            make_float4(x0(row[0]), x0(row[1]), x0(row[2]), x0(row[3]));
    }
  }
  if (!g.write_q) return;
  const int part = (warp & 7) >> 2;  // which four of the eight 16-blocks this thread takes
  uint32_t code[8];                  // the codes of those four blocks: 32 consecutive bytes of the operand row
  uint32_t sfw = 0;
  if (warp < 8) {
    // blocks along the columns of X (contraction axis of G1): thread = row
    const int rr = (warp & 3) * 32 + lane;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int kb = part * 4 + q;
      float v[16];
      if (tall) {
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = x0(xs[rr * P + kb * 16 + i]);
      } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float4 t = *reinterpret_cast<const float4*>(xs + rr * P + kb * 16 + i * 4);
          v[4 * i] = x0(t.x); v[4 * i + 1] = x0(t.y); v[4 * i + 2] = x0(t.z); v[4 * i + 3] = x0(t.w);
        }
      }
      uint32_t sb;
      float unused;
      if (PF) sb = quantize_block16_opts(v, g.q, sg, code[2 * q], code[2 * q + 1], unused);
      else sb = quantize_block16(v, six_sg, sg, code[2 * q], code[2 * q + 1]);
      sfw |= sb << (8 * q);
    }
    uint4* dst = reinterpret_cast<uint4*>(m.qx_codes + (r0 + rr) * (l / 2) + (c0 + part * 64) / 2);
    dst[0] = make_uint4(code[0], code[1], code[2], code[3]);
    dst[1] = make_uint4(code[4], code[5], code[6], code[7]);
    *reinterpret_cast<uint32_t*>(m.qx_sf + sf_offset(r0 + rr, c0 / 16 + part * 4, l / 16)) = sfw;
  } else {
    // blocks along the rows of X (contraction axis of G3): thread = column of X = row of X^T
    const int cc = (warp & 3) * 32 + lane;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int gq = part * 4 + q;
      float v[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) v[i] = x0(xs[(gq * 16 + i) * P + cc]);
      uint32_t sb;
      float unused;
      if (PF) sb = quantize_block16_opts(v, g.q, sg, code[2 * q], code[2 * q + 1], unused);
      else sb = quantize_block16(v, six_sg, sg, code[2 * q], code[2 * q + 1]);
      sfw |= sb << (8 * q);
    }
    uint4* dst = reinterpret_cast<uint4*>(m.qt_codes + (c0 + cc) * (s / 2) + (r0 + part * 64) / 2);
    dst[0] = make_uint4(code[0], code[1], code[2], code[3]);
    dst[1] = make_uint4(code[4], code[5], code[6], code[7]);
    *reinterpret_cast<uint32_t*>(m.qt_sf + sf_offset(c0 + cc, r0 / 16 + part * 4, s / 16)) = sfw;
  }
}

}  // namespace

cudaError_t prologue_set_attributes() {
  cudaError_t e = cudaFuncSetAttribute(kp_prep_operands<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * kPitchWide * 4);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(kp_prep_operands<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * kPitchWide * 4);
}

// Enqueue the prologue for `count` matrices of one shape (s, l) and one parameter set.
cudaError_t launch_prologue_group(const PrologueItem* items, int count, int write_q, const QuantOpts& q,
                                  cudaStream_t st) {
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
    const int64_t cap = pl.s0 * pl.l0 / 8 < pl.s * pl.s ? pl.s0 * pl.l0 / 8 : pl.s * pl.s;
    g.cand_cap = (uint32_t)cap;
    g.eps = pl.eps;
    g.stat_blocks = pl.stat_blocks;
    g.write_q = write_q;
    g.zero_words = (int)(pl.zero_bytes / 4);
    g.ix = pl.ix;
    g.q = q;
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
      m.cand = reinterpret_cast<uint32_t*>(it.ws + L.A);
      m.qx_codes = it.ws + L.qX_codes; m.qx_sf = it.ws + L.qX_scales;
      m.qt_codes = it.ws + L.qXt_codes[0]; m.qt_sf = it.ws + L.qXt_scales[0];
      m.tall = it.pl->tall;
      m.clear_status = it.clear_status ? 1 : 0;
      m.store_x = it.store_x ? 1 : 0;
      m.x_rows = it.x_rows; m.x_cols = it.x_cols;
      m.hist_top = it.hist_top;
      if (!it.hist_top) all_counted = false;
    }
    const int sms = pl.sms;
    int64_t hb = (g.n4 + 512 * 4 - 1) / (512 * 4);
    const int hist_blocks = (int)(hb < (int64_t)sms * 4 ? (hb < 1 ? 1 : hb) : (int64_t)sms * 4);
    const dim3 gy1(1, (unsigned)nn), gh((unsigned)hist_blocks, (unsigned)nn), gs((unsigned)g.stat_blocks, (unsigned)nn);
    {
      ProfScope ps(FP4_PROF_CLIP, st);
      kp_init<<<dim3(4, (unsigned)nn), 256, 0, st>>>(g);
      count_launches(1);
      if (g.clip) {
        if (!all_counted) kp_hist_top<<<gh, 512, 0, st>>>(g);
        kp_pick_top<<<gy1, 256, 0, st>>>(g);
        count_launches(all_counted ? 1 : 2);
      }
    }
    {
      ProfScope ps(FP4_PROF_STATS, st);
      kp_compact_stats<<<gs, 256, 0, st>>>(g);
      kp_finalize<<<gy1, 1024, 0, st>>>(g);
      count_launches(2);
    }
    {
      ProfScope ps(FP4_PROF_PREP, st);
      const dim3 gp((unsigned)(pl.l / 128), (unsigned)(pl.s / 128), (unsigned)nn);
      if (q.rht || q.four_six) kp_prep_operands<true><<<gp, 512, 128 * kPitchWide * 4, st>>>(g);
      else kp_prep_operands<false><<<gp, 512, 128 * kPitchWide * 4, st>>>(g);
      count_launches(1);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace fp4
