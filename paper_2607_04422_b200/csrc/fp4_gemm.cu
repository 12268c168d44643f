// Block-scaled NVFP4 GEMM on the 5th-generation tensor cores, with the fused
// epilogues of the Newton-Schulz iteration (Section 3.4, display equations):
//
//   G1:  A  = qX qX^T                      -> A (FP32), qA = Q_1x16(A), amax(A)
//   G2:  B  = b A + c qA qA^{16x1}         -> qB = Q_1x16(B)
//   G3:  X+ = a X + qB qX^{16x1}           -> X+ (FP32), Q_1x16(X+), Q_16x1(X+), amax(X+)
//
// Every product is "row operand times column operand transposed" with both operands
// K-major (16-element blocks along the contraction axis), which is the form
// tcgen05.mma kind::mxf4nvf4 consumes.  A and B are symmetric, so G1 and G2 compute the
// tiles on and above the diagonal only and write the quantised mirror image of each
// off-diagonal tile themselves (a block of 16 along the mirror's rows is a block of 16
// down this tile's columns).
//
// One CTA owns 128 x 128 output tiles.  Warp roles: 0 = TMA producer of operand stages,
// 1 = MMA issuer (one thread) and TMEM owner, 2 = TMA producer of the FP32 tile the
// epilogue combines with, 3..6 = epilogue (TMEM lane quadrant = warp % 4).  Two CTAs
// share an SM, so one CTA's epilogue overlaps the other's main loop.
#include "fp4_kernels.h"

namespace fp4 {

namespace {

constexpr int BM = 128, BN = 128, BK = 128;
#ifndef FP4_STAGES
#define FP4_STAGES 4
#endif
constexpr int STAGES = FP4_STAGES;
constexpr int OPER_BYTES = BM * BK / 2;      // 8192: one operand tile of a stage (64-byte rows)
constexpr int SF_BYTES = 2 * 512;            // two scale atoms (128 rows x 8 blocks) per operand and stage
constexpr uint32_t STAGE_TX = 2 * OPER_BYTES + 2 * SF_BYTES;
constexpr int CHUNK = 16;                    // FP32 columns per epilogue step
constexpr int CHUNK_BYTES = BM * CHUNK * 4;  // 8192
constexpr int NCHUNK = BN / CHUNK;

constexpr int OFF_A = 0;
constexpr int OFF_B = OFF_A + STAGES * OPER_BYTES;
constexpr int OFF_SFA = OFF_B + STAGES * OPER_BYTES;
constexpr int OFF_SFB = OFF_SFA + STAGES * SF_BYTES;
constexpr int OFF_AUX = OFF_SFB + STAGES * SF_BYTES;
constexpr int OFF_OUT = OFF_AUX + 2 * CHUNK_BYTES;
constexpr int OFF_BAR = OFF_OUT + 2 * CHUNK_BYTES;
constexpr int SMEM_BYTES = OFF_BAR + 256 + 1024;  // + slack to align the base to 1024

constexpr int NTHREADS = 224;
constexpr int EPI_THREADS = 128;
constexpr uint32_t TMEM_COLS = 256;
constexpr uint32_t TMEM_SF_COL = 128;  // scale factors: 16 columns per stage after the accumulator

// instruction descriptor: E2M1 x E2M1, UE4M3 scales, both operands K-major, M = N = 128
constexpr uint32_t IDESC = (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | (0u << 23) |
                           ((uint32_t)(BM >> 4) << 24);

struct Barriers {
  uint64_t full[STAGES];
  uint64_t empty[STAGES];
  uint64_t acc_full;
  uint64_t acc_empty;
  uint64_t aux_full[2];
  uint64_t aux_empty[2];
  uint32_t tmem_base;
  uint32_t abort_flag;
};

__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Wait on an mbarrier phase for at most two seconds; false on give-up (own time-out or
// another thread's abort flag).
__device__ __noinline__ bool wait_slow(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag) {
  const uint64_t t0 = globaltimer_ns();
  for (;;) {
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (globaltimer_ns() - t0 > 2000000000ull) {
      *abort_flag = 1;
      return false;
    }
  }
}
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  return wait_slow(bar, parity, abort_flag);
}

// barrier over the epilogue threads that also ANDs a predicate
__device__ __forceinline__ bool epi_barrier_and(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %1, 0;\n\t"
      "barrier.cta.red.and.pred q, 1, 128, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)pred)
      : "memory");
  return r != 0;
}

__device__ __forceinline__ void decode_tile(int t, int tiles_n, int symmetric, int& ti, int& tj) {
  if (!symmetric) {
    ti = t / tiles_n;
    tj = t - ti * tiles_n;
  } else {
    int row = 0, rem = t;
    while (rem >= tiles_n - row) { rem -= tiles_n - row; ++row; }
    ti = row;
    tj = row + rem;
  }
}

template <int MODE>
__global__ void __launch_bounds__(NTHREADS, 2)
k_gemm(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
       const __grid_constant__ CUtensorMap tmAux, const __grid_constant__ CUtensorMap tmOut, const GemmArgs args) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Barriers* bars = reinterpret_cast<Barriers*>(smem + OFF_BAR);
  volatile uint32_t* abort_flag = &bars->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_tiles = args.symmetric ? args.tiles_n * (args.tiles_n + 1) / 2 : args.tiles_m * args.tiles_n;
  const int num_kb = args.K / BK;
  constexpr bool HAS_AUX = (MODE == kG2 || MODE == kG3);
  constexpr bool STORE_F32 = (MODE == kPlain || MODE == kG1 || MODE == kG3);

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { mbar_init(&bars->full[i], 1); mbar_init(&bars->empty[i], 1); }
    mbar_init(&bars->acc_full, 1);
    mbar_init(&bars->acc_empty, EPI_THREADS);
    for (int i = 0; i < 2; ++i) { mbar_init(&bars->aux_full[i], 1); mbar_init(&bars->aux_empty[i], EPI_THREADS); }
    bars->abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    if (HAS_AUX) tma_prefetch_desc(&tmAux);
    if (STORE_F32) tma_prefetch_desc(&tmOut);
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------ operand producer
    if (elect_one()) {
      int st = 0; uint32_t ph = 0; bool ok = true;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
        int ti, tj;
        decode_tile(t, args.tiles_n, args.symmetric, ti, tj);
        const uint8_t* sfa = args.sfa + (size_t)ti * (args.K / 64) * 512;
        const uint8_t* sfb = args.sfb + (size_t)tj * (args.K / 64) * 512;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!wait_bar(&bars->empty[st], ph ^ 1, abort_flag)) { ok = false; break; }
          mbar_expect_tx(&bars->full[st], STAGE_TX);
          tma_load_2d(smem + OFF_A + st * OPER_BYTES, &tmA, kb * (BK / 2), ti * BM, &bars->full[st]);
          tma_load_2d(smem + OFF_B + st * OPER_BYTES, &tmB, kb * (BK / 2), tj * BN, &bars->full[st]);
          bulk_load_1d(smem + OFF_SFA + st * SF_BYTES, sfa + (size_t)kb * SF_BYTES, SF_BYTES, &bars->full[st]);
          bulk_load_1d(smem + OFF_SFB + st * SF_BYTES, sfb + (size_t)kb * SF_BYTES, SF_BYTES, &bars->full[st]);
          if (++st == STAGES) { st = 0; ph ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (elect_one()) {
      int st = 0; uint32_t ph = 0, acc_ph = 0; bool ok = true;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
        if (!wait_bar(&bars->acc_empty, acc_ph ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!wait_bar(&bars->full[st], ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sf_t = tmem_base + TMEM_SF_COL + st * 16;
#pragma unroll
          for (int a = 0; a < 2; ++a) {
            tc_cp_sf(sf_t + a * 4, umma_desc(smem_u32(smem + OFF_SFA + st * SF_BYTES + a * 512), 128, 0));
            tc_cp_sf(sf_t + 8 + a * 4, umma_desc(smem_u32(smem + OFF_SFB + st * SF_BYTES + a * 512), 128, 0));
          }
          const uint64_t adesc = umma_desc(smem_u32(smem + OFF_A + st * OPER_BYTES), 512, 4);
          const uint64_t bdesc = umma_desc(smem_u32(smem + OFF_B + st * OPER_BYTES), 512, 4);
#pragma unroll
          for (int k = 0; k < 2; ++k) {
            // 64 elements = 32 bytes further along K: +2 in the 16-byte address field
            tc_mma_nvf4(tmem_base, adesc + 2 * k, bdesc + 2 * k, IDESC, sf_t + k * 4, sf_t + 8 + k * 4,
                        (kb | k) != 0 ? 1u : 0u);
          }
          tc_commit(&bars->empty[st]);
          if (++st == STAGES) { st = 0; ph ^= 1; }
        }
        if (!ok) break;
        tc_commit(&bars->acc_full);
        acc_ph ^= 1;
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------ producer of the FP32 tile
    if (HAS_AUX && elect_one()) {
      uint32_t it = 0; bool ok = true;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
        int ti, tj;
        decode_tile(t, args.tiles_n, args.symmetric, ti, tj);
        for (int c = 0; c < NCHUNK; ++c, ++it) {
          const int b = it & 1;
          if (!wait_bar(&bars->aux_empty[b], ((it >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
          mbar_expect_tx(&bars->aux_full[b], CHUNK_BYTES);
          tma_load_2d(smem + OFF_AUX + b * CHUNK_BYTES, &tmAux, tj * BN + c * CHUNK, ti * BM, &bars->aux_full[b]);
        }
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue
    const int quad = warp & 3;
    const int row = quad * 32 + lane;           // row of the tile this thread owns (TMEM lane)
    const int et = (warp - 3) * 32 + lane;      // index among the epilogue threads
    const bool leader = (et == 0);

    // per-call scalars (written by earlier kernels of the stream)
    float scale, sg_out = 1.0f;
    float* sc = args.scalars;
    if (MODE == kPlain) {
      scale = __fmul_rn(args.sg_a, args.sg_b);
    } else if (MODE == kG1) {
      const float sgx = sc[args.ix.sg_X0 + args.iter];
      const float ax = sc[args.ix.amax_X0 + args.iter];
      scale = __fmul_rn(sgx, sgx);
      float bound = __fmul_rn(__fmul_rn(__fmul_rn(2.0f, args.l_cols), ax), ax);
      sg_out = scale_predicted(fminf(bound, 4.0f));
      if (blockIdx.x == 0 && leader) sc[args.ix.sg_A0 + args.iter] = sg_out;
    } else if (MODE == kG2) {
      const float sga = sc[args.ix.sg_A0 + args.iter];
      const float aa = sc[args.ix.amax_A0 + args.iter];
      scale = __fmul_rn(sga, sga);
      float bound = __fmul_rn(__fadd_rn(fabsf(args.cb), __fmul_rn(4.0f, fabsf(args.cc))), aa);
      sg_out = scale_predicted(bound);
      if (blockIdx.x == 0 && leader) sc[args.ix.sg_B0 + args.iter] = sg_out;
    } else {
      const float sgb = sc[args.ix.sg_B0 + args.iter];
      const float sgx = sc[args.ix.sg_X0 + args.iter];
      const float ax = sc[args.ix.amax_X0 + args.iter];
      scale = __fmul_rn(sgb, sgx);
      float bound = __fmul_rn(__fmul_rn(4.0f, fabsf(args.ca)), ax);
      sg_out = scale_predicted(bound);
      if (blockIdx.x == 0 && leader) sc[args.ix.sg_X0 + args.iter + 1] = sg_out;
    }
    const float six_sg = __fmul_rn(6.0f, sg_out);
    const bool do_q = (MODE != kPlain) && args.write_q;

    uint32_t acc_ph = 0, it = 0;
    float amax = 0.0f;
    bool ok = true;
    for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
      int ti, tj;
      decode_tile(t, args.tiles_n, args.symmetric, ti, tj);
      const bool mirror = do_q && (MODE == kG3 || (args.symmetric && ti != tj));
      // give-up decisions are made warp-uniform: the TMEM loads below are warp-collective
      bool tile_ok = __all_sync(0xffffffffu, wait_bar(&bars->acc_full, acc_ph, abort_flag));
      acc_ph ^= 1;
      tc_fence_after();
      const int64_t grow = (int64_t)ti * BM + row;  // global row of this thread
      uint32_t sfw = 0;
      for (int c = 0; c < NCHUNK; ++c, ++it) {
        const int b = it & 1;
        float v[16];
        if (tile_ok) {
          float acc[16];
          tc_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + c * CHUNK, acc);
          if (c == NCHUNK - 1) {  // accumulator drained: the next tile's MMAs may start
            tc_fence_before();
            mbar_arrive(&bars->acc_empty);
          }
          if (HAS_AUX) {
            tile_ok = __all_sync(0xffffffffu, wait_bar(&bars->aux_full[b], (it >> 1) & 1, abort_flag));
            if (tile_ok) {
              const uint8_t* arow = smem + OFF_AUX + b * CHUNK_BYTES + row * 64;
              const int sw = (row >> 1) & 3;
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                float4 x = *reinterpret_cast<const float4*>(arow + ((j ^ sw) << 4));
                float e[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  const float p = __fmul_rn(acc[4 * j + q], scale);
                  if (MODE == kG2) v[4 * j + q] = __fadd_rn(__fmul_rn(args.cb, e[q]), __fmul_rn(args.cc, p));
                  else v[4 * j + q] = __fadd_rn(__fmul_rn(args.ca, e[q]), p);
                }
              }
              mbar_arrive(&bars->aux_empty[b]);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = __fmul_rn(acc[i], scale);
          }
        }
        if (tile_ok) {
          if (MODE == kG1 || MODE == kG3) {
#pragma unroll
            for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(v[i]));
          }
          if (do_q) {
            // blocks of 16 along this tile's columns: in-thread
            uint32_t lo, hi;
            uint32_t sb = quantize_block16(v, six_sg, sg_out, lo, hi);
            const int64_t gcol = (int64_t)tj * BN + c * CHUNK;
            *reinterpret_cast<uint2*>(args.rq_codes + grow * (args.rq_K / 2) + gcol / 2) = make_uint2(lo, hi);
            sfw |= sb << (8 * (c & 3));
            if ((c & 3) == 3) {
              *reinterpret_cast<uint32_t*>(args.rq_sf + sf_offset(grow, (gcol >> 4) & ~3ll, args.rq_K >> 4)) = sfw;
              sfw = 0;
            }
          }
          if (STORE_F32 || mirror) {
            // stage the FP32 chunk in the 64-byte-swizzled layout TMA stores from
            uint8_t* orow = smem + OFF_OUT + b * CHUNK_BYTES + row * 64;
            const int sw = (row >> 1) & 3;
#pragma unroll
            for (int j = 0; j < 4; ++j)
              *reinterpret_cast<float4*>(orow + ((j ^ sw) << 4)) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            fence_proxy_async_smem();
          }
        }
        // the previous chunk's store must have read its staging buffer before the next
        // chunk overwrites it
        if (STORE_F32 && leader) bulk_wait_read<0>();
        if (!epi_barrier_and(tile_ok)) { ok = false; break; }
        if (STORE_F32 && leader) {
          tma_store_2d(&tmOut, tj * BN + c * CHUNK, ti * BM, smem + OFF_OUT + b * CHUNK_BYTES);
          bulk_commit();
        }
        if (mirror) {
          // blocks of 16 down this tile's rows: thread = (column cc, row group g)
          const int cc = et & 15, g = et >> 4;
          const uint8_t* obase = smem + OFF_OUT + b * CHUNK_BYTES;
          float w[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int r = g * 16 + i;
            w[i] = *reinterpret_cast<const float*>(obase + r * 64 + ((((cc >> 2) ^ ((r >> 1) & 3))) << 4) + (cc & 3) * 4);
          }
          uint32_t lo, hi;
          uint32_t sb = quantize_block16(w, six_sg, sg_out, lo, hi);
          const int64_t trow = (int64_t)tj * BN + c * CHUNK + cc;  // row of the mirrored / transposed tensor
          const int64_t tcol = (int64_t)ti * BM + g * 16;
          *reinterpret_cast<uint2*>(args.cq_codes + trow * (args.cq_K / 2) + tcol / 2) = make_uint2(lo, hi);
          args.cq_sf[sf_offset(trow, tcol >> 4, args.cq_K >> 4)] = (uint8_t)sb;
        }
      }
    }
    if (MODE == kG1 || MODE == kG3) {
#pragma unroll
      for (int o = 16; o; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
      if (lane == 0) {
        const int slot = (MODE == kG1) ? args.ix.amax_A0 + args.iter : args.ix.amax_X0 + args.iter + 1;
        atomicMax(reinterpret_cast<uint32_t*>(sc + slot), __float_as_uint(amax));
      }
    }
    if (STORE_F32 && leader) bulk_wait_all<0>();
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (threadIdx.x == 0 && bars->abort_flag) report_timeout(args.status);
}

template <int MODE>
cudaError_t launch_mode(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmAux,
                        const CUtensorMap& tmOut, const GemmArgs& args, int sms, cudaStream_t st) {
  const int num_tiles = args.symmetric ? args.tiles_n * (args.tiles_n + 1) / 2 : args.tiles_m * args.tiles_n;
  int grid = 2 * sms;
  if (grid > num_tiles) grid = num_tiles;
  count_launches(1);
  k_gemm<MODE><<<grid, NTHREADS, SMEM_BYTES, st>>>(tmA, tmB, tmAux, tmOut, args);
  return cudaGetLastError();
}

}  // namespace

cudaError_t gemm_set_attributes() {
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(k_gemm<kPlain>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm<kG1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm<kG2>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm<kG3>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  return cudaSuccess;
}

cudaError_t launch_gemm(GemmMode mode, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmAux,
                        const CUtensorMap& tmOut, const GemmArgs& args, int sms, cudaStream_t st) {
  switch (mode) {
    case kPlain: return launch_mode<kPlain>(tmA, tmB, tmAux, tmOut, args, sms, st);
    case kG1: return launch_mode<kG1>(tmA, tmB, tmAux, tmOut, args, sms, st);
    case kG2: return launch_mode<kG2>(tmA, tmB, tmAux, tmOut, args, sms, st);
    default: return launch_mode<kG3>(tmA, tmB, tmAux, tmOut, args, sms, st);
  }
}

}  // namespace fp4
