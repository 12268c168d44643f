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
// epilogue combines with, 3 = TMA-store issuer, 4..11 = drain (TMEM lane quadrant =
// warp % 4; two sets of four split a tile's columns), 12..19 = finish.  The epilogue is a pipeline over a ring of 8 KB chunk buffers
// (16 FP32 columns x 128 rows) connected by mbarriers only: TMA load of the FP32 tile
// chunk -> drain (combine, quantise along the row, write the result chunk in place) ->
// TMA store and, concurrently, finish (quantise down the columns) -> slot free.  One
// persistent CTA per SM with three accumulator buffers in TMEM: the MMAs of the next tiles
// run while a tile is drained, so the operand ring never idles.
#include "fp4_gemm_common.cuh"

namespace fp4 {

namespace {

#ifndef FP4_BK
#define FP4_BK 256
#endif
#ifndef FP4_STAGES
#define FP4_STAGES 4
#endif
#ifndef FP4_RING
#define FP4_RING 10
#endif
constexpr int BM = 128, BN = 128, BK = FP4_BK;  // BK elements of K per stage: 64- or 128-byte operand rows
static_assert(BK == 128 || BK == 256, "operand rows of a stage are one TMA swizzle span");
constexpr int KSTEPS = BK / 64;               // MMAs (K = 64) per stage
constexpr uint32_t OPER_SWIZZLE = (BK == 256) ? 2u : 4u;  // UMMA layout type: 128- or 64-byte swizzle
constexpr uint32_t OPER_SBO = 8 * (BK / 2);   // bytes between 8-row groups of an operand tile
constexpr int STAGES = FP4_STAGES;          // operand stages of the main loop
constexpr int RING = FP4_RING;              // FP32 chunk buffers of the epilogue
constexpr int OPER_BYTES = BM * BK / 2;      // one operand tile of a stage
constexpr int SF_BYTES = KSTEPS * 512;       // one scale atom (128 rows x 4 blocks) per MMA, operand and stage
constexpr int CHUNK = 16;                    // FP32 columns per epilogue step
constexpr int CHUNK_BYTES = BM * CHUNK * 4;  // 8192
constexpr int NCHUNK = BN / CHUNK;

constexpr int OFF_A = 0;
constexpr int OFF_B = OFF_A + STAGES * OPER_BYTES;
constexpr int OFF_SFA = OFF_B + STAGES * OPER_BYTES;
constexpr int OFF_SFB = OFF_SFA + STAGES * SF_BYTES;
constexpr int OFF_RING = OFF_SFB + STAGES * SF_BYTES;
constexpr int OFF_BAR = OFF_RING + RING * CHUNK_BYTES;
constexpr int SMEM_BYTES = OFF_BAR + 512 + 1024;  // + slack to align the base to 1024
static_assert(SMEM_BYTES <= 232448, "one CTA per SM: at most 227 KB of dynamic shared memory");

// warps: 0 operand producer, 1 MMA issuer, 2 producer of the FP32 tile, 3 TMA-store issuer,
// 4..11 drain (TMEM -> registers -> ring; warps 4..7 take columns 0..63 of a tile, 8..11
// columns 64..127), 12..19 finish (transposed quantisation from the ring, same split)
constexpr int NTHREADS = 640;
constexpr int NACC = 3;                  // accumulator buffers: the MMAs of the next tiles run during a drain
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t TMEM_SF_COL = 384;    // scale factors after the accumulators
constexpr uint32_t SF_COLS = KSTEPS * 8; // per stage: 4 columns per MMA for each operand
static_assert(NACC * BN + STAGES * SF_COLS <= 512, "tensor memory columns");
constexpr int HALF_CHUNKS = NCHUNK / 2;
static_assert(RING % 2 == 0, "the ring is split between the two column halves of a tile");
constexpr int RING_HALF = RING / 2;

// Ring slot and use count of chunk c of the seq-th tile of this CTA.  Each column half of a
// tile has its own slots, used strictly in order by that half's drain and finish warps, so
// every waiter sees every phase of the barriers it waits on.
__device__ __forceinline__ void chunk_slot(uint32_t seq, int c, int& b, uint32_t& use) {
  const int h = c / HALF_CHUNKS;
  const uint32_t j = seq * HALF_CHUNKS + (uint32_t)(c - h * HALF_CHUNKS);
  b = h * RING_HALF + (int)(j % RING_HALF);
  use = j / RING_HALF;
}
// the single-thread roles walk the chunks of a tile alternating between the two halves
__device__ __forceinline__ int interleaved_chunk(int i) { return (i & 1) * HALF_CHUNKS + (i >> 1); }

// instruction descriptor: E2M1 x E2M1, UE4M3 scales, both operands K-major, M = N = 128
constexpr uint32_t IDESC = (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | (0u << 23) |
                           ((uint32_t)(BM >> 4) << 24);

struct Barriers {
  uint64_t full[STAGES];     // operand stage landed (TMA bytes)
  uint64_t empty[STAGES];    // operand stage consumed (MMA commit)
  uint64_t acc_full[NACC];   // accumulator complete (MMA commit)
  uint64_t acc_empty[NACC];  // accumulator drained (8 drain warps)
  uint64_t aux_full[RING];   // FP32 tile chunk landed in a ring slot (TMA bytes)
  uint64_t v_ready[RING];    // result chunk written to the slot (the 4 drain warps of its half)
  uint64_t slot_free[RING];  // slot read by everyone: the 4 finish warps of its half + the store warp
  uint32_t tmem_base;
  uint32_t abort_flag;
};
static_assert(sizeof(Barriers) <= 512, "barrier block");

template <int MODE, bool PF>
__global__ void __launch_bounds__(NTHREADS, 1)
k_gemm(const __grid_constant__ ProblemPack pack, const __grid_constant__ GemmLaunch args) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Barriers* bars = reinterpret_cast<Barriers*>(smem + OFF_BAR);
  volatile uint32_t* abort_flag = &bars->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const GemmProblem* probs = pack.p;
  const int tiles_per_problem = args.symmetric ? args.tiles_n * (args.tiles_n + 1) / 2 : args.tiles_m * args.tiles_n;
  const int num_tiles = tiles_per_problem * args.num_problems;
#ifdef FP4_DEBUG_ONE_KBLOCK
  const int num_kb = 1;  // timing experiments only: epilogue cost without the main loop
#else
  const int num_kb = (args.K + BK - 1) / BK;  // K is a multiple of 128: the last stage may be half full
#endif
  constexpr bool HAS_AUX = (MODE == kG2 || MODE == kG3);
  constexpr bool STORE_F32 = (MODE == kPlain || MODE == kG1 || MODE == kG3);
  const bool do_q = (MODE != kPlain) && args.write_q;

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { mbar_init(&bars->full[i], 1); mbar_init(&bars->empty[i], 1); }
    for (int i = 0; i < NACC; ++i) { mbar_init(&bars->acc_full[i], 1); mbar_init(&bars->acc_empty[i], 8); }
    for (int i = 0; i < RING; ++i) {
      mbar_init(&bars->aux_full[i], 1);
      mbar_init(&bars->v_ready[i], 4);
      mbar_init(&bars->slot_free[i], 5);
    }
    bars->abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;
  pdl_wait();   // set-up done; from here on the kernel reads what the launches before it wrote

  if (warp == 0) {
    // ------------------------------------------------------------ operand producer
    if (elect_one()) {
      int st = 0; uint32_t ph = 0; bool ok = true;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
        int p, ti, tj;
        decode_tile(t, args, tiles_per_problem, p, ti, tj);
        const GemmProblem* pr = probs + p;
        const uint8_t* sfa = pr->sfa + (size_t)ti * (args.K / 64) * 512;
        const uint8_t* sfb = pr->sfb + (size_t)tj * (args.K / 64) * 512;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!wait_bar(&bars->empty[st], ph ^ 1, abort_flag)) { ok = false; break; }
          // a half-full last stage: the operand boxes are zero-filled beyond K (and still
          // credit their full size), only the scale atoms that exist are fetched
          const int kvalid = args.K - kb * BK < BK ? args.K - kb * BK : BK;
          const uint32_t sf_bytes = (uint32_t)(kvalid / 64) * 512;
          mbar_expect_tx(&bars->full[st], 2 * OPER_BYTES + 2 * sf_bytes);
          tma_load_2d(smem + OFF_A + st * OPER_BYTES, &pr->tmA, kb * (BK / 2), ti * BM, &bars->full[st]);
          tma_load_2d(smem + OFF_B + st * OPER_BYTES, &pr->tmB, kb * (BK / 2), tj * BN, &bars->full[st]);
          bulk_load_1d(smem + OFF_SFA + st * SF_BYTES, sfa + (size_t)kb * SF_BYTES, sf_bytes, &bars->full[st]);
          bulk_load_1d(smem + OFF_SFB + st * SF_BYTES, sfb + (size_t)kb * SF_BYTES, sf_bytes, &bars->full[st]);
          if (++st == STAGES) { st = 0; ph ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (elect_one()) {
      int st = 0; uint32_t ph = 0, seq = 0; bool ok = true;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++seq) {
        const uint32_t ab = seq % NACC, ause = seq / NACC;
        if (!wait_bar(&bars->acc_empty[ab], (ause & 1) ^ 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + ab * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!wait_bar(&bars->full[st], ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sf_t = tmem_base + TMEM_SF_COL + st * SF_COLS;
          const int ksteps = (args.K - kb * BK < BK ? args.K - kb * BK : BK) / 64;
#pragma unroll
          for (int a = 0; a < KSTEPS; ++a) {
            if (a < ksteps) tc_cp_sf(sf_t + a * 4, umma_desc(smem_u32(smem + OFF_SFA + st * SF_BYTES + a * 512), 128, 0));
            if (a < ksteps) tc_cp_sf(sf_t + KSTEPS * 4 + a * 4,
                                     umma_desc(smem_u32(smem + OFF_SFB + st * SF_BYTES + a * 512), 128, 0));
          }
          const uint64_t adesc = umma_desc(smem_u32(smem + OFF_A + st * OPER_BYTES), OPER_SBO, OPER_SWIZZLE);
          const uint64_t bdesc = umma_desc(smem_u32(smem + OFF_B + st * OPER_BYTES), OPER_SBO, OPER_SWIZZLE);
#pragma unroll
          for (int k = 0; k < KSTEPS; ++k) {
            // 64 elements = 32 bytes further along K: +2 in the 16-byte address field
            if (k < ksteps)
              tc_mma_nvf4(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC, sf_t + k * 4, sf_t + KSTEPS * 4 + k * 4,
                          (kb | k) != 0 ? 1u : 0u);
          }
          tc_commit(&bars->empty[st]);
          if (++st == STAGES) { st = 0; ph ^= 1; }
        }
        if (!ok) break;
        tc_commit(&bars->acc_full[ab]);
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------ producer of the FP32 tile
    // Loads the chunk the epilogue combines with (A for G2, X for G3) into the ring slot
    // that will afterwards hold the result chunk, as soon as the slot is free: the loads
    // of a tile run ahead of its main loop.
    if (HAS_AUX && elect_one()) {
      uint32_t seq = 0; bool ok = true;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++seq) {
        int p, ti, tj;
        decode_tile(t, args, tiles_per_problem, p, ti, tj);
        const GemmProblem* pr = probs + p;
        for (int i = 0; i < NCHUNK; ++i) {
          const int c = interleaved_chunk(i);
          int b; uint32_t use;
          chunk_slot(seq, c, b, use);
          if (!wait_bar(&bars->slot_free[b], (use & 1) ^ 1, abort_flag)) { ok = false; break; }
          mbar_expect_tx(&bars->aux_full[b], CHUNK_BYTES);
          tma_load_2d(smem + OFF_RING + b * CHUNK_BYTES, &pr->tmAux, tj * BN + c * CHUNK, ti * BM, &bars->aux_full[b]);
        }
      }
    }
  } else if (warp == 3) {
    // ------------------------------------------------------------ TMA-store issuer
    // Stores each finished chunk and hands the slot back once the store has read it.
    if (elect_one()) {
      uint32_t seq = 0; bool ok = true;
      int prev_slot = -1;
      for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++seq) {
        int p, ti, tj;
        decode_tile(t, args, tiles_per_problem, p, ti, tj);
        const GemmProblem* pr = probs + p;
        for (int i = 0; i < NCHUNK; ++i) {
          const int c = interleaved_chunk(i);
          int b; uint32_t use;
          chunk_slot(seq, c, b, use);
          if (!wait_bar(&bars->v_ready[b], use & 1, abort_flag)) { ok = false; break; }
          // a chunk that starts outside the stored matrix (zero padding of the work shape) is dropped
          if (STORE_F32 && args.out_h == 0 && tj * BN + c * CHUNK < pr->out_cols && ti * BM < pr->out_rows) {
            tma_store_2d(&pr->tmOut, tj * BN + c * CHUNK, ti * BM, smem + OFF_RING + b * CHUNK_BYTES);
            bulk_commit();
            bulk_wait_read<1>();  // every store but the newest has read its slot
            if (prev_slot >= 0) mbar_arrive(&bars->slot_free[prev_slot]);
            prev_slot = b;
          } else {
            mbar_arrive(&bars->slot_free[b]);
          }
        }
      }
      if (STORE_F32) {
        bulk_wait_read<0>();
        if (prev_slot >= 0) mbar_arrive(&bars->slot_free[prev_slot]);
        bulk_wait_all<0>();
      }
    }
  } else if (warp < 12) {
    // ------------------------------------------------------------ drain warps
    // TMEM -> registers (thread = row), combine with the FP32 tile, quantise the blocks
    // that run along the row, write the result chunk into the ring slot.  Warps 4..7 take
    // the chunks of columns 0..63, warps 8..11 those of columns 64..127.
    const int half = (warp - 4) >> 2;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    float scale = 0.0f, sg_out = 1.0f, inv_sg = 1.0f;
    uint32_t rcp_base = 0;
    float ca = 0.0f, cb = 0.0f, cc = 0.0f;
    float tau = 0.0f, inv = 0.0f;  // first G3 stage on the raw input: X0 = clamp(G, tau) * inv
    bool raw = false;
    const GemmProblem* pr = nullptr;
    int cur_p = -1;
    const int sw = (row >> 1) & 3;
    const uint32_t tm_lane = tmem_base + ((uint32_t)(quad * 32) << 16);

    uint32_t seq = 0;
    float amax = 0.0f;
    bool ok = true;
    for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++seq) {
      int p, ti, tj;
      decode_tile(t, args, tiles_per_problem, p, ti, tj);
      if (p != cur_p) {
        // a new matrix: hand in the running maximum of the previous one, fetch this one's scalars
        if ((MODE == kG1 || MODE == kG3) && cur_p >= 0) {
#pragma unroll
          for (int o = 16; o; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
          if (lane == 0) {
            const int slot = (MODE == kG1) ? args.ix.amax_A0 + args.iter : args.ix.amax_X0 + args.iter + 1;
            atomicMax(reinterpret_cast<uint32_t*>(pr->scalars + slot), __float_as_uint(amax));
          }
          amax = 0.0f;
        }
        cur_p = p;
        pr = probs + p;
        // the CTA that owns a matrix's first tile publishes its output scale
        epilogue_scalars<MODE>(*pr, args, scale, sg_out, t == p * tiles_per_problem && threadIdx.x == 128);
        inv_sg = __frcp_rn(sg_out);  // exact: the predicted scales are powers of two
        rcp_base = rcp_base_of(sg_out);
        ca = pr->ca; cb = pr->cb; cc = pr->cc;
        raw = (MODE == kG3) && pr->aux_raw != 0;
        if (raw) {
          tau = args.clip ? pr->scalars[args.ix.tau] : __int_as_float(0x7f800000);
          inv = pr->scalars[args.ix.inv];
        }
      }
      const bool mirror = do_q && (MODE == kG3 || (args.symmetric && ti != tj));
      // give-up decisions are made warp-uniform: the TMEM loads below are warp-collective
      const uint32_t ab = seq % NACC, ause = seq / NACC;
      ok = __all_sync(0xffffffffu, wait_bar(&bars->acc_full[ab], ause & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      const int64_t grow = (int64_t)ti * BM + row;
      const uint32_t tm_acc = tm_lane + ab * BN;
      uint32_t sfw = 0;
      uint32_t acc[16];
      tc_ld16_issue(tm_acc + half * HALF_CHUNKS * CHUNK, acc);
      for (int c = half * HALF_CHUNKS; c < (half + 1) * HALF_CHUNKS; ++c) {
        int b; uint32_t use;
        chunk_slot(seq, c, b, use);
        uint8_t* slot_row = smem + OFF_RING + b * CHUNK_BYTES + row * 64;
        float v[16];
        // the slot: holds the FP32 tile chunk (G2, G3) or must be free (G1, plain)
        if (HAS_AUX) ok = __all_sync(0xffffffffu, wait_bar(&bars->aux_full[b], use & 1, abort_flag));
        else ok = __all_sync(0xffffffffu, wait_bar(&bars->slot_free[b], (use & 1) ^ 1, abort_flag));
        if (!ok) break;
        tc_wait_ld16(acc);
        if (HAS_AUX) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            float4 x = *reinterpret_cast<const float4*>(slot_row + ((j ^ sw) << 4));
            float e[4] = {x.x, x.y, x.z, x.w};
            if (MODE == kG3 && raw) {
#pragma unroll
              for (int q = 0; q < 4; ++q) e[q] = __fmul_rn(fminf(fmaxf(e[q], -tau), tau), inv);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const float prod = __fmul_rn(__uint_as_float(acc[4 * j + q]), scale);
              if (MODE == kG2) v[4 * j + q] = __fadd_rn(__fmul_rn(cb, e[q]), __fmul_rn(cc, prod));
              else v[4 * j + q] = __fadd_rn(__fmul_rn(ca, e[q]), prod);
            }
          }
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] = __fmul_rn(__uint_as_float(acc[i]), scale);
        }
        // the next chunk's accumulator columns are fetched while this chunk is finished
        if (c + 1 < (half + 1) * HALF_CHUNKS) {
          tc_ld16_issue(tm_acc + (c + 1) * CHUNK, acc);
        } else {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&bars->acc_empty[ab]);  // this warp is done with the accumulator
        }
        if (STORE_F32 && MODE != kPlain && args.out_h == 2) {
          // BF16 storage kept in an FP32 tensor: this thread stores the rounded values of its row itself
          const int64_t gcol0 = (int64_t)tj * BN + c * CHUNK;
          if (grow < pr->out_rows && gcol0 < pr->out_cols) {
            float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(pr->out_direct) + grow * pr->out_direct_ld + gcol0);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const uint32_t w0 = cvt_bf16x2(v[4 * j], v[4 * j + 1]), w1 = cvt_bf16x2(v[4 * j + 2], v[4 * j + 3]);
              dst[j] = make_float4(bf16_lo(w0), bf16_hi(w0), bf16_lo(w1), bf16_hi(w1));
            }
          }
        }
        if ((STORE_F32 && args.out_h == 0) || mirror) {
#pragma unroll
          for (int j = 0; j < 4; ++j)
            *reinterpret_cast<float4*>(slot_row + ((j ^ sw) << 4)) =
                make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
          fence_proxy_async_smem();
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->v_ready[b]);
        if (do_q) {
          uint32_t lo, hi;
          float bmax;
          uint32_t sb;
          if (PF) sb = quantize_block16_opts(v, args.q, sg_out, lo, hi, bmax);
          else sb = quantize_block16_pow2(v, sg_out, inv_sg, rcp_base, lo, hi, bmax);
          if (MODE == kG1 || MODE == kG3) amax = fmaxf(amax, bmax);
          const int64_t gcol = (int64_t)tj * BN + c * CHUNK;
          *reinterpret_cast<uint2*>(pr->rq_codes + grow * (args.rq_K / 2) + gcol / 2) = make_uint2(lo, hi);
          sfw |= sb << (8 * (c & 3));
          if ((c & 3) == 3) {
            *reinterpret_cast<uint32_t*>(pr->rq_sf + sf_offset(grow, (gcol >> 4) & ~3ll, args.rq_K >> 4)) = sfw;
            sfw = 0;
          }
        }
      }
    }
    if ((MODE == kG1 || MODE == kG3) && cur_p >= 0) {
#pragma unroll
      for (int o = 16; o; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
      if (lane == 0) {
        const int slot = (MODE == kG1) ? args.ix.amax_A0 + args.iter : args.ix.amax_X0 + args.iter + 1;
        atomicMax(reinterpret_cast<uint32_t*>(pr->scalars + slot), __float_as_uint(amax));
      }
    }
  } else {
    // ------------------------------------------------------------ finish warps
    // Blocks of 16 that run down this tile's rows (the transposed operand copy in G3, the
    // mirrored triangle in G1/G2): thread = (column cc of the chunk, row group g).
    const int half = (warp - 12) >> 2;
    const int et = ((warp - 12) & 3) * 32 + lane;
    const int cc = et & 15, g = et >> 4;
    const int rot = (lane >> 4) & 1;
    float scale, sg_out = 1.0f, inv_sg = 1.0f;
    uint32_t rcp_base = 0;
    const GemmProblem* pr = nullptr;
    int cur_p = -1;
    uint32_t seq = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++seq) {
      int p, ti, tj;
      decode_tile(t, args, tiles_per_problem, p, ti, tj);
      if (p != cur_p) {
        cur_p = p;
        pr = probs + p;
        epilogue_scalars<MODE>(*pr, args, scale, sg_out, false);
        inv_sg = __frcp_rn(sg_out);
        rcp_base = rcp_base_of(sg_out);
      }
      const bool mirror = do_q && (MODE == kG3 || (args.symmetric && ti != tj));
      for (int c = half * HALF_CHUNKS; c < (half + 1) * HALF_CHUNKS; ++c) {
        int b; uint32_t use;
        chunk_slot(seq, c, b, use);
        ok = __all_sync(0xffffffffu, wait_bar(&bars->v_ready[b], use & 1, abort_flag));
        if (!ok) break;
        if (mirror) {
          const uint8_t* obase = smem + OFF_RING + b * CHUNK_BYTES;
          float w[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            // the upper half-warp starts one row later (and wraps), so that the two half-warps
            // read rows of different parity, i.e. different banks
            const int r = g * 16 + ((i + rot) & 15);
            w[i] = *reinterpret_cast<const float*>(obase + r * 64 + ((((cc >> 2) ^ ((r >> 1) & 3))) << 4) + (cc & 3) * 4);
          }
          uint32_t lo, hi;
          float bmax;
          uint32_t sb;
          if (PF) {
            // the transform and the error sums need the block in row order
            float x[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) x[i] = rot ? w[(i + 15) & 15] : w[i];
            sb = quantize_block16_opts(x, args.q, sg_out, lo, hi, bmax);
          } else {
            sb = quantize_block16_pow2(w, sg_out, inv_sg, rcp_base, lo, hi, bmax);
            if (rot) {
              // the codes were packed one row early: rotate the 16 nibbles back into row order
              const uint32_t nlo = (lo << 4) | (hi >> 28), nhi = (hi << 4) | (lo >> 28);
              lo = nlo; hi = nhi;
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(&bars->slot_free[b]);  // the slot's values are in registers
          const int64_t trow = (int64_t)tj * BN + c * CHUNK + cc;  // row of the mirrored / transposed tensor
          const int64_t tcol = (int64_t)ti * BM + g * 16;
          *reinterpret_cast<uint2*>(pr->cq_codes + trow * (args.cq_K / 2) + tcol / 2) = make_uint2(lo, hi);
          pr->cq_sf[sf_offset(trow, tcol >> 4, args.cq_K >> 4)] = (uint8_t)sb;
        } else {
          __syncwarp();
          if (lane == 0) mbar_arrive(&bars->slot_free[b]);
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (threadIdx.x == 0 && bars->abort_flag) report_timeout(args.status);
}

template <int MODE, bool PF>
cudaError_t launch_mode(const ProblemPack& pack, const GemmLaunch& L, int sms, cudaStream_t st) {
  const int tpp = L.symmetric ? L.tiles_n * (L.tiles_n + 1) / 2 : L.tiles_m * L.tiles_n;
  const int num_tiles = tpp * L.num_problems;
  int grid = sms;
  if (grid > num_tiles) grid = num_tiles;
  count_launches(1);
  launch_chained(k_gemm<MODE, PF>, dim3(grid), dim3(NTHREADS), SMEM_BYTES, st, pack, L);
  return cudaGetLastError();
}

}  // namespace

int gemm_stage_k() { return BK; }

cudaError_t gemm_set_attributes() {
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(k_gemm<kPlain, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm<kG1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm<kG1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm<kG2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm<kG2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm<kG3, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm<kG3, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  return cudaSuccess;
}

cudaError_t launch_gemm(GemmMode mode, const ProblemPack& pack, const GemmLaunch& launch, int sms, cudaStream_t st) {
  if (launch.num_problems < 1 || launch.num_problems > kPackMax) return cudaErrorInvalidValue;
  const bool pf = launch.q.rht || launch.q.four_six;
  switch (mode) {
    case kPlain: return launch_mode<kPlain, false>(pack, launch, sms, st);
    case kG1: return pf ? launch_mode<kG1, true>(pack, launch, sms, st) : launch_mode<kG1, false>(pack, launch, sms, st);
    case kG2: return pf ? launch_mode<kG2, true>(pack, launch, sms, st) : launch_mode<kG2, false>(pack, launch, sms, st);
    default: return pf ? launch_mode<kG3, true>(pack, launch, sms, st) : launch_mode<kG3, false>(pack, launch, sms, st);
  }
}

}  // namespace fp4
