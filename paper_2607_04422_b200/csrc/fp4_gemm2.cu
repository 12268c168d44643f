// The same block-scaled NVFP4 GEMM and fused Newton-Schulz epilogues as fp4_gemm.cu
// (Section 3.4, display equations), for shapes whose dimensions are multiples of 256:
// a pair of CTAs on two SMs (a cluster of 2) computes one 256 x 256 output tile with
// tcgen05.mma.cta_group::2.  Each CTA holds 128 rows of the row operand and 128 of the 256
// rows of the column operand in its shared memory, so every byte fetched from L2 and every
// byte the tensor core reads from shared memory feeds twice as many multiply-adds as in the
// 128 x 128 single-CTA kernel, whose main loop is bound by exactly that traffic.
//
// Per CTA: accumulator 128 lanes x 256 FP32 columns in tensor memory, drained in sixteen
// 16-column chunks by sixteen epilogue warps: four teams of four warps, a team owns four
// chunks of a tile, a warp of a team the 32 accumulator lanes of its quadrant.  For one chunk
// a warp combines its 32 x 16 block with the FP32 tile, quantises it along the rows, stages
// it in shared memory for the TMA store and, reading its own block back column-wise,
// quantises it down the columns (the transposed / mirrored operand copy): both
// quantisations of a block stay inside one warp, no hand-over between warps.  Only the even
// CTA of a pair issues MMAs; both CTAs run every other role on their own 128 rows.  TMA
// loads of both CTAs signal the even CTA's stage barrier; MMA completion is multicast to the
// stage and accumulator barriers of both CTAs.
#include "fp4_gemm_common.cuh"

namespace fp4 {

namespace {

#ifndef FP4_STAGES2
#define FP4_STAGES2 4
#endif
#ifndef FP4_RING2
#define FP4_RING2 8
#endif
constexpr int PM = 256, PN = 256;              // output tile of a CTA pair
constexpr int BM = 128;                        // rows per CTA
constexpr int BK = 256;                        // elements of K per stage: 128-byte operand rows
constexpr int KSTEPS = BK / 64;
constexpr int STAGES = FP4_STAGES2;
constexpr int RING = FP4_RING2;
constexpr int OPER_BYTES = BM * BK / 2;        // 16 KB: 128 rows of one operand
constexpr int SF_ATOMS = KSTEPS * 512;         // scale atoms of one 128-row block and stage
constexpr int SF_BYTES = 3 * SF_ATOMS;         // row operand: own block; column operand: both blocks
constexpr uint32_t STAGE_BYTES_CTA = 2 * OPER_BYTES + SF_BYTES;
constexpr int CHUNK = 16;
constexpr int CHUNK_BYTES = BM * CHUNK * 4;    // 8 KB
constexpr int NCHUNK = PN / CHUNK;             // 16
constexpr int TEAMS = 4;                       // epilogue teams (of four warps) per CTA
constexpr int TEAM_CHUNKS = NCHUNK / TEAMS;    // 4: one 64-column group, one 32-bit word of row scales
static_assert(RING % TEAMS == 0, "the ring is split between the teams");
constexpr int RING_TEAM = RING / TEAMS;

// Two consecutive tiles use two accumulator buffers that share OV_CHUNKS chunks of tensor
// memory (512 columns cannot hold two 256-column accumulators plus the scale factors):
// buffer 0 = columns [0, 256), buffer 1 = columns [240, 496), scale factors [496, 508).
// The shared columns are buffer 0's last chunk and buffer 1's first; the half that owns them
// drains them first and reports it, then the next tile's MMAs may start while the rest of
// the tile is still being drained.  The time from "accumulator complete" to that report is
// on the critical path of every tile (drain of the shared chunk, then the next main loop),
// which is why the scale factors get only the 12 columns one MMA needs.
#ifndef FP4_OV_CHUNKS
#define FP4_OV_CHUNKS 1
#endif
constexpr int OV_CHUNKS = FP4_OV_CHUNKS;
constexpr uint32_t ACC1_COL = PN - OV_CHUNKS * CHUNK;  // 240

static_assert(OV_CHUNKS <= TEAM_CHUNKS, "the shared chunks belong to one team");
static_assert(TEAM_CHUNKS == 4, "a team writes one 32-bit word of row scales per row and tile");
// chunk handled at position i by team t in a tile that uses buffer `par`: buffer 0 shares its
// last chunks, which the last team therefore takes first; buffer 1 shares its first chunks
__device__ __forceinline__ int team_chunk(int par, int t, int i) {
  if (par == 0 && t == TEAMS - 1)
    return i < OV_CHUNKS ? NCHUNK - OV_CHUNKS + i : t * TEAM_CHUNKS + (i - OV_CHUNKS);
  return t * TEAM_CHUNKS + i;
}
// Ring slot and use count of position i of team t in the seq-th tile of this CTA.  Each team
// has its own slots, used strictly in order, so every waiter sees every phase of the
// barriers it waits on.
__device__ __forceinline__ void chunk_slot(uint32_t seq, int t, int i, int& b, uint32_t& use) {
  const uint32_t j = seq * TEAM_CHUNKS + (uint32_t)i;
  b = t * RING_TEAM + (int)(j % RING_TEAM);
  use = j / RING_TEAM;
}

constexpr int OFF_A = 0;
constexpr int OFF_B = OFF_A + STAGES * OPER_BYTES;
constexpr int OFF_SF = OFF_B + STAGES * OPER_BYTES;
constexpr int OFF_RING = OFF_SF + STAGES * SF_BYTES;
constexpr int OFF_BAR = OFF_RING + RING * CHUNK_BYTES;
constexpr int SMEM_BYTES = OFF_BAR + 512 + 1024;
static_assert(SMEM_BYTES <= 232448, "at most 227 KB of dynamic shared memory");

constexpr int NTHREADS = 128 + TEAMS * 128;  // four single-thread roles, then the epilogue teams
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t TMEM_SF_COL = ACC1_COL + PN;  // scale factors after the second accumulator buffer
// Scale factors of ONE MMA (K = 64): 4 columns (row operand) + 8 (column operand, N = 256).  Copies and
// MMAs execute in issue order, so the copies for the next MMA may target the same columns.
constexpr uint32_t SF_COLS = 12;
static_assert(TMEM_SF_COL + SF_COLS <= 512, "tensor memory columns");

// instruction descriptor: E2M1 x E2M1, UE4M3 scales, K-major operands, M = 256 (pair), N = 256
constexpr uint32_t IDESC = (1u << 7) | (1u << 10) | ((uint32_t)(PN >> 3) << 17) | ((uint32_t)(PM >> 4) << 24);

struct Barriers {
  uint64_t full[STAGES];     // even CTA: both CTAs' operand bytes of a stage have landed
  uint64_t empty[STAGES];    // stage consumed (MMA commit, multicast to both CTAs)
  uint64_t acc_full[2];      // accumulator buffer complete (MMA commit, multicast)
  uint64_t acc_empty[2];     // even CTA: buffer drained by all epilogue warps of the pair
  uint64_t ov_free;          // even CTA: the columns shared with the other buffer are drained (8 warps)
  uint64_t aux_full[RING];
  uint64_t v_ready[RING];
  uint64_t slot_free[RING];
  uint32_t tmem_base;
  uint32_t abort_flag;
};
static_assert(sizeof(Barriers) <= 512, "barrier block");

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of `p` (a shared-memory object of this CTA) in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(const void* p, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
  return r;
}
// Arrive on a barrier of (possibly) the peer CTA.  Relaxed: the barriers signalled this way guard
// tensor memory that the arriving warp has finished reading (tcgen05.wait::ld has returned), not data
// in memory; a release at cluster scope would first wait for all of the thread's earlier global
// stores to be performed, thousands of cycles on the critical path of every tile.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load whose completion bytes are credited to a barrier that may live in the peer CTA
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const void* tmap, int x, int y, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%2, %3}], [%4];" ::"r"(smem_u32(smem_dst)),
      "l"(tmap), "r"(x), "r"(y), "r"(bar_cluster)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t* smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)),
               "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_cp_sf2(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void tc_mma_nvf4_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::mxf4nvf4.block_scale.block16 [%0], %1, %2, %3, [%5], [%6], p;\n\t}" ::"r"(
          d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
      : "memory");
}
// arrive on the barrier at this shared-memory offset in both CTAs of the pair when all MMAs
// issued so far have completed
__device__ __forceinline__ void tc_commit_pair(uint64_t* bar) {
  const uint16_t mask = 3;
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
          smem_u32(bar)),
      "h"(mask)
      : "memory");
}

// BH: instantiation with BF16 storage of the FP32 tiles (args.aux_h / args.out_h may be set)
template <int MODE, bool PF, bool BH>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NTHREADS, 1)
k_gemm_pair(const __grid_constant__ GemmProblem single, const GemmProblem* __restrict__ table, const GemmLaunch args) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Barriers* bars = reinterpret_cast<Barriers*>(smem + OFF_BAR);
  volatile uint32_t* abort_flag = &bars->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = (rank == 0);
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const GemmProblem* probs = table ? table : &single;
  // args.tiles_m / tiles_n count 256 x 256 tiles here
  // only the two symmetric products are ever launched with triangle tiles: a compile-time fact for the others
  const bool sym = (MODE == kG1 || MODE == kG2) && args.symmetric != 0;
  const int tiles_per_problem = sym ? args.tiles_n * (args.tiles_n + 1) / 2 : args.tiles_m * args.tiles_n;
  const int num_tiles = tiles_per_problem * args.num_problems;
  const int num_kb = args.K / BK;
  constexpr bool HAS_AUX = (MODE == kG2 || MODE == kG3);
  constexpr bool STORE_F32 = (MODE == kPlain || MODE == kG1 || MODE == kG3);
  const bool do_q = (MODE != kPlain) && args.write_q;

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { mbar_init(&bars->full[i], 1); mbar_init(&bars->empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&bars->acc_full[i], 1); mbar_init(&bars->acc_empty[i], 2 * 4 * TEAMS); }
    mbar_init(&bars->ov_free, 8);
    for (int i = 0; i < RING; ++i) {
      mbar_init(&bars->aux_full[i], 1);
      mbar_init(&bars->v_ready[i], 4);
      mbar_init(&bars->slot_free[i], 5);
    }
    bars->abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc2(&bars->tmem_base, TMEM_COLS);
    tmem_relinquish2();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer's barriers are initialised before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------ operand producer (both CTAs)
    if (elect_one()) {
      int st = 0; uint32_t ph = 0; bool ok = true;
      for (int t = pair; t < num_tiles && ok; t += num_pairs) {
        int p, ti, tj;
        decode_tile(t, args, tiles_per_problem, p, ti, tj, sym);
        const GemmProblem* pr = probs + p;
        const int arow = ti * PM + (int)rank * BM;   // this CTA's rows of the row operand
        const int brow = tj * PN + (int)rank * BM;   // this CTA's half of the column operand
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!wait_bar(&bars->empty[st], ph ^ 1, abort_flag)) { ok = false; break; }
          const uint32_t full_leader = map_to_cta(&bars->full[st], 0);
          if (leader) mbar_expect_tx(&bars->full[st], 2 * STAGE_BYTES_CTA);
          tma_load_2d_pair(smem + OFF_A + st * OPER_BYTES, &pr->tmA, kb * (BK / 2), arow, full_leader);
          tma_load_2d_pair(smem + OFF_B + st * OPER_BYTES, &pr->tmB, kb * (BK / 2), brow, full_leader);
          // scale atoms: 64-bit elements, one row of the map per 128-row block
          uint8_t* sf = smem + OFF_SF + st * SF_BYTES;
          tma_load_2d_pair(sf, &pr->tmSfa, kb * (SF_ATOMS / 8), arow / 128, full_leader);
          tma_load_2d_pair(sf + SF_ATOMS, &pr->tmSfb, kb * (SF_ATOMS / 8), tj * 2, full_leader);
          tma_load_2d_pair(sf + 2 * SF_ATOMS, &pr->tmSfb, kb * (SF_ATOMS / 8), tj * 2 + 1, full_leader);
          if (++st == STAGES) { st = 0; ph ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (even CTA only)
    if (leader && elect_one()) {
      int st = 0; uint32_t ph = 0, seq = 0; bool ok = true;
      for (int t = pair; t < num_tiles && ok; t += num_pairs, ++seq) {
        const uint32_t par = seq & 1, buse = seq >> 1;
        // this buffer's previous tile is drained, and so are the columns it shares with the
        // buffer of the tile before this one
        if (!wait_bar(&bars->acc_empty[par], (buse & 1) ^ 1, abort_flag)) { ok = false; break; }
        if (seq > 0 && !wait_bar(&bars->ov_free, (seq - 1) & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + par * ACC1_COL;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!wait_bar(&bars->full[st], ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sf_t = tmem_base + TMEM_SF_COL;
          const uint8_t* sf = smem + OFF_SF + st * SF_BYTES;
          const uint64_t adesc = umma_desc(smem_u32(smem + OFF_A + st * OPER_BYTES), 1024, 2);
          const uint64_t bdesc = umma_desc(smem_u32(smem + OFF_B + st * OPER_BYTES), 1024, 2);
#pragma unroll
          for (int k = 0; k < KSTEPS; ++k) {
            tc_cp_sf2(sf_t, umma_desc(smem_u32(sf + k * 512), 128, 0));
            tc_cp_sf2(sf_t + 4, umma_desc(smem_u32(sf + SF_ATOMS + k * 512), 128, 0));
            tc_cp_sf2(sf_t + 8, umma_desc(smem_u32(sf + 2 * SF_ATOMS + k * 512), 128, 0));
            tc_mma_nvf4_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC, sf_t, sf_t + 4, (kb | k) != 0 ? 1u : 0u);
          }
          tc_commit_pair(&bars->empty[st]);
          if (++st == STAGES) { st = 0; ph ^= 1; }
        }
        if (!ok) break;
        tc_commit_pair(&bars->acc_full[par]);
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------ producer of the FP32 tile
    // One thread serves the rings of all teams without blocking on any: it polls the next
    // slot of each team in turn and loads a chunk as soon as its slot is free.
    if (HAS_AUX && elect_one()) {
      const uint32_t my_tiles = pair < num_tiles ? (uint32_t)((num_tiles - pair + num_pairs - 1) / num_pairs) : 0u;
      const uint32_t total = my_tiles * TEAM_CHUNKS;
      uint32_t n[TEAMS], seq_dec[TEAMS];
      int pp[TEAMS], tis[TEAMS], tjs[TEAMS];
#pragma unroll
      for (int h = 0; h < TEAMS; ++h) { n[h] = 0; seq_dec[h] = 0xFFFFFFFFu; pp[h] = tis[h] = tjs[h] = 0; }
      uint32_t idle = 0, done = 0;
      uint64_t t_idle = 0;
      while (done < TEAMS * total) {
        bool progressed = false;
#pragma unroll
        for (int h = 0; h < TEAMS; ++h) {
          if (n[h] >= total) continue;
          const uint32_t seq = n[h] / TEAM_CHUNKS;
          const int i = (int)(n[h] % TEAM_CHUNKS);
          int b; uint32_t use;
          chunk_slot(seq, h, i, b, use);
          if (!mbar_try_wait(&bars->slot_free[b], (use & 1) ^ 1)) continue;
          if (seq_dec[h] != seq) {
            decode_tile(pair + (int)seq * num_pairs, args, tiles_per_problem, pp[h], tis[h], tjs[h], sym);
            seq_dec[h] = seq;
          }
          const GemmProblem* pr = probs + pp[h];
          const int bi = tis[h] * 2 + (int)rank;
          const int c = team_chunk((int)(seq & 1), h, i);
          const int bj = tjs[h] * 2 + c / 8;
          if (sym && bj < bi) {
            // a 128 x 128 block below the diagonal: nothing to combine, the slot is passed on empty
            mbar_arrive(&bars->aux_full[b]);
          } else {
            if (BH && args.aux_h) {
              // the tile is kept in BF16: four boxes of 32 rows x 32 bytes, each at the start of the 2 KB
              // of the slot that the warp of those rows later stages its FP32 block in (no warp's
              // staging can then overwrite rows another warp has not read yet)
              mbar_expect_tx(&bars->aux_full[b], CHUNK_BYTES / 2);
              tma_load_2d(smem + OFF_RING + b * CHUNK_BYTES, &pr->tmH, tjs[h] * PN + c * CHUNK, bi * BM, &bars->aux_full[b]);
            } else {
              mbar_expect_tx(&bars->aux_full[b], CHUNK_BYTES);
              tma_load_2d(smem + OFF_RING + b * CHUNK_BYTES, &pr->tmAux, tjs[h] * PN + c * CHUNK, bi * BM, &bars->aux_full[b]);
            }
          }
          ++n[h];
          ++done;
          progressed = true;
        }
        if (progressed) { idle = 0; continue; }
#ifdef FP4_POLL_SLEEP
        __nanosleep(FP4_POLL_SLEEP);
#endif
        if ((++idle & 1023u) == 0) {
          if (*abort_flag) break;
          const uint64_t now = globaltimer_ns();
          if (idle == 1024u) t_idle = now;
          else if (now - t_idle > 2000000000ull) { *abort_flag = 1; break; }
        }
      }
    }
  } else if (warp == 3) {
    // ------------------------------------------------------------ TMA-store issuer
    // One thread, all teams, polling like the producer above; up to three stores are in
    // flight, a slot is handed back once two newer stores have been issued or, when no chunk
    // is waiting to be sent, as soon as its store has read it.
    if (elect_one()) {
      const uint32_t my_tiles = pair < num_tiles ? (uint32_t)((num_tiles - pair + num_pairs - 1) / num_pairs) : 0u;
      const uint32_t total = my_tiles * TEAM_CHUNKS;
      uint32_t n[TEAMS], seq_dec[TEAMS];
      int pp[TEAMS], tis[TEAMS], tjs[TEAMS];
#pragma unroll
      for (int h = 0; h < TEAMS; ++h) { n[h] = 0; seq_dec[h] = 0xFFFFFFFFu; pp[h] = tis[h] = tjs[h] = 0; }
      int q0 = -1, q1 = -1;  // slots of the two newest stores, not yet handed back
      uint32_t idle = 0, done = 0;
      uint64_t t_idle = 0;
      while (done < TEAMS * total) {
        bool progressed = false;
#pragma unroll
        for (int h = 0; h < TEAMS; ++h) {
          if (n[h] >= total) continue;
          const uint32_t seq = n[h] / TEAM_CHUNKS;
          const int i = (int)(n[h] % TEAM_CHUNKS);
          int b; uint32_t use;
          chunk_slot(seq, h, i, b, use);
          if (!mbar_try_wait(&bars->v_ready[b], use & 1)) continue;
          if (seq_dec[h] != seq) {
            decode_tile(pair + (int)seq * num_pairs, args, tiles_per_problem, pp[h], tis[h], tjs[h], sym);
            seq_dec[h] = seq;
          }
          const GemmProblem* pr = probs + pp[h];
          const int bi = tis[h] * 2 + (int)rank;
          const int c = team_chunk((int)(seq & 1), h, i);
          const bool below = sym && (tjs[h] * 2 + c / 8) < bi;
          // a chunk that starts outside the stored matrix (zero padding of the work shape) is dropped
          const bool inside = tjs[h] * PN + c * CHUNK < pr->out_cols && bi * BM < pr->out_rows;
          if (STORE_F32 && !below && inside) {
            if (BH && args.out_h == 1) {
              // the result was staged in BF16, 32 rows x 32 bytes at the start of each warp's part of the slot
              tma_store_2d(&pr->tmH, tjs[h] * PN + c * CHUNK, bi * BM, smem + OFF_RING + b * CHUNK_BYTES);
            } else {
              tma_store_2d(&pr->tmOut, tjs[h] * PN + c * CHUNK, bi * BM, smem + OFF_RING + b * CHUNK_BYTES);
            }
            bulk_commit();
            bulk_wait_read<2>();  // every store but the two newest has read its slot
            if (q0 >= 0) mbar_arrive(&bars->slot_free[q0]);
            q0 = q1; q1 = b;
          } else {
            mbar_arrive(&bars->slot_free[b]);
          }
          ++n[h];
          ++done;
          progressed = true;
        }
        if (progressed) { idle = 0; continue; }
#ifdef FP4_POLL_SLEEP
        __nanosleep(FP4_POLL_SLEEP);
#endif
        if (STORE_F32 && q1 >= 0) {
          // nothing to send right now: do not sit on the slots of the newest stores (their team may
          // need them back before anyone issues another store)
          bulk_wait_read<0>();
          if (q0 >= 0) mbar_arrive(&bars->slot_free[q0]);
          mbar_arrive(&bars->slot_free[q1]);
          q0 = q1 = -1;
          continue;
        }
        if ((++idle & 1023u) == 0) {
          if (*abort_flag) break;
          const uint64_t now = globaltimer_ns();
          if (idle == 1024u) t_idle = now;
          else if (now - t_idle > 2000000000ull) { *abort_flag = 1; break; }
        }
      }
      if (STORE_F32) {
        bulk_wait_read<0>();
        if (q0 >= 0) mbar_arrive(&bars->slot_free[q0]);
        if (q1 >= 0) mbar_arrive(&bars->slot_free[q1]);
        bulk_wait_all<0>();
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    const int team = (warp - 4) >> 2;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    // column pass: lane = (column cq of the chunk, 16-row group g of this warp's 32 rows)
    const int cq = lane & 15, g = lane >> 4;
    float scale = 0.0f, sg_out = 1.0f, inv_sg = 1.0f;
    uint32_t rcp_base = 0;
    float ca = 0.0f, cb = 0.0f, cc = 0.0f;
    float tau = 0.0f, inv = 0.0f;  // first G3 stage on the raw input: X0 = clamp(G, tau) * inv
    bool raw = false;
    const GemmProblem* pr = nullptr;
    int cur_p = -1;
    const int sw = (row >> 1) & 3;
    // column pass: byte offset of (first row of this lane's 16-row group, column cq) in a slot, and the
    // swizzled offsets of the column's 16-byte group for the four values of bits 1-2 of the row
    const int col_off = (quad * 32 + g * 16) * 64 + (cq & 3) * 4;
    int col_sw[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) col_sw[k] = ((cq >> 2) ^ k) << 4;
    const uint32_t tm_lane = tmem_base + ((uint32_t)(quad * 32) << 16);
    const uint32_t acc_empty_leader0 = map_to_cta(&bars->acc_empty[0], 0);
    const uint32_t acc_empty_leader1 = map_to_cta(&bars->acc_empty[1], 0);
    const uint32_t ov_free_leader = map_to_cta(&bars->ov_free, 0);

    uint32_t seq = 0;
    float amax = 0.0f;
    bool ok = true;
    for (int t = pair; t < num_tiles && ok; t += num_pairs, ++seq) {
      int p, ti, tj;
      decode_tile(t, args, tiles_per_problem, p, ti, tj, sym);
      if (p != cur_p) {
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
        epilogue_scalars<MODE>(*pr, args, scale, sg_out,
                               leader && t == p * tiles_per_problem && threadIdx.x == 128);
        inv_sg = __frcp_rn(sg_out);  // exact: the predicted scales are powers of two
        rcp_base = rcp_base_of(sg_out);
        ca = pr->ca; cb = pr->cb; cc = pr->cc;
        raw = (MODE == kG3) && pr->aux_raw != 0;
        if (raw) {
          tau = args.clip ? pr->scalars[args.ix.tau] : __int_as_float(0x7f800000);
          inv = pr->scalars[args.ix.inv];
        }
      }
      const int bi = ti * 2 + (int)rank;                               // 128-row block of this CTA
      const int bj = tj * 2 + (team * TEAM_CHUNKS * CHUNK) / 128;      // 128-column block of this team's chunks
      const bool below = sym && bj < bi;                    // redundant block of a diagonal tile
      const bool mirror = do_q && !below && (MODE == kG3 || (sym && bi != bj));
      const bool hout = BH && STORE_F32 && MODE != kPlain && args.out_h == 1 && !below;  // result stored as BF16
      const bool stage = !below && ((STORE_F32 && !hout) || mirror);
      const int par = (int)(seq & 1);
      ok = __all_sync(0xffffffffu, wait_bar(&bars->acc_full[par], (seq >> 1) & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      const int64_t grow = (int64_t)bi * BM + row;
      // store addresses of this tile: row-quantised codes of this thread's row; column-quantised
      // codes and scale of (tensor row = tile column cq, 16-block = this lane's row group)
      uint8_t* rq_row = nullptr; uint8_t* cq_col = nullptr; uint8_t* cq_sfp = nullptr;
      if (do_q) {
        rq_row = pr->rq_codes + grow * (args.rq_K / 2) + ((int64_t)tj * PN) / 2;
        const int64_t tcol = (int64_t)bi * BM + quad * 32 + g * 16;
        const int64_t kb = tcol >> 4, kblocks = args.cq_K >> 4;
        cq_col = pr->cq_codes + ((int64_t)tj * PN + cq) * (args.cq_K / 2) + tcol / 2;
        cq_sfp = pr->cq_sf + ((int64_t)tj * 2 * (kblocks >> 2) + (kb >> 2)) * 512 + (kb & 3) + cq * 16;
      }
      const uint32_t tm_acc = tm_lane + par * ACC1_COL;
      const bool owns_overlap = (team == (par == 0 ? TEAMS - 1 : 0));
      uint32_t sfw = 0;
      uint32_t acc[16];
      tc_ld16_issue(tm_acc + team_chunk(par, team, 0) * CHUNK, acc);
      for (int i = 0; i < TEAM_CHUNKS; ++i) {
        const int c = team_chunk(par, team, i);
        int b; uint32_t use;
        chunk_slot(seq, team, i, b, use);
        uint8_t* slot = smem + OFF_RING + b * CHUNK_BYTES;
        uint8_t* slot_row = slot + row * 64;
        float v[16];
        if (HAS_AUX) ok = __all_sync(0xffffffffu, wait_bar(&bars->aux_full[b], use & 1, abort_flag));
        else ok = __all_sync(0xffffffffu, wait_bar(&bars->slot_free[b], (use & 1) ^ 1, abort_flag));
        if (!ok) break;
        tc_wait_ld16(acc);
        if (BH && HAS_AUX && !below && args.aux_h) {
          // the FP32 tile is kept in BF16: this lane's row is 32 bytes at the start of its warp's part of the slot
          const uint8_t* hrow = slot + row * 32;
          const uint4 h0 = *reinterpret_cast<const uint4*>(hrow);
          const uint4 h1 = *reinterpret_cast<const uint4*>(hrow + 16);
          const uint32_t hw[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
          bar_sync(1 + team, 128);  // the four warps have their rows before any of them stages FP32 values over them
#pragma unroll
          for (int q = 0; q < 16; ++q) {
            const float e = (q & 1) ? bf16_hi(hw[q >> 1]) : bf16_lo(hw[q >> 1]);
            const float prod = __fmul_rn(__uint_as_float(acc[q]), scale);
            if (MODE == kG2) v[q] = __fadd_rn(__fmul_rn(cb, e), __fmul_rn(cc, prod));
            else v[q] = __fadd_rn(__fmul_rn(ca, e), prod);
          }
        } else if (HAS_AUX && !below) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float4 x = *reinterpret_cast<const float4*>(slot_row + ((j ^ sw) << 4));
            float e[4] = {x.x, x.y, x.z, x.w};
            if (MODE == kG3 && raw) {
#pragma unroll
              for (int q = 0; q < 4; ++q) e[q] = __fmul_rn(fminf(fmaxf(e[q], -tau), tau), inv);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              // every product and the sum rounded on its own (scalar intrinsics: never contracted)
              const float prod = __fmul_rn(__uint_as_float(acc[4 * j + q]), scale);
              if (MODE == kG2) v[4 * j + q] = __fadd_rn(__fmul_rn(cb, e[q]), __fmul_rn(cc, prod));
              else v[4 * j + q] = __fadd_rn(__fmul_rn(ca, e[q]), prod);
            }
          }
        } else {
#pragma unroll
          for (int k = 0; k < 16; ++k) v[k] = __fmul_rn(__uint_as_float(acc[k]), scale);
        }
        uint32_t hout_w[8];  // the row rounded to BF16 (before a quantiser option may transform v in place)
        if (hout) {
#pragma unroll
          for (int q = 0; q < 8; ++q) hout_w[q] = cvt_bf16x2(v[2 * q], v[2 * q + 1]);
        }
        if (owns_overlap && i == OV_CHUNKS - 1) {
          // the columns shared with the other buffer are in registers: the next tile may use them
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(ov_free_leader);
        }
        if (i + 1 < TEAM_CHUNKS) {
          tc_ld16_issue(tm_acc + team_chunk(par, team, i + 1) * CHUNK, acc);
        } else {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(par ? acc_empty_leader1 : acc_empty_leader0);  // done with the buffer
        }
        if (stage) {
#pragma unroll
          for (int j = 0; j < 4; ++j)
            *reinterpret_cast<float4*>(slot_row + ((j ^ sw) << 4)) =
                make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
          fence_proxy_async_smem();
        }
        __syncwarp();
        if (!hout && lane == 0) mbar_arrive(&bars->v_ready[b]);  // the store issuer may send the chunk
        // Blocks of 16 down the rows of this warp's own 32 x 16 block (the transposed operand
        // copy in G3, the mirrored triangle in G1/G2), read back from the staging slot: row
        // k of the block is at k * 64 bytes, its 16-byte column group XOR-swizzled with bits
        // 1-2 of k.  (The two half-warps read rows 16 apart, a two-way bank conflict on these
        // sixteen 4-byte loads; avoiding it costs more instructions than it saves.)
        float w[16];
        if (mirror) {
          const uint8_t* colp = slot + col_off;
#pragma unroll
          for (int k = 0; k < 16; ++k)
            w[k] = *reinterpret_cast<const float*>(colp + k * 64 + (col_sw[(k >> 1) & 3]));
        }
        if (hout) {
          bar_sync(1 + team, 128);  // the four warps have read their FP32 blocks back
          // BF16 storage: the FP32 block has been read back (or was never staged); the rounded result
          // takes its place, 32 bytes per row at the start of this warp's part of the slot, and
          // the store issuer sends the four warps' rows as four boxes
          uint8_t* hrow = slot + row * 32;
          *reinterpret_cast<uint4*>(hrow) = make_uint4(hout_w[0], hout_w[1], hout_w[2], hout_w[3]);
          *reinterpret_cast<uint4*>(hrow + 16) = make_uint4(hout_w[4], hout_w[5], hout_w[6], hout_w[7]);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) { mbar_arrive(&bars->v_ready[b]); mbar_arrive(&bars->slot_free[b]); }  // done with the slot
        }
        if (!below && do_q) {
          uint32_t lo, hi;
          float bmax;
          uint32_t sb;
          if (PF) sb = quantize_block16_opts(v, args.q, sg_out, lo, hi, bmax);
          else sb = quantize_block16_pow2(v, sg_out, inv_sg, rcp_base, lo, hi, bmax);
          if (MODE == kG1 || MODE == kG3) amax = fmaxf(amax, bmax);
          *reinterpret_cast<uint2*>(rq_row + c * (CHUNK / 2)) = make_uint2(lo, hi);
          sfw |= sb << (8 * (c & 3));
        }
        if (!hout) {
          __syncwarp();
          if (lane == 0) mbar_arrive(&bars->slot_free[b]);  // this warp's part of the slot is in registers
        }
        if (mirror) {
          uint32_t lo, hi;
          float bmax;
          uint32_t sb;
          if (PF) sb = quantize_block16_opts(w, args.q, sg_out, lo, hi, bmax);
          else sb = quantize_block16_pow2(w, sg_out, inv_sg, rcp_base, lo, hi, bmax);
          // tensor row = tj * 256 + c * 16 + cq: its codes are c * 16 rows further on; in the scale
          // atoms, c / 8 selects the 128-row atom, c % 2 the upper 16 of 32 rows, (c % 8) / 2 the 32-row group
          *reinterpret_cast<uint2*>(cq_col + (int64_t)c * CHUNK * (args.cq_K / 2)) = make_uint2(lo, hi);
          cq_sfp[(int64_t)(c >> 3) * (args.cq_K >> 6) * 512 + (c & 1) * 256 + ((c & 7) >> 1) * 4] = (uint8_t)sb;
        }
      }
      if (ok && do_q && !below) {
        // the scale word of this team's 64 columns of the row
        const int64_t kb0 = ((int64_t)tj * PN + team * TEAM_CHUNKS * CHUNK) >> 4;
        *reinterpret_cast<uint32_t*>(pr->rq_sf + sf_offset(grow, kb0, args.rq_K >> 4)) = sfw;
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
  }

  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // neither CTA leaves while the other may still signal it or read its shared memory
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc2(tmem_base, TMEM_COLS);
  }
  if (threadIdx.x == 0 && bars->abort_flag) report_timeout(args.status);
}

template <int MODE, bool PF, bool BH>
cudaError_t launch_pair_mode(const GemmProblem* single, const GemmProblem* table, const GemmLaunch& L, int sms,
                             cudaStream_t st) {
  const int tpp = L.symmetric ? L.tiles_n * (L.tiles_n + 1) / 2 : L.tiles_m * L.tiles_n;
  const int num_tiles = tpp * L.num_problems;
  int pairs = sms / 2;
  if (pairs > num_tiles) pairs = num_tiles;
  count_launches(1);
  static const GemmProblem kNone = {};
  k_gemm_pair<MODE, PF, BH><<<2 * pairs, NTHREADS, SMEM_BYTES, st>>>(single ? *single : kNone, table, L);
  return cudaGetLastError();
}

}  // namespace

cudaError_t gemm_pair_set_attributes() {
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kPlain, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG1, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG1, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG1, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG1, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG2, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG2, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG2, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG2, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG3, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG3, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG3, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG3, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES))) return e;
  return cudaSuccess;
}

// `launch` carries tile counts in 128-blocks; all of M, N, K must be multiples of 256.
cudaError_t launch_gemm_pair(GemmMode mode, const GemmProblem* single, const GemmProblem* table,
                             const GemmLaunch& launch, int sms, cudaStream_t st) {
  if ((single == nullptr) == (table == nullptr)) return cudaErrorInvalidValue;
  if ((launch.tiles_m & 1) || (launch.tiles_n & 1) || (launch.K % BK)) return cudaErrorInvalidValue;
  GemmLaunch L = launch;
  L.tiles_m = launch.tiles_m / 2;
  L.tiles_n = launch.tiles_n / 2;
  const bool pf = launch.q.rht || launch.q.four_six;
  const bool bh = launch.aux_h != 0 || launch.out_h != 0;
#define FP4_PAIR_CASE(M)                                                                                    \
  return pf ? (bh ? launch_pair_mode<M, true, true>(single, table, L, sms, st)                               \
                  : launch_pair_mode<M, true, false>(single, table, L, sms, st))                             \
            : (bh ? launch_pair_mode<M, false, true>(single, table, L, sms, st)                              \
                  : launch_pair_mode<M, false, false>(single, table, L, sms, st))
  switch (mode) {
    case kPlain: return launch_pair_mode<kPlain, false, false>(single, table, L, sms, st);
    case kG1: FP4_PAIR_CASE(kG1);
    case kG2: FP4_PAIR_CASE(kG2);
    default: FP4_PAIR_CASE(kG3);
  }
#undef FP4_PAIR_CASE
}

}  // namespace fp4
