// The block-scaled NVFP4 GEMM with the fused Newton-Schulz epilogues (Section 3.4, display
// equations) for shapes whose dimensions are multiples of 256: a pair of CTAs on two SMs (a
// cluster of 2) computes one 256 x 256 output tile with tcgen05.mma.cta_group::2.  Each CTA
// holds 128 rows of the row operand and 128 of the 256 rows of the column operand in its
// shared memory, so every byte fetched from L2 and every byte the tensor core reads from
// shared memory feeds twice as many multiply-adds as in the 128 x 128 single-CTA kernel.
//
// Per CTA: accumulator 128 lanes x 256 FP32 columns in tensor memory, drained by sixteen
// epilogue warps that share nothing with one another.  A warp owns the 32 accumulator lanes
// of its quadrant and 64 of the 256 columns, and walks them in four chunks of 16 columns.
// For a chunk it fetches the 32 x 16 block of the FP32 tile it combines with by TMA into its
// own buffer (two chunks ahead), combines it with the accumulator block, quantises the block
// along the rows, writes the result into the same buffer, sends it off with its own TMA
// store, reads the buffer back column-wise and quantises down the columns (the transposed
// operand copy in G3, the mirrored triangle in G1/G2).  The NVFP4 codes of a warp's 32 x 64
// part of a tile are collected in shared memory and leave as two TMA stores per tile.  The
// only barriers between warps are those of the accumulator hand-over with the MMA issuer.
//
// Only the even CTA of a pair issues MMAs; both CTAs run every other role on their own 128
// rows.  TMA loads of both CTAs signal the even CTA's stage barrier; MMA completion is
// multicast to the stage and accumulator barriers of both CTAs.
#include "fp4_gemm_common.cuh"

namespace fp4 {

namespace {

#ifndef FP4_BK_AUX
#define FP4_BK_AUX 256
#endif
#ifndef FP4_STAGES_AUX
#define FP4_STAGES_AUX 3
#endif
#ifndef FP4_STAGES_NOAUX
#define FP4_STAGES_NOAUX 4
#endif
constexpr int PM = 256, PN = 256;              // output tile of a CTA pair
constexpr int BM = 128;                        // rows per CTA
constexpr int MAX_STAGES = 8;
constexpr int CHUNK = 16;                      // FP32 columns per epilogue step
constexpr int NCHUNK = PN / CHUNK;             // 16
constexpr int TEAMS = 4;                       // column groups of a tile: 64 columns = one word of row scales
constexpr int TEAM_CHUNKS = NCHUNK / TEAMS;    // 4
constexpr int EPI_WARPS = 4 * TEAMS;           // one warp per (column group, lane quadrant)
constexpr int XBUF_BYTES = 32 * CHUNK * 4;     // a warp's FP32 chunk buffer, 2 KB: 32 rows x 64 bytes (64-byte swizzle)
constexpr int RQ_BYTES = 32 * 32;              // row-quantised codes of 32 rows x 64 columns
// What a warp alone would write as partial 32-byte sectors is collected for one 128-column half of the
// CTA's tile (two column groups = eight warps) and leaves as whole sectors: the column-quantised codes
// [128 tile columns][64 bytes = the CTA's 128 rows], their scale bytes (two atoms) and the row scales
// (two atoms).  Writes of part of a sector make the L2 fetch the rest from memory first.
constexpr int HALF_CQ_BYTES = 128 * 64;
constexpr int HALF_SF_BYTES = 2 * 512;
constexpr int HALF_AREA = HALF_CQ_BYTES + 2 * HALF_SF_BYTES;
static_assert(TEAM_CHUNKS == 4, "the chunk loop is written for four chunks");

// Two consecutive tiles use two accumulator buffers that share one chunk of tensor memory
// (512 columns cannot hold two 256-column accumulators plus the scale factors):
// buffer 0 = columns [0, 256), buffer 1 = columns [240, 496), scale factors [496, 508).
// The shared columns are buffer 0's last chunk and buffer 1's first.  Column group 0 of the
// epilogue takes the tile's chunks in the order 15, 14, ... on buffer 0 and 0, 1, ... on buffer
// 1, so its four warps always drain the shared chunk first and report it; the next tile's MMAs
// may then start while the rest of the tile is still being drained.
constexpr uint32_t ACC1_COL = PN - CHUNK;      // 240

// Shared-memory layout, per epilogue mode.  The main loop is bound by how many operand bytes a pair of
// SMs keeps in flight (the plain product runs at 2.9 / 3.9 / 4.7 PFLOP/s with 2 / 3 / 4 stages), so every
// mode takes as many stages as its epilogue leaves room for: the modes that combine with an FP32 tile
// (G2, G3) need two chunk buffers per warp - one in work, one being fetched - and fit three stages; the
// others (G1, the plain product) stage their result in one buffer and fit four.
template <int MODE>
struct Lay {
  static constexpr bool HAS_AUX = (MODE == kG2 || MODE == kG3);
  static constexpr int BK = HAS_AUX ? FP4_BK_AUX : 256;        // elements of K per stage: 64- or 128-byte operand rows
  static_assert(BK == 128 || BK == 256, "operand rows of a stage are one TMA swizzle span");
  static constexpr int KSTEPS = BK / 64;                       // MMAs (K = 64) per stage
  static constexpr uint32_t OPER_SWIZZLE = (BK == 256) ? 2u : 4u;  // UMMA layout type: 128- or 64-byte swizzle
  static constexpr uint32_t OPER_SBO = 8 * (BK / 2);           // bytes between 8-row groups of an operand tile
  static constexpr int OPER_BYTES = BM * BK / 2;               // 128 rows of one operand
  static constexpr int SF_ATOMS = KSTEPS * 512;                // scale atoms of one 128-row block and stage
  static constexpr int SF_BYTES = 3 * SF_ATOMS;                // row operand: own block; column operand: both blocks
  static constexpr uint32_t STAGE_BYTES_CTA = 2 * OPER_BYTES + SF_BYTES;
  static constexpr int STAGES = HAS_AUX ? FP4_STAGES_AUX : FP4_STAGES_NOAUX;
  static constexpr int XBUF = HAS_AUX ? 2 : 1;                 // FP32 chunk buffers per warp
  static constexpr int WARP_AREA = XBUF * XBUF_BYTES + RQ_BYTES;
  static constexpr int OFF_A = 0;
  static constexpr int OFF_B = OFF_A + STAGES * OPER_BYTES;
  static constexpr int OFF_SF = OFF_B + STAGES * OPER_BYTES;
  static constexpr int OFF_EPI = OFF_SF + STAGES * SF_BYTES;
  static constexpr int OFF_HALF = OFF_EPI + EPI_WARPS * WARP_AREA;
  static constexpr int OFF_BAR = OFF_HALF + 2 * HALF_AREA;
  static constexpr int SMEM_BYTES = OFF_BAR + 512 + 1024;
  static_assert(STAGES <= MAX_STAGES, "barrier arrays");
  static_assert(OFF_EPI % 1024 == 0 && WARP_AREA % 1024 == 0, "chunk buffers keep the swizzle phase");
  static_assert(OFF_HALF % 1024 == 0 && HALF_AREA % 1024 == 0, "code staging keeps the swizzle phase");
  static_assert(SMEM_BYTES <= 232448, "at most 227 KB of dynamic shared memory");
};

constexpr int ROLE_WARPS = 3;                  // operand producer, MMA issuer, issuer of the half-tile stores
constexpr int NTHREADS = (ROLE_WARPS + EPI_WARPS) * 32;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t TMEM_SF_COL = ACC1_COL + PN;  // scale factors after the second accumulator buffer
// Scale factors of ONE MMA (K = 64): 4 columns (row operand) + 8 (column operand, N = 256).  Copies and
// MMAs execute in issue order, so the copies for the next MMA may target the same columns.
constexpr uint32_t SF_COLS = 12;
static_assert(TMEM_SF_COL + SF_COLS <= 512, "tensor memory columns");

// instruction descriptor: E2M1 x E2M1, UE4M3 scales, K-major operands, M = 256 (pair), N = 256
constexpr uint32_t IDESC = (1u << 7) | (1u << 10) | ((uint32_t)(PN >> 3) << 17) | ((uint32_t)(PM >> 4) << 24);

struct Barriers {
  uint64_t full[MAX_STAGES]; // even CTA: both CTAs' operand bytes of a stage have landed
  uint64_t empty[MAX_STAGES];  // stage consumed (MMA commit, multicast to both CTAs)
  uint64_t acc_full[2];      // accumulator buffer complete (MMA commit, multicast)
  uint64_t acc_empty[2];     // even CTA: buffer drained by all epilogue warps of the pair
  uint64_t ov_free;          // even CTA: the columns shared with the other buffer are drained (8 warps)
  uint64_t xfull[EPI_WARPS * 2];  // a warp's chunk buffer holds the FP32 block it asked for
  uint64_t half_done[2];     // the eight warps of a half have staged their quantised output of the tile
  uint64_t half_free[2];     // the stores of the half's staging area have read it
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
// The same load with an L2 eviction-priority hint (a policy made by createpolicy)
__device__ __forceinline__ void tma_load_2d_pair_hint(void* smem_dst, const void* tmap, int x, int y, uint32_t bar_cluster,
                                                      uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%2, %3}], [%4], %5;" ::"r"(smem_u32(smem_dst)),
      "l"(tmap), "r"(x), "r"(y), "r"(bar_cluster), "l"(policy)
      : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
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

// ---- shared-memory accesses of the epilogue by 32-bit shared address.  Not given a "memory"
// clobber: they are volatile, so they keep their order among themselves and with the barrier
// and fence wrappers (all volatile too), while plain arithmetic may move across them.
__device__ __forceinline__ void lds128(uint32_t a, float& x, float& y, float& z, float& w) {
  asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(x), "=f"(y), "=f"(z), "=f"(w) : "r"(a));
}
__device__ __forceinline__ void lds128u(uint32_t a, uint32_t& x, uint32_t& y, uint32_t& z, uint32_t& w) {
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(x), "=r"(y), "=r"(z), "=r"(w) : "r"(a));
}
__device__ __forceinline__ float lds32(uint32_t a) {
  float x;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(x) : "r"(a));
  return x;
}
__device__ __forceinline__ void sts128(uint32_t a, float x, float y, float z, float w) {
  asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(a), "f"(x), "f"(y), "f"(z), "f"(w));
}
__device__ __forceinline__ void sts128u(uint32_t a, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(x), "r"(y), "r"(z), "r"(w));
}
__device__ __forceinline__ void sts32(uint32_t a, uint32_t x) {
  asm volatile("st.shared.b32 [%0], %1;" ::"r"(a), "r"(x));
}
__device__ __forceinline__ void sts8(uint32_t a, uint32_t x) {
  asm volatile("st.shared.b8 [%0], %1;" ::"r"(a), "r"(x));
}
// contiguous bytes shared -> global (16-byte aligned, a multiple of 16 bytes), part of the thread's bulk group
__device__ __forceinline__ void bulk_store_s(void* gdst, uint32_t smem_src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_src), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void sts64u(uint32_t a, uint32_t x, uint32_t y) {
  asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(a), "r"(x), "r"(y));
}
// TMA by 32-bit shared addresses
__device__ __forceinline__ void tma_load_2d_s(uint32_t smem_dst, const void* tmap, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%2, %3}], [%4];" ::"r"(smem_dst),
      "l"(tmap), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_store_2d_s(const void* tmap, int x, int y, uint32_t smem_src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];" ::"l"(tmap),
               "r"(x), "r"(y), "r"(smem_src)
               : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_s(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_s(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
#ifdef FP4_TRACE
// Diagnostics build only: cycles each role spends waiting, summed per warp.
__device__ unsigned long long g_trace[160 * 18 * 8];
#define TR_DECL unsigned long long tr_[8] = {0, 0, 0, 0, 0, 0, 0, 0}; long long tr_t0_ = clock64(), tr_s_ = 0;
#define TR_BEGIN tr_s_ = clock64();
#define TR_END(k) tr_[k] += (unsigned long long)(clock64() - tr_s_);
#define TR_COUNT(k) tr_[k] += 1;
#define TR_FLUSH if ((threadIdx.x & 31) == 0) { tr_[7] = (unsigned long long)(clock64() - tr_t0_); for (int k_ = 0; k_ < 8; ++k_) g_trace[(blockIdx.x * 18 + (threadIdx.x >> 5)) * 8 + k_] = tr_[k_]; }
#else
#define TR_DECL
#define TR_BEGIN
#define TR_END(k)
#define TR_COUNT(k)
#define TR_FLUSH
#endif

// warp index, known to the compiler to be the same in all lanes
__device__ __forceinline__ int uniform_warp_index() { return __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0); }

// 32 bytes per lane, global memory
__device__ __forceinline__ void ldg256(const void* p, uint32_t (&r)[8]) {
  asm volatile("ld.global.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "l"(p));
  asm volatile("ld.global.v4.b32 {%0, %1, %2, %3}, [%4+16];" : "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]) : "l"(p));
}
__device__ __forceinline__ void stg256(void* p, const uint32_t (&r)[8]) {
  asm volatile("st.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
  asm volatile("st.global.v4.b32 [%0+16], {%1, %2, %3, %4};" ::"l"(p), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}

// BH: instantiation with BF16 storage of the FP32 tiles (args.aux_h / args.out_h may be set)
// UPD: the last G3 stage of a call that also applies Root's parameter update (args.update): every lane
//   loads the 16 BF16 weights under its row of a chunk (one 32-byte sector, fetched a chunk ahead),
//   forms W * decay - step * X+ from the values it holds and stores the sector back.
template <int MODE, bool PF, bool BH, bool UPD = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NTHREADS, 1)
k_gemm_pair(const __grid_constant__ ProblemPack pack, const __grid_constant__ GemmLaunch args) {
  using L = Lay<MODE>;
  constexpr int STAGES = L::STAGES, XBUF = L::XBUF, WARP_AREA = L::WARP_AREA;
  constexpr int BK = L::BK, KSTEPS = L::KSTEPS, OPER_BYTES = L::OPER_BYTES, SF_ATOMS = L::SF_ATOMS, SF_BYTES = L::SF_BYTES;
  constexpr uint32_t STAGE_BYTES_CTA = L::STAGE_BYTES_CTA, OPER_SBO = L::OPER_SBO, OPER_SWIZZLE = L::OPER_SWIZZLE;
  constexpr int OFF_A = L::OFF_A, OFF_B = L::OFF_B, OFF_SF = L::OFF_SF, OFF_EPI = L::OFF_EPI, OFF_HALF = L::OFF_HALF,
                OFF_BAR = L::OFF_BAR;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Barriers* bars = reinterpret_cast<Barriers*>(smem + OFF_BAR);
  volatile uint32_t* abort_flag = &bars->abort_flag;

  const int warp = uniform_warp_index(), lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = (rank == 0);
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const GemmProblem* probs = pack.p;
  // args.tiles_m / tiles_n count 256 x 256 tiles here
  // only the two symmetric products are ever launched with triangle tiles: a compile-time fact for the others
  const bool sym = (MODE == kG1 || MODE == kG2) && args.symmetric != 0;
  const int tiles_per_problem = sym ? args.tiles_n * (args.tiles_n + 1) / 2 : args.tiles_m * args.tiles_n;
  const int num_tiles = tiles_per_problem * args.num_problems;
  const int num_kb = args.K / BK;
  constexpr bool HAS_AUX = (MODE == kG2 || MODE == kG3);
  constexpr bool STORE_F32 = (MODE == kPlain || MODE == kG1 || MODE == kG3);
  const bool do_q = (MODE != kPlain) && !UPD && args.write_q;  // the update variant is launched without quantised outputs
  // Measurement of the tensor-pipe ceiling (plain product only): each CTA pair fetches the first stages of
  // its first tile once and every later MMA runs on those resident stages - no operand traffic, same
  // instruction stream, same epilogue.
  const bool dry = (MODE == kPlain) && args.dry_operands != 0;

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { mbar_init(&bars->full[i], 1); mbar_init(&bars->empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&bars->acc_full[i], 1); mbar_init(&bars->acc_empty[i], 2 * EPI_WARPS); }
    mbar_init(&bars->ov_free, 8);
    for (int i = 0; i < EPI_WARPS * 2; ++i) mbar_init(&bars->xfull[i], 1);
    for (int i = 0; i < 2; ++i) { mbar_init(&bars->half_done[i], EPI_WARPS / 2); mbar_init(&bars->half_free[i], 1); }
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
  pdl_wait();          // set-up done; from here on the kernel reads what the launches before it wrote

  if (warp == 0) {
    // ------------------------------------------------------------ operand producer (both CTAs)
    if (elect_one()) {
      int st = 0; uint32_t ph = 0;
      TR_DECL
      // G3's operands (qB and the transposed copy of qX, some 20 MB per matrix) are re-read by every tile
      // while 200 MB of FP32 X stream through the L2 beside them: a stage completes when its last byte
      // has arrived, so even a small share of operand lines evicted to DRAM makes almost every stage wait
      // for DRAM.  Loading them with evict-last priority took 6 % off G3; the same hint on the symmetric
      // products' operands, and evict-first on the FP32 tiles, measured slower and are not used.
      const uint64_t keep = l2_policy_evict_last();
#define TMA_OPERAND(dst, map, x, y, bar)                                          \
  do {                                                                            \
    if (MODE == kG3) tma_load_2d_pair_hint(dst, map, x, y, bar, keep);            \
    else tma_load_2d_pair(dst, map, x, y, bar);                                   \
  } while (0)
      for (int t = pair; t < (dry ? min(num_tiles, pair + 1) : num_tiles); t += num_pairs) {
        int p, ti, tj;
        decode_tile(t, args, tiles_per_problem, p, ti, tj, sym);
        const GemmProblem* pr = probs + p;
        const int arow = ti * PM + (int)rank * BM;   // this CTA's rows of the row operand
        const int brow = tj * PN + (int)rank * BM;   // this CTA's half of the column operand
        for (int kb = 0; kb < (dry ? min(num_kb, STAGES) : num_kb); ++kb) {
          TR_BEGIN
          wait_or_abort(&bars->empty[st], ph ^ 1, abort_flag);
          TR_END(0)
          const uint32_t full_leader = map_to_cta(&bars->full[st], 0);
          if (leader) mbar_expect_tx(&bars->full[st], 2 * STAGE_BYTES_CTA);
          TMA_OPERAND(smem + OFF_A + st * OPER_BYTES, &pr->tmA, kb * (BK / 2), arow, full_leader);
          TMA_OPERAND(smem + OFF_B + st * OPER_BYTES, &pr->tmB, kb * (BK / 2), brow, full_leader);
          // scale atoms: 64-bit elements, one row of the map per 128-row block
          uint8_t* sf = smem + OFF_SF + st * SF_BYTES;
          TMA_OPERAND(sf, &pr->tmSfa, kb * (SF_ATOMS / 8), arow / 128, full_leader);
          TMA_OPERAND(sf + SF_ATOMS, &pr->tmSfb, kb * (SF_ATOMS / 8), tj * 2, full_leader);
          TMA_OPERAND(sf + 2 * SF_ATOMS, &pr->tmSfb, kb * (SF_ATOMS / 8), tj * 2 + 1, full_leader);
          if (++st == STAGES) { st = 0; ph ^= 1; }
        }
      }
      TR_FLUSH
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (even CTA only)
    if (leader && elect_one()) {
      int st = 0; uint32_t ph = 0, seq = 0;
      TR_DECL
      for (int t = pair; t < num_tiles; t += num_pairs, ++seq) {
        const uint32_t par = seq & 1, buse = seq >> 1;
        TR_COUNT(6)
        TR_BEGIN
        // this buffer's previous tile is drained, and so are the columns it shares with the
        // buffer of the tile before this one
        wait_or_abort(&bars->acc_empty[par], (buse & 1) ^ 1, abort_flag);
        TR_END(0)
        TR_BEGIN
        if (seq > 0) wait_or_abort(&bars->ov_free, (seq - 1) & 1, abort_flag);
        TR_END(1)
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + par * ACC1_COL;
        for (int kb = 0; kb < num_kb; ++kb) {
          TR_BEGIN
          if (!dry || (seq == 0 && kb < STAGES)) wait_or_abort(&bars->full[st], ph, abort_flag);
          TR_END(2)
          tc_fence_after();
          const uint32_t sf_t = tmem_base + TMEM_SF_COL;
          const uint8_t* sf = smem + OFF_SF + st * SF_BYTES;
          const uint64_t adesc = umma_desc(smem_u32(smem + OFF_A + st * OPER_BYTES), OPER_SBO, OPER_SWIZZLE);
          const uint64_t bdesc = umma_desc(smem_u32(smem + OFF_B + st * OPER_BYTES), OPER_SBO, OPER_SWIZZLE);
#pragma unroll
          for (int k = 0; k < KSTEPS; ++k) {
            tc_cp_sf2(sf_t, umma_desc(smem_u32(sf + k * 512), 128, 0));
            tc_cp_sf2(sf_t + 4, umma_desc(smem_u32(sf + SF_ATOMS + k * 512), 128, 0));
            tc_cp_sf2(sf_t + 8, umma_desc(smem_u32(sf + 2 * SF_ATOMS + k * 512), 128, 0));
            tc_mma_nvf4_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, IDESC, sf_t, sf_t + 4, (kb | k) != 0 ? 1u : 0u);
          }
          if (!dry) tc_commit_pair(&bars->empty[st]);
          if (++st == STAGES) { st = 0; ph ^= 1; }
        }
        tc_commit_pair(&bars->acc_full[par]);
      }
      TR_FLUSH
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------ issuer of the half-tile stores
    // When the eight warps of a half have staged their part of a tile, one thread sends the staging area
    // off: column-quantised codes by TMA (64-byte rows), the two kinds of scale bytes as whole atoms.
    if (do_q && elect_one()) {
      uint32_t seq = 0;
      for (int t = pair; t < num_tiles; t += num_pairs, ++seq) {
        int p, ti, tj;
        decode_tile(t, args, tiles_per_problem, p, ti, tj, sym);
        const GemmProblem* pr = probs + p;
        const int bi = ti * 2 + (int)rank;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int hcol = (seq & 1) ? h : 1 - h;          // which 128 columns of the tile this half holds
          const int bj = tj * 2 + hcol;
          const bool below = sym && bj < bi;
          const bool mirror = !below && (MODE == kG3 || (sym && bi != bj));
          wait_or_abort(&bars->half_done[h], seq & 1, abort_flag);
          if (!below) {
            const uint32_t st = smem_u32(smem + OFF_HALF + h * HALF_AREA);
            bulk_store_s(pr->rq_sf + ((int64_t)bi * (args.rq_K >> 6) + bj * 2) * 512, st + HALF_CQ_BYTES + HALF_SF_BYTES,
                         HALF_SF_BYTES);
            if (mirror) {
              tma_store_2d_s(&pr->tmCq, bi * (BM / 2), bj * 128, st);
              bulk_store_s(pr->cq_sf + ((int64_t)bj * (args.cq_K >> 6) + bi * 2) * 512, st + HALF_CQ_BYTES, HALF_SF_BYTES);
            }
          }
        }
        bulk_commit();
        bulk_wait_read<0>();
        mbar_arrive(&bars->half_free[0]);
        mbar_arrive(&bars->half_free[1]);
      }
      bulk_wait_all<0>();
    }
  } else {
    // ------------------------------------------------------------ epilogue warps
    const int ew = warp - ROLE_WARPS;
    const int team = ew >> 2;      // which 64 columns of a tile (mirrored on buffer 0, see below)
    const int quad = warp & 3;     // tensor-memory lane quadrant this warp may read
    // column pass: lane = (column cq of the chunk, 16-row group g of this warp's 32 rows)
    const int cq = lane & 15, g = lane >> 4;
    const uint32_t area = smem_u32(smem + OFF_EPI + ew * WARP_AREA);
    const uint32_t rq_st = area + XBUF * XBUF_BYTES;   // [32 rows][32 bytes]
    const int half = team >> 1;                         // the staging area this warp shares with seven others
    const uint32_t half_st = smem_u32(smem + OFF_HALF + half * HALF_AREA);
    const uint32_t half_done = smem_u32(&bars->half_done[half]), half_free = smem_u32(&bars->half_free[half]);
    const uint32_t xfull0 = smem_u32(&bars->xfull[ew * 2]);
    // row pass: this lane's row of a chunk buffer is 64 bytes whose 16-byte groups are XOR-swizzled with
    // bits 1-2 of the row; group j of the row sits at row_addr ^ (j << 4)
    const uint32_t row_addr = area + lane * 64 + (((lane >> 1) & 3) << 4);
    // column pass: row k of the lane's 16-row group is at col_addr[(k >> 1) & 3] + k * 64
    uint32_t col_addr[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) col_addr[k] = area + g * 16 * 64 + (cq & 3) * 4 + (((cq >> 2) ^ k) << 4);
    const uint32_t tm_lane = tmem_base + ((uint32_t)(quad * 32) << 16);
    const uint32_t acc_empty_leader0 = map_to_cta(&bars->acc_empty[0], 0);
    const uint32_t acc_empty_leader1 = map_to_cta(&bars->acc_empty[1], 0);
    const uint32_t ov_free_leader = map_to_cta(&bars->ov_free, 0);
    // A tall input is worked on as its transpose.  The first G3 stage reads the caller's matrix through a
    // transposing box and the last one writes the caller's result the same way, so neither
    // an FP32 copy of X0 nor a final transpose pass is needed (per-problem flags aux_tr / out_tr).
    constexpr bool TR = (MODE == kG3);
    const bool auxh = BH && HAS_AUX && args.aux_h != 0;                               // the combined tile is BF16
    const bool hout = BH && STORE_F32 && MODE != kPlain && args.out_h == 1;           // the result is stored as BF16

    float scale = 0.0f, sg_out = 1.0f, inv_sg = 1.0f;
    uint32_t rcp_base = 0;
    float ca = 0.0f, cb = 0.0f, cc = 0.0f;
    bool scale_pow2 = false;
    uint64_t scale2 = 0, ca2 = 0, cb2 = 0, ccs2 = 0;
    float tau = 0.0f, inv = 0.0f;  // first G3 stage on the raw input: X0 = clamp(G, tau) * inv
    bool raw = false, aux_tr = false, out_tr = false;
    const GemmProblem* pr = nullptr;
    int cur_p = -1;
    float amax = 0.0f;

    // The block of the FP32 tile for chunk slot `e` (0..3 = position among the 64 columns) of the tile
    // (problem q, tile row bi2 of 128, 64-column group at column x64): fetched into buffer b.  A block
    // below the diagonal of a symmetric product has nothing to fetch: its slot is passed on empty.
    auto fetch = [&](const GemmProblem* q, int x64, int y32, int e, bool skip, int b) {
      if (lane == 0) {
        const uint32_t bar = xfull0 + b * 8;
        if (skip) {
          mbar_arrive_s(bar);
        } else if (auxh) {
          mbar_expect_tx_s(bar, XBUF_BYTES / 2);
          tma_load_2d_s(area + b * XBUF_BYTES, &q->tmH, x64 + e * CHUNK, y32, bar);
        } else if (TR && q->aux_tr) {
          // the tile comes from a matrix stored the other way round (a tall input): the same 2 KB arrive as
          // 16 rows (columns of the tile) of 32 elements (its rows)
          mbar_expect_tx_s(bar, XBUF_BYTES);
          tma_load_2d_s(area + b * XBUF_BYTES, &q->tmAux, y32, x64 + e * CHUNK, bar);
        } else {
          mbar_expect_tx_s(bar, XBUF_BYTES);
          tma_load_2d_s(area + b * XBUF_BYTES, &q->tmAux, x64 + e * CHUNK, y32, bar);
        }
      }
    };
    // geometry of a tile for this warp
    struct Geo { int p, ti, tj, x64, y32; bool below; };
    auto geometry = [&](int t, uint32_t seq_) {
      Geo q;
      decode_tile(t, args, tiles_per_problem, q.p, q.ti, q.tj, sym);
      const int cgx = (seq_ & 1) ? team : TEAMS - 1 - team;       // column group: mirrored on buffer 0
      const int bi_ = q.ti * 2 + (int)rank;
      q.x64 = q.tj * PN + cgx * (TEAM_CHUNKS * CHUNK);
      q.y32 = bi_ * BM + quad * 32;
      q.below = sym && (q.tj * 2 + (cgx >> 1)) < bi_;              // redundant block of a diagonal tile
      return q;
    };

    uint32_t seq = 0;
    int t = pair;
    Geo cur;
    TR_DECL
    if (t < num_tiles) {
      cur = geometry(t, 0);
      if (HAS_AUX) {
        // chunk position e of slot i: i on buffer 1, 3 - i on buffer 0 (seq = 0 uses buffer 0)
        fetch(probs + cur.p, cur.x64, cur.y32, 3, cur.below, 0);
        fetch(probs + cur.p, cur.x64, cur.y32, 2, cur.below, 1);
      }
    }
    for (; t < num_tiles; t += num_pairs, ++seq) {
      const int p = cur.p, tj = cur.tj;
      const int x64 = cur.x64, y32 = cur.y32;
      const bool below = cur.below;
      // the next tile of this pair: its first two blocks are fetched during this tile's last two chunks
      const bool has_next = t + num_pairs < num_tiles;
      Geo nxt = cur;
      if (has_next) nxt = geometry(t + num_pairs, seq + 1);
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
                               leader && t == p * tiles_per_problem && threadIdx.x == ROLE_WARPS * 32);
        inv_sg = __frcp_rn(sg_out);  // exact: the predicted scales are powers of two
        rcp_base = rcp_base_of(sg_out);
        ca = pr->ca; cb = pr->cb; cc = pr->cc;
        // a power-of-two scale (every tensor scale produced inside the loop is one) multiplies exactly
        scale_pow2 = (__float_as_uint(scale) & 0x007FFFFFu) == 0 && scale > 1e-30f && scale < 1e30f;
        scale2 = pack2(scale, scale);
        ca2 = pack2(ca, ca); cb2 = pack2(cb, cb);
        const float ccs = __fmul_rn(cc, scale);
        ccs2 = pack2(ccs, ccs);
        raw = (MODE == kG3) && pr->aux_raw != 0;
        aux_tr = TR && pr->aux_tr != 0;
        out_tr = TR && pr->out_tr != 0;
        if (raw) {
          tau = args.clip ? pr->scalars[args.ix.tau] : __int_as_float(0x7f800000);
          inv = pr->scalars[args.ix.inv];
        }
      }
      const int par = (int)(seq & 1);
      const int flip = par ? 0 : 3;                                     // chunk position of slot i: i ^ flip
      const int bi = cur.ti * 2 + (int)rank;                            // 128-row block of this CTA
      const int cg = x64 / (TEAM_CHUNKS * CHUNK) & 3;                   // 64-column group within the tile
      const int bj = tj * 2 + (cg >> 1);                                // 128-column block of this warp's columns
      const bool mirror = do_q && !below && (MODE == kG3 || (sym && bi != bj));
      // the FP32 (or BF16) result leaves by TMA - unless the caller wants the parameter update only
      const bool store_out = STORE_F32 && !(UPD && args.no_out && pr->W != nullptr);
      const bool stage = (store_out && !hout) || mirror;
      const bool rows_in = y32 < pr->out_rows;                          // else: zero padding of the work shape
      TR_COUNT(6)
      TR_BEGIN
      wait_or_abort(&bars->acc_full[par], (seq >> 1) & 1, abort_flag);
      TR_END(0)
      tc_fence_after();
      const uint32_t acc_empty_leader = par ? acc_empty_leader1 : acc_empty_leader0;

      if (below) {
        // nothing of this block is needed: hand the accumulator back, keep the chunk slots turning
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (team == 0) mbar_arrive_cluster(ov_free_leader);
          mbar_arrive_cluster(acc_empty_leader);
        }
        if (do_q) {
          // Nothing is staged, but the half's count still has to fill once per tile - and only after the
          // store issuer has seen the previous tile's phase (two of these tiles can follow each other, and
          // a barrier that completes twice unobserved looks unchanged to a parity wait).
          wait_or_abort(half_free, (seq & 1) ^ 1, abort_flag);
          if (lane == 0) mbar_arrive_s(half_done);
        }
        if (HAS_AUX) {
#pragma unroll
          for (int i = 0; i < TEAM_CHUNKS; ++i) {
            wait_or_abort(xfull0 + (i & 1) * 8, (uint32_t)(i >> 1), abort_flag);
            if (i < 2) fetch(pr, x64, y32, (i + 2) ^ flip, true, i & 1);
            else if (has_next) fetch(probs + nxt.p, nxt.x64, nxt.y32, (i - 2) ^ (flip ^ 3), nxt.below, i & 1);
          }
        }
        cur = nxt;
        continue;
      }

      // store addresses of this tile: the scale word of this lane's row; scale byte of (tensor row =
      // tile column cq, 16-block = this lane's row group) in the column-quantised output
      // where this lane's outputs go in the half's staging area (cgl: which of its two column groups)
      //   codes of (tile column = cgl * 64 + e * 16 + cq, rows quad * 32 + g * 16 ...): 64-byte rows, the
      //     16-byte groups XOR-swizzled with bits 1-2 of the row index (which are those of cq);
      //   their scale byte: atom quad / 2 (128 tile columns x 4 blocks of 16 rows), row e % 2 * 16 + cq,
      //     group cgl * 2 + e / 2, byte quad % 2 * 2 + g;
      //   the scale word of this lane's row: atom cgl, row lane, group quad.
      const int cgl = cg & 1;
      const uint32_t cq_st = half_st + (cgl * 64 + cq) * 64 + ((quad ^ ((cq >> 1) & 3)) << 4) + g * 8;
      const uint32_t csf_st = half_st + HALF_CQ_BYTES + (quad >> 1) * 512 + cq * 16 + cgl * 8 + (quad & 1) * 2 + g;
      const uint32_t rsf_st = half_st + HALF_CQ_BYTES + HALF_SF_BYTES + cgl * 512 + lane * 16 + quad * 4;
      const uint32_t tm_acc = tm_lane + par * ACC1_COL + cg * (TEAM_CHUNKS * CHUNK);
      uint32_t sfw = 0;
      uint32_t acc[16];
      // parameter update: this lane's row of the weight under the tile, one 32-byte piece per chunk
      uint16_t* wrow = nullptr;
      uint32_t wnext[8];
      if (UPD) {
        if (pr->W && rows_in && y32 + lane < pr->out_rows) wrow = pr->W + ((int64_t)y32 + lane) * pr->W_ld + x64;
        if (wrow && x64 + flip * CHUNK < pr->out_cols) ldg256(wrow + flip * CHUNK, wnext);
      }
      tc_ld16_issue(tm_acc + flip * CHUNK, acc);
#pragma unroll
      for (int i = 0; i < TEAM_CHUNKS; ++i) {
        const int e = i ^ flip;                         // position of this chunk among the warp's 64 columns
        const int b = i & 1;
        const uint32_t boff = (XBUF == 2 ? b : 0) * XBUF_BYTES;   // without a fetched tile: one staging buffer
        const int xcol = x64 + e * CHUNK;
        float v[16];
        if (HAS_AUX) {
          TR_BEGIN
          wait_or_abort(xfull0 + b * 8, (uint32_t)(i >> 1), abort_flag);
          TR_END(1)
        }
        // ---- combine the accumulator block with the FP32 tile
        if (BH && HAS_AUX && auxh) {
          // the tile is kept in BF16: this lane's row is 32 bytes of the first half of the buffer
          uint32_t hw[8];
          lds128u(area + boff + lane * 32, hw[0], hw[1], hw[2], hw[3]);
          lds128u(area + boff + lane * 32 + 16, hw[4], hw[5], hw[6], hw[7]);
          tc_wait_ld16(acc);
#pragma unroll
          for (int q = 0; q < 16; ++q) {
            const float x = (q & 1) ? bf16_hi(hw[q >> 1]) : bf16_lo(hw[q >> 1]);
            const float prod = __fmul_rn(__uint_as_float(acc[q]), scale);
            if (MODE == kG2) v[q] = __fadd_rn(__fmul_rn(cb, x), __fmul_rn(cc, prod));
            else v[q] = __fadd_rn(__fmul_rn(ca, x), prod);
          }
          __syncwarp();  // every lane has its row before FP32 rows are staged over them
        } else if (HAS_AUX) {
          float x[16];
          if (TR && aux_tr) {
            // the block lies transposed in the buffer: element (row = lane, column j) at j * 128 + lane * 4
#pragma unroll
            for (int j = 0; j < 16; ++j) x[j] = lds32(area + boff + j * 128 + lane * 4);
            __syncwarp();  // every lane has its row before the result rows are staged over the block
          } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              lds128((row_addr + boff) ^ (j << 4), x[4 * j], x[4 * j + 1], x[4 * j + 2], x[4 * j + 3]);
          }
          TR_BEGIN
          tc_wait_ld16(acc);
          TR_END(2)
          if (MODE == kG3 && raw) {
#pragma unroll
            for (int q = 0; q < 16; ++q) x[q] = __fmul_rn(fminf(fmaxf(x[q], -tau), tau), inv);
          }
          if (scale_pow2) {
            // The product acc * scale is exact when scale is a power of two, so
            //   G3: fl(fl(a x) + fl(acc scale)) = fma(acc, scale, fl(a x))
            //   G2: fl(c fl(acc scale)) = fl((c scale) acc), with c scale exact as well (ccs)
            // and the result has the bits of the three separately rounded operations.  Two lanes per
            // instruction; no packed product ever feeds a packed sum (that pair could be contracted).
#pragma unroll
            for (int q = 0; q < 16; q += 2) {
              if (MODE == kG2) {
                float t0, t1, u0, u1;
                unpack2(mul2(cb2, pack2(x[q], x[q + 1])), t0, t1);
                unpack2(mul2(ccs2, pack2(__uint_as_float(acc[q]), __uint_as_float(acc[q + 1]))), u0, u1);
                v[q] = __fadd_rn(t0, u0);
                v[q + 1] = __fadd_rn(t1, u1);
              } else {
                const uint64_t ax = mul2(ca2, pack2(x[q], x[q + 1]));
                unpack2(fma2(pack2(__uint_as_float(acc[q]), __uint_as_float(acc[q + 1])), scale2, ax), v[q], v[q + 1]);
              }
            }
          } else {
#pragma unroll
            for (int q = 0; q < 16; ++q) {
              // every product and the sum rounded on its own (scalar intrinsics: never contracted)
              const float prod = __fmul_rn(__uint_as_float(acc[q]), scale);
              if (MODE == kG2) v[q] = __fadd_rn(__fmul_rn(cb, x[q]), __fmul_rn(cc, prod));
              else v[q] = __fadd_rn(__fmul_rn(ca, x[q]), prod);
            }
          }
        } else {
          tc_wait_ld16(acc);
#pragma unroll
          for (int k = 0; k < 16; ++k) v[k] = __fmul_rn(__uint_as_float(acc[k]), scale);
        }
        // ---- the accumulator columns are in registers
        if (i == 0 && team == 0) {
          // ... among them those shared with the other buffer: the next tile may use them
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(ov_free_leader);
        }
        if (i + 1 < TEAM_CHUNKS) {
          tc_ld16_issue(tm_acc + ((i + 1) ^ flip) * CHUNK, acc);
        } else {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(acc_empty_leader);  // done with the buffer
        }
        if (UPD) {
          uint32_t wcur[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) wcur[q] = wnext[q];
          const bool upd_here = wrow && xcol < pr->out_cols;
          if (i + 1 < TEAM_CHUNKS) {
            const int e1 = (i + 1) ^ flip;
            if (wrow && x64 + e1 * CHUNK < pr->out_cols) ldg256(wrow + e1 * CHUNK, wnext);
          }
          if (upd_here) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
              wcur[q] = cvt_bf16x2(param_update_value(bf16_lo(wcur[q]), v[2 * q], args.upd_decay, args.upd_step),
                                   param_update_value(bf16_hi(wcur[q]), v[2 * q + 1], args.upd_decay, args.upd_step));
            stg256(wrow + e * CHUNK, wcur);
          }
        }
        uint32_t hw_out[8];  // the row rounded to BF16 (before a quantiser option may transform v in place)
        if (BH && hout) {
#pragma unroll
          for (int q = 0; q < 8; ++q) hw_out[q] = cvt_bf16x2(v[2 * q], v[2 * q + 1]);
        }
        // ---- stage the block (for the TMA store and / or the column pass) and send it off
        const bool send = rows_in && xcol < pr->out_cols;
        if (TR && out_tr) {
          // the caller's matrix is the transpose: the block leaves as 16 rows of 32 elements
#pragma unroll
          for (int j = 0; j < 16; ++j) sts32(area + boff + j * 128 + lane * 4, __float_as_uint(v[j]));
          fence_proxy_async_smem();
        } else if (stage) {
#pragma unroll
          for (int j = 0; j < 4; ++j)
            sts128((row_addr + boff) ^ (j << 4), v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
          if (store_out && !hout) fence_proxy_async_smem();
        }
        __syncwarp();
        if (store_out && !hout && send && lane == 0) {
          if (TR && out_tr) tma_store_2d_s(&pr->tmOut, y32, xcol, area + boff);
          else tma_store_2d_s(&pr->tmOut, xcol, y32, area + boff);
          bulk_commit();
        }
        // ---- blocks of 16 down the rows of this warp's own 32 x 16 block (the transposed operand
        // copy in G3, the mirrored triangle in G1/G2), read back from the buffer.  (The two
        // half-warps read rows 16 apart, a two-way bank conflict on these sixteen 4-byte loads.)
        float w[16];
        if (mirror) {
#pragma unroll
          for (int k = 0; k < 16; ++k) w[k] = lds32(col_addr[(k >> 1) & 3] + boff + k * 64);
        }
        if (BH && hout && store_out) {
          // BF16 storage: the rounded rows take the place of the FP32 block once it has been read back,
          // 32 bytes per row at the start of the buffer
          __syncwarp();
          sts128u(area + boff + lane * 32, hw_out[0], hw_out[1], hw_out[2], hw_out[3]);
          sts128u(area + boff + lane * 32 + 16, hw_out[4], hw_out[5], hw_out[6], hw_out[7]);
          fence_proxy_async_smem();
          __syncwarp();
          if (send && lane == 0) {
            tma_store_2d_s(&pr->tmH, xcol, y32, area + boff);
            bulk_commit();
          }
        }
        // ---- quantise along the row
        uint32_t rlo = 0, rhi = 0;
        if (do_q) {
          float bmax;
          uint32_t sb;
          if (PF) sb = quantize_block16_opts<MODE != kG3>(v, args.q, sg_out, rlo, rhi, bmax);
          else sb = quantize_block16_pow2(v, sg_out, inv_sg, rcp_base, rlo, rhi, bmax);
          if (MODE == kG1 || MODE == kG3) amax = fmaxf(amax, bmax);
          sfw |= sb << (8 * e);
        }
        // ---- the buffer is free once every lane has read its column and the store has read the
        // block; the block two chunks ahead is fetched into it.  (Waiting for the store's read here
        // also covers the code stores of the previous tile before the first chunk writes codes.)
        // The column reads above belong to the generic proxy, the fetch below writes the buffer through the
        // async proxy: without a fence between them nothing orders the two (the reads were seen to be
        // scheduled after the fetch, and now and then the new block arrived first).
        if (HAS_AUX) fence_proxy_async_smem();
        __syncwarp();
        TR_BEGIN
        if (lane == 0 && (STORE_F32 || i == 0)) bulk_wait_read<0>();
        TR_END(3)
        if (XBUF == 1) __syncwarp();  // one buffer: the next chunk is staged over this one, after the store's read
        if (HAS_AUX) {
          if (i < 2) fetch(pr, x64, y32, (i + 2) ^ flip, false, b);
          else if (has_next) fetch(probs + nxt.p, nxt.x64, nxt.y32, (i - 2) ^ (flip ^ 3), nxt.below, b);
        }
        if (do_q) {
          if (i == 0) {
            __syncwarp();
            // the stores of the previous tile have read the half's staging area
            wait_or_abort(half_free, (seq & 1) ^ 1, abort_flag);
          }
          sts64u(rq_st + lane * 32 + e * 8, rlo, rhi);
        }
        // ---- quantise down the columns
        if (mirror) {
          uint32_t lo, hi;
          float bmax;
          uint32_t sb;
          if (PF) sb = quantize_block16_opts<MODE != kG3>(w, args.q, sg_out, lo, hi, bmax);
          else sb = quantize_block16_pow2(w, sg_out, inv_sg, rcp_base, lo, hi, bmax);
          sts64u(cq_st + e * (CHUNK * 64), lo, hi);
          // tensor row = x64 + e * 16 + cq: e % 2 selects the upper 16 of 32 rows of its scale atom,
          // e / 2 the 32-row group
          sts8(csf_st + (e & 1) * 256 + (e >> 1) * 4, sb);
        }
      }
      if (do_q) {
        // the scale word of this warp's 64 columns of the row; the codes of the warp's part of the tile
        sts32(rsf_st, sfw);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_s(half_done);
          tma_store_2d_s(&pr->tmRq, x64 >> 1, y32, rq_st);
          bulk_commit();
        }
      }
      cur = nxt;
    }
    if ((MODE == kG1 || MODE == kG3) && cur_p >= 0) {
#pragma unroll
      for (int o = 16; o; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
      if (lane == 0) {
        const int slot = (MODE == kG1) ? args.ix.amax_A0 + args.iter : args.ix.amax_X0 + args.iter + 1;
        atomicMax(reinterpret_cast<uint32_t*>(pr->scalars + slot), __float_as_uint(amax));
      }
    }
    TR_FLUSH
    if (lane == 0) bulk_wait_all<0>();  // this warp's stores have left shared memory and are complete
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

template <int MODE, bool PF, bool BH, bool UPD = false>
cudaError_t launch_pair_mode(const ProblemPack& pack, const GemmLaunch& L, int sms, cudaStream_t st) {
  const int tpp = L.symmetric ? L.tiles_n * (L.tiles_n + 1) / 2 : L.tiles_m * L.tiles_n;
  const int num_tiles = tpp * L.num_problems;
  int pairs = sms / 2;
  if (pairs > num_tiles) pairs = num_tiles;
  count_launches(1);
  launch_chained(k_gemm_pair<MODE, PF, BH, UPD>, dim3(2 * pairs), dim3(NTHREADS), Lay<MODE>::SMEM_BYTES, st, pack, L);
  return cudaGetLastError();
}

}  // namespace

#ifdef FP4_TRACE
extern "C" int fp4_trace_read(unsigned long long* dst, int clear) {
  if (cudaMemcpyFromSymbol(dst, g_trace, sizeof(g_trace)) != cudaSuccess) return 1;
  if (clear) {
    static unsigned long long zero[160 * 18 * 8];
    if (cudaMemcpyToSymbol(g_trace, zero, sizeof(zero)) != cudaSuccess) return 1;
  }
  return 0;
}
#endif

cudaError_t gemm_pair_set_attributes() {
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kPlain, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<kPlain>::SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG1, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<kG1>::SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG1, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<kG1>::SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG1, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<kG1>::SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG1, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<kG1>::SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG2, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<kG2>::SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG2, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<kG2>::SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG2, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<kG2>::SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG2, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<kG2>::SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG3, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<kG3>::SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG3, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<kG3>::SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG3, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<kG3>::SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG3, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<kG3>::SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG3, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<kG3>::SMEM_BYTES))) return e;
  if ((e = cudaFuncSetAttribute(k_gemm_pair<kG3, false, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Lay<kG3>::SMEM_BYTES))) return e;
  return cudaSuccess;
}

// Elements of K per operand stage of a mode: the operand and scale descriptors of a problem are built
// with boxes of that depth.
int gemm_pair_stage_k(GemmMode mode) {
  switch (mode) {
    case kG1: return Lay<kG1>::BK;
    case kG2: return Lay<kG2>::BK;
    case kG3: return Lay<kG3>::BK;
    default: return Lay<kPlain>::BK;
  }
}

// `launch` carries tile counts in 128-blocks; all of M, N, K must be multiples of 256.
cudaError_t launch_gemm_pair(GemmMode mode, const ProblemPack& pack, const GemmLaunch& launch, int sms,
                             cudaStream_t st) {
  if ((launch.tiles_m & 1) || (launch.tiles_n & 1) || (launch.K % 256)) return cudaErrorInvalidValue;
  if (launch.num_problems < 1 || launch.num_problems > kPackMax) return cudaErrorInvalidValue;
  GemmLaunch L = launch;
  L.tiles_m = launch.tiles_m / 2;
  L.tiles_n = launch.tiles_n / 2;
  const bool pf = launch.q.rht || launch.q.four_six;
  const bool bh = launch.aux_h != 0 || launch.out_h != 0;
#define FP4_PAIR_CASE(M)                                                                \
  return pf ? (bh ? launch_pair_mode<M, true, true>(pack, L, sms, st)                    \
                  : launch_pair_mode<M, true, false>(pack, L, sms, st))                  \
            : (bh ? launch_pair_mode<M, false, true>(pack, L, sms, st)                   \
                  : launch_pair_mode<M, false, false>(pack, L, sms, st))
  if (launch.update) {
    // the last G3 stage with the parameter update: nothing is quantised there (write_q = 0)
    if (mode != kG3 || launch.write_q) return cudaErrorInvalidValue;
    return bh ? launch_pair_mode<kG3, false, true, true>(pack, L, sms, st)
              : launch_pair_mode<kG3, false, false, true>(pack, L, sms, st);
  }
  switch (mode) {
    case kPlain: return launch_pair_mode<kPlain, false, false>(pack, L, sms, st);
    case kG1: FP4_PAIR_CASE(kG1);
    case kG2: FP4_PAIR_CASE(kG2);
    default: FP4_PAIR_CASE(kG3);
  }
#undef FP4_PAIR_CASE
}

}  // namespace fp4
