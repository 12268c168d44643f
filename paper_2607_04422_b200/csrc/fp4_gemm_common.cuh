// Device helpers shared by the two GEMM kernels (one CTA per tile / a pair of CTAs per tile).
#pragma once

#include "fp4_kernels.h"

namespace fp4 {

__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// Wait on an mbarrier phase for at most limit_ns; false on give-up (own time-out or another
// thread's abort flag).
static __device__ __noinline__ bool wait_limited(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                 uint64_t limit_ns) {
  const uint64_t t0 = globaltimer_ns();
  for (;;) {
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (globaltimer_ns() - t0 > limit_ns) {
      *abort_flag = 1;
      return false;
    }
  }
}
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // two seconds
static __device__ __forceinline__ bool wait_slow(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag) {
  return wait_limited(bar, parity, abort_flag, kWaitLimitNs);
}
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  return wait_slow(bar, parity, abort_flag);
}

// The same wait for callers that do not branch on the outcome: when a wait gives up (its own
// time-out, or another thread of the CTA gave up before) the abort flag is set and every later
// wait of the CTA falls through at once, so the kernel runs to its end on whatever data it has
// and the host reads FP4_ERR_DEVICE_TIMEOUT from the status word.  The polls carry a suspend-time
// hint: the thread sleeps in hardware until the phase completes instead of spinning.
__device__ __forceinline__ bool mbar_try_wait_hint(uint32_t bar_addr, uint32_t parity, uint32_t hint_ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar_addr), "r"(parity), "r"(hint_ns)
      : "memory");
  return ok != 0;
}
static __device__ __noinline__ void wait_slow_abort(uint32_t bar_addr, uint32_t parity, volatile uint32_t* abort_flag) {
  const uint64_t t0 = globaltimer_ns();
  for (;;) {
    if (*abort_flag) return;
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait_hint(bar_addr, parity, 4000u)) return;
    if (globaltimer_ns() - t0 > kWaitLimitNs) {
      *abort_flag = 1;
      return;
    }
  }
}
__device__ __forceinline__ void wait_or_abort(uint32_t bar_addr, uint32_t parity, volatile uint32_t* abort_flag) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar_addr), "r"(parity)
      : "memory");
  if (!ok) wait_slow_abort(bar_addr, parity, abort_flag);
}
__device__ __forceinline__ void wait_or_abort(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag) {
  wait_or_abort(smem_u32(bar), parity, abort_flag);
}

// tile index of a launch -> (problem, tile row, tile column)
__device__ __forceinline__ void decode_tile(int t, const GemmLaunch& L, int tiles_per_problem, int& p, int& ti,
                                            int& tj, bool sym) {
  p = t / tiles_per_problem;
  t -= p * tiles_per_problem;
  const int tiles_n = L.tiles_n;
  if (!sym) {
    ti = t / tiles_n;
    tj = t - ti * tiles_n;
  } else {
    int row = 0, rem = t;
    while (rem >= tiles_n - row) { rem -= tiles_n - row; ++row; }
    ti = row;
    tj = row + rem;
  }
}
__device__ __forceinline__ void decode_tile(int t, const GemmLaunch& L, int tiles_per_problem, int& p, int& ti,
                                            int& tj) {
  decode_tile(t, L, tiles_per_problem, p, ti, tj, L.symmetric != 0);
}

// Per-call scalars of an epilogue: the factor that turns the accumulator into the
// product (tensor scales of the two operands) and the tensor scale of the quantised
// output, predicted from the running maxima (power of two); the bound is widened by
// args.q.widen when the output is rotated before quantisation (|x H| <= 4 amax(x)).
template <int MODE>
__device__ __forceinline__ void epilogue_scalars(const GemmProblem& pr, const GemmLaunch& args, float& scale,
                                                 float& sg_out, bool publish) {
  float* sc = pr.scalars;
  sg_out = 1.0f;
  if (MODE == kPlain) {
    scale = __fmul_rn(pr.sg_a, pr.sg_b);
  } else if (MODE == kG1) {
    const float sgx = sc[args.ix.sg_X0 + args.iter];
    const float ax = sc[args.ix.amax_X0 + args.iter];
    scale = __fmul_rn(sgx, sgx);
    float bound = __fmul_rn(__fmul_rn(__fmul_rn(2.0f, args.l_cols), ax), ax);
    sg_out = scale_predicted(__fmul_rn(args.q.widen, fminf(bound, 4.0f)));
    if (publish) sc[args.ix.sg_A0 + args.iter] = sg_out;
  } else if (MODE == kG2) {
    const float sga = sc[args.ix.sg_A0 + args.iter];
    const float aa = sc[args.ix.amax_A0 + args.iter];
    scale = __fmul_rn(sga, sga);
    float bound = __fmul_rn(__fadd_rn(fabsf(pr.cb), __fmul_rn(4.0f, fabsf(pr.cc))), aa);
    sg_out = scale_predicted(__fmul_rn(args.q.widen, bound));
    if (publish) sc[args.ix.sg_B0 + args.iter] = sg_out;
  } else {
    const float sgb = sc[args.ix.sg_B0 + args.iter];
    const float sgx = sc[args.ix.sg_X0 + args.iter];
    const float ax = sc[args.ix.amax_X0 + args.iter];
    scale = __fmul_rn(sgb, sgx);
    float bound = __fmul_rn(__fmul_rn(4.0f, fabsf(pr.ca)), ax);
    sg_out = scale_predicted(__fmul_rn(args.q.widen, bound));
    if (publish) sc[args.ix.sg_X0 + args.iter + 1] = sg_out;
  }
}

}  // namespace fp4
