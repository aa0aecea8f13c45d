// Device-side helpers shared by the LANTERN kernels: warp reductions and scans, the JSD mass bound, mbarrier + bulk-copy (TMA) wrappers for sm_100a.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace lantern {

constexpr int kWarp = 32;
constexpr unsigned kFull = 0xffffffffu;

// ---------------------------------------------------------------------------------------
// warp primitives
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFull, v, o));
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}
__device__ __forceinline__ double warp_incl_scan(double v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    double t = __shfl_up_sync(kFull, v, o);
    if (lane >= o) v += t;
  }
  return v;
}

// ---------------------------------------------------------------------------------------
// JSD bound (Section 5.3.2).  Moving mass S onto a token of probability q0 changes the
// distribution by JSD (natural logarithm; only the collapsed tokens contribute)
//   f(S) = 1/2 [ S ln 2 + q0 ln(1 - x) + (q0 + S) ln(1 + x) ],   x = S / (2 q0 + S),
// since (q0 + S) / mid = 1 + x and q0 / mid = 1 - x for mid = q0 + S/2.  f is increasing and
// convex in S with f' = 1/2 [ln 2 + ln(1 + x)], so "f(S) < delta" is "S < S*" with f(S*) = delta,
// and the prefix test stays a comparison of a running sum with one number per draft.  S* by
// Newton's method from the upper bound 2 delta / ln 2 (f >= S ln2 / 2): four steps in single
// precision, one in double precision (|f(S*) - delta| below 1e-8 over delta in [1e-7, 2],
// q0 in [0, 1] on a CPU replica; the decision window is 1e-6).  Called by one thread per draft, which publishes the result: kept out of line
// so that the callers' register budgets do not see it.
// ---------------------------------------------------------------------------------------
static __device__ __noinline__ double jsd_mass_bound(double delta, double q0) {
  const double LN2 = 0.69314718055994530942;
  if (!(delta > 0.0)) return 0.0;
  if (!(q0 > 0.0)) return delta / LN2;   // f(S) = S ln 2 exactly
  const float LN2F = 0.693147182464599609375f;
  const float qf = static_cast<float>(q0), df = static_cast<float>(delta);
  float Sf = 2.0f * df / LN2F;
#pragma unroll 1
  for (int it = 0; it < 4; ++it) {
    const float x = Sf / (2.0f * qf + Sf);
    const float lp = log1pf(x);
    const float t = Sf * LN2F + (qf + Sf) * lp + qf * log1pf(-x);
    Sf -= (0.5f * t - df) / (0.5f * (LN2F + lp));
    Sf = Sf > 0.0f ? Sf : 0.0f;
  }
  double S = Sf > 0.0f ? static_cast<double>(Sf) : delta / LN2;
  {
    const double x = S / (2.0 * q0 + S);
    const double lp = log1p(x);
    const double t = S * LN2 + (q0 + S) * lp + q0 * log1p(-x);
    S -= (0.5 * t - delta) / (0.5 * (LN2 + lp));
  }
  return S;
}

// The same bound found by a whole warp (all 32 lanes call it and get the same value): f is increasing and
// S ln2 / 2 <= f(S) <= S ln 2, so the root lies in [delta / ln 2, 2 delta / ln 2]; three rounds in which the 32
// lanes evaluate f (single precision) at 32 points of the current interval and a ballot picks the
// sub-interval narrow it by 33^3, and one Newton step in double precision finishes.  A third of the
// latency of the one-thread iteration above, which sits on every context's critical path.
static __device__ __forceinline__ double jsd_mass_bound_warp(double delta, double q0, int lane) {
  const double LN2 = 0.69314718055994530942;
  if (!(delta > 0.0)) return 0.0;
  if (!(q0 > 0.0)) return delta / LN2;   // f(S) = S ln 2 exactly
  const float LN2F = 0.693147182464599609375f;
  const float qf = static_cast<float>(q0), df = static_cast<float>(delta);
  float lo = df / LN2F, w = lo;          // the root lies in [lo, lo + w]
#pragma unroll 1
  for (int round = 0; round < 3; ++round) {
    const float step = w * (1.0f / 33.0f);
    const float Sf = lo + step * static_cast<float>(lane + 1);
    const float x = Sf / (2.0f * qf + Sf);
    const float t = Sf * LN2F + (qf + Sf) * log1pf(x) + (x < 1.0f ? qf * log1pf(-x) : 0.0f);   // q0 ln(1 - x) -> 0 with q0
    const int below = __popc(__ballot_sync(0xffffffffu, 0.5f * t < df));   // f is increasing: a prefix of the lanes
    lo += step * static_cast<float>(below);
    w = step;
  }
  double S = static_cast<double>(lo) + 0.5 * static_cast<double>(w);
  {
    const double x = S / (2.0 * q0 + S);
    const double lp = log1p(x);
    const double t = S * LN2 + (q0 + S) * lp + q0 * log1p(-x);
    S -= (0.5 * t - delta) / (0.5 * (LN2 + lp));
  }
  return S;
}

// ---------------------------------------------------------------------------------------
// shared-memory barrier (mbarrier) and bulk asynchronous copy global -> shared
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
               : "memory");
}
// One bulk copy of `bytes` (multiple of 16, both addresses 16-byte aligned) that reports its
// completion to `bar`.  No multicast: the destination is this CTA's own shared memory.
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_addr(dst_smem)),
               "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar))
               : "memory");
}
// Bounded wait for phase `parity` of `bar`.  Returns false if the limit ran out.  Each try may suspend
// the thread in hardware for up to `suspend_ns` (it wakes when the phase completes), so a long wait costs
// few issue slots; the hint is an upper limit, the loop bound is what ends a wait that never completes.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint32_t max_tries = (1u << 21),
                                          uint32_t suspend_ns = 4000) {
  const uint32_t a = smem_addr(bar);
  for (uint32_t i = 0; i < max_tries; ++i) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(a), "r"(parity), "r"(suspend_ns)
        : "memory");
    if (ok) return true;
  }
  return false;
}

}  // namespace lantern
