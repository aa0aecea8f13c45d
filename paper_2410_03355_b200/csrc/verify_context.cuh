// Fused context pass of the LANTERN verification step (included by verify.cu).
//
// Persistent kernel, one CTA per SM.  The CTA holds TWO independent consumer groups of eight
// warps, each working on its own context in its own staging area of shared memory, and two
// producer warps (one thread each) that hand out contexts and issue the bulk asynchronous
// copies (TMA, completion on an mbarrier, no multicast) of a group's next rows as soon as the
// group releases its area.  The two groups drift apart in phase, so the latency-bound deciding
// part of one context overlaps the issue-bound streaming part of the other and the copy of a
// third: the SM is rarely idle although every context is a chain of dependent steps.
//
// Streaming part (per thread, on its own tokens, in passes of at most 32 tokens): guidance
// combine, the thread's own maximum, numerators 2^((z - max) log2 e) through the hardware ex2
// unit, partial sums -- no cross-thread step at all, so the warps stream at full rate.  The
// numerators E are stored over the context's own raw target rows (every thread overwrites only
// bytes that it alone has read) and stay in the units of their (pass, thread) slice; a
// per-slice factor, tabulated once the common maximum is known, brings them to common units
// when they are used.  Sums
// over many numerators average the ex2 unit's ~1e-7 rounding out; the two single probabilities
// that decide a position, q(x~) and p(x~), are recomputed by one thread in double precision.
//
// Deciding part, per child (Section 4.3 / Algorithm 2, second block): gather of the neighbour
// row's numerators, double-precision scan against the strict bound, accept test; on rejection
// the residual [q_{k,delta}(.|D = x~) - p]_+ in one register pass (drafter numerators are
// recomputed from the raw drafter row, which stays in shared memory), its total, and either the
// inverse-CDF draw or the write-back for the next sibling.
#pragma once

// Which contexts are evaluated.  Algorithm 1 stops at the first rejection, so a context behind a
// rejected node is never tested by the method.  Work items come in breadth-first order per sequence
// (see the plan kernel); when a context has been decided, its group marks the contexts behind every
// child it did not accept as dead (a sequence's contexts are numbered in pre-order for this, so that a
// subtree is one contiguous range of marks), and a producer that meets a dead context leaves it out.  A context whose parent is still undecided when its turn comes is
// evaluated anyway: with few sequences per call that keeps every SM busy (all contexts of a tree run
// side by side), with many sequences it is rare, and the walk kernel reads only records on the
// accepted path either way, so the result never depends on what was speculated.
#define LANTERN_CONTEXT_KERNEL_REVISION 18   // bump on every change to this file

namespace lantern {

constexpr int GT = 256;         // threads of one consumer group
constexpr int GW = GT / 32;     // warps of one consumer group
constexpr int LOG_GT = 8;
constexpr int NGRP = 2;         // consumer groups per CTA
constexpr int MAXU = 16;        // (pass, warp) slices of a context, at most
constexpr int kNone = 0x7fffffff;
// A residual whose total weight is at most this fraction of the current target's mass defines no
// distribution to draw from (the single-precision residual pass resolves totals to a few 1e-7 of that
// mass): the walk stops there and the next token comes from the context's own target.
constexpr double kDegenerate = 1e-5;
constexpr int CTX_THREADS = NGRP * GT + NGRP * 32;   // consumers, then one producer warp per group

// Thread t of a group owns, for chunk c, the eight consecutive tokens [(c*GT + t)*8, +8), i.e. 16-byte
// group g = c*GT + t of a bf16 row.  E is laid over the context's own raw target rows: with bf16 logits
// the low four numerators of g replace g's bytes in row slot 0 and the high four replace g's bytes in
// row slot 1; with fp32 logits the eight numerators replace g's own 32 bytes of row slot 0.
// Float index of token x inside the staging area:
template <bool BF16>
__device__ __forceinline__ int ephys(int x, int row_floats) {
  if (BF16) return ((x >> 2) & 1) * row_floats + ((x >> 3) << 2) + (x & 3);
  return x;
}
// index of the (pass, thread) slice that owns token x in the factor table; LOG_CP = log2(chunks per pass)
template <int LOG_CP>
__device__ __forceinline__ int owner_slice(int x) {
  const int g = x >> 3;
  return ((g >> (LOG_GT + LOG_CP)) << LOG_GT) | (g & (GT - 1));
}

__device__ __forceinline__ void gbar(int grp);   // barrier among the threads of one consumer group (below)

}  // namespace lantern
#include "verify_context_topk.cuh"
namespace lantern {

struct GroupShared {
  double wzq[GW], wzp[GW];      // per-warp sums of numerators, common units
  double wt[8 * GW];            // per-(chunk, warp) totals for scans and block sums
  double sbefore[GW];           // prefix sum just before a warp's first failing neighbour
  double acc_e, acc_p;          // double-precision numerators of the tested x~, common units
  double hist[32];              // drafter/target scale ratio of each earlier rejection round of this context
  float fqt[2 * GT];            // factor of every (pass, thread) slice: its units -> common units
  float wmq[GW], wmp[GW];       // per-warp maxima of the slices' shift constants
  int first[GW];                // a warp's first failing neighbour slot
  int badslot[GW];              // a warp's first neighbour slot with an entry outside [0, V)
  int cand[GW];
  int acc_valid;                // acc_e / acc_p are usable for the current child
  int tok;
  int fail;                     // a bounded wait for the target rows ran out (sticky)
  GroupTopk tk;                 // scratch of the top-k threshold search (TOPK variants)
  GroupItem work[2];            // descriptor of context i in work[i & 1]: the next one is published while the current one runs
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 2^(z log2(e) - shift) for one value, to about 1.5e-7: the exponent is formed in double precision,
// split into an fp32 head for the ex2 unit and a tail that is applied to first order.
__device__ __forceinline__ double exp2_single(float z, float shift) {
  const double x = static_cast<double>(z) * 1.4426950408889634074 - static_cast<double>(shift);
  const float xh = static_cast<float>(x);
  if (xh < -1000.0f) return 0.0;   // far below the flush-to-zero range; also keeps -inf from turning into inf - inf
  const float xl = static_cast<float>(x - static_cast<double>(xh));
  const float y = ex2_approx(xh);
  return static_cast<double>(__fmaf_rn(y, xl * 0.693147182464599609375f, y));
}

// one row of a context into one row slot of a staging area, in bulk copies of at most 16 KB
__device__ __forceinline__ void ctx_issue_row(unsigned char* dst, const unsigned char* src, int rowbytes, uint64_t* bar) {
  for (int off = 0; off < rowbytes; off += 16384) {
    const int n = min(16384, rowbytes - off);
    bulk_load(dst + off, src + off, static_cast<uint32_t>(n), bar);
  }
}
// the drafter row of a context, into row slot 2
__device__ __forceinline__ void ctx_issue_drafter(const VerifyParams& P, int item, unsigned char* stage, int rowbytes,
                                                  uint64_t* bar) {
  mbar_expect_tx(bar, static_cast<uint32_t>(rowbytes));
  ctx_issue_row(stage + 2 * rowbytes, static_cast<const unsigned char*>(P.draft) + static_cast<size_t>(item) * rowbytes,
                rowbytes, bar);
}
// the target rows of a context (conditional, and unconditional if there is one), into row slots 0 and 1
template <bool UNC>
__device__ __forceinline__ void ctx_issue_target(const VerifyParams& P, int item, unsigned char* stage, int rowbytes,
                                                 uint64_t* bar) {
  mbar_expect_tx(bar, static_cast<uint32_t>((UNC ? 2 : 1) * rowbytes));
  const size_t row_off = static_cast<size_t>(item) * rowbytes;
  const unsigned char* t = static_cast<const unsigned char*>(P.target) + row_off;
  ctx_issue_row(stage, t, rowbytes, bar);
  if (UNC) ctx_issue_row(stage + rowbytes, t + static_cast<size_t>(P.B) * P.R * rowbytes, rowbytes, bar);
}

// Ask L2 for the rows of a context ahead of time: the bulk copy that later brings them into shared
// memory (it cannot start before the group has released its staging area) then finds them on chip.
template <bool BF16, bool UNC>
__device__ __forceinline__ void ctx_prefetch_rows(const VerifyParams& P, int item, int rowbytes) {
  const size_t row_off = static_cast<size_t>(item) * rowbytes;
  const size_t branch = static_cast<size_t>(P.B) * P.R * rowbytes;
  const unsigned char* t = static_cast<const unsigned char*>(P.target) + row_off;
  const unsigned char* d = static_cast<const unsigned char*>(P.draft) + row_off;
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(t), "r"(rowbytes) : "memory");
  if (UNC) asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(t + branch), "r"(rowbytes) : "memory");
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(d), "r"(rowbytes) : "memory");
}

// one logit of a row in global memory, widened to fp32
template <bool BF16>
__device__ __forceinline__ float ctx_raw_logit(const void* base, size_t elem) {
  if (BF16) return __uint_as_float(static_cast<uint32_t>(__ldg(static_cast<const unsigned short*>(base) + elem)) << 16);
  return __ldg(static_cast<const float*>(base) + elem);
}

// Packed pairs of fp32 values (Blackwell's two-wide fp32 instructions): each lane is rounded exactly
// like the scalar instruction, so results do not depend on the packing.
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// barrier among the 256 threads of consumer group `grp` (hardware barrier 1 + grp)
__device__ __forceinline__ void gbar(int grp) { asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "n"(GT) : "memory"); }
// the same barrier, returning the AND of every thread's predicate
__device__ __forceinline__ bool gbar_and(int grp, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 p, %1, 0;\n\t"
      "bar.red.and.pred q, %2, %3, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r)
      : "r"(static_cast<uint32_t>(pred)), "r"(1 + grp), "n"(GT)
      : "memory");
  return r != 0;
}
// a load that stays where it is written (issued early on purpose; the value is used much later)
__device__ __forceinline__ int ld_nc_here(const int32_t* p) {
  int v;
  asm volatile("ld.global.nc.s32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// CH = 8-token chunks per thread (1, 2, 4 or 8); a thread streams them in NP passes of CP chunks.
// TONE = the temperature is exactly 1 (the paper's sampling setting): no division is compiled in.
// JSD selects the Section 5.3.2 bound at compile time, so that the default path carries none of its code.
// TOPK applies the per-row thresholds of the top-k logit filter (Appendix B.2; written by
// lantern_topk_kernel): processed logits below a row's threshold count as -inf.
template <int CH, bool BF16, bool UNC, bool TONE, bool JSD, bool TOPK>
__global__ void __launch_bounds__(CTX_THREADS, 1) lantern_context_kernel(VerifyParams P) {
  constexpr int NP = CH > 4 ? 2 : 1;          // passes
  constexpr int CP = CH / NP;                 // chunks per pass
  constexpr int LOG_CP = CP == 4 ? 2 : (CP == 2 ? 1 : 0);
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ GroupShared SG[NGRP];
  // per group: drafter row landed / target rows landed / drafter slot free / target slots (E) free
  __shared__ __align__(8) uint64_t bar_full_d[NGRP], bar_full_t[NGRP], bar_empty_d[NGRP], bar_empty_t[NGRP];

  const int tid = threadIdx.x, lane = tid & 31;
  const int V = P.V, N = P.N, R = P.R, k = P.k;
  const int rowbytes = V * (BF16 ? 2 : 4);
  const int stage_bytes = (3 * rowbytes + 127) & ~127;   // row slots: conditional, unconditional, drafter
  const int row_floats = rowbytes >> 2;
  auto EI = [&](int x) { return ephys<BF16>(x, row_floats); };
  const float L_hi = 1.44269502162933349609375f;   // fl32(log2 e)
  const float ninf = __int_as_float(0xff800000);

  if (tid == 0) {
    for (int g = 0; g < NGRP; ++g) {
      mbar_init(&bar_full_d[g], 1);
      mbar_init(&bar_full_t[g], 1);
      mbar_init(&bar_empty_d[g], GW);
      mbar_init(&bar_empty_t[g], GW);
      SG[g].fail = 0;
      SG[g].tk.n_list[0] = SG[g].tk.n_list[1] = 0;
    }
    fence_mbar_init();
    fence_proxy_async();
  }
  if (TOPK && tid < NGRP * GT) SG[tid >> LOG_GT].tk.hist[0][tid & (GT - 1)] = SG[tid >> LOG_GT].tk.hist[1][tid & (GT - 1)] = 0;
  __syncthreads();

  // ======================= producer warps =======================
  // One warp per consumer group hands out work and keeps that group's copies going.  Its 32 lanes look
  // at up to 32 consecutive work slots at a time (a batch: the first one dealt statically, later ones
  // from a global counter, in sizes that shrink towards the end of the list so that the groups finish
  // together), drop the empty and the dead ones, and lane 0 feeds the rest to the group one by one:
  // the drafter row as soon as the group has streamed the previous one, the target rows as soon as the
  // group releases its staging area.  The next batch is loaded while the current one is being worked
  // on, so that no round trip to the work list is on the critical path.
  if (tid >= NGRP * GT) {
    const int grp = (tid - NGRP * GT) >> 5;
    GroupShared& S = SG[grp];
    const int total = P.counters->n_rank * P.B;  // occupied part of the slot array
    const int G = gridDim.x * NGRP;              // producers in the grid
    const int me = blockIdx.x * NGRP + grp;
    const uint32_t tries = P.wait_tries;
    // Slots per batch.  Few live contexts per batch (two; one towards the end of the list, so that the groups
    // finish together): a batch is worked through in order, and the longer that takes the more of its
    // contexts meet an undecided parent and are evaluated for nothing.  But as many slots as it has taken so
    // far to find that many live ones: tree workloads leave most slots empty or dead, and every batch costs a
    // round trip to the work list.
    int slots_seen = 0, live_seen = 0;
    auto batch_size = [&](int at) {
      const int share = (total - at) / (4 * G);
      const int live = share < 1 ? 1 : (share > 2 ? 2 : share);
      const int s = live * ((slots_seen + 1) / (live_seen + 1));
      return s < 1 ? 1 : (s > 32 ? 32 : s);
    };
    struct Cand {
      int item, cbase, nchild_node0, span0, tok0, mark;
      float r0, u_final;
    };
    auto load_cand = [&](int start, int size) -> Cand {
      Cand c;
      c.item = -1;
      c.cbase = c.nchild_node0 = c.span0 = c.tok0 = c.mark = 0;
      c.r0 = c.u_final = 0.0f;
      const int w = start + lane;
      if (lane < size && w < total) {
        const int4 lo = __ldg(reinterpret_cast<const int4*>(P.work + w));
        const int4 hi = __ldg(reinterpret_cast<const int4*>(P.work + w) + 1);
        c.item = lo.x, c.cbase = lo.y, c.nchild_node0 = lo.z, c.span0 = lo.w;
        c.tok0 = hi.x, c.r0 = __int_as_float(hi.y), c.u_final = __int_as_float(hi.z), c.mark = hi.w;
      }
      return c;
    };
    auto is_dead = [&](int mark) -> bool {
      return *reinterpret_cast<const volatile unsigned char*>(P.dead + mark) != 0;
    };
    int n_eval = 0, n_skip = 0;
    // live candidates of a batch, as a lane mask
    auto filter = [&](const Cand& c) -> unsigned {
      const bool has = c.item >= 0;
      const bool dead = has && is_dead(c.mark);
      n_skip += __popc(__ballot_sync(kFull, dead));
      const unsigned live = __ballot_sync(kFull, has && !dead);
      live_seen += __popc(live);
      return live;
    };
    const int b0 = batch_size(0);
    Cand cur = load_cand(me * b0, b0);
    bool cur_end = me * b0 >= total;
    int seen = G * b0;
    // start of the next dynamic batch (lane 0 asks, everybody hears)
    auto grab = [&](int& size) -> int {
      size = batch_size(seen < total ? seen : total);
      int st = 0;
      if (lane == 0) st = G * b0 + atomicAdd(&P.counters->work_next, size);
      st = __shfl_sync(kFull, st, 0);
      seen = st;
      slots_seen += size;
      return st;
    };
    int nsize = 0;
    int nstart = grab(nsize);
    Cand nxt = load_cand(nstart, nsize);
    bool nxt_end = nstart >= total;
    unsigned mask = filter(cur);
    int i = 0;        // contexts handed to the group so far
    bool clean = true;
    auto next_batch = [&]() {   // make `mask` non-empty if any live context is left
      while (mask == 0 && !cur_end) {
        cur = nxt;
        cur_end = nxt_end;
        if (!cur_end) {
          nstart = grab(nsize);
          nxt = load_cand(nstart, nsize);
          nxt_end = nstart >= total;
        }
        mask = filter(cur);
      }
    };
    for (;;) {
      next_batch();
      if (mask == 0) break;
      const int l = __ffs(mask) - 1;
      mask &= mask - 1;
      // Top-k filter: where the two thresholds of this context lie, from a sample of its rows in global memory
      // (they have been asked into L2 already) -- found now, while the group is busy with the context before.
      float br_d[4] = {0.0f, 0.0f, 0.0f, 0.0f}, br_t[4] = {0.0f, 0.0f, 0.0f, 0.0f};
      if (TOPK) {
        const int item_l = __shfl_sync(kFull, cur.item, l);
        const size_t row = static_cast<size_t>(item_l) * V;
        const size_t branch = static_cast<size_t>(P.B) * R * V;
        auto raw8 = [&](const void* base, size_t elem, float (&z)[8]) {
          if (BF16) {
            const uint4 x = __ldg(reinterpret_cast<const uint4*>(static_cast<const unsigned short*>(base) + elem));
            const uint32_t xw[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              z[2 * q] = __uint_as_float(xw[q] << 16);
              z[2 * q + 1] = __uint_as_float(xw[q] & 0xffff0000u);
            }
          } else {
            const float4 x0 = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(base) + elem));
            const float4 x1 = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(base) + elem) + 1);
            z[0] = x0.x, z[1] = x0.y, z[2] = x0.z, z[3] = x0.w, z[4] = x1.x, z[5] = x1.y, z[6] = x1.z, z[7] = x1.w;
          }
        };
        auto zd_g = [&](int g, float (&z)[8]) {      // the same operations as the streaming loop, lane by lane
          raw8(P.draft, row + static_cast<size_t>(g) * 8, z);
          if (!TONE) {
#pragma unroll
            for (int e = 0; e < 8; ++e) z[e] = __fdiv_rn(z[e], P.T);
          }
        };
        auto zt_g = [&](int g, float (&z)[8]) {
          raw8(P.target, row + static_cast<size_t>(g) * 8, z);
          if (UNC) {
            float u[8];
            raw8(P.target, branch + row + static_cast<size_t>(g) * 8, u);
#pragma unroll
            for (int e = 0; e < 8; ++e) z[e] = __fmaf_rn(P.cfg_scale, __fsub_rn(z[e], u[e]), u[e]);
          }
          if (!TONE) {
#pragma unroll
            for (int e = 0; e < 8; ++e) z[e] = __fdiv_rn(z[e], P.T);
          }
        };
        tkg_warp_bracket(zd_g, P.top_k, V, lane, br_d);
        tkg_warp_bracket(zt_g, P.top_k, V, lane, br_t);
      }
      // The drafter slot is free once every warp of the group has streamed the previous context's
      // drafter row (nothing reads it afterwards), i.e. while that context is still being decided:
      // the next drafter row travels early, and the group streams it while its target rows are copied.
      if (i >= 1 && !mbar_wait(&bar_empty_d[grp], (i - 1) & 1, tries)) {
        clean = false;   // the group never released its slot: it has given up, and so does its producer
        break;
      }
      // as late as possible: has the context died meanwhile, has the call been given up?
      const int gone = (lane == l && is_dead(cur.mark)) ? 1 : 0;
      const int stop = *reinterpret_cast<const volatile int*>(&P.counters->abort);
      if (__any_sync(kFull, stop != 0)) break;
      if (__any_sync(kFull, gone)) {
        ++n_skip;
        continue;
      }
      GroupItem it;
      it.item = __shfl_sync(kFull, cur.item, l);
      it.cbase = __shfl_sync(kFull, cur.cbase, l);
      const int nn0 = __shfl_sync(kFull, cur.nchild_node0, l);
      it.nchild = nn0 >> 16;
      it.node0 = nn0 & 0xffff;
      it.span0 = __shfl_sync(kFull, cur.span0, l);
      it.tok0 = __shfl_sync(kFull, cur.tok0, l);
      it.r0 = __shfl_sync(kFull, cur.r0, l);
      it.u_final = __shfl_sync(kFull, cur.u_final, l);
#pragma unroll
      for (int q = 0; q < 4; ++q) it.bracket[0][q] = br_d[q], it.bracket[1][q] = br_t[q];
      bool ok = true;
      if (lane == 0) {
        S.work[i & 1] = it;                   // published by the mbarrier operation of the copy below
        const bool withheld = it.item == P.withhold_item;   // self-test of the bounded waits: nothing is copied
        fence_proxy_async();
        if (!withheld) ctx_issue_drafter(P, it.item, smem + grp * stage_bytes, rowbytes, &bar_full_d[grp]);
        // the target slots (later E) are free once every warp of the group has finished the previous context
        if (i >= 1 && !mbar_wait(&bar_empty_t[grp], (i - 1) & 1, tries)) ok = false;
        if (ok && !withheld) {
          fence_proxy_async();
          ctx_issue_target<UNC>(P, it.item, smem + grp * stage_bytes, rowbytes, &bar_full_t[grp]);
        }
      }
      ok = __shfl_sync(kFull, ok ? 1 : 0, 0) != 0;
      ++n_eval;
      ++i;
      if (!ok) {
        clean = false;
        break;
      }
      // Look ahead: the next live context (a batch swap, if the current batch is used up, happens here, where
      // nothing waits for it) and an L2 prefetch of its rows -- of a context that has passed the dead check,
      // so that hardly any prefetched row goes unused.
      next_batch();
      if (mask) {
        const int item_ahead = __shfl_sync(kFull, cur.item, __ffs(mask) - 1);
        if (lane == 0) ctx_prefetch_rows<BF16, UNC>(P, item_ahead, rowbytes);
      }
    }
    if (lane == 0) {
      if (clean) {   // the group is waiting for its next context: hand it the terminator
        if (i == 0 || mbar_wait(&bar_empty_d[grp], (i - 1) & 1, tries)) {
          S.work[i & 1].item = -1;
          __threadfence_block();
          mbar_arrive(&bar_full_d[grp]);
        }
      }
      if (n_eval) atomicAdd(&P.counters->n_evaluated, n_eval);
      if (n_skip) atomicAdd(&P.counters->n_skipped, n_skip);
    }
    return;
  }

  // ======================= consumer groups =======================
  const int grp = tid >> LOG_GT;        // which group
  const int gt = tid & (GT - 1);        // thread within the group
  const int gw = gt >> 5;               // warp within the group
  GroupShared& S = SG[grp];
  unsigned char* stage = smem + grp * stage_bytes;    // this group's rows, later its E
  float* E = reinterpret_cast<float*>(stage);
  // staging rows: 0 = conditional target, 1 = unconditional target (if any), 2 = drafter
  const unsigned char* rc = stage;
  const unsigned char* ru = stage + rowbytes;
  unsigned char* rd = stage + 2 * rowbytes;
  constexpr bool T_is_one = TONE;
  // The eight raw drafter logits of 16-byte group g of a row in global memory (a rejection reads the
  // drafter row again from there -- normally from L2 -- because its slot already belongs to the next context)
  struct DraftRaw {
    uint4 a, b;   // b: second half of an fp32 group
  };
  auto draft_fetch = [&](const unsigned char* row, int g) {
    DraftRaw d;
    d.b = make_uint4(0, 0, 0, 0);
    if (BF16) {
      d.a = __ldg(reinterpret_cast<const uint4*>(row + static_cast<size_t>(g) * 16));
    } else {
      d.a = __ldg(reinterpret_cast<const uint4*>(row + static_cast<size_t>(g) * 32));
      d.b = __ldg(reinterpret_cast<const uint4*>(row + static_cast<size_t>(g) * 32 + 16));
    }
    return d;
  };
  // the same eight as processed logits (z_p = l_d / T)
  auto draft_chunk = [&](const DraftRaw& d, float (&out)[8]) {
    if (BF16) {
      const uint32_t dw[4] = {d.a.x, d.a.y, d.a.z, d.a.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        out[2 * i] = __uint_as_float(dw[i] << 16);
        out[2 * i + 1] = __uint_as_float(dw[i] & 0xffff0000u);
      }
    } else {
      const uint32_t dw[8] = {d.a.x, d.a.y, d.a.z, d.a.w, d.b.x, d.b.y, d.b.z, d.b.w};
#pragma unroll
      for (int e = 0; e < 8; ++e) out[e] = __uint_as_float(dw[e]);
    }
    if (!T_is_one) {
#pragma unroll
      for (int e = 0; e < 8; ++e) out[e] = __fdiv_rn(out[e], P.T);
    }
  };
  const uint32_t tries = P.wait_tries;
  // A bounded wait that runs out ends the group: the context keeps the "not evaluated" record the plan
  // gave it (the walk reports INTERNAL for a sequence that reaches it), the call is given up (no producer
  // hands out further work), and one thread gives the copies that may still be on their way into this
  // group's staging area the same bounded wait before the group leaves.
  auto give_up = [&](int iter, bool drafter_too) {
    if (gt == 0) {
      *reinterpret_cast<volatile int*>(&P.counters->abort) = 1;
      if (drafter_too) mbar_wait(&bar_full_d[grp], iter & 1, tries);
      mbar_wait(&bar_full_t[grp], iter & 1, tries);
      if (!drafter_too) mbar_wait(&bar_full_d[grp], (iter + 1) & 1, tries);   // the next drafter row may be under way
    }
  };
  for (int iter = 0;; ++iter) {
    // One warp watches the copy's mbarrier (bounded wait); the group barrier then releases everybody
    // at once and tells every thread alike whether the rows have landed.
    bool landed = true;
    if (gw == 0) landed = mbar_wait(&bar_full_d[grp], iter & 1, tries);
    const bool arrived = gbar_and(grp, landed);
    if (!arrived) {   // the drafter row did not land within the limit
      give_up(iter, true);
      break;
    }
    const GroupItem cur = S.work[iter & 1];
    const int item = cur.item;
    if (item < 0) break;
    float tq = 0.0f, tp = 0.0f;   // top-k thresholds of this context's target and drafter rows (found below)
    const int b = item / R;
    const ChildInfo* kids = P.children + cur.cbase;
    const int nchild = cur.nchild;

    // first child: its neighbour row (four slots per thread) and, for thread 0, its raw logits; issued
    // now, used after the streaming part
    int node = cur.node0;
    int xt = cur.tok0;
    float r = cur.r0;
    int nb[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int j = 4 * gt + 1 + i;
      nb[i] = (j < k) ? ld_nc_here(P.nbr + static_cast<size_t>(xt) * k + j) : -1;
    }
    // (the drafter logit of x~ goes to every thread: the drafter row does not stay in shared memory)
    float raw_c = 0.0f, raw_u = 0.0f;
    float raw_d = ctx_raw_logit<BF16>(P.draft, static_cast<size_t>(item) * V + xt);
    if (gt == 0) {
      const size_t e = static_cast<size_t>(item) * V + xt;
      raw_c = ctx_raw_logit<BF16>(P.target, e);
      if (UNC) raw_u = ctx_raw_logit<BF16>(P.target, static_cast<size_t>(P.B) * R * V + e);
    }

    // ---------------- streaming part, thread-local, NP passes of CP chunks ----------------
    // values travel as packed pairs (tokens 2i, 2i+1 of a chunk)
    uint64_t a2[CP * 4];
    float mlq_mine[NP], mlp_mine[NP];   // this thread's shift constants fl(max * log2 e), per pass
    float tq_mine[NP], tp_mine[NP];     // and its sums of numerators, in its own units
    const uint64_t L2 = pack2(L_hi, L_hi);
    // four packed pairs of processed logits of 16-byte group g of a row
    auto pairs_of = [&](const unsigned char* row, int g, uint64_t (&o)[4]) {
      if (BF16) {
        const uint4 x = *reinterpret_cast<const uint4*>(row + g * 16);
        const uint32_t xw[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) o[i] = pack2(__uint_as_float(xw[i] << 16), __uint_as_float(xw[i] & 0xffff0000u));
      } else {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float4 x = *reinterpret_cast<const float4*>(row + g * 32 + h * 16);
          o[2 * h] = pack2(x.x, x.y);
          o[2 * h + 1] = pack2(x.z, x.w);
        }
      }
    };
    auto divide_T = [&](uint64_t v) {
      float lo, hi;
      unpack2(v, lo, hi);
      return pack2(__fdiv_rn(lo, P.T), __fdiv_rn(hi, P.T));
    };
    if (TOPK) {   // the drafter row's top-k threshold, from the staged row (the row came early)
      auto zd = [&](int g, float (&z)[8]) {
        uint64_t d2[4];
        pairs_of(rd, g, d2);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint64_t l2 = d2[i];
          if (!T_is_one) l2 = divide_T(l2);
          unpack2(l2, z[2 * i], z[2 * i + 1]);
        }
      };
      tp = tkg_kth_largest(zd, cur.bracket[0], P.top_k, V, CH, S.tk, 0, grp, gt, &P.counters->n_slow_topk);
    }
    // --- drafter first (its row came early): slice maximum and partial sum of numerators ---
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      float mp = ninf;
#pragma unroll
      for (int c = 0; c < CP; ++c) {
        const int g = (p * CP + c) * GT + gt;
        if (g * 8 < V) {
          uint64_t d2[4];
          pairs_of(rd, g, d2);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint64_t l2 = d2[i];
            if (!T_is_one) l2 = divide_T(l2);
            float lo, hi;
            unpack2(l2, lo, hi);
            if (TOPK) {   // below the row's top-k threshold: -inf
              lo = lo < tp ? ninf : lo, hi = hi < tp ? ninf : hi;
              l2 = pack2(lo, hi);
            }
            a2[c * 4 + i] = l2;
            mp = max3(mp, lo, hi);
          }
        } else {
#pragma unroll
          for (int i = 0; i < 4; ++i) a2[c * 4 + i] = pack2(ninf, ninf);
        }
      }
      mp = fmaxf(mp, -1.0e37f);
      const float mlp_w = mp * L_hi;
      mlp_mine[p] = mlp_w;
      const uint64_t nml2 = pack2(-mlp_w, -mlp_w);
      uint64_t t2 = pack2(0.0f, 0.0f);
#pragma unroll
      for (int c = 0; c < CP; ++c) {
        uint64_t e2[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float lo, hi;
          unpack2(fma2(a2[c * 4 + i], L2, nml2), lo, hi);
          e2[i] = pack2(ex2_approx(lo), ex2_approx(hi));
        }
        t2 = add2(t2, add2(add2(e2[0], e2[1]), add2(e2[2], e2[3])));
      }
      float tlo, thi;
      unpack2(t2, tlo, thi);
      tp_mine[p] = tlo + thi;
    }

    // The drafter slot is not read again for this context (a rejection fetches the drafter logits from
    // global memory): hand it back, so that the next context's drafter row is copied while this one is decided.
    __syncwarp();
    if (lane == 0) mbar_arrive(&bar_empty_d[grp]);
    // The target rows were issued when the previous context was released; they arrive while the drafter
    // row is streamed.  Every thread waits for itself (bounded); a wait that runs out is reported after
    // the next group barrier, where every thread sees it alike.
    if (!mbar_wait(&bar_full_t[grp], iter & 1, tries)) S.fail = 1;
    if (TOPK) {   // the target row's threshold, on the guided (and tempered) logits the streaming loop forms
      const uint64_t s2 = pack2(P.cfg_scale, P.cfg_scale);
      auto zt = [&](int g, float (&z)[8]) {
        uint64_t c2[4], u2[4];
        pairs_of(rc, g, c2);
        if (UNC) pairs_of(ru, g, u2);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          uint64_t l2 = c2[i];
          if (UNC) l2 = fma2(s2, sub2(c2[i], u2[i]), u2[i]);
          if (!T_is_one) l2 = divide_T(l2);
          unpack2(l2, z[2 * i], z[2 * i + 1]);
        }
      };
      tq = tkg_kth_largest(zt, cur.bracket[1], P.top_k, V, CH, S.tk, 1, grp, gt, &P.counters->n_slow_topk);
    }
    // --- target: guidance combine, slice maximum, numerators, partial sum; E replaces the raw rows ---
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      const uint64_t s2 = pack2(P.cfg_scale, P.cfg_scale);
      float mq = ninf;
#pragma unroll
      for (int c = 0; c < CP; ++c) {
        const int g = (p * CP + c) * GT + gt;
        if (g * 8 < V) {
          uint64_t c2[4], u2[4];
          pairs_of(rc, g, c2);
          if (UNC) pairs_of(ru, g, u2);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            uint64_t l2 = c2[i];
            if (UNC) l2 = fma2(s2, sub2(c2[i], u2[i]), u2[i]);   // l_u + s (l_c - l_u)
            if (!T_is_one) l2 = divide_T(l2);
            if (TOPK) {   // below the row's top-k threshold: -inf (a NaN stays, to be reported)
              float lo, hi;
              unpack2(l2, lo, hi);
              l2 = pack2(lo < tq ? ninf : lo, hi < tq ? ninf : hi);
            }
            a2[c * 4 + i] = l2;
            float lo, hi;
            unpack2(l2, lo, hi);
            mq = max3(mq, lo, hi);
          }
        } else {
#pragma unroll
          for (int i = 0; i < 4; ++i) a2[c * 4 + i] = pack2(ninf, ninf);
        }
      }
      // a slice without any finite logit (padding, masked tokens) still needs a finite shift
      mq = fmaxf(mq, -1.0e37f);
      const float mlq_w = mq * L_hi;
      mlq_mine[p] = mlq_w;
      const uint64_t nml2 = pack2(-mlq_w, -mlq_w);
      uint64_t t2 = pack2(0.0f, 0.0f);
#pragma unroll
      for (int c = 0; c < CP; ++c) {
        float e[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float lo, hi;
          unpack2(fma2(a2[c * 4 + i], L2, nml2), lo, hi);
          e[2 * i] = ex2_approx(lo);
          e[2 * i + 1] = ex2_approx(hi);
        }
        t2 = add2(t2, add2(add2(pack2(e[0], e[1]), pack2(e[2], e[3])), add2(pack2(e[4], e[5]), pack2(e[6], e[7]))));
        const int g = (p * CP + c) * GT + gt;
        if (g * 8 < V) {
          *reinterpret_cast<float4*>(E + EI(g * 8)) = make_float4(e[0], e[1], e[2], e[3]);
          *reinterpret_cast<float4*>(E + EI(g * 8 + 4)) = make_float4(e[4], e[5], e[6], e[7]);
        }
      }
      float tlo, thi;
      unpack2(t2, tlo, thi);
      tq_mine[p] = tlo + thi;
    }
    // ---------------- group statistics ----------------
    // common maxima first (one warp reduction, then eight values read by everybody), then the slices'
    // factors and the normalisers
    float mlq_g, mlp_g;
    {
      float mq_t = mlq_mine[0], mp_t = mlp_mine[0];
#pragma unroll
      for (int p = 1; p < NP; ++p) {
        mq_t = fmaxf(mq_t, mlq_mine[p]);
        mp_t = fmaxf(mp_t, mlp_mine[p]);
      }
      mq_t = warp_max(mq_t);
      mp_t = warp_max(mp_t);
      if (lane == 0) {
        S.wmq[gw] = mq_t;
        S.wmp[gw] = mp_t;
      }
    }
    gbar(grp);   // [stats 1] per-warp maxima, and E, are visible
    if (S.fail) {   // the target rows did not land within the limit
      give_up(iter, false);
      break;
    }
    mlq_g = S.wmq[0];
    mlp_g = S.wmp[0];
#pragma unroll
    for (int w = 1; w < GW; ++w) {
      mlq_g = fmaxf(mlq_g, S.wmq[w]);
      mlp_g = fmaxf(mlp_g, S.wmp[w]);
    }
    float fq_mine[NP], fp_mine[NP];
    double Zq = 0.0, Zp = 0.0;
#pragma unroll
    for (int p = 0; p < NP; ++p) {
      fq_mine[p] = ex2_approx(mlq_mine[p] - mlq_g);
      fp_mine[p] = ex2_approx(mlp_mine[p] - mlp_g);
      S.fqt[p * GT + gt] = fq_mine[p];
      Zq += static_cast<double>(fq_mine[p]) * static_cast<double>(tq_mine[p]);
      Zp += static_cast<double>(fp_mine[p]) * static_cast<double>(tp_mine[p]);
    }
    Zq = warp_sum(Zq);
    Zp = warp_sum(Zp);
    if (lane == 0) {
      S.wzq[gw] = Zq;
      S.wzp[gw] = Zp;
    }
    gbar(grp);   // [stats 2] factor table and per-warp sums are visible
    Zq = 0.0;
    Zp = 0.0;
#pragma unroll
    for (int w = 0; w < GW; ++w) {
      Zq += S.wzq[w];
      Zp += S.wzp[w];
    }

    int status = 0;              // bits every thread sets alike
    int accepted = -1;
    bool record_written = false;
    if (!(Zq > 0.0 && Zq < 1e300 && Zp > 0.0 && Zp < 1e300)) {
      status |= LANTERN_ST_NONFINITE;
    } else {
      // current normalisers: q'(x) = E(x) * fq[slice of x] / Zq_c,  p'(x) = ep(x) * fp[slice of x] / Zp_c
      // (Zp_c = 0 stands for a drafter distribution that has no mass left).  Comparisons are written on
      // the unnormalised sums, so that no thread divides on the way to a decision.
      double Zq_c = Zq, Zp_c = Zp;
      const double delta = static_cast<double>(P.delta);
      if (gt == 0) {   // the two single probabilities of the first child, in double precision
        float zq = raw_c;
        if (UNC) zq = __fmaf_rn(P.cfg_scale, __fsub_rn(raw_c, raw_u), raw_u);
        float zp = raw_d;
        if (!T_is_one) {
          zq = __fdiv_rn(zq, P.T);
          zp = __fdiv_rn(zp, P.T);
        }
        if (TOPK) {   // these come from global memory, unfiltered
          zq = zq < tq ? ninf : zq;
          zp = zp < tp ? ninf : zp;
        }
        S.acc_e = exp2_single(zq, mlq_g);
        S.acc_p = exp2_single(zp, mlp_g);
        S.acc_valid = 1;
      }

      for (int ci = 0; ci < nchild; ++ci) {
        if (gt == 0) atomicAdd(&P.counters->n_tested, 1);   // work accounting (a fire-and-forget reduction)
        const int32_t* nrow = P.nbr + static_cast<size_t>(xt) * k;
        // the next sibling's description, wanted only after a rejection: in flight meanwhile
        ChildInfo sib = {0, 0, 0.0f, 0};
        if (ci + 1 < nchild) {
          const int4 v = __ldg(reinterpret_cast<const int4*>(kids + ci + 1));
          sib.node = v.x, sib.token = v.y, sib.r = __int_as_float(v.z);
        }
        // bulk numerators of x~ itself, common units (drafter: from its raw logit; no mass is left once x~
        // was rejected as an earlier sibling of this context, or where the top-k filter cut it)
        float px_bulk, e_xt_bulk;
        {
          float dz = raw_d;
          if (!T_is_one) dz = __fdiv_rn(dz, P.T);
          if (TOPK) dz = dz < tp ? ninf : dz;
          for (int j = 0; j < ci; ++j)
            if (__ldg(&kids[j].token) == xt) dz = ninf;
          px_bulk = ex2_approx(__fmaf_rn(dz, L_hi, -mlp_g));
          e_xt_bulk = E[EI(xt)] * S.fqt[owner_slice<LOG_CP>(xt)];
        }

        // ---- A_{k,delta}(x~): gather + prefix scan with the strict bound ----
        double thr = delta * Zq_c;   // the bound in the units of the unnormalised sums
        // Section 5.3.2: the mass whose JSD is delta; the group's last warp finds it together, published by
        // [scan 1] through the last slot of wt[], which nothing else touches between the start of a child and
        // its [scan 2]
        if (JSD && gw == GW - 1) {
          const double sstar = jsd_mass_bound_warp(delta, static_cast<double>(e_xt_bulk) / Zq_c, lane) * Zq_c;
          if (lane == 0) S.wt[8 * GW - 1] = sstar;
        }
        double carry = 0.0, sm = 0.0;
        int m = k - 1;
        bool cut = false;
        for (int base = 0; base < k - 1 && !cut; base += 4 * GT) {
          double pre4[4];       // inclusive prefix over this thread's four slots
          bool val4[4];
          double run = 0.0;
          int my_bad = kNone;   // first of this thread's slots whose entry lies outside [0, V): it carries no mass
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int j = base + 4 * gt + 1 + i;
            val4[i] = j < k;
            const int n = base == 0 ? nb[i] : (val4[i] ? __ldg(nrow + j) : -1);
            const bool inr = val4[i] && static_cast<unsigned>(n) < static_cast<unsigned>(V);
            if (val4[i] && !inr && my_bad == kNone) my_bad = j;
            run += inr ? static_cast<double>(E[EI(n)] * S.fqt[owner_slice<LOG_CP>(n)]) : 0.0;
            pre4[i] = run;
          }
          const double incl = warp_incl_scan(run, lane);
          if (lane == 31) S.wt[gw] = incl;
          gbar(grp);   // [scan 1]
          if (JSD && base == 0) thr = S.wt[8 * GW - 1];
          double pre = 0.0, tot = 0.0;
#pragma unroll
          for (int w = 0; w < GW; ++w) {
            const double t = S.wt[w];
            if (w < gw) pre += t;
            tot += t;
          }
          const double before = carry + pre + (incl - run);   // prefix before this thread's first slot
          int my_first = kNone;
          double my_before = 0.0;
#pragma unroll
          for (int i = 3; i >= 0; --i) {
            const double Sj = before + pre4[i];
            if (val4[i] && !(Sj < thr)) {
              my_first = base + 4 * gt + 1 + i;
              my_before = i > 0 ? before + pre4[i > 0 ? i - 1 : 0] : before;
            }
          }
          const int wfirst = __reduce_min_sync(kFull, my_first);
          if (wfirst != kNone && my_first == wfirst) {
            S.first[gw] = wfirst;
            S.sbefore[gw] = my_before;
          } else if (wfirst == kNone && lane == 0) {
            S.first[gw] = kNone;
          }
          const int wbad = __reduce_min_sync(kFull, my_bad);
          if (lane == 0) S.badslot[gw] = wbad;
          gbar(grp);   // [scan 2]
          int gfirst = kNone, src = 0, gbad = kNone;
#pragma unroll
          for (int w = GW - 1; w >= 0; --w) {
            const int f = S.first[w];
            if (f != kNone && f <= gfirst) {
              gfirst = f;
              src = w;
            }
            gbad = min(gbad, S.badslot[w]);
          }
          // a bad entry is reported where Algorithm 2's loop meets it, i.e. ahead of the slot that ends the set
          if (gbad < gfirst) status |= LANTERN_ST_BAD_TABLE;
          if (gfirst != kNone) {
            m = gfirst - 1;
            sm = S.sbefore[src];
            cut = true;
          } else {
            carry += tot;
            sm = carry;
          }
        }
        if (k == 1) gbar(grp);   // publish S.acc_* when the scan loop did not run
        // the two single probabilities: thread 0's double-precision values where it has them; a bulk
        // value of exactly zero (token inside an earlier A, or rejected before) stays zero
        const bool acc = S.acc_valid != 0;
        const double e_xt = (acc && e_xt_bulk != 0.0f) ? S.acc_e : static_cast<double>(e_xt_bulk);
        const double p_xt = (acc && px_bulk != 0.0f) ? S.acc_p : static_cast<double>(px_bulk);
        // Section 4.3: accept iff r p(x~) < sum_A q, i.e. r p_xt / Zp_c < (e_xt + sm) / Zq_c, both sides times Zq_c Zp_c
        const double qa_un = e_xt + sm;
        const bool accept = Zp_c > 0.0 ? static_cast<double>(r) * p_xt * Zq_c < qa_un * Zp_c : 0.0 < qa_un;
        if (gt == 0 && (P.out_qa || P.out_px || P.out_m)) {
          const size_t o = static_cast<size_t>(b) * N + node;
          if (P.out_qa) P.out_qa[o] = static_cast<float>(qa_un / Zq_c);
          if (P.out_px) P.out_px[o] = Zp_c > 0.0 ? static_cast<float>(p_xt / Zp_c) : 0.0f;
          if (P.out_m) P.out_m[o] = m;
        }
        if (accept) {
          accepted = node;
          break;
        }
        // ---- rejected: residual [q_{k,delta}(.|D = x~) - p]_+ ----
        // the drafter logits of the first pass: asked for at once, in flight while A is flagged and across the barrier
        const unsigned char* drow = static_cast<const unsigned char*>(P.draft) + static_cast<size_t>(item) * rowbytes;
        DraftRaw dnext[CP];
#pragma unroll
        for (int c = 0; c < CP; ++c) {
          const int g = c * GT + gt;
          dnext[c] = draft_fetch(drow, g * 8 < V ? g : gt);
        }
        // members of A (x~ included) leave no residual mass: flag them with a negative sign
        for (int base = 0; base < m; base += 4 * GT) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int j = base + 4 * gt + 1 + i;
            if (j <= m) {
              const int n = base == 0 ? nb[i] : __ldg(nrow + j);
              if (static_cast<unsigned>(n) < static_cast<unsigned>(V)) E[EI(n)] = -fabsf(E[EI(n)]);
            }
          }
        }
        if (gt == 0) E[EI(xt)] = -fabsf(E[EI(xt)]);
        // x~ leaves the drafter distribution for the following siblings: the residual pass below strikes
        // every token rejected so far (children 0..ci) from the drafter logits it fetches.  Which of this
        // thread's chunks hold one:
        uint32_t struck = 0;
        for (int j = 0; j <= ci; ++j) {
          const int t = j == ci ? xt : __ldg(&kids[j].token);
          if (((t >> 3) & (GT - 1)) == gt) struck |= 1u << (t >> (3 + LOG_GT));
        }
        const bool last = (ci + 1 == nchild);
        if (!last) {   // next sibling's neighbour row, in flight during the residual pass
          node = sib.node;
          xt = sib.token;
          r = sib.r;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int j = 4 * gt + 1 + i;
            nb[i] = (j < k) ? ld_nc_here(P.nbr + static_cast<size_t>(xt) * k + j) : -1;
          }
          raw_d = ctx_raw_logit<BF16>(P.draft, static_cast<size_t>(item) * V + xt);
          if (gt == 0) {   // its raw target logits, for the double-precision replay below
            const size_t e = static_cast<size_t>(item) * V + xt;
            raw_c = ctx_raw_logit<BF16>(P.target, e);
            if (UNC) raw_u = ctx_raw_logit<BF16>(P.target, static_cast<size_t>(P.B) * R * V + e);
          }
        }
        gbar(grp);   // [flags]
        // w = E - (p'/q' scale ratio) * ep in common units, i.e. E - ratio * ep in the slice's own units
        // of E; the residual replaces E (it is the next sibling's target, or what the draw reads)
        const float ratio_g = Zp_c > 0.0 ? static_cast<float>(Zq_c / Zp_c) : 0.0f;
        float cs[CH];
        double wsum = 0.0, psum = 0.0;
#pragma unroll
        for (int p = 0; p < NP; ++p) {
          // (a slice whose numerators are all negligible has factor 0; nothing of it survives anyway)
          const float ratio = fq_mine[p] > 0.0f ? ratio_g * (fp_mine[p] / fq_mine[p]) : 0.0f;
          float wp_ = 0.0f, pp_ = 0.0f;
          DraftRaw dcur[CP];
#pragma unroll
          for (int c = 0; c < CP; ++c) {
            dcur[c] = dnext[c];
            if (p + 1 < NP) {   // the next pass's logits travel during this pass
              const int g = ((p + 1) * CP + c) * GT + gt;
              dnext[c] = draft_fetch(drow, g * 8 < V ? g : gt);
            }
          }
#pragma unroll
          for (int c = 0; c < CP; ++c) {
            const int g = (p * CP + c) * GT + gt;
            float w8[8];
            if (g * 8 < V) {
              const float4 lo = *reinterpret_cast<const float4*>(E + EI(g * 8));
              const float4 hi = *reinterpret_cast<const float4*>(E + EI(g * 8 + 4));
              const float e8[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
              float ep8[8];
              draft_chunk(dcur[c], ep8);
              if (TOPK) {   // below the row's top-k threshold: -inf
#pragma unroll
                for (int e = 0; e < 8; ++e) ep8[e] = ep8[e] < tp ? ninf : ep8[e];
              }
              if ((struck >> (p * CP + c)) & 1u) {   // a token rejected in this context sits in this chunk
                for (int j = 0; j <= ci; ++j) {
                  const int t = __ldg(&kids[j].token);
                  if ((t >> 3) == g) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) ep8[e] = (t & 7) == e ? ninf : ep8[e];
                  }
                }
              }
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                ep8[e] = ex2_approx(__fmaf_rn(ep8[e], L_hi, -mlp_mine[p]));
                w8[e] = fmaxf(0.0f, __fmaf_rn(-ratio, ep8[e], e8[e]));
              }
              pp_ += sum8(ep8);
              *reinterpret_cast<float4*>(E + EI(g * 8)) = make_float4(w8[0], w8[1], w8[2], w8[3]);
              *reinterpret_cast<float4*>(E + EI(g * 8 + 4)) = make_float4(w8[4], w8[5], w8[6], w8[7]);
            } else {
#pragma unroll
              for (int e = 0; e < 8; ++e) w8[e] = 0.0f;
            }
            cs[p * CP + c] = sum8(w8);
            wp_ += cs[p * CP + c];
          }
          wsum += static_cast<double>(wp_) * static_cast<double>(fq_mine[p]);
          psum += static_cast<double>(pp_) * static_cast<double>(fp_mine[p]);
        }
        double W, Sp;
        if (!last) {
          const double ww = warp_sum(wsum);
          const double wp = warp_sum(psum);
          if (lane == 0) {
            S.wt[gw] = ww;
            S.wt[GW + gw] = wp;
          }
          gbar(grp);   // [totals] also publishes the written-back residual
          W = 0.0;
          Sp = 0.0;
#pragma unroll
          for (int w = 0; w < GW; ++w) {
            W += S.wt[w];
            Sp += S.wt[GW + w];
          }
          if (!(W > kDegenerate * Zq_c)) {
            status |= LANTERN_ST_DEGENERATE;
            break;
          }
          if (gt == 0) {
            // The next sibling's own two probabilities in double precision: its numerators from the raw
            // logits, carried through every rejection round so far (E <- max(0, E - ratio_i * ep)); the
            // totals W, Sp are sums of thousands of terms and do not suffer from cancellation.
            if (ci < 32) {
              S.hist[ci] = static_cast<double>(ratio_g);
              float zq = raw_c;
              if (UNC) zq = __fmaf_rn(P.cfg_scale, __fsub_rn(raw_c, raw_u), raw_u);
              float zp = raw_d;
              if (!T_is_one) {
                zq = __fdiv_rn(zq, P.T);
                zp = __fdiv_rn(zp, P.T);
              }
              if (TOPK) {   // these come from global memory, unfiltered
                zq = zq < tq ? ninf : zq;
                zp = zp < tp ? ninf : zp;
              }
              double e = exp2_single(zq, mlq_g);
              const double pe = exp2_single(zp, mlp_g);
              for (int i = 0; i <= ci; ++i) e = fmax(0.0, e - S.hist[i] * pe);
              S.acc_e = e;
              S.acc_p = pe;
              S.acc_valid = 1;
            } else {
              S.acc_valid = 0;
            }
          }
          Zq_c = W;
          Zp_c = Sp > 0.0 ? Sp : 0.0;
          continue;
        }
        // ---- last child rejected: draw the replacement token from the residual (Algorithm 1) ----
        double csd[CH], incl[CH], excl[CH] = {};
#pragma unroll
        for (int c = 0; c < CH; ++c) {
          csd[c] = static_cast<double>(cs[c]) * static_cast<double>(fq_mine[c / CP]);
          incl[c] = warp_incl_scan(csd[c], lane);
          if (lane == 31) S.wt[c * GW + gw] = incl[c];
        }
        gbar(grp);   // [draw 1]
        {
          // exclusive prefix over (chunk, warp) in chunk-major order; 32 entries per round
          double carry2 = 0.0;
#pragma unroll
          for (int half = 0; half < (CH * GW + 31) / 32; ++half) {
            const int e = half * 32 + lane;
            const double t = e < CH * GW ? S.wt[e] : 0.0;
            const double in = warp_incl_scan(t, lane);
            const double ex = carry2 + in - t;
#pragma unroll
            for (int c = 0; c < CH; ++c) {
              const int want = c * GW + gw;
              const double got = __shfl_sync(kFull, ex, want & 31);
              if ((want >> 5) == half) excl[c] = got + incl[c] - csd[c];
            }
            carry2 += __shfl_sync(kFull, in, 31);
          }
          W = carry2;
        }
        if (!(W > kDegenerate * Zq_c)) {
          status |= LANTERN_ST_DEGENERATE;
          break;
        }
        const double target = static_cast<double>(cur.u_final) * W;
        int cand = kNone;
#pragma unroll
        for (int c = CH - 1; c >= 0; --c)
          if (excl[c] + csd[c] > target) cand = c * GT + gt;
        const int wmin = __reduce_min_sync(kFull, cand);
        if (lane == 0) S.cand[gw] = wmin;
        if (gt == 0) S.tok = -1;
        gbar(grp);   // [draw 2]
        const int win = __reduce_min_sync(kFull, lane < GW ? S.cand[lane] : kNone);
        if (win == kNone) {
          // rounding left no slot above the target: the largest token of positive weight
          int lastp = -1;
          for (int c = 0; c < CH; ++c) {
            const int g = c * GT + gt;
            if (g * 8 < V && cs[c] > 0.0f)
              for (int e = 0; e < 8; ++e)
                if (E[EI(g * 8 + e)] > 0.0f) lastp = g * 8 + e;
          }
          if (lastp >= 0) atomicMax(&S.tok, lastp);
          gbar(grp);
          if (gt == 0) {
            Record rec = {-1, S.tok, status | (S.tok < 0 ? LANTERN_ST_DEGENERATE : 0), 0};
            P.records[item] = rec;
          }
        } else if ((win & (GT - 1)) == gt) {
          const int wc = win >> LOG_GT;
          const int g = wc * GT + gt;
          double ex_c = 0.0, fqd = 0.0;
#pragma unroll
          for (int c = 0; c < CH; ++c)
            if (c == wc) {
              ex_c = excl[c];
              fqd = static_cast<double>(fq_mine[c / CP]);
            }
          int tok = -1, lastpos = -1;
          double cum = ex_c;
          for (int e = 0; e < 8; ++e) {
            const float wv = E[EI(g * 8 + e)];
            cum += static_cast<double>(wv) * fqd;
            if (wv > 0.0f) lastpos = e;
            if (tok < 0 && cum > target) tok = e;
          }
          if (tok < 0) tok = lastpos;
          Record rec = {-1, g * 8 + tok, status, 0};
          P.records[item] = rec;
        }
        record_written = true;
      }
    }
    if (!record_written && gt == 0) {
      Record rec = {accepted, -1, status, 0};
      P.records[item] = rec;
    }
    // Algorithm 1 goes on from the accepted child only: every context behind another child is dead.  In
    // pre-order those are one contiguous range per child.
    for (int j = 0; j < nchild; ++j) {
      int node_j = cur.node0, span_j = cur.span0;
      if (j > 0) {
        const int4 kid = __ldg(reinterpret_cast<const int4*>(kids + j));
        node_j = kid.x, span_j = kid.w;
      }
      if (node_j != accepted) {
        unsigned char* first = P.dead + static_cast<size_t>(b) * R + (span_j >> 16);
        for (int o = gt; o < (span_j & 0xffff); o += GT) first[o] = 1;
      }
    }
    // this context's staging area (rows and E) is no longer needed by this warp
    __syncwarp();
    if (lane == 0) mbar_arrive(&bar_empty_t[grp]);
  }
}

}  // namespace lantern
