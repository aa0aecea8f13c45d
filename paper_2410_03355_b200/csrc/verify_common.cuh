// Shared by every translation unit of the verification step: workspace structures, kernel
// parameters, block-level reductions / scans / draws of the 1024-thread kernels, and the entry
// through which the host reaches the fused context kernel's compile-time variants.
#pragma once

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "lantern.h"
#include "lantern_device.cuh"

namespace lantern {

constexpr int NT = 1024;        // threads per CTA of the context / bonus kernels
constexpr int NW = NT / 32;
constexpr int LOG_NT = 10;
constexpr int MAX_N = 1024;

struct Counters {               // first 256 bytes of the workspace, zeroed per call
  int work_next;                // dynamic part of the work counter
  int n_heavy;                  // contexts with >= 2 children (handed out first)
  int n_light;                  // contexts with exactly 1 child
  int n_bonus;                  // sequences whose walk ended on a childless context
};

struct Record {                 // result of one context
  int accepted;                 // accepted child node; -1 if every child was rejected; kLeaf if it has none
  int token;                    // replacement token if every child was rejected
  int status;                   // LANTERN_ST_* bits found in this context
  int pad;
};
constexpr int kLeaf = -2;

struct ChildInfo {              // one drafted node, stored in the order its parent context tries it
  int node;                     // node index within the sequence
  int token;                    // x~
  float r;                      // its acceptance uniform
  int pad;
};

struct WorkItem {               // one context with children: everything its CTA needs, in one 32-byte load
  int item;                     // b * R + c  (row index of the context); -1 = none
  int cbase;                    // index of its first child in the ChildInfo array
  int nchild;
  int node0;                    // first child, inlined
  int tok0;
  float r0;
  float u_final;                // the sequence's uniform for the final draw
  int pad;
};

struct VerifyParams {
  const void* target;
  const void* draft;
  const int32_t* tokens;
  const int32_t* parents;
  const int32_t* nbr;
  const float* uniforms;
  int32_t* out_len;
  int32_t* out_tok;
  int32_t* out_path;
  int32_t* out_status;
  float* out_qa;
  float* out_px;
  int32_t* out_m;
  // workspace pieces
  Counters* counters;
  WorkItem* work;               // [B*N]: heavy items from the front, light items from the back
  ChildInfo* children;          // [B, N]
  Record* records;              // [B, R]
  int32_t* seq_status;          // [B]
  int32_t* bonus_seq;           // [B]
  int32_t* bonus_ctx;           // [B]
  int B, N, R, V, k;
  float cfg_scale, T, delta;
  int divergence;               // LANTERN_DIV_TVD or LANTERN_DIV_JSD: what delta bounds
  int top_k;                    // logit filter; 0 = off (then thr_q, thr_p are null)
  float* thr_q;                 // [B, R] top_k-th largest processed target logit of a context row
  float* thr_p;                 // [B, R] the same for the drafter row
};

// ---------------------------------------------------------------------------------------
// layout of a row held by a CTA: thread t owns, for chunk c, the eight consecutive tokens
// [(c*NT + t)*8, +8).  In shared memory the numerators E are stored so that both 16-byte
// halves of a thread's chunk are bank-conflict free: physical float index of token x below.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ int phys(int x) {
  const int g = x >> 3;
  const int c = g >> LOG_NT;
  const int t = g & (NT - 1);
  const int h = (x >> 2) & 1;
  return ((((c << 1) | h) << LOG_NT) + t) << 2 | (x & 3);
}

struct BlockScratch {
  double wt[2 * NW];            // per-(chunk, warp) totals
  double wbase[2 * NW];         // their exclusive prefix
  double sp[NW];
  double total;
  double total2;
  double sm;
  float fm[2 * NW];
  float px;
  int first;
  int win;
  int tok;
  int item;
  int bad;
};

// max of two values over the block
__device__ __forceinline__ void block_max2(float& a, float& b, BlockScratch& S, int lane, int warp) {
  a = warp_max(a);
  b = warp_max(b);
  if (lane == 0) {
    S.fm[warp] = a;
    S.fm[NW + warp] = b;
  }
  __syncthreads();
  a = warp_max(S.fm[lane]);
  b = warp_max(S.fm[NW + lane]);
  __syncthreads();
}

// sum of two doubles over the block
__device__ __forceinline__ void block_sum2(double& a, double& b, BlockScratch& S, int lane, int warp) {
  a = warp_sum(a);
  b = warp_sum(b);
  if (lane == 0) {
    S.wt[warp] = a;
    S.wt[NW + warp] = b;
  }
  __syncthreads();
  a = warp_sum(S.wt[lane]);
  b = warp_sum(S.wt[NW + lane]);
  __syncthreads();
}

__device__ __forceinline__ float sum8(const float* v) {
  return ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
}

// Exclusive prefix (over the order chunk-major, then thread) of per-chunk sums cs[c], the
// grand total in S.total, and the block sum of `extra` in S.total2.
template <int CH>
__device__ __forceinline__ void block_scan_chunks(const double (&cs)[CH], double (&excl)[CH], double extra,
                                                  BlockScratch& S, int lane, int warp) {
  double incl[CH];
#pragma unroll
  for (int c = 0; c < CH; ++c) {
    incl[c] = warp_incl_scan(cs[c], lane);
    if (lane == 31) S.wt[c * NW + warp] = incl[c];
  }
  extra = warp_sum(extra);
  if (lane == 0) S.sp[warp] = extra;
  __syncthreads();
  if (warp == 0) {
    double carry = 0.0;
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      const double t = S.wt[c * NW + lane];
      const double in = warp_incl_scan(t, lane);
      S.wbase[c * NW + lane] = carry + in - t;
      carry += __shfl_sync(kFull, in, 31);
    }
    const double e = warp_sum(S.sp[lane]);
    if (lane == 0) {
      S.total = carry;
      S.total2 = e;
    }
  }
  __syncthreads();
#pragma unroll
  for (int c = 0; c < CH; ++c) excl[c] = S.wbase[c * NW + warp] + incl[c] - cs[c];
}

// Inverse CDF over the weights w (registers, layout above): smallest token whose inclusive
// cumulative weight exceeds target; if rounding leaves none, the largest token of positive
// weight; -1 if there is no positive weight.  Must be called by the whole block.
template <int CH>
__device__ __forceinline__ int block_draw(const float (&w)[CH * 8], const double (&cs)[CH], const double (&excl)[CH],
                                          double target, int V, BlockScratch& S, int tid) {
  if (tid == 0) {
    S.win = 0x7fffffff;
    S.tok = -1;
  }
  __syncthreads();
  int cand = 0x7fffffff;
#pragma unroll
  for (int c = CH - 1; c >= 0; --c)
    if (excl[c] + cs[c] > target) cand = c * NT + tid;
  const int wmin = __reduce_min_sync(kFull, cand);
  if ((tid & 31) == 0 && wmin != 0x7fffffff) atomicMin(&S.win, wmin);
  __syncthreads();
  const int win = S.win;
  if (win == 0x7fffffff) {
    int last = -1;
#pragma unroll
    for (int c = 0; c < CH; ++c)
#pragma unroll
      for (int e = 0; e < 8; ++e)
        if (w[c * 8 + e] > 0.0f) last = (c * NT + tid) * 8 + e;
    if (last >= V) last = -1;
    if (last >= 0) atomicMax(&S.tok, last);
  } else if ((win & (NT - 1)) == tid) {
    const int wc = win >> LOG_NT;
    int tok = -1, lastpos = -1;
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      if (c == wc) {
        double cum = excl[c];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float wv = w[c * 8 + e];
          cum += static_cast<double>(wv);
          if (wv > 0.0f) lastpos = e;
          if (tok < 0 && cum > target) tok = e;
        }
      }
    }
    if (tok < 0) tok = lastpos;
    S.tok = win * 8 + tok;
  }
  __syncthreads();
  return S.tok;
}

// Launch of the fused context kernel (verify_context.cuh).  Its variants -- temperature 1 compiled
// out or not (TONE), TVD or JSD bound, top-k thresholds applied or not -- are compiled in separate
// translation units (verify_context_v*.cu) so that they build in parallel; this function picks one.
cudaError_t launch_context_kernel(const VerifyParams& P, int CH, bool bf16, bool uncond, bool tone, bool jsd, bool topk,
                                  int grid, size_t smem_bytes, cudaStream_t st);

}  // namespace lantern
