// Shared by every translation unit of the verification step: workspace structures, kernel
// parameters, and the entry through which the host reaches the fused context kernel's
// compile-time variants.
#pragma once

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "lantern.h"
#include "lantern_device.cuh"

namespace lantern {

constexpr int MAX_N = 1024;

struct Counters {               // first 256 bytes of the workspace, zeroed per call
  int work_next;                // dynamic part of the work counter
  int n_heavy;                  // contexts with >= 2 children (first in the compact list)
  int n_light;                  // contexts with exactly 1 child
  int n_bonus;                  // sequences whose next token is drawn from a context's own target
  int n_rank;                   // largest number of contexts with children in one sequence
  int n_evaluated;              // contexts the fused pass evaluated
  int n_skipped;                // contexts it left out because the walk cannot reach them
  int n_tested;                 // drafted nodes it tested
  int status_or;                // OR of every sequence's status bits (written by the walk and later kernels)
  int abort;                    // a bounded wait ran out somewhere: no further work is handed out
  int n_slow_topk;              // rows whose top-k threshold needed the slow exact search
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
  int span;                     // the contexts behind the node, in pre-order: (first position << 16) | count
};

struct WorkItem {               // one context with children: everything its CTA needs, in one 32-byte load
  int item;                     // b * R + c  (row index of the context); -1 = none
  int cbase;                    // index of its first child in the ChildInfo array
  int nchild_node0;             // (number of children << 16) | first child's node index
  int span0;                    // first child's ChildInfo::span
  int tok0;                     // first child's token and uniform, inlined
  float r0;
  float u_final;                // the sequence's uniform for the final draw
  int mark;                     // index of the context's own entry in the array of dead marks
};

struct GroupItem {              // the same, as a producer hands it to its consumer group through shared memory
  int item, cbase, nchild, node0, tok0, span0;
  float r0, u_final;
  float bracket[2][4];          // top-k filter only: where the thresholds of the drafter row [0] and the target row [1] lie
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
  WorkItem* work;               // [N, B]: slot r * B + b holds the r-th context with children of sequence b in
                                //         breadth-first order (by depth, then by index); item = -1 where there is none
  int32_t* ctx_slots;           // [B*N]: the occupied slots, heavy ones from the front, light ones from the back
  unsigned char* dead;          // [B, R], a sequence's contexts in pre-order: 1 once the walk is known not to reach one
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
  uint32_t wait_tries;          // limit of every bounded mbarrier wait, in tries
  int withhold_item;            // self-test only: the copies of this context are never issued (-1 = none)
};

__device__ __forceinline__ float sum8(const float* v) {
  return ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
}


// Launch of the fused context kernel (verify_context.cuh).  Its variants -- temperature 1 compiled
// out or not (TONE), TVD or JSD bound, top-k thresholds applied or not -- are compiled in separate
// translation units (verify_context_v*.cu) so that they build in parallel; this function picks one.
cudaError_t launch_context_kernel(const VerifyParams& P, int CH, bool bf16, bool uncond, bool tone, bool jsd, bool topk,
                                  int grid, size_t smem_bytes, cudaStream_t st);

}  // namespace lantern
