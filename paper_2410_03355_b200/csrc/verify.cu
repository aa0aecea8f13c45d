// LANTERN relaxed verification step on sm_100a: plan -> fused context pass -> walk -> bonus.
//
// One "context" is a row of logits that has at least one drafted child.  The fused pass is
// a persistent kernel, one CTA per SM: a bulk asynchronous copy (TMA, completion on an
// mbarrier) brings the context's two target rows and its drafter row into shared memory
// while the CTA is still working on the previous context; the rows are then read ONCE into
// registers, guidance-combined, turned into softmax numerators, and every child of the
// context is tested on chip:
//     A_{k,delta}(x~)  : gather of the target numerators at the token's neighbour row and a
//                        block-wide prefix scan with the strict bound (Algorithm 2, 2nd block)
//     accept test      : r * p(x~) < sum_A q                     (Section 4.3, final rule)
//     on rejection     : residual [q_{k,delta}(.|D=x~) - p]_+ over all V tokens, its total,
//                        and either the next sibling's test on the renormalised residual or
//                        the inverse-CDF draw of the replacement token   (Section 4.3, Alg. 1)
// Each context leaves a 16-byte record; a tiny walk kernel follows the records from the root
// (Algorithm 1's loop), and a last kernel draws the bonus token where the walk ended on a
// context without children (Algorithm 1, line after the loop).
//
// Precision: processed logits are fp32 (difference, fused multiply-add, division, each
// rounded once); exponentials come from the fp32 ex2 unit (about 3e-7 relative); every sum over more
// than eight terms and every threshold comparison is done in double precision.
#include "verify_common.cuh"

#include <stddef.h>

namespace lantern {

// ---------------------------------------------------------------------------------------
// kernel 1: plan.  One warp per sequence: validate tokens / parents / uniforms, bucket the
// nodes by parent context (children in node order), initialise the per-node outputs, and write
// one self-contained work item per context with children.
//
// Work items are laid out so that the fused pass meets a sequence's contexts in the order
// Algorithm 1's loop can reach them: slot r * B + b holds the r-th context with children of
// sequence b in breadth-first order (by depth, then by index).  A context whose parent node has
// already been rejected when its turn comes is never evaluated (see verify_context.cuh); the
// order only decides how often that is known in time, never the result.
// Every context with children starts with a record that says "not evaluated" (INTERNAL), which
// the fused pass overwrites; contexts without children are marked as leaves.
// ---------------------------------------------------------------------------------------
constexpr int PLAN_WARPS = 4;
constexpr int kPlanArrays = 13;  // per-warp arrays of N + 2 ints in shared memory

__global__ void __launch_bounds__(PLAN_WARPS * 32) lantern_plan_kernel(VerifyParams P) {
  extern __shared__ int plan_smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.x * PLAN_WARPS + warp;
  if (b >= P.B) return;
  const int N = P.N, R = P.R, B = P.B;
  int* cnt = plan_smem + warp * kPlanArrays * (R + 1);   // cnt[c]: number of children of context c
  int* cur = cnt + (R + 1);                    // fill cursor, ends as the end offset of context c
  int* dep = cur + (R + 1);                    // depth of context c (root = 0), later its breadth-first rank
  int* lvl = dep + (R + 1);                    // per depth: where its nodes lie in the (depth, index) order
  int* siz = lvl + (R + 1);                    // number of contexts in the subtree of context c, itself included
  int* din = siz + (R + 1);                    // depth-first (pre-order) position of context c
  int* tmp = din + (R + 1);                    // per context: children placed so far; later running sums of sizes
  int* anc = tmp + (R + 1);                    // pointer jumping: an ancestor of node i; later the (depth, index) order
  int* s_par = anc + (R + 1);                  // the sequence's parents, tokens and uniforms, staged once by all
  int* s_tok = s_par + (R + 1);                //   lanes: the serial parts below then run out of shared memory
  int* s_uni = s_tok + (R + 1);
  int* s_pos = s_uni + (R + 1);                // place of node i in the child lists
  int* s_first = s_pos + (R + 1);              // first child (smallest node index) of context c
  for (int i = lane; i <= R; i += 32) cnt[i] = 0, siz[i] = 1, s_first[i] = -1;
  __syncwarp();
  int status = 0;
  const float qnan = __int_as_float(0x7fc00000);
  for (int i = lane; i < N; i += 32) {
    const size_t o = static_cast<size_t>(b) * N + i;
    const int tok = P.tokens[o];
    if (static_cast<unsigned>(tok) >= static_cast<unsigned>(P.V)) status |= LANTERN_ST_BAD_TOKEN;
    const int par = P.parents ? P.parents[o] : i - 1;
    if (par < -1 || par >= i) status |= LANTERN_ST_BAD_PARENT;
    else atomicAdd(&cnt[par + 1], 1);
    s_par[i] = par;
    s_tok[i] = tok;
    if (P.out_path) P.out_path[o] = -1;
    if (P.out_qa) P.out_qa[o] = qnan;
    if (P.out_px) P.out_px[o] = qnan;
    if (P.out_m) P.out_m[o] = -1;
  }
  if (P.uniforms) {   // greedy decoding draws nothing and passes no uniforms
    for (int i = lane; i <= N; i += 32) {
      const float r = P.uniforms[static_cast<size_t>(b) * R + i];
      if (!(r >= 0.0f && r < 1.0f)) status |= LANTERN_ST_BAD_UNIFORM;
      s_uni[i] = __float_as_int(r);
    }
  } else {
    for (int i = lane; i <= N; i += 32) s_uni[i] = 0;
  }
  for (int c = lane; c < R; c += 32) P.dead[static_cast<size_t>(b) * R + c] = 0;
  status = __reduce_or_sync(kFull, status);
  __syncwarp();
  if (lane == 0) P.seq_status[b] = status;
  if (status) {   // the walk reports the fault; no work is queued for this sequence
    for (int r = lane; r < N; r += 32) P.work[static_cast<size_t>(r) * B + b].item = -1;
    return;
  }

  ChildInfo* kids = P.children + static_cast<size_t>(b) * N;
  // Children of each context in node order (cur, s_pos, s_first), subtree sizes and pre-order positions
  // (siz, din: the contexts behind a node then occupy one contiguous range of positions, which is what lets
  // the fused pass strike a whole rejected subtree with a few byte stores), and the breadth-first rank of every
  // context with children (dep).  All of it by the whole warp, 32 nodes at a time.
  int n_ctx = 0;
  const unsigned below = (1u << lane) - 1u;
  if (!P.parents) {
    // a chain: context c has the one child c, lies c deep, and has the R - c contexts from itself on behind it
    for (int c = lane; c < R; c += 32) {
      cur[c] = c < N ? c + 1 : N;
      siz[c] = R - c;
      din[c] = c;
      dep[c] = c;
      if (c < N) s_pos[c] = c, s_first[c] = c;
    }
    n_ctx = N;
  } else {
    // -- child-list offsets: cur[c] = end of the children of context c
    int carry = 0;
    for (int base = 0; base < R; base += 32) {
      const int c = base + lane;
      int incl = c < R ? cnt[c] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += t;
      }
      if (c < R) cur[c] = carry + incl, tmp[c] = 0;
      carry += __shfl_sync(kFull, incl, 31);
    }
    __syncwarp();
    // -- place of every node among its siblings (tmp[c]: children of c placed so far), first child
    for (int base = 0; base < N; base += 32) {
      const int i = base + lane;
      const unsigned act = __ballot_sync(kFull, i < N);
      if (i < N) {
        const int pc = s_par[i] + 1;
        const unsigned peers = __match_any_sync(act, pc);
        const int before = tmp[pc];
        const int rk = before + __popc(peers & below);
        s_pos[i] = cur[pc] - cnt[pc] + rk;
        if (rk == 0) s_first[pc] = i;
        __syncwarp(act);
        if ((peers & below) == 0) tmp[pc] = before + __popc(peers);
      }
      __syncwarp();
    }
    // -- depth of every context by pointer jumping: dep[i + 1] = distance from node i to anc[i] (or to the root)
    for (int i = lane; i < N; i += 32) anc[i] = s_par[i], dep[i + 1] = 1;
    if (lane == 0) dep[0] = 0;
    __syncwarp();
    for (int round = 0; round < 12; ++round) {   // every round at least doubles the distance covered: 2^11 > 1024
      bool more = false;
      for (int base = 0; base < N; base += 32) {
        const int i = base + lane;
        const int a = i < N ? anc[i] : -1;
        int da = 0, aa = -1;
        if (a >= 0) da = dep[a + 1], aa = anc[a];   // a < i: a pair that is consistent whether or not a has moved this round
        __syncwarp();
        if (a >= 0) {
          dep[i + 1] += da;
          anc[i] = aa;
          more |= aa >= 0;
        }
        __syncwarp();
      }
      if (!__any_sync(kFull, more)) break;
    }
    int maxd = 0;
    for (int i = lane; i < N; i += 32) maxd = max(maxd, dep[i + 1]);
    maxd = __reduce_max_sync(kFull, maxd);
    // -- nodes ordered by (depth, index): lvl[d] counts, then is the cursor, and ends as the end of level d
    for (int d = lane; d <= maxd; d += 32) lvl[d] = 0;
    __syncwarp();
    for (int i = lane; i < N; i += 32) atomicAdd(&lvl[dep[i + 1]], 1);
    __syncwarp();
    carry = 0;
    for (int base = 0; base <= maxd; base += 32) {
      const int d = base + lane;
      const int n = d <= maxd ? lvl[d] : 0;
      int incl = n;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += t;
      }
      if (d <= maxd) lvl[d] = carry + incl - n;
      carry += __shfl_sync(kFull, incl, 31);
    }
    __syncwarp();
    int* order = anc;   // (the ancestors are no longer needed)
    for (int base = 0; base < N; base += 32) {
      const int i = base + lane;
      const unsigned act = __ballot_sync(kFull, i < N);
      if (i < N) {
        const int d = dep[i + 1];
        const unsigned peers = __match_any_sync(act, d);
        const int before = lvl[d];
        order[before + __popc(peers & below)] = i;
        __syncwarp(act);
        if ((peers & below) == 0) lvl[d] = before + __popc(peers);
      }
      __syncwarp();
    }
    // -- subtree sizes, deepest level first (level d occupies order[lvl[d - 1] .. lvl[d]))
    for (int d = maxd; d >= 1; --d) {
      for (int pos = lvl[d - 1] + lane; pos < lvl[d]; pos += 32) {
        const int i = order[pos];
        atomicAdd(&siz[s_par[i] + 1], siz[i + 1]);
      }
      __syncwarp();
    }
    // -- sizes in child-list order and their running sum: tmp[pos] = sizes of everything placed before pos
    for (int i = lane; i < N; i += 32) tmp[s_pos[i]] = siz[i + 1];
    __syncwarp();
    carry = 0;
    for (int base = 0; base < N; base += 32) {
      const int pos = base + lane;
      const int n = pos < N ? tmp[pos] : 0;
      int incl = n;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += t;
      }
      if (pos < N) tmp[pos] = carry + incl - n;
      carry += __shfl_sync(kFull, incl, 31);
    }
    if (lane == 0) din[0] = 0;
    __syncwarp();
    // -- pre-order positions, top level first: after the parent come the subtrees of the earlier siblings
    for (int d = 1; d <= maxd; ++d) {
      for (int pos = lvl[d - 1] + lane; pos < lvl[d]; pos += 32) {
        const int i = order[pos];
        const int pc = s_par[i] + 1;
        din[i + 1] = din[pc] + 1 + tmp[s_pos[i]] - tmp[cur[pc] - cnt[pc]];
      }
      __syncwarp();
    }
    // -- breadth-first rank of the contexts with children: the root, then the nodes by (depth, index)
    n_ctx = cnt[0] > 0 ? 1 : 0;
    for (int base = 0; base < N; base += 32) {
      const int pos = base + lane;
      const int i = pos < N ? order[pos] : 0;
      const bool has = pos < N && cnt[i + 1] > 0;
      const unsigned bal = __ballot_sync(kFull, has);
      if (has) dep[i + 1] = n_ctx + __popc(bal & below);   // the depth is no longer needed: dep[c] becomes the rank
      n_ctx += __popc(bal);
    }
  }
  // (thousands of warps would otherwise queue up on one address: most find the maximum already there)
  if (lane == 0 && n_ctx > *reinterpret_cast<volatile int*>(&P.counters->n_rank)) atomicMax(&P.counters->n_rank, n_ctx);
  __syncwarp();         // the shared arrays are complete
  for (int i = lane; i < N; i += 32) {   // the child lists, written by all lanes
    ChildInfo ci = {i, s_tok[i], __int_as_float(s_uni[i]), (din[i + 1] << 16) | siz[i + 1]};
    kids[s_pos[i]] = ci;
  }
  for (int r = n_ctx + lane; r < N; r += 32) P.work[static_cast<size_t>(r) * B + b].item = -1;
  const float u_final = __int_as_float(s_uni[N]);
  const int cap = B * N;
  for (int base = 0; base < R; base += 32) {
    const int c = base + lane;
    const int n = c < R ? cnt[c] : 0;
    const unsigned heavy = __ballot_sync(kFull, n >= 2);
    const unsigned light = __ballot_sync(kFull, n == 1);
    int hb = 0, lb = 0;
    if (P.ctx_slots && lane == 0) {
      if (heavy) hb = atomicAdd(&P.counters->n_heavy, __popc(heavy));
      if (light) lb = atomicAdd(&P.counters->n_light, __popc(light));
    }
    hb = __shfl_sync(kFull, hb, 0);
    lb = __shfl_sync(kFull, lb, 0);
    const unsigned below = (1u << lane) - 1u;
    if (c < R) {
      if (n == 0) {
        Record leaf = {kLeaf, -1, 0, 0};
        P.records[static_cast<size_t>(b) * R + c] = leaf;
      } else {
        Record pending = {-1, -1, LANTERN_ST_INTERNAL, 0};   // stands until the fused pass has evaluated the context
        P.records[static_cast<size_t>(b) * R + c] = pending;
        const int start = cur[c] - n;
        const int f = s_first[c];             // the context's first child (smallest node index)
        WorkItem w = {b * R + c, b * N + start, (n << 16) | f, (din[f + 1] << 16) | siz[f + 1], s_tok[f],
                      __int_as_float(s_uni[f]), u_final, b * R + din[c]};
        const int slot = dep[c] * B + b;
        P.work[slot] = w;
        if (P.ctx_slots) P.ctx_slots[n >= 2 ? hb + __popc(heavy & below) : cap - 1 - (lb + __popc(light & below))] = slot;
      }
    }
  }
}

}  // namespace lantern

// kernel 2: the fused context pass
#include "verify_context.cuh"
// greedy decoding (temperature 0)
#include "verify_greedy.cuh"
#include "verify_bonus.cuh"
#include "verify_topk.cuh"

namespace lantern {

// ---------------------------------------------------------------------------------------
// kernel 3: walk (Algorithm 1's loop over the records; one thread per sequence)
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) lantern_walk_kernel(VerifyParams P) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= P.B) return;
  const int N = P.N, R = P.R;
  int status = P.seq_status[b];
  int len = 0, next = -1;
  if (status == 0) {
    int cur = 0;
    for (int step = 0; step <= N; ++step) {
      const Record rec = P.records[static_cast<size_t>(b) * R + cur];
      bool from_q = rec.accepted == kLeaf;   // no drafts left on this path: bonus token from q
      if (!from_q) {
        status |= rec.status;
        // a residual without weight: the next token comes from the context's own target as well
        from_q = (rec.status & LANTERN_ST_DEGENERATE) && !(rec.status & (LANTERN_ST_NONFINITE | LANTERN_ST_INTERNAL));
      }
      if (from_q) {
        const int slot = atomicAdd(&P.counters->n_bonus, 1);
        P.bonus_seq[slot] = b;
        P.bonus_ctx[slot] = cur;
        break;
      }
      if (rec.status & (LANTERN_ST_NONFINITE | LANTERN_ST_INTERNAL)) break;
      if (rec.accepted >= 0) {
        // an accepted node is a child of this context: its index is at least the context's, and the path
        // holds at most N nodes; anything else is not a record the fused pass wrote
        if (rec.accepted < cur || rec.accepted >= N || len >= N) {
          status |= LANTERN_ST_INTERNAL;
          break;
        }
        if (P.out_path) P.out_path[static_cast<size_t>(b) * N + len] = rec.accepted;
        ++len;
        cur = rec.accepted + 1;
        continue;
      }
      next = rec.token;
      break;
    }
  }
  P.out_len[b] = len;
  P.out_tok[b] = next;
  if (P.out_status) P.out_status[b] = status;
  if (status) atomicOr(&P.counters->status_or, status);
}

// ---------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------
static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct WsLayout {
  size_t counters, work, slots, children, records, dead, seqst, bseq, bctx, thrq, thrp, total;
};

static WsLayout ws_layout(int B, int N, bool topk = false) {
  const size_t R = static_cast<size_t>(N) + 1, b = static_cast<size_t>(B);
  const size_t n1 = N > 0 ? N : 1;
  WsLayout L;
  size_t o = 0;
  L.counters = o; o += 256;
  L.work = o;     o += align_up(b * n1 * sizeof(WorkItem), 256);
  L.slots = o;    o += align_up(b * n1 * 4, 256);
  L.children = o; o += align_up(b * n1 * sizeof(ChildInfo), 256);
  L.records = o;  o += align_up(b * R * sizeof(Record), 256);
  L.dead = o;     o += align_up(b * R, 256);
  L.seqst = o;    o += align_up(b * 4, 256);
  L.bseq = o;     o += align_up(b * 4, 256);
  L.bctx = o;     o += align_up(b * 4, 256);
  L.thrq = o;     o += topk ? align_up(b * R * 4, 256) : 0;
  L.thrp = o;     o += topk ? align_up(b * R * 4, 256) : 0;
  L.total = o;
  return L;
}

static thread_local cudaEvent_t g_ev_before = nullptr, g_ev_after = nullptr;

// limit of the kernels' bounded waits and the self-test's withheld context (lantern_debug_wait_test)
constexpr uint32_t kDefaultWaitTries = 1u << 21;
static thread_local uint32_t g_wait_tries = kDefaultWaitTries;
static thread_local int g_withhold_item = -1;

// thresholds of the top-k filter: mode 0 = rows of the contexts with children (after the plan),
// mode 1 = rows of the bonus draws (after the walk)
template <bool BF16, bool UNC>
static cudaError_t launch_topk(const VerifyParams& P, int mode, long long jobs, int sms, cudaStream_t st) {
  auto kt = lantern_topk_kernel<BF16, UNC>;
  const size_t smem = static_cast<size_t>(P.V) * (UNC ? 2 : 1) * (BF16 ? 2 : 4);   // one job's raw rows
  cudaError_t e = cudaFuncSetAttribute(kt, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kt, TKT, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorInvalidConfiguration;
  const long long slots = static_cast<long long>(sms) * per_sm;
  const int grid = static_cast<int>(jobs < slots ? (jobs > 0 ? jobs : 1) : slots);
  kt<<<grid, TKT, smem, st>>>(P, mode);
  return cudaGetLastError();
}

// the variants of the fused context kernel live in verify_context_v<tone + 2 jsd + 4 topk>.cu
#define LANTERN_DECLARE_VARIANT(n) \
  cudaError_t launch_context_v##n(const VerifyParams&, int, bool, bool, int, size_t, cudaStream_t);
LANTERN_DECLARE_VARIANT(0) LANTERN_DECLARE_VARIANT(1) LANTERN_DECLARE_VARIANT(2) LANTERN_DECLARE_VARIANT(3)
LANTERN_DECLARE_VARIANT(4) LANTERN_DECLARE_VARIANT(5) LANTERN_DECLARE_VARIANT(6) LANTERN_DECLARE_VARIANT(7)
#undef LANTERN_DECLARE_VARIANT

cudaError_t launch_context_kernel(const VerifyParams& P, int CH, bool bf16, bool uncond, bool tone, bool jsd, bool topk,
                                  int grid, size_t smem_bytes, cudaStream_t st) {
  switch ((tone ? 1 : 0) | (jsd ? 2 : 0) | (topk ? 4 : 0)) {
    case 0: return launch_context_v0(P, CH, bf16, uncond, grid, smem_bytes, st);
    case 1: return launch_context_v1(P, CH, bf16, uncond, grid, smem_bytes, st);
    case 2: return launch_context_v2(P, CH, bf16, uncond, grid, smem_bytes, st);
    case 3: return launch_context_v3(P, CH, bf16, uncond, grid, smem_bytes, st);
    case 4: return launch_context_v4(P, CH, bf16, uncond, grid, smem_bytes, st);
    case 5: return launch_context_v5(P, CH, bf16, uncond, grid, smem_bytes, st);
    case 6: return launch_context_v6(P, CH, bf16, uncond, grid, smem_bytes, st);
    default: return launch_context_v7(P, CH, bf16, uncond, grid, smem_bytes, st);
  }
}

template <bool BF16, bool UNC, bool TOPK>
static cudaError_t launch_bonus(const VerifyParams& P, int sms, cudaStream_t st) {
  auto kb = lantern_bonus_stream_kernel<BF16, UNC, TOPK>;
  const size_t smem = static_cast<size_t>(P.V) * (UNC ? 2 : 1) * (BF16 ? 2 : 4);   // one context's raw target rows
  cudaError_t e = cudaFuncSetAttribute(kb, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kb, BNT, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorInvalidConfiguration;
  const long long slots = static_cast<long long>(sms) * per_sm;
  const int grid = static_cast<int>(P.B < slots ? P.B : slots);
  kb<<<grid, BNT, smem, st>>>(P);
  return cudaGetLastError();
}

template <bool BF16, bool UNC, bool TOPK>
static cudaError_t launch_verify(const VerifyParams& P, int CH, bool tone, bool jsd, long long items, int sms,
                                 int grid_ctx, size_t smem_bytes, cudaStream_t st) {
  cudaError_t e;   // (with the top-k filter the fused pass finds the thresholds of its contexts itself)
  if (g_ev_before && g_ev_after) cudaEventRecord(g_ev_before, st);
  e = launch_context_kernel(P, CH, BF16, UNC, tone, jsd, TOPK, grid_ctx, smem_bytes, st);
  if (e != cudaSuccess) return e;
  if (g_ev_before && g_ev_after) cudaEventRecord(g_ev_after, st);
  lantern_walk_kernel<<<(P.B + 127) / 128, 128, 0, st>>>(P);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (TOPK) {
    e = launch_topk<BF16, UNC>(P, 1, P.B, sms, st);
    if (e != cudaSuccess) return e;
  }
  return launch_bonus<BF16, UNC, TOPK>(P, sms, st);
}

template <bool BF16, bool UNC, bool TOPK>
static cudaError_t launch_greedy(const VerifyParams& P, long long items, int sms, int grid_bonus, cudaStream_t st) {
  auto kc = lantern_greedy_context_kernel<BF16, UNC, TOPK>;
  // a ring of staging areas per CTA, each holding the raw target rows of one context; sized so that
  // three CTAs share an SM where the rows allow it
  const size_t area = static_cast<size_t>(P.V) * (UNC ? 2 : 1) * (BF16 ? 2 : 4);
  int ring = static_cast<int>((72 * 1024) / area);
  ring = ring < 1 ? 1 : (ring > GRING_MAX ? GRING_MAX : ring);
  const size_t smem = ring * area;
  cudaError_t e = cudaFuncSetAttribute(kc, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  int per_sm = 0;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kc, GCT, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorInvalidConfiguration;
  const long long slots = static_cast<long long>(sms) * per_sm;
  const int grid_ctx = static_cast<int>(items < slots ? items : slots);
  if (TOPK) {
    e = launch_topk<BF16, UNC>(P, 0, items, sms, st);
    if (e != cudaSuccess) return e;
  }
  if (g_ev_before && g_ev_after) cudaEventRecord(g_ev_before, st);
  kc<<<grid_ctx, GCT, smem, st>>>(P, ring);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (g_ev_before && g_ev_after) cudaEventRecord(g_ev_after, st);
  lantern_walk_kernel<<<(P.B + 127) / 128, 128, 0, st>>>(P);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  lantern_greedy_bonus_kernel<BF16, UNC><<<grid_bonus, GRT, 0, st>>>(P);   // the arg max is never filtered out
  return cudaGetLastError();
}

}  // namespace lantern

using namespace lantern;

static bool shape_ok(int B, int N, int V, int k, int dtype) {
  if (dtype != LANTERN_F32 && dtype != LANTERN_BF16) return false;
  if (B < 0 || N < 0 || N > MAX_N || V < 8 || V > 16384 || (V % 8) != 0 || k < 1 || k > V) return false;
  return static_cast<long long>(B) * (N + 1) < (1ll << 31);
}

extern "C" size_t lantern_verify_workspace_bytes(int B, int N, int V, int k, int dtype) {
  if (!shape_ok(B, N, V, k, dtype)) return 0;
  return ws_layout(B > 0 ? B : 1, N).total;
}

extern "C" int lantern_verify_launch_count(int greedy, int top_k_active) {
  // memset, plan, fused pass (or greedy pass), walk, bonus; with the filter one threshold kernel more: ahead
  // of the greedy pass, or ahead of the bonus draw in sampling (the fused pass finds its own thresholds)
  (void)greedy;
  return 5 + (top_k_active ? 1 : 0);
}

extern "C" lantern_status lantern_last_status(const void* workspace, void* cuda_stream, int32_t* out_bits) {
  if (!workspace) return LANTERN_E_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int32_t bits = 0;
  const unsigned char* c = static_cast<const unsigned char*>(workspace) + offsetof(Counters, status_or);
  if (cudaMemcpyAsync(&bits, c, sizeof(bits), cudaMemcpyDeviceToHost, st) != cudaSuccess) return LANTERN_E_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return LANTERN_E_CUDA;
  if (out_bits) *out_bits = bits;
  return bits ? LANTERN_E_DATA : LANTERN_OK;
}

extern "C" lantern_status lantern_verify_counts(const void* workspace, void* cuda_stream, int64_t* out_counts) {
  if (!workspace || !out_counts) return LANTERN_E_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  Counters c;
  if (cudaMemcpyAsync(&c, workspace, sizeof(c), cudaMemcpyDeviceToHost, st) != cudaSuccess) return LANTERN_E_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return LANTERN_E_CUDA;
  // sampling keeps no count of its own: every context with children is either evaluated or left out
  const int64_t listed = static_cast<int64_t>(c.n_heavy) + c.n_light;
  out_counts[0] = listed ? listed : static_cast<int64_t>(c.n_evaluated) + c.n_skipped;
  out_counts[1] = c.n_evaluated;
  out_counts[2] = c.n_skipped;
  out_counts[3] = c.n_bonus;
  out_counts[4] = c.n_tested;
  out_counts[5] = c.n_slow_topk;
  return LANTERN_OK;
}

extern "C" lantern_status lantern_debug_wait_test(int max_tries, int withhold_context) {
  if (max_tries < 0) return LANTERN_E_PARAM;
  g_wait_tries = max_tries == 0 ? kDefaultWaitTries : static_cast<uint32_t>(max_tries);
  g_withhold_item = withhold_context;
  return LANTERN_OK;
}

extern "C" int lantern_kernel_revision(void) { return LANTERN_CONTEXT_KERNEL_REVISION; }

extern "C" lantern_status lantern_verify_profile_events(void* before_fused, void* after_fused) {
  if ((before_fused == nullptr) != (after_fused == nullptr)) return LANTERN_E_NULL;
  g_ev_before = static_cast<cudaEvent_t>(before_fused);
  g_ev_after = static_cast<cudaEvent_t>(after_fused);
  return LANTERN_OK;
}

static lantern_status verify_impl(const void* target_logits, const void* draft_logits, int dtype, float cfg_scale,
                                  int has_uncond, float T, const int32_t* draft_tokens, const int32_t* tree_parents,
                                  const int32_t* neighbor_idx, int k, float delta, int divergence, int top_k,
                                  const float* uniforms, int B, int N, int V, int32_t* out_accept_len,
                                  int32_t* out_next_token, int32_t* out_accept_path, int32_t* out_status,
                                  float* out_node_qa, float* out_node_px, int32_t* out_node_m, void* workspace,
                                  size_t workspace_bytes, void* cuda_stream);

extern "C" lantern_status lantern_verify(const void* target_logits, const void* draft_logits, int dtype,
                                         float cfg_scale, int has_uncond, float T, const int32_t* draft_tokens,
                                         const int32_t* tree_parents, const int32_t* neighbor_idx, int k,
                                         float delta, const float* uniforms, int B, int N, int V,
                                         int32_t* out_accept_len, int32_t* out_next_token,
                                         int32_t* out_accept_path, int32_t* out_status, float* out_node_qa,
                                         float* out_node_px, int32_t* out_node_m, void* workspace,
                                         size_t workspace_bytes, void* cuda_stream) {
  return lantern_verify_ex(target_logits, draft_logits, dtype, cfg_scale, has_uncond, T, draft_tokens, tree_parents,
                           neighbor_idx, k, delta, LANTERN_DIV_TVD, 0, uniforms, B, N, V, out_accept_len,
                           out_next_token, out_accept_path, out_status, out_node_qa, out_node_px, out_node_m,
                           workspace, workspace_bytes, cuda_stream);
}

extern "C" size_t lantern_verify_workspace_bytes_ex(int B, int N, int V, int k, int dtype, int top_k) {
  if (!shape_ok(B, N, V, k, dtype) || top_k < 0) return 0;
  return ws_layout(B > 0 ? B : 1, N, top_k > 0).total;
}

extern "C" lantern_status lantern_verify_ex(const void* target_logits, const void* draft_logits, int dtype,
                                         float cfg_scale, int has_uncond, float T, const int32_t* draft_tokens,
                                         const int32_t* tree_parents, const int32_t* neighbor_idx, int k,
                                         float delta, int divergence, int top_k, const float* uniforms, int B,
                                         int N, int V, int32_t* out_accept_len, int32_t* out_next_token,
                                         int32_t* out_accept_path, int32_t* out_status, float* out_node_qa,
                                         float* out_node_px, int32_t* out_node_m, void* workspace,
                                         size_t workspace_bytes, void* cuda_stream) {
  if (divergence != LANTERN_DIV_TVD && divergence != LANTERN_DIV_JSD) return LANTERN_E_PARAM;
  if (top_k < 0) return LANTERN_E_PARAM;
  return verify_impl(target_logits, draft_logits, dtype, cfg_scale, has_uncond, T, draft_tokens, tree_parents,
                     neighbor_idx, k, delta, divergence, top_k, uniforms, B, N, V, out_accept_len, out_next_token,
                     out_accept_path, out_status, out_node_qa, out_node_px, out_node_m, workspace,
                     workspace_bytes, cuda_stream);
}

static lantern_status verify_impl(const void* target_logits, const void* draft_logits, int dtype,
                                         float cfg_scale, int has_uncond, float T, const int32_t* draft_tokens,
                                         const int32_t* tree_parents, const int32_t* neighbor_idx, int k,
                                         float delta, int divergence, int top_k, const float* uniforms, int B, int N, int V,
                                         int32_t* out_accept_len, int32_t* out_next_token,
                                         int32_t* out_accept_path, int32_t* out_status, float* out_node_qa,
                                         float* out_node_px, int32_t* out_node_m, void* workspace,
                                         size_t workspace_bytes, void* cuda_stream) {
  if (dtype != LANTERN_F32 && dtype != LANTERN_BF16) return LANTERN_E_PARAM;
  if (B < 0 || N < 0 || N > MAX_N || V < 8 || V > 16384 || (V % 8) != 0 || k < 1 || k > V) return LANTERN_E_SHAPE;
  if (static_cast<long long>(B) * (N + 1) >= (1ll << 31)) return LANTERN_E_SHAPE;
  if (!(T >= 0.0f) || !(delta >= 0.0f) || !isfinite(T) || !isfinite(delta)) return LANTERN_E_PARAM;
  if (has_uncond && !isfinite(cfg_scale)) return LANTERN_E_PARAM;
  const bool greedy = T == 0.0f;   // Section 4.3, last sentence: no drafter distribution, no random numbers
  const int esize = dtype == LANTERN_BF16 ? 2 : 4;
  const int nrows = has_uncond ? 3 : 2;
  const int CH = V > 4 * GT * 8 ? 8 : (V > 2 * GT * 8 ? 4 : (V > GT * 8 ? 2 : 1));   // 8-token chunks per thread
  // one staging area of three row slots per consumer group; the numerators are kept over the rows they came from
  const size_t smem_bytes = NGRP * ((static_cast<size_t>(3) * V * esize + 127) & ~static_cast<size_t>(127));
  (void)nrows;
  if (!greedy && (smem_bytes > 192 * 1024 || (dtype == LANTERN_F32 && V > 8192))) return LANTERN_E_SHAPE;   // plus the kernel's static part: within the 227 KB of a CTA
  if (B == 0) return LANTERN_OK;
  if (!target_logits || !neighbor_idx || !out_accept_len || !out_next_token) return LANTERN_E_NULL;
  if (!greedy && !uniforms) return LANTERN_E_NULL;
  if (N > 0 && (!draft_tokens || (!greedy && !draft_logits))) return LANTERN_E_NULL;
  if ((reinterpret_cast<uintptr_t>(target_logits) & 15) || (reinterpret_cast<uintptr_t>(draft_logits) & 15))
    return LANTERN_E_ALIGN;
  const bool topk = top_k > 0 && top_k < V;   // top_k >= V keeps every logit
  const WsLayout L = ws_layout(B, N, top_k > 0);
  if (!workspace || workspace_bytes < L.total || (reinterpret_cast<uintptr_t>(workspace) & 255))
    return LANTERN_E_WORKSPACE;

  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  VerifyParams P;
  P.target = target_logits;
  P.draft = draft_logits;
  P.tokens = draft_tokens;
  P.parents = tree_parents;
  P.nbr = neighbor_idx;
  P.uniforms = greedy ? nullptr : uniforms;
  P.out_len = out_accept_len;
  P.out_tok = out_next_token;
  P.out_path = out_accept_path;
  P.out_status = out_status;
  P.out_qa = out_node_qa;
  P.out_px = out_node_px;
  P.out_m = out_node_m;
  P.counters = reinterpret_cast<Counters*>(ws + L.counters);
  P.work = reinterpret_cast<WorkItem*>(ws + L.work);
  P.children = reinterpret_cast<ChildInfo*>(ws + L.children);
  P.records = reinterpret_cast<Record*>(ws + L.records);
  P.seq_status = reinterpret_cast<int32_t*>(ws + L.seqst);
  P.bonus_seq = reinterpret_cast<int32_t*>(ws + L.bseq);
  P.bonus_ctx = reinterpret_cast<int32_t*>(ws + L.bctx);
  P.B = B;
  P.N = N;
  P.R = N + 1;
  P.V = V;
  P.k = k;
  P.cfg_scale = cfg_scale;
  P.T = T;
  P.delta = delta;
  P.divergence = divergence;
  P.top_k = topk ? top_k : 0;
  P.thr_q = topk ? reinterpret_cast<float*>(ws + L.thrq) : nullptr;
  P.thr_p = topk ? reinterpret_cast<float*>(ws + L.thrp) : nullptr;
  // only the threshold kernel of greedy decoding with the logit filter walks the compact list
  P.ctx_slots = (greedy && topk) ? reinterpret_cast<int32_t*>(ws + L.slots) : nullptr;
  P.dead = ws + L.dead;
  P.wait_tries = g_wait_tries;
  P.withhold_item = g_withhold_item;

  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return LANTERN_E_CUDA;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return LANTERN_E_CUDA;
  if (sms < 1) return LANTERN_E_CUDA;

  if (cudaMemsetAsync(P.counters, 0, 256, st) != cudaSuccess) return LANTERN_E_CUDA;
  const size_t plan_smem = static_cast<size_t>(PLAN_WARPS) * kPlanArrays * (N + 2) * sizeof(int);
  if (plan_smem > 48 * 1024 &&
      cudaFuncSetAttribute(lantern_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           static_cast<int>(plan_smem)) != cudaSuccess)
    return LANTERN_E_CUDA;
  lantern_plan_kernel<<<(B + PLAN_WARPS - 1) / PLAN_WARPS, PLAN_WARPS * 32, plan_smem, st>>>(P);
  if (cudaGetLastError() != cudaSuccess) return LANTERN_E_CUDA;

  const long long items = static_cast<long long>(B) * (N > 0 ? N : 1);   // upper bound of contexts with children
  const long long ctas = (items + NGRP - 1) / NGRP;   // every CTA runs NGRP contexts at a time
  const int grid_ctx = static_cast<int>(ctas < sms ? ctas : sms);
  const int grid_bonus = B < 4 * sms ? B : 4 * sms;   // greedy bonus: 256-thread CTAs
  cudaError_t e;
  const bool bf = dtype == LANTERN_BF16, un = has_uncond != 0;
  if (greedy) {
#define LANTERN_GREEDY(KV)                                                                                   \
  (bf ? (un ? launch_greedy<true, true, KV>(P, items, sms, grid_bonus, st) : launch_greedy<true, false, KV>(P, items, sms, grid_bonus, st)) \
      : (un ? launch_greedy<false, true, KV>(P, items, sms, grid_bonus, st) : launch_greedy<false, false, KV>(P, items, sms, grid_bonus, st)))
    e = topk ? LANTERN_GREEDY(true) : LANTERN_GREEDY(false);
#undef LANTERN_GREEDY
    return e == cudaSuccess ? LANTERN_OK : LANTERN_E_CUDA;
  }
  // every combination of the compile-time variants exists: T = 1 never meets the division code
  const bool tone = T == 1.0f, jsd = divergence == LANTERN_DIV_JSD;
#define LANTERN_DISPATCH2(KV)                                                                        \
  (bf ? (un ? launch_verify<true, true, KV>(P, CH, tone, jsd, items, sms, grid_ctx, smem_bytes, st)   \
            : launch_verify<true, false, KV>(P, CH, tone, jsd, items, sms, grid_ctx, smem_bytes, st)) \
      : (un ? launch_verify<false, true, KV>(P, CH, tone, jsd, items, sms, grid_ctx, smem_bytes, st)  \
            : launch_verify<false, false, KV>(P, CH, tone, jsd, items, sms, grid_ctx, smem_bytes, st)))
  e = topk ? LANTERN_DISPATCH2(true) : LANTERN_DISPATCH2(false);
#undef LANTERN_DISPATCH2
  return e == cudaSuccess ? LANTERN_OK : LANTERN_E_CUDA;
}

// ---------------------------------------------------------------------------------------
// lantern_verify_static: same computation, scratch taken from a fixed array in the device
// image instead of a caller workspace (for callers that must not allocate device memory).
// ---------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_workspace[LANTERN_STATIC_WORKSPACE_BYTES];

// In host code `g_static_workspace` is only a handle for the symbol, never an address a kernel
// could use; the device address is asked for once per device and remembered here.
static void* g_static_workspace_ptr[64] = {};

static lantern_status static_workspace_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return LANTERN_E_CUDA;
  if (dev >= 64) return LANTERN_E_SHAPE;   // the table of addresses below serves ordinals 0..63
  void* p = __atomic_load_n(&g_static_workspace_ptr[dev], __ATOMIC_ACQUIRE);
  if (!p) {
    if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || !p) return LANTERN_E_CUDA;
    __atomic_store_n(&g_static_workspace_ptr[dev], p, __ATOMIC_RELEASE);   // same value whoever wins
  }
  *out = p;
  return LANTERN_OK;
}

extern "C" lantern_status lantern_verify_static(const void* target_logits, const void* draft_logits, int dtype,
                                                float cfg_scale, int has_uncond, float T,
                                                const int32_t* draft_tokens, const int32_t* tree_parents,
                                                const int32_t* neighbor_idx, int k, float delta,
                                                const float* uniforms, int B, int N, int V,
                                                int32_t* out_accept_len, int32_t* out_next_token,
                                                int32_t* out_accept_path, int32_t* out_status, float* out_node_qa,
                                                float* out_node_px, int32_t* out_node_m, void* cuda_stream) {
  if (B < 0 || N < 0 || N > MAX_N) return LANTERN_E_SHAPE;
  // the fixed array bounds the call size: refuse anything whose scratch would not fit
  if (B > 0 && ws_layout(B, N).total > static_cast<size_t>(LANTERN_STATIC_WORKSPACE_BYTES)) return LANTERN_E_WORKSPACE;
  void* ws = nullptr;
  const lantern_status rc = static_workspace_address(&ws);
  if (rc != LANTERN_OK) return rc;
  // lantern_verify zeroes the counters at the head of the scratch on the stream before its first
  // kernel, so whatever the previous call left in the array does not matter.
  return lantern_verify(target_logits, draft_logits, dtype, cfg_scale, has_uncond, T, draft_tokens, tree_parents,
                        neighbor_idx, k, delta, uniforms, B, N, V, out_accept_len, out_next_token, out_accept_path,
                        out_status, out_node_qa, out_node_px, out_node_m, ws, LANTERN_STATIC_WORKSPACE_BYTES,
                        cuda_stream);
}

extern "C" const char* lantern_status_string(lantern_status s) {
  switch (s) {
    case LANTERN_OK: return "ok";
    case LANTERN_E_NULL: return "a required pointer is NULL";
    case LANTERN_E_SHAPE: return "a size is outside the supported range";
    case LANTERN_E_PARAM: return "a scalar parameter is invalid";
    case LANTERN_E_WORKSPACE: return "workspace missing, too small or misaligned";
    case LANTERN_E_CUDA: return "a CUDA runtime call failed";
    case LANTERN_E_DATA: return "a fault in the data was found on the device (see out_status)";
    case LANTERN_E_ALIGN: return "a pointer is not 16-byte aligned";
    case LANTERN_E_UNIMPLEMENTED: return "not implemented in this build";
    default: return "unknown status";
  }
}
