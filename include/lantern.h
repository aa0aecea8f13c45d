/*
 * lantern.h -- C ABI of the LANTERN relaxed speculative-verification library (CUDA, sm_100a).
 *
 * The library implements the verification side of "LANTERN" (arXiv 2410.03355): the one-time
 * latent-neighbourhood table B_k of a VQ codebook and, per verification step, the relaxed
 * acceptance test over the TVD-bounded neighbourhood A_{k,delta}, the relaxed residual
 * resampling on rejection, and the walk of a chain or tree of drafts to the first rejection.
 *
 * Notation (the paper's): q = target distribution, p = drafter distribution, x~ = draft token,
 * B_k(x~) = k nearest codes of x~ in the codebook, itself included (Section 4.2),
 * A_{k,delta}(x~) = the distance-ordered prefix of B_k(x~) whose moved mass stays below
 * delta (Section 4.3; Algorithm 2).
 *
 * Conventions common to all calls
 *   - Every data pointer is a DEVICE pointer owned by the caller; the library neither
 *     allocates, frees nor keeps it.  `workspace` is caller-owned device scratch of at least
 *     the size the matching *_workspace_bytes() call returns; its contents are undefined
 *     before and after a call, and two calls in flight at once need distinct workspaces.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the default stream).  Work is
 *     enqueued on it and the call returns without waiting for it.
 *   - Return value: LANTERN_OK, or a negative code found on the host before anything is
 *     launched (outputs untouched).  Faults that live in the data (a token out of range, a
 *     NaN logit ...) never trap: they set bits in out_status[b] and give that sequence the
 *     fallback result accept_len = number of drafts accepted before the fault, next_token = -1
 *     (a token no vocabulary holds, so that a caller who does not look at out_status cannot
 *     mistake it for a result).  lantern_last_status() tells in one word whether any sequence
 *     of a call carried such a bit.
 */
#ifndef LANTERN_H_
#define LANTERN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t lantern_status;

enum {
  LANTERN_OK = 0,
  LANTERN_E_NULL = -1,          /* a required pointer is NULL */
  LANTERN_E_SHAPE = -2,         /* a size is out of the supported range (see each call) */
  LANTERN_E_PARAM = -3,         /* a scalar parameter is invalid (T <= 0, delta < 0, NaN ...) */
  LANTERN_E_WORKSPACE = -4,     /* workspace missing, too small or misaligned */
  LANTERN_E_CUDA = -5,          /* a CUDA runtime call failed (no device, launch error) */
  LANTERN_E_DATA = -6,          /* lantern_last_status: some sequence of the call carries a status bit */
  LANTERN_E_UNIMPLEMENTED = -7, /* valid request this build does not cover (none at present) */
  LANTERN_E_ALIGN = -8          /* a pointer is not 16-byte aligned */
};

/* storage type of logits */
enum { LANTERN_F32 = 0, LANTERN_BF16 = 1 };

/* bits of out_status[b] */
enum {
  LANTERN_ST_BAD_TOKEN = 1,     /* a draft token outside [0, V) */
  LANTERN_ST_BAD_PARENT = 2,    /* a parent index outside [-1, own index) */
  LANTERN_ST_BAD_UNIFORM = 4,   /* a uniform outside [0, 1) */
  LANTERN_ST_NONFINITE = 8,     /* NaN / +inf logit, or a row with no finite logit, on the walked path */
  LANTERN_ST_DEGENERATE = 16,   /* a residual without weight was met; next_token was drawn from q instead (see lantern_verify) */
  LANTERN_ST_BAD_TABLE = 32,    /* a neighbour entry outside [0, V) was met while a set A was grown (it carries no mass) */
  LANTERN_ST_INTERNAL = 64      /* an on-chip copy did not complete within its wait limit: the sequence was not finished */
};

/* Human-readable name of a return code (static storage). */
const char* lantern_status_string(lantern_status s);

/* ------------------------------------------------------------------------------------------
 * Neighbour table.  Algorithm 2, block "Precompute B_k for all tokens" (Appendix D.2), with
 * the l2 latent distance of Section 5.1.
 *
 * For every code i: squared l2 distance to every code j, accumulated in fp32 in dimension
 * order as acc = fma(a_d - b_d, a_d - b_d, acc); the k smallest (distance, index) pairs with
 * i itself forced into slot 0; stored in increasing distance, ties by smaller index.
 *
 *   codebook   [V, D] row-major fp32, finite values
 *   V, D, k    1 <= k <= V <= 32768, 1 <= D <= 4096, k <= 4097
 *   idx        out [V, k] int32; idx[i,0] == i
 *   dist       out [V, k] fp32 squared distances, dist[i,0] == 0; may be NULL
 *   workspace  lantern_build_workspace_bytes(V, D, k) bytes (0 for D <= 32: may then be NULL)
 * ---------------------------------------------------------------------------------------- */
size_t lantern_build_workspace_bytes(int V, int D, int k);

lantern_status lantern_build_neighbors(const float* codebook, int V, int D, int k, int32_t* idx, float* dist,
                                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Neighbour table under a named latent proximity (Section 5.3.1 compares the l2 distance with
 * cosine similarity).  LANTERN_METRIC_L2 is lantern_build_neighbors.  LANTERN_METRIC_COSINE
 * scales every code to unit length first -- squared norm accumulated in fp32 in dimension order
 * by one fused multiply-add per dimension, one square root, one division per component; a zero
 * code stays zero -- and builds the same table on the scaled codes: on unit vectors the squared
 * distance is 2 - 2 cos, so rows come in decreasing cosine similarity, ties by smaller index,
 * and dist holds 2 - 2 cos.
 *
 *   workspace  lantern_build_workspace_bytes_metric(V, D, k, metric) bytes, 256-byte aligned
 *              (for the cosine metric it also holds the scaled codes)
 *   other arguments, limits and return codes as for lantern_build_neighbors; an unknown metric
 *   returns LANTERN_E_PARAM
 * ---------------------------------------------------------------------------------------- */
enum { LANTERN_METRIC_L2 = 0, LANTERN_METRIC_COSINE = 1 };

size_t lantern_build_workspace_bytes_metric(int V, int D, int k, int metric);

lantern_status lantern_build_neighbors_metric(const float* codebook, int V, int D, int k, int metric, int32_t* idx,
                                              float* dist, void* workspace, size_t workspace_bytes,
                                              void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * One verification step.  Algorithm 1, verification loop and the bonus-token line after it,
 * with the acceptance rule and residual of Section 4.3 and A_{k,delta} built as in
 * Algorithm 2's second block.
 *
 * Per sequence b the drafts form a tree of N nodes (a chain when tree_parents is NULL).
 * Context row 0 is the root; row i+1 is the context that follows node i.  Node i is tested
 * in the context of its parent with
 *     q = softmax((l_u + s (l_c - l_u)) / T)   of that row's target logits (guidance scales of
 *                                              Appendix B.2; l_c alone when has_uncond == 0)
 *     p = softmax(draft row / T)
 * and is accepted iff  r_i * p(x~) < sum_{x in A_{k,delta}(x~)} q(x).  Children of one context
 * are tried in node order; a rejection replaces q by the normalised residual
 * [q_{k,delta}(.|D = x~) - p]_+ and removes x~ from p before the next sibling.  The walk
 * follows accepted nodes; where every child is rejected the next token is drawn from the
 * last residual, and where the walk reaches a node without children it is drawn from that
 * row's q, both by inverse CDF at uniforms[b, N].
 *
 * A residual whose total weight is at most 1e-5 of the mass of the distribution it was taken
 * from defines nothing to draw from (Algorithm 1's else-branch presumes a positive weight; the
 * case needs a drafted token outside the drafter's own support, or two distributions that agree
 * to single precision): the walk stops at that context, LANTERN_ST_DEGENERATE is set, and the
 * next token is drawn from the context's own q at uniforms[b, N] -- a valid token.
 *
 * A neighbour entry outside [0, V) carries no mass; LANTERN_ST_BAD_TABLE is set when Algorithm 2's
 * loop meets one, i.e. in a slot ahead of the one that ends the set (entries behind it are not read).
 *
 * Only contexts that the walk can reach need evaluating, and with many sequences per call the
 * library leaves out most of the others (see out_node_* below); the results never depend on it.
 *
 *   target_logits  [C, B, N+1, V], C = 2 (conditional, unconditional) if has_uncond else 1
 *   draft_logits   [B, N+1, V] (already guided); rows of contexts without children are not read;
 *                  may be NULL when N == 0
 *   dtype          LANTERN_F32 or LANTERN_BF16, for both logit tensors; bases 16-byte aligned
 *   cfg_scale      s, read only if has_uncond
 *   T              temperature > 0, or exactly 0 for greedy decoding (Section 4.3, last sentence):
 *                  q is then the softmax at temperature 1, node i is accepted iff
 *                  sum_{A_{k,delta}(x~)} q >= max_x q(x) (x~ is an arg max of q_{k,delta}(.|D = x~),
 *                  ties accept), children are tried in node order against the same q, and the
 *                  next token is arg max q of the context where the walk stops (smallest index
 *                  on ties).  draft_logits and uniforms are not read and may be NULL;
 *                  out_node_px is written as 0; V <= 16384 for both logit types
 *   draft_tokens   [B, N] int32 in [0, V)
 *   tree_parents   [B, N] int32, -1 = child of the root, else an index < own index; NULL = chain
 *   neighbor_idx   [V, k] int32 as written by lantern_build_neighbors (slot 0 = the token itself)
 *   k, delta       1 <= k <= V; delta >= 0 (delta = 0 or k = 1 gives standard speculative sampling)
 *   uniforms       [B, N+1] fp32 in [0, 1): entry i tests node i, entry N is the final draw
 *   B, N, V        B >= 0; 0 <= N <= 1024; V a multiple of 8, 8 <= V <= 16384 with bf16 logits and
 *                  8 <= V <= 8192 with fp32 logits (two staging areas of three logit rows each
 *                  must fit in shared memory); anything else returns LANTERN_E_SHAPE
 *   out_accept_len  [B] number of accepted nodes
 *   out_next_token  [B] resampled or bonus token (-1 with a fault bit in out_status)
 *   out_accept_path [B, N] node ids of the accepted path in order, -1 padded; may be NULL
 *   out_status      [B] LANTERN_ST_* bits; may be NULL
 *   out_node_qa, out_node_px  [B, N] fp32: sum_A q and p(x~) as used in each node's test;
 *   out_node_m                [B, N] int32: |A_{k,delta}(x~)| - 1.  Written for every node the
 *                  walk tests (the children of each context on the accepted path, up to and
 *                  including the first accepted one).  Other nodes hold either NaN / -1 or the
 *                  values of a test made ahead of time that the walk did not need.  Each may be NULL.
 *   workspace       lantern_verify_workspace_bytes(B, N, V, k, dtype) bytes, 256-byte aligned
 *
 * The call only enqueues work on cuda_stream (one memset and four or five kernels): it allocates
 * nothing, reads nothing back and does not wait for the stream, and it re-initialises the part
 * of the workspace it relies on.  It may therefore be recorded by a stream capture and replayed
 * as a CUDA graph on inputs rewritten in place; make one call with the same shape, logit type
 * and options outside the capture first (kernel attributes are set then).
 *
 * lantern_verify_workspace_bytes returns 0 for sizes lantern_verify would refuse.
 * ---------------------------------------------------------------------------------------- */
size_t lantern_verify_workspace_bytes(int B, int N, int V, int k, int dtype);

lantern_status lantern_verify(const void* target_logits, const void* draft_logits, int dtype, float cfg_scale,
                              int has_uncond, float T, const int32_t* draft_tokens, const int32_t* tree_parents,
                              const int32_t* neighbor_idx, int k, float delta, const float* uniforms, int B,
                              int N, int V, int32_t* out_accept_len, int32_t* out_next_token,
                              int32_t* out_accept_path, int32_t* out_status, float* out_node_qa,
                              float* out_node_px, int32_t* out_node_m, void* workspace, size_t workspace_bytes,
                              void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * lantern_verify with the variants of the paper's ablations and generation settings.
 *
 *   divergence  what delta bounds when A_{k,delta}(x~) is grown (Section 5.3.2):
 *               LANTERN_DIV_TVD  the total variation distance between q and q_{k,delta}(.|D = x~),
 *                                i.e. the mass moved onto x~ (Section 4.3; lantern_verify);
 *               LANTERN_DIV_JSD  their Jensen-Shannon divergence with the natural logarithm,
 *                                JSD = 1/2 [ S ln 2 + q0 ln(q0 / mid) + (q0 + S) ln((q0 + S) / mid) ],
 *                                q0 = q(x~), S = the moved mass, mid = q0 + S / 2 (only the collapsed
 *                                tokens differ between the two distributions).  Neighbours are
 *                                still added in order of distance until the first one that would
 *                                reach delta.
 *   top_k       logit filter of the generation settings (Appendix B.2: top-k 1000 or 2000, top-p 1):
 *               processed logits below the top_k-th largest of their row count as -inf, for the
 *               target and for the drafter alike, before the softmax; logits equal to the
 *               top_k-th largest are all kept.  0, or any value >= V, switches the filter off.
 *   workspace   lantern_verify_workspace_bytes_ex(B, N, V, k, dtype, top_k) bytes, 256-byte aligned
 *
 * Everything else, and every return code, is as for lantern_verify; an unknown divergence or a
 * negative top_k returns LANTERN_E_PARAM.
 * ---------------------------------------------------------------------------------------- */
enum { LANTERN_DIV_TVD = 0, LANTERN_DIV_JSD = 1 };

size_t lantern_verify_workspace_bytes_ex(int B, int N, int V, int k, int dtype, int top_k);

lantern_status lantern_verify_ex(const void* target_logits, const void* draft_logits, int dtype, float cfg_scale,
                                 int has_uncond, float T, const int32_t* draft_tokens, const int32_t* tree_parents,
                                 const int32_t* neighbor_idx, int k, float delta, int divergence, int top_k,
                                 const float* uniforms, int B, int N, int V, int32_t* out_accept_len,
                                 int32_t* out_next_token, int32_t* out_accept_path, int32_t* out_status,
                                 float* out_node_qa, float* out_node_px, int32_t* out_node_m, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * All-token aggregation: for every token x of every given context row,
 *     out_agg[r, x] = sum_{y in A_{k,delta}(x)} q_r(y),   out_m[r, x] = |A_{k,delta}(x)| - 1,
 * with q_r the row's target distribution (guidance and temperature as in lantern_verify) and
 * A_{k,delta}(x) grown as in Algorithm 2's second block (TVD bound).  The paper's method never
 * needs this for more than the drafted tokens -- lantern_verify does not use it; the entry point
 * exists to measure the V x k gather-sum that the full aggregation amounts to.
 *
 *   logits        [C, rows, V], C = 2 (conditional, unconditional) if has_uncond else 1; 16-byte aligned
 *   neighbor_idx  [V, k] int32 as written by lantern_build_neighbors; 16-byte aligned
 *   rows, V, k    rows >= 0; V a multiple of 8, 8 <= V <= 16384; 1 <= k <= V
 *   T, delta      T > 0; delta >= 0
 *   out_agg       [rows, V] fp32 (NaN for a row with a NaN / +inf logit or no finite logit)
 *   out_m         [rows, V] int32, may be NULL (-1 for such a row)
 *   out_status    [rows] LANTERN_ST_NONFINITE / LANTERN_ST_BAD_TABLE bits, may be NULL
 * No workspace.  Asynchronous on cuda_stream.
 * ---------------------------------------------------------------------------------------- */
lantern_status lantern_aggregate_all(const void* logits, int dtype, float cfg_scale, int has_uncond, float T,
                                     const int32_t* neighbor_idx, int k, float delta, int rows, int V,
                                     float* out_agg, int32_t* out_m, int32_t* out_status, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * lantern_verify without a caller-supplied workspace.  (The paper has no counterpart: this
 * entry point exists for integration reasons only and computes exactly what lantern_verify
 * computes.)
 *
 * Who needs it: code that may not allocate device memory at the point where it verifies
 * drafts -- a serving loop whose HBM was handed out in full at start-up (KV cache, activation
 * arenas) so that a cudaMalloc would fail or fragment it, a plug-in that runs under an
 * allocator it does not own, or a latency-critical step that cannot afford the device-wide
 * synchronisation a cudaMalloc / cudaFree implies.  Such callers still own the inputs and
 * outputs; only the scratch that lantern_verify asks for is taken off their hands.
 *
 * The scratch lives in a fixed array inside the library's device image,
 * LANTERN_STATIC_WORKSPACE_BYTES (6 MiB) large: every GPU on which the library is loaded
 * holds those 6 MiB until the process exits.  The call makes no cudaMalloc / cudaFree and
 * calls nothing that allocates.
 *
 *   - Sizes: lantern_verify_workspace_bytes(B, N, V, k, dtype) must not exceed
 *     LANTERN_STATIC_WORKSPACE_BYTES (e.g. B = 8192, N = 7 or B = 1024, N = 60 fit);
 *     otherwise the call returns LANTERN_E_WORKSPACE and does nothing.  All other argument
 *     rules and return codes are those of lantern_verify.
 *   - First call on a device: the library looks up the device address of its array (once per
 *     device, with that device current, no allocation) and keeps it for the life of the process.
 *     Make that first call outside any stream capture.  The address does not survive a
 *     cudaDeviceReset of that device: do not reset a device between calls.  Device ordinals
 *     0..63 are served; a higher ordinal returns LANTERN_E_SHAPE.
 *   - The array is shared by every call on that device and keeps the previous call's contents;
 *     the call itself resets the few words that must start at zero.  Two such calls that may
 *     run on the GPU at the same time (different streams, different host threads) would write
 *     the same scratch and corrupt each other: serialise them, or use lantern_verify with
 *     separate workspaces.
 * ---------------------------------------------------------------------------------------- */
#define LANTERN_STATIC_WORKSPACE_BYTES (6u << 20)

lantern_status lantern_verify_static(const void* target_logits, const void* draft_logits, int dtype,
                                     float cfg_scale, int has_uncond, float T, const int32_t* draft_tokens,
                                     const int32_t* tree_parents, const int32_t* neighbor_idx, int k, float delta,
                                     const float* uniforms, int B, int N, int V, int32_t* out_accept_len,
                                     int32_t* out_next_token, int32_t* out_accept_path, int32_t* out_status,
                                     float* out_node_qa, float* out_node_px, int32_t* out_node_m,
                                     void* cuda_stream);

/* Revision number of the fused verification kernel; bumped whenever that kernel changes, so that
 * stored profiler counters can be matched to the code they were taken on. */
int lantern_kernel_revision(void);

/* Number of kernels (and memsets) one verification call enqueues: memset, plan, fused pass or greedy
 * pass, walk, bonus; a call whose top-k filter is active (0 < top_k < V) enqueues one threshold kernel
 * more (ahead of the greedy pass; in sampling ahead of the bonus draw -- the fused pass finds the
 * thresholds of its own contexts).  For launch accounting. */
int lantern_verify_launch_count(int greedy, int top_k_active);

/* ------------------------------------------------------------------------------------------
 * Summary of the data faults of the last verification call that used `workspace` (the per-sequence
 * detail is in that call's out_status).  Waits for `cuda_stream`, on which that call was enqueued.
 *
 *   out_bits   receives the OR of the LANTERN_ST_* bits of all sequences of the call; may be NULL
 *   returns    LANTERN_OK if no sequence carried a bit, LANTERN_E_DATA if one did,
 *              LANTERN_E_NULL / LANTERN_E_CUDA otherwise
 * ---------------------------------------------------------------------------------------- */
lantern_status lantern_last_status(const void* workspace, void* cuda_stream, int32_t* out_bits);

/* Work accounting of the last verification call that used `workspace` (waits for `cuda_stream`):
 *   out_counts[0]  contexts with at least one drafted child (in sampling: [1] + [2], which falls short of it
 *                  only if the call was abandoned after a wait ran out)
 *   out_counts[1]  of those, the ones the fused pass evaluated
 *   out_counts[2]  the ones it left out because the walk could not reach them (Algorithm 1 stops
 *                  at the first rejection)
 *   out_counts[3]  next tokens drawn from a context's own q (bonus draws and degenerate residuals)
 *   out_counts[4]  drafted nodes the fused pass tested
 *   out_counts[5]  rows whose top-k threshold needed the slow exact search (with a top-k filter only)
 * out_counts holds six entries. */
lantern_status lantern_verify_counts(const void* workspace, void* cuda_stream, int64_t* out_counts);

/* Self-test of the kernels' bounded waits (not part of the method).  Every wait for an on-chip copy
 * gives up after a number of tries (2^21 by default, each suspended for up to 4 us); a sequence whose
 * copy never completes ends with LANTERN_ST_INTERNAL instead of hanging the GPU.  This call sets, for
 * the calling host thread's later sampling calls, the number of tries (0 = the default) and the index
 * b * (N + 1) + c of one context whose copies the fused pass deliberately never starts (-1 = none), so
 * that the path can be exercised without any fault: nothing is left in flight, the affected group
 * gives up, the rest of the call is abandoned cleanly, and the device stays usable. */
lantern_status lantern_debug_wait_test(int max_tries, int withhold_context);

/* Measurement hook (not part of the method): when both arguments are non-NULL cudaEvent_t
 * handles, every later lantern_verify call made by the calling host thread records
 * `before_fused` on its stream right before the fused context kernel and `after_fused` right
 * after it, so that a benchmark can time that kernel alone with CUDA events.  Pass two NULLs
 * to switch it off.  The events are owned by the caller. */
lantern_status lantern_verify_profile_events(void* before_fused, void* after_fused);

#ifdef __cplusplus
}
#endif
#endif /* LANTERN_H_ */
