// LANTERN relaxed speculative verification -- CPU oracle.
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, single-threaded statement of
// what the method computes, written from the paper's definitions.  It shares no code with
// the CUDA library and is never on the product path; only tests, the smoke check and the
// CPU-baseline leg of the benchmark may call it.
//
// What follows the paper, and where:
//   * neighbour table B_k            -- Algorithm 2, "Precompute B_k" block (Appendix D.2)
//   * neighbourhood A_{k,delta}      -- Section 4.3 and Algorithm 2, "Dynamically calculate" block
//   * relaxed acceptance / residual  -- Section 4.3, final acceptance condition; q_k in Section 4.3
//   * chain walk and bonus token     -- Algorithm 1 (verification loop and the line after it)
//   * standard speculative sampling  -- Section 2 (the k = 1 / delta = 0 special case)
//
// Notation follows the paper: q = target distribution, p = drafter distribution,
// B_k(x~) = the k nearest codes of x~ including itself, A_{k,delta}(x~) = its TVD-bounded prefix.
//
// Readings taken where the paper leaves a choice (each is restated where it is used):
//   R1  distance = squared l2, accumulated in fp32 in dimension order with one fused
//       multiply-add per dimension; ties broken by smaller index; self always in slot 0.
//   R2  guidance: l = l_u + s*(l_c - l_u); then z = l / T; then softmax.  The processed
//       logit z is an fp32 quantity (difference, fused multiply-add and division each
//       rounded once to fp32); everything after it is double precision.
//   R3  A_{k,delta} is a prefix of the distance order, built with a break at the first
//       neighbour that would reach the bound; the bound is strict; x~ itself is always in.
//   R4  D_TV(q_{k,delta}, q) equals the moved mass sum_{x in A, x != x~} q(x), so the
//       "TVD increment for adding x" of Algorithm 2 is q(x).
//   R5  only the target is summed over A; the denominator is p(x~) alone.
//   R6  trees: children of a context are tested in node order; after a rejection the
//       target becomes the normalised relaxed residual and the drafter has the rejected
//       token removed and is renormalised (multi-round rejection); a chain is the tree
//       with parent(i) = i - 1.
//   R7  the uniform r lies in [0,1); accept iff r * p(x~) < sum_A q  (no division).
//   R8  inverse CDF: the smallest token whose inclusive cumulative weight exceeds
//       u * (total weight); if rounding leaves none, the largest token of positive weight.
//   R10 a residual whose total weight does not exceed `degenerate_eps` (1e-5 of the unit mass
//       unless the caller says otherwise) defines no distribution to draw from: the relaxed
//       target and the drafter coincide there.  The walk stops at that context, the status
//       bit is set, and the next token is drawn from the context's own target q -- the one
//       distribution Algorithm 1 does define for a context (its line after the loop).
//
// Parity pins: every exported function is pinned by tests/test_oracle_*.py against closed
// forms, brute force, a separately written textbook speculative sampler, and Monte-Carlo
// chi-square tests of the emitted-token law.  What the paper cannot pin (absolute accept
// rates on synthetic logits; the conventions R2 and R6 beyond their losslessness at
// delta = 0) is "parity unpinned" against the paper and fixed by these readings.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

namespace {

enum { DT_F32 = 0, DT_BF16 = 1 };

enum {
  ST_BAD_TOKEN = 1,        // a draft token outside [0, V)
  ST_BAD_PARENT = 2,       // a parent index not in [-1, own index)
  ST_BAD_UNIFORM = 4,      // a uniform outside [0, 1) or NaN
  ST_NONFINITE = 8,        // NaN / +inf logit or empty softmax in a visited context
  ST_DEGENERATE = 16,      // residual of (near) zero total weight: next token drawn from q (R10)
  ST_BAD_TABLE = 32        // a neighbour entry outside [0, V)
};

inline float load_logit(const void* base, int dtype, size_t i) {
  if (dtype == DT_F32) return static_cast<const float*>(base)[i];
  uint32_t bits = static_cast<uint32_t>(static_cast<const uint16_t*>(base)[i]) << 16;
  float f;
  std::memcpy(&f, &bits, 4);
  return f;
}

// R2: processed target logit as an fp32 value.
inline float target_z(float lc, float lu, int has_uncond, float s, float T) {
  float l = lc;
  if (has_uncond) {
    float d = lc - lu;
    l = std::fmaf(s, d, lu);
  }
  return l / T;
}

// softmax of fp32 processed logits in double precision; returns false if not well defined.
bool softmax(const std::vector<float>& z, std::vector<double>& out, double* Z_out) {
  const size_t V = z.size();
  double m = -std::numeric_limits<double>::infinity();
  for (size_t x = 0; x < V; ++x) {
    if (std::isnan(z[x])) return false;
    if (static_cast<double>(z[x]) > m) m = z[x];
  }
  if (!std::isfinite(m)) return false;
  double Z = 0.0;
  out.resize(V);
  for (size_t x = 0; x < V; ++x) {
    out[x] = std::exp(static_cast<double>(z[x]) - m);
    Z += out[x];
  }
  if (!(Z > 0.0) || !std::isfinite(Z)) return false;
  for (size_t x = 0; x < V; ++x) out[x] /= Z;
  if (Z_out) *Z_out = Z;
  return true;
}

// R8.  margin (optional) = distance of the target point to the nearer CDF edge of the
// chosen token, in units of the total weight.
int inverse_cdf(const std::vector<double>& w, double u, double* margin) {
  const int V = static_cast<int>(w.size());
  double tot = 0.0;
  for (int x = 0; x < V; ++x) tot += w[x];
  if (margin) *margin = std::numeric_limits<double>::infinity();
  if (!(tot > 0.0)) return -1;
  const double target = u * tot;
  double cum = 0.0;
  int last_pos = -1;
  for (int x = 0; x < V; ++x) {
    const double lo = cum;
    cum += w[x];
    if (w[x] > 0.0) last_pos = x;
    if (cum > target) {
      if (margin) *margin = std::min(target - lo, cum - target) / tot;
      return x;
    }
  }
  if (margin) *margin = 0.0;
  return last_pos;
}

}  // namespace

extern "C" {

// variants (declared ahead of their first use)
enum { DIV_TVD = 0, DIV_JSD = 1 };
static void top_k_filter(std::vector<float>& z, int K);
int oracle_row_distribution_topk(const void* row_c, const void* row_u, int dtype, int has_uncond,
                                 float cfg_scale, float T, int top_k, int V, double* out);
double oracle_jsd_collapsed(double q0, double S);
int oracle_a_set_div(const double* q, int V, const int32_t* nbr_row, int k, double delta, int divergence,
                     double q0, double* moved, double* cut_margin, int* bad_entry);


// ---------------------------------------------------------------------------------------
// Algorithm 2, first block: for every code, its k nearest codes (itself included), stored
// in increasing distance.  R1 fixes the key.  Returns 0, or -1 on bad arguments.
// ---------------------------------------------------------------------------------------
// `rows` (nrows entries) selects which codes to compute; row r of idx / dist then belongs to
// code rows[r].  rows == nullptr computes all V codes in order.
int oracle_build_neighbors_rows(const float* codebook, int V, int D, int k, const int32_t* rows, int nrows,
                                int32_t* idx, float* dist) {
  if (!codebook || !idx || V < 1 || D < 1 || k < 1 || k > V) return -1;
  if (!rows) nrows = V;
  for (size_t e = 0; e < static_cast<size_t>(V) * D; ++e)
    if (!std::isfinite(codebook[e])) return -2;  // distances would not be ordered
  std::vector<float> key(V);
  std::vector<int32_t> order(V);
  for (int r = 0; r < nrows; ++r) {
    const int i = rows ? rows[r] : r;
    if (i < 0 || i >= V) return -1;
    const float* a = codebook + static_cast<size_t>(i) * D;
    for (int j = 0; j < V; ++j) {
      const float* b = codebook + static_cast<size_t>(j) * D;
      float acc = 0.0f;
      for (int d = 0; d < D; ++d) {
        float t = a[d] - b[d];
        acc = std::fmaf(t, t, acc);
      }
      key[j] = acc;
    }
    int n = 0;
    for (int j = 0; j < V; ++j)
      if (j != i) order[n++] = j;
    std::sort(order.begin(), order.begin() + n, [&](int32_t x, int32_t y) {
      if (key[x] != key[y]) return key[x] < key[y];
      return x < y;
    });
    int32_t* row = idx + static_cast<size_t>(r) * k;
    row[0] = i;
    for (int j = 1; j < k; ++j) row[j] = order[j - 1];
    if (dist) {
      float* drow = dist + static_cast<size_t>(r) * k;
      for (int j = 0; j < k; ++j) drow[j] = key[row[j]];
    }
  }
  return 0;
}

// ---------------------------------------------------------------------------------------
// Cosine variant of the latent proximity (Section 5.3.1): every code is scaled to unit length
// and B_k is then built on the scaled codes with the same distance routine -- on unit vectors
// the squared distance is 2 - 2 cos, so the order is that of decreasing cosine similarity.
// Canonical fp32 sequence: squared norm accumulated in dimension order with one fused
// multiply-add per dimension, one square root, one division per component.  A zero code stays
// zero (its similarity to everything is taken as 0).
// ---------------------------------------------------------------------------------------
int oracle_normalize_rows(const float* codebook, int V, int D, float* out) {
  if (!codebook || !out || V < 1 || D < 1) return -1;
  for (int i = 0; i < V; ++i) {
    const float* a = codebook + static_cast<size_t>(i) * D;
    float n2 = 0.0f;
    for (int d = 0; d < D; ++d) n2 = std::fmaf(a[d], a[d], n2);
    const float n = std::sqrt(n2);
    for (int d = 0; d < D; ++d) out[static_cast<size_t>(i) * D + d] = n > 0.0f ? a[d] / n : 0.0f;
  }
  return 0;
}

int oracle_build_neighbors(const float* codebook, int V, int D, int k, int32_t* idx, float* dist) {
  return oracle_build_neighbors_rows(codebook, V, D, k, nullptr, V, idx, dist);
}

// Number of rows whose neighbour order under double-precision distances differs from the
// fp32 order of R1 (a report on how much R1's precision matters; not part of the method).
int64_t oracle_count_order_differences(const float* codebook, int V, int D, int k, const int32_t* idx) {
  int64_t diff = 0;
  std::vector<double> key(V);
  std::vector<int32_t> order(V);
  for (int i = 0; i < V; ++i) {
    for (int j = 0; j < V; ++j) {
      double acc = 0.0;
      for (int d = 0; d < D; ++d) {
        double t = static_cast<double>(codebook[static_cast<size_t>(i) * D + d]) -
                   static_cast<double>(codebook[static_cast<size_t>(j) * D + d]);
        acc += t * t;
      }
      key[j] = acc;
    }
    int n = 0;
    for (int j = 0; j < V; ++j)
      if (j != i) order[n++] = j;
    std::sort(order.begin(), order.begin() + n, [&](int32_t x, int32_t y) {
      if (key[x] != key[y]) return key[x] < key[y];
      return x < y;
    });
    const int32_t* row = idx + static_cast<size_t>(i) * k;
    bool same = row[0] == i;
    for (int j = 1; j < k && same; ++j) same = row[j] == order[j - 1];
    if (!same) ++diff;
  }
  return diff;
}

// ---------------------------------------------------------------------------------------
// Softmax of processed logits for one context row (R2); exported so tests can look at q, p.
// row_c / row_u are the conditional / unconditional rows (row_u ignored unless has_uncond).
// ---------------------------------------------------------------------------------------
int oracle_row_distribution(const void* row_c, const void* row_u, int dtype, int has_uncond,
                            float cfg_scale, float T, int V, double* out) {
  return oracle_row_distribution_topk(row_c, row_u, dtype, has_uncond, cfg_scale, T, 0, V, out);
}

int oracle_row_distribution_topk(const void* row_c, const void* row_u, int dtype, int has_uncond,
                                 float cfg_scale, float T, int top_k, int V, double* out) {
  if (!(T > 0.0f) || V < 1 || top_k < 0) return -1;
  std::vector<float> z(V);
  for (int x = 0; x < V; ++x) {
    float lc = load_logit(row_c, dtype, x);
    float lu = has_uncond ? load_logit(row_u, dtype, x) : 0.0f;
    z[x] = target_z(lc, lu, has_uncond, cfg_scale, T);
  }
  top_k_filter(z, top_k);
  std::vector<double> q;
  if (!softmax(z, q, nullptr)) return -2;
  std::memcpy(out, q.data(), sizeof(double) * V);
  return 0;
}

// ---------------------------------------------------------------------------------------
// Algorithm 2, second block (R3, R4): size of A_{k,delta}(x~) beyond x~ and its moved mass.
// q is a distribution over V tokens; nbr_row = B_k(x~) in increasing distance, slot 0 = x~.
// Returns m = number of neighbours taken (0..k-1); *moved = sum of their q.
// ---------------------------------------------------------------------------------------
int oracle_a_set(const double* q, int V, const int32_t* nbr_row, int k, double delta, double* moved,
                 double* cut_margin, int* bad_entry) {
  return oracle_a_set_div(q, V, nbr_row, k, delta, DIV_TVD, 0.0, moved, cut_margin, bad_entry);
}

// ---------------------------------------------------------------------------------------
// Jensen-Shannon divergence (natural logarithm) between q and q_{k,delta}(.|D = x~) when A
// holds x~ with q(x~) = q0 and further tokens of total mass S (Section 5.3.2 names the
// divergence; the formula is its definition written out on the only tokens where the two
// distributions differ).  With mid = (q + q')/2:
//   a token y of A other than x~ has q' = 0, mid = q(y)/2: it adds q(y) ln 2;
//   x~ has q = q0, q' = q0 + S, mid = q0 + S/2;
//   everywhere else q = q' and the terms vanish.
// The natural logarithm is the base under which the paper's matched pairs agree (Table 3:
// TVD 0.3 <-> JSD 0.2, TVD 0.2 <-> JSD 0.13, and S ln 2 = 0.208, 0.139 for small q0).
// ---------------------------------------------------------------------------------------
double oracle_jsd_collapsed(double q0, double S) {
  const double Q = q0 + S, mid = q0 + 0.5 * S;
  double t = S * std::log(2.0);
  if (q0 > 0.0) t += q0 * std::log(q0 / mid);
  if (Q > 0.0) t += Q * std::log(Q / mid);
  return 0.5 * t;
}

// Algorithm 2's second block with the bound taken on the named divergence: TVD (the moved
// mass, R4) or JSD.  q0 = q(x~) is used by JSD only.  cut_margin is in the divergence's units.
int oracle_a_set_div(const double* q, int V, const int32_t* nbr_row, int k, double delta, int divergence,
                     double q0, double* moved, double* cut_margin, int* bad_entry) {
  auto div = [&](double mass) { return divergence == DIV_JSD ? oracle_jsd_collapsed(q0, mass) : mass; };
  double s = 0.0;
  int m = 0;
  if (bad_entry) *bad_entry = 0;
  for (int j = 1; j < k; ++j) {
    const int32_t n = nbr_row[j];
    double qn = 0.0;
    if (n < 0 || n >= V) {
      if (bad_entry) *bad_entry = 1;  // contributes no mass
    } else {
      qn = q[n];
    }
    if (div(s + qn) < delta) {  // strict bound (R3)
      s += qn;
      m = j;
    } else {
      if (moved) *moved = s;
      if (cut_margin) *cut_margin = std::min(std::fabs(div(s) - delta), std::fabs(div(s + qn) - delta));
      return m;  // break at the first neighbour that does not fit
    }
  }
  if (moved) *moved = s;
  if (cut_margin) *cut_margin = std::fabs(div(s) - delta);
  return m;
}

// ---------------------------------------------------------------------------------------
// Top-k logit filter (Appendix B.2: the generation settings use top-k 1000 / 2000 and top-p
// 1.0, i.e. no nucleus cut): processed logits below the K-th largest become -inf; logits equal
// to it are all kept.  K <= 0 or K >= V leaves the row as it is.  Applied to the target's and the
// drafter's processed logits alike, before the softmax.
// ---------------------------------------------------------------------------------------
static void top_k_filter(std::vector<float>& z, int K) {
  const int V = static_cast<int>(z.size());
  if (K <= 0 || K >= V) return;
  for (float v : z)
    if (v != v) return;  // NaN: the softmax reports the row
  std::vector<float> t(z);
  std::nth_element(t.begin(), t.begin() + (K - 1), t.end(), [](float a, float b) { return a > b; });
  const float kth = t[K - 1];
  for (float& v : z)
    if (v < kth) v = -std::numeric_limits<float>::infinity();
}

// ---------------------------------------------------------------------------------------
// One verification call: Algorithm 1's verification loop with the Section 4.3 rule,
// extended to trees by R6.  All pointers are host pointers.
//
// Layouts: target_logits [C, B, N+1, V] with C = 2 (cond, uncond) if has_uncond else 1;
// draft_logits [B, N+1, V] (already guided); row 0 is the root context, row i+1 the context
// after node i; draft_tokens, tree_parents [B, N] (tree_parents may be null = chain);
// neighbor_idx [V, k]; uniforms [B, N+1] (entry i tests node i, entry N is the final draw).
//
// Outputs [B]: accept_len, next_token, status;  accept_path [B, N] (-1 padded, may be null).
// Trace outputs (each may be null), per node [B, N]:
//   tr_tested  1 if the walk tested the node, else 0
//   tr_qa      sum of the current target over A_{k,delta}(x~)
//   tr_px      current drafter probability of x~
//   tr_m       |A_{k,delta}(x~)| - 1
//   tr_margin  min(|r - qa/px|, cut margin, |W - degenerate_eps| after a rejection)
//              (distance of the node's decisions to flipping)
//   tr_qa_mag  magnitude of the terms qa was formed from: equal to qa for the first child of a
//              context; after sibling rejections the target is a difference (q' - p')/W, and this
//              is the sum over A of the minuend-plus-subtrahend magnitudes carried through the
//              rounds.  A diagnostic for setting a floating-point tolerance, not part of the method.
// per sequence [B]:
//   tr_w       total weight of the last residual (0 if none)
//   tr_draw_margin  margin of the final inverse-CDF draw
// Returns 0 or a negative code for bad arguments.
// ---------------------------------------------------------------------------------------
// oracle_verify_ex adds the variants: `divergence` (DIV_TVD: Section 4.3 as written; DIV_JSD:
// Section 5.3.2's alternative bound), `top_k` (Appendix B.2's logit filter; 0 = none) and
// `degenerate_eps` (R10's threshold on a residual's total weight, in units of the unit mass).
int oracle_verify_ex(const void* target_logits, const void* draft_logits, int dtype, float cfg_scale,
                     int has_uncond, float T, const int32_t* draft_tokens, const int32_t* tree_parents,
                     const int32_t* neighbor_idx, int k, float delta_f, int divergence, int top_k,
                     const float* uniforms, int B, int N, int V, int32_t* out_accept_len,
                     int32_t* out_next_token, int32_t* out_accept_path, int32_t* out_status, uint8_t* tr_tested,
                     double* tr_qa, double* tr_px, int32_t* tr_m, double* tr_margin, double* tr_w,
                     double* tr_draw_margin, double* tr_qa_mag, double degenerate_eps) {
  if (B < 0 || N < 0 || V < 1 || k < 1 || k > V) return -2;
  if (!(T > 0.0f) || !(delta_f >= 0.0f) || !(degenerate_eps >= 0.0)) return -3;
  if ((divergence != DIV_TVD && divergence != DIV_JSD) || top_k < 0) return -3;
  if (B == 0) return 0;
  if (!target_logits || !neighbor_idx || !uniforms || !out_accept_len || !out_next_token) return -1;
  if (N > 0 && (!draft_logits || !draft_tokens)) return -1;
  if (dtype != DT_F32 && dtype != DT_BF16) return -3;

  const double delta = static_cast<double>(delta_f);
  const int R = N + 1;
  const size_t rowsz = static_cast<size_t>(V);
  const size_t branch = static_cast<size_t>(B) * R * rowsz;  // elements per guidance branch

  std::vector<float> z(V);
  std::vector<double> q, q_ctx, p, w(V), mag(V);
  std::vector<std::vector<int>> kids(R);

  for (int b = 0; b < B; ++b) {
    int status = 0;
    int32_t* path = out_accept_path ? out_accept_path + static_cast<size_t>(b) * N : nullptr;
    if (path) std::fill(path, path + N, -1);
    for (int i = 0; i < N; ++i) {
      const size_t o = static_cast<size_t>(b) * N + i;
      if (tr_tested) tr_tested[o] = 0;
      if (tr_qa) tr_qa[o] = 0.0;
      if (tr_px) tr_px[o] = 0.0;
      if (tr_m) tr_m[o] = -1;
      if (tr_margin) tr_margin[o] = std::numeric_limits<double>::infinity();
      if (tr_qa_mag) tr_qa_mag[o] = 0.0;
    }
    if (tr_w) tr_w[b] = 0.0;
    if (tr_draw_margin) tr_draw_margin[b] = std::numeric_limits<double>::infinity();

    // host-checkable data faults of this sequence
    for (auto& v : kids) v.clear();
    for (int i = 0; i < N; ++i) {
      const int32_t tok = draft_tokens[static_cast<size_t>(b) * N + i];
      if (tok < 0 || tok >= V) status |= ST_BAD_TOKEN;
      const int32_t par = tree_parents ? tree_parents[static_cast<size_t>(b) * N + i] : i - 1;
      if (par < -1 || par >= i) status |= ST_BAD_PARENT;
      else kids[par + 1].push_back(i);  // ascending node order by construction
    }
    for (int i = 0; i <= N; ++i) {
      const float r = uniforms[static_cast<size_t>(b) * R + i];
      if (!(r >= 0.0f && r < 1.0f)) status |= ST_BAD_UNIFORM;
    }
    if (status) {
      out_accept_len[b] = 0;
      out_next_token[b] = -1;
      if (out_status) out_status[b] = status;
      continue;
    }

    const double u_final = uniforms[static_cast<size_t>(b) * R + N];
    int cur = 0;  // current context row
    int accept_len = 0;
    int next_token = -1;
    for (;;) {
      const size_t row = (static_cast<size_t>(b) * R + cur) * rowsz;
      // target distribution of the current context (R2)
      for (int x = 0; x < V; ++x) {
        float lc = load_logit(target_logits, dtype, row + x);
        float lu = has_uncond ? load_logit(target_logits, dtype, branch + row + x) : 0.0f;
        z[x] = target_z(lc, lu, has_uncond, cfg_scale, T);
      }
      top_k_filter(z, top_k);
      if (!softmax(z, q, nullptr)) {
        status |= ST_NONFINITE;
        break;
      }
      if (kids[cur].empty()) {
        // Algorithm 1, line after the verification loop: all drafts on the path accepted,
        // draw the extra token from the unmodified target.
        double mg;
        next_token = inverse_cdf(q, u_final, &mg);
        if (tr_draw_margin) tr_draw_margin[b] = mg;
        break;
      }
      for (int x = 0; x < V; ++x) z[x] = load_logit(draft_logits, dtype, row + x) / T;
      top_k_filter(z, top_k);
      if (!softmax(z, p, nullptr)) {
        status |= ST_NONFINITE;
        break;
      }

      int accepted = -1;
      bool degenerate = false;
      q_ctx = q;  // the context's own target, kept for R10
      if (tr_qa_mag) mag.assign(q.begin(), q.end());
      for (int c : kids[cur]) {
        const int32_t xt = draft_tokens[static_cast<size_t>(b) * N + c];
        const double r = uniforms[static_cast<size_t>(b) * R + c];
        const int32_t* nrow = neighbor_idx + static_cast<size_t>(xt) * k;
        // A_{k,delta}(x~) on the current target (R3, R4)
        double moved = 0.0, cut_margin = 0.0;
        int bad = 0;
        const int m = oracle_a_set_div(q.data(), V, nrow, k, delta, divergence, q[xt], &moved, &cut_margin, &bad);
        if (bad) status |= ST_BAD_TABLE;
        const double qa = q[xt] + moved;  // sum over A_{k,delta}(x~), x~ included (R5)
        const double px = p[xt];
        const size_t o = static_cast<size_t>(b) * N + c;
        if (tr_tested) tr_tested[o] = 1;
        if (tr_qa) tr_qa[o] = qa;
        if (tr_px) tr_px[o] = px;
        if (tr_m) tr_m[o] = m;
        if (tr_qa_mag) {
          double g = mag[xt];
          for (int j = 1; j <= m; ++j)
            if (nrow[j] >= 0 && nrow[j] < V) g += mag[nrow[j]];
          tr_qa_mag[o] = g;
        }
        if (tr_margin) {
          double am = px > 0.0 ? std::fabs(r - qa / px) : std::numeric_limits<double>::infinity();
          tr_margin[o] = std::min(am, k > 1 ? cut_margin : std::numeric_limits<double>::infinity());
        }
        // Section 4.3, final rule (R7): accept with probability min(1, qa / px)
        if (r * px < qa) {
          accepted = c;
          break;
        }
        // rejected: relaxed residual [q_{k,delta}(.|D = x~) - p]_+ (Section 4.3)
        for (int x = 0; x < V; ++x) w[x] = q[x];
        w[xt] = qa;
        for (int j = 1; j <= m; ++j) {
          const int32_t n = nrow[j];
          if (n >= 0 && n < V && n != xt) w[n] = 0.0;
        }
        double W = 0.0;
        for (int x = 0; x < V; ++x) {
          w[x] = std::max(0.0, w[x] - p[x]);
          W += w[x];
        }
        if (tr_w) tr_w[b] = W;
        if (tr_margin) tr_margin[o] = std::min(tr_margin[o], std::fabs(W - degenerate_eps));
        if (!(W > degenerate_eps)) {
          // R10.  A rejection of a token the drafter could have produced leaves at least
          // p(x~) - sum_A q of residual mass, so this is reached only through a drafted token
          // outside the drafter's support with target and drafter equal elsewhere, or through
          // two distributions that agree to within the threshold.
          status |= ST_DEGENERATE;
          degenerate = true;
          break;
        }
        if (tr_qa_mag)
          for (int x = 0; x < V; ++x) mag[x] = w[x] > 0.0 ? (mag[x] + p[x]) / W : 0.0;
        for (int x = 0; x < V; ++x) q[x] = w[x] / W;
        // R6: the rejected token leaves the drafter distribution
        p[xt] = 0.0;
        double S = 0.0;
        for (int x = 0; x < V; ++x) S += p[x];
        if (S > 0.0) {
          for (int x = 0; x < V; ++x) p[x] /= S;
        } else {
          std::fill(p.begin(), p.end(), 0.0);
        }
      }
      if (degenerate) {  // R10: no residual to draw from; the context's own target serves
        double mg;
        next_token = inverse_cdf(q_ctx, u_final, &mg);
        if (tr_draw_margin) tr_draw_margin[b] = mg;
        break;
      }
      if (accepted >= 0) {
        if (path) path[accept_len] = accepted;
        ++accept_len;
        cur = accepted + 1;
        continue;
      }
      // every child rejected: the next token comes from the last residual (Algorithm 1, else-branch)
      double mg;
      next_token = inverse_cdf(q, u_final, &mg);
      if (tr_draw_margin) tr_draw_margin[b] = mg;
      break;
    }
    out_accept_len[b] = accept_len;
    out_next_token[b] = next_token;
    if (out_status) out_status[b] = status;
  }
  return 0;
}

// ---------------------------------------------------------------------------------------
// Greedy decoding (Section 4.3, last sentence: accept x~ iff x~ = argmax_x q_{k,delta}(x|D = x~)).
//
// Reading taken (the paper gives no more than that sentence): q is the softmax of the guided
// target logits at temperature 1; A_{k,delta}(x~) is built on it as for sampling; since
// q_{k,delta} puts sum_A q on x~, zero on the rest of A and q elsewhere, x~ is an arg max iff
// sum_A q >= q(x) for every x outside A (ties accept).  Children of a context are tried in node
// order against the same q (there is no residual in greedy decoding); where every child is
// rejected, and where the walk reaches a context without children, the next token is
// argmax_x q(x), smallest index on ties -- after a rejection that is also argmax of
// q_{k,delta}(.|D = x~), because the arg max of q cannot lie inside a rejected A.
// No drafter distribution and no random numbers are involved.
//
// Layouts as in oracle_verify.  Trace outputs per node [B, N] (each may be null): tr_tested,
// tr_qa (sum_A q), tr_m (|A| - 1), tr_margin (min of the cut margin and |sum_A q - max_{x not in A} q|).
// ---------------------------------------------------------------------------------------
int oracle_verify_greedy_ex(const void* target_logits, int dtype, float cfg_scale, int has_uncond,
                            const int32_t* draft_tokens, const int32_t* tree_parents, const int32_t* neighbor_idx,
                            int k, float delta_f, int divergence, int top_k, int B, int N, int V,
                            int32_t* out_accept_len, int32_t* out_next_token, int32_t* out_accept_path,
                            int32_t* out_status, uint8_t* tr_tested, double* tr_qa, int32_t* tr_m,
                            double* tr_margin) {
  if (B < 0 || N < 0 || V < 1 || k < 1 || k > V) return -2;
  if (!(delta_f >= 0.0f)) return -3;
  if ((divergence != DIV_TVD && divergence != DIV_JSD) || top_k < 0) return -3;
  if (B == 0) return 0;
  if (!target_logits || !neighbor_idx || !out_accept_len || !out_next_token) return -1;
  if (N > 0 && !draft_tokens) return -1;
  if (dtype != DT_F32 && dtype != DT_BF16) return -3;
  const double delta = static_cast<double>(delta_f);
  const int R = N + 1;
  const size_t branch = static_cast<size_t>(B) * R * V;
  std::vector<float> z(V);
  std::vector<double> q;
  std::vector<char> inA(V);
  std::vector<std::vector<int>> kids(R);
  for (int b = 0; b < B; ++b) {
    int status = 0;
    int32_t* path = out_accept_path ? out_accept_path + static_cast<size_t>(b) * N : nullptr;
    if (path) std::fill(path, path + N, -1);
    for (int i = 0; i < N; ++i) {
      const size_t o = static_cast<size_t>(b) * N + i;
      if (tr_tested) tr_tested[o] = 0;
      if (tr_qa) tr_qa[o] = 0.0;
      if (tr_m) tr_m[o] = -1;
      if (tr_margin) tr_margin[o] = std::numeric_limits<double>::infinity();
    }
    for (auto& v : kids) v.clear();
    for (int i = 0; i < N; ++i) {
      const int32_t tok = draft_tokens[static_cast<size_t>(b) * N + i];
      if (tok < 0 || tok >= V) status |= ST_BAD_TOKEN;
      const int32_t par = tree_parents ? tree_parents[static_cast<size_t>(b) * N + i] : i - 1;
      if (par < -1 || par >= i) status |= ST_BAD_PARENT;
      else kids[par + 1].push_back(i);
    }
    if (status) {
      out_accept_len[b] = 0;
      out_next_token[b] = -1;
      if (out_status) out_status[b] = status;
      continue;
    }
    int cur = 0, accept_len = 0, next_token = -1;
    for (;;) {
      const size_t row = (static_cast<size_t>(b) * R + cur) * V;
      for (int x = 0; x < V; ++x) {
        float lc = load_logit(target_logits, dtype, row + x);
        float lu = has_uncond ? load_logit(target_logits, dtype, branch + row + x) : 0.0f;
        z[x] = target_z(lc, lu, has_uncond, cfg_scale, 1.0f);
      }
      top_k_filter(z, top_k);
      if (!softmax(z, q, nullptr)) {
        status |= ST_NONFINITE;
        break;
      }
      int best = 0;
      for (int x = 1; x < V; ++x)
        if (q[x] > q[best]) best = x;   // smallest index on ties
      int accepted = -1;
      for (int c : kids[cur]) {
        const int32_t xt = draft_tokens[static_cast<size_t>(b) * N + c];
        const int32_t* nrow = neighbor_idx + static_cast<size_t>(xt) * k;
        double moved = 0.0, cut_margin = 0.0;
        int bad = 0;
        const int m = oracle_a_set_div(q.data(), V, nrow, k, delta, divergence, q[xt], &moved, &cut_margin, &bad);
        if (bad) status |= ST_BAD_TABLE;
        const double qa = q[xt] + moved;
        std::fill(inA.begin(), inA.end(), 0);
        inA[xt] = 1;
        for (int j = 1; j <= m; ++j)
          if (nrow[j] >= 0 && nrow[j] < V) inA[nrow[j]] = 1;
        double outside = -1.0;   // max of q outside A (none: -1, so that x~ is accepted)
        for (int x = 0; x < V; ++x)
          if (!inA[x] && q[x] > outside) outside = q[x];
        const size_t o = static_cast<size_t>(b) * N + c;
        if (tr_tested) tr_tested[o] = 1;
        if (tr_qa) tr_qa[o] = qa;
        if (tr_m) tr_m[o] = m;
        if (tr_margin) tr_margin[o] = std::min(std::fabs(qa - outside), k > 1 ? cut_margin : std::numeric_limits<double>::infinity());
        if (qa >= outside) {   // x~ is an arg max of q_{k,delta}(.|D = x~)
          accepted = c;
          break;
        }
      }
      if (accepted >= 0) {
        if (path) path[accept_len] = accepted;
        ++accept_len;
        cur = accepted + 1;
        continue;
      }
      next_token = best;   // every child rejected, or no child: arg max of the target
      break;
    }
    out_accept_len[b] = accept_len;
    out_next_token[b] = next_token;
    if (out_status) out_status[b] = status;
  }
  return 0;
}

int oracle_verify(const void* target_logits, const void* draft_logits, int dtype, float cfg_scale,
                  int has_uncond, float T, const int32_t* draft_tokens, const int32_t* tree_parents,
                  const int32_t* neighbor_idx, int k, float delta_f, const float* uniforms, int B, int N,
                  int V, int32_t* out_accept_len, int32_t* out_next_token, int32_t* out_accept_path,
                  int32_t* out_status, uint8_t* tr_tested, double* tr_qa, double* tr_px, int32_t* tr_m,
                  double* tr_margin, double* tr_w, double* tr_draw_margin, double* tr_qa_mag) {
  return oracle_verify_ex(target_logits, draft_logits, dtype, cfg_scale, has_uncond, T, draft_tokens, tree_parents,
                          neighbor_idx, k, delta_f, DIV_TVD, 0, uniforms, B, N, V, out_accept_len, out_next_token,
                          out_accept_path, out_status, tr_tested, tr_qa, tr_px, tr_m, tr_margin, tr_w,
                          tr_draw_margin, tr_qa_mag, 1e-5);
}

int oracle_verify_greedy(const void* target_logits, int dtype, float cfg_scale, int has_uncond,
                         const int32_t* draft_tokens, const int32_t* tree_parents, const int32_t* neighbor_idx,
                         int k, float delta_f, int B, int N, int V, int32_t* out_accept_len,
                         int32_t* out_next_token, int32_t* out_accept_path, int32_t* out_status,
                         uint8_t* tr_tested, double* tr_qa, int32_t* tr_m, double* tr_margin) {
  return oracle_verify_greedy_ex(target_logits, dtype, cfg_scale, has_uncond, draft_tokens, tree_parents,
                                 neighbor_idx, k, delta_f, DIV_TVD, 0, B, N, V, out_accept_len, out_next_token,
                                 out_accept_path, out_status, tr_tested, tr_qa, tr_m, tr_margin);
}

// ---------------------------------------------------------------------------------------
// All-token aggregation (not part of the paper's method: a benchmark of the V x k gather-sum
// that building A_{k,delta}(x) for EVERY token x of a row amounts to; the verification step
// only ever needs it for the drafted tokens).  For one context row with distribution q:
//     agg[x] = sum_{y in A_{k,delta}(x)} q(y),   m[x] = |A_{k,delta}(x)| - 1,
// with A_{k,delta}(x) built exactly as in Algorithm 2's second block (oracle_a_set).
// rows_c / rows_u: [rows, V] logits; agg [rows, V] double; m [rows, V] int32 (may be null);
// margin [rows, V] double: distance of each cut to flipping (may be null).
// ---------------------------------------------------------------------------------------
int oracle_aggregate_all(const void* rows_c, const void* rows_u, int dtype, int has_uncond, float cfg_scale,
                         float T, const int32_t* neighbor_idx, int k, float delta_f, int rows, int V, double* agg,
                         int32_t* m_out, double* margin) {
  if (rows < 0 || V < 1 || k < 1 || k > V || !(T > 0.0f) || !(delta_f >= 0.0f)) return -2;
  if (rows == 0) return 0;
  if (!rows_c || !neighbor_idx || !agg || (has_uncond && !rows_u)) return -1;
  const double delta = static_cast<double>(delta_f);
  std::vector<float> z(V);
  std::vector<double> q;
  for (int r = 0; r < rows; ++r) {
    const size_t off = static_cast<size_t>(r) * V;
    for (int x = 0; x < V; ++x) {
      float lc = load_logit(rows_c, dtype, off + x);
      float lu = has_uncond ? load_logit(rows_u, dtype, off + x) : 0.0f;
      z[x] = target_z(lc, lu, has_uncond, cfg_scale, T);
    }
    if (!softmax(z, q, nullptr)) return -4;
    for (int x = 0; x < V; ++x) {
      double moved = 0.0, cm = 0.0;
      const int m = oracle_a_set(q.data(), V, neighbor_idx + static_cast<size_t>(x) * k, k, delta, &moved, &cm, nullptr);
      agg[off + x] = q[x] + moved;
      if (m_out) m_out[off + x] = m;
      if (margin) margin[off + x] = k > 1 ? cm : std::numeric_limits<double>::infinity();
    }
  }
  return 0;
}

}  // extern "C"
