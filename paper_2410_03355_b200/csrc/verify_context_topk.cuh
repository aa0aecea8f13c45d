// Top-k threshold of one staged row, found by the consumer group that is about to stream the row
// (Appendix B.2: logits below the K-th largest of their row count as -inf; ties at that value are kept).
// Included by verify_context.cuh; used by the TOPK variants of the fused kernel only.
//
// The row sits in shared memory as raw logits; `zchunk(g, z)` turns 16-byte group g into its eight
// processed logits (guidance combine, temperature) with exactly the roundings of the streaming loop.
// Steps, all exact in the end (the sample only decides where to look):
//   1. the group's producer warp, while the group is still busy with the context before, takes a
//      512-value sample spread over the row (from global memory) and finds, by bisection with warp-wide
//      counts, two values (lo, hi) whose sample ranks lie three standard deviations to either side of
//      the rank the K-th largest is expected to have in the sample; they travel with the work item;
//   2. every thread goes over its 64 values once, without a branch: it counts those >= hi and notes
//      down, one byte each, which of its values lie in [lo, hi); the notes of all threads are then
//      gathered into one list (one counter update per warp), so that what follows is evenly spread;
//   3. if the K-th largest does lie in [lo, hi) -- count(>= hi) < K <= count(>= lo) -- the listed values go
//      into a 256-bin histogram over [lo, hi) (a monotone map, so bins are ordered like the values),
//      every warp finds the bin holding the wanted rank by a suffix scan of its own, the values of
//      that bin (a handful) are put side by side, and every warp ranks them with shuffles;
//   4. otherwise (a sample that misleads, more notes than fit, a crowded bin) the value is found by plain
//      bisection on the order-preserving bit patterns, one pass over the row per step: slow, exact,
//      and bounded by 32 passes.  lantern_verify_counts reports how many rows needed it.
#pragma once

namespace lantern {

constexpr int TKG_OWN = 24;         // bracket values a thread can note down (about five are expected)
constexpr int TKG_LIST = 2048;      // bracket values of the whole row
constexpr int TKG_BINS = 256;
constexpr int TKG_TINY = 32;        // values of the wanted bin that one warp can rank
static_assert(TKG_BINS == GT, "every thread of a group clears one bin");

struct GroupTopk {
  // During the pass: code[i * GT + t] = which of its 64 values thread t found inside the bracket as its i-th.
  // Afterwards the same bytes hold, per entry of `list`, the bin its value fell into.
  unsigned char code[TKG_OWN * GT];
  unsigned short list[TKG_LIST];    // (thread << 8) | code of every bracket value, in no particular order
  int hist[2][TKG_BINS];            // [0] serves the drafter row of a context, [1] its target row: a call never
  float tiny[2][TKG_TINY];          //     clears what a slow warp may still be reading from the call before
  int n_tiny[2], n_list[2];
  int wsum[GW][2];
};

// order-preserving bit pattern of a processed logit: NaN lowest, -0 as +0
__device__ __forceinline__ uint32_t tkg_key(float z) {
  if (z != z) return 0u;
  if (z == 0.0f) z = 0.0f;
  const uint32_t u = __float_as_uint(z);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float tkg_value(uint32_t key) {
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// Two values whose ranks among the warp's sample values (16 per lane, NaN = absent) are within `slack` of
// r_hi and r_lo: both searches advance in the same passes.  Where a search finds no such value (equal
// sample values) it ends on the side that widens the bracket.
__device__ __forceinline__ void tkg_sample_bracket(const float (&s)[16], uint32_t kmin, uint32_t kmax, int r_hi, int r_lo,
                                                   int slack, bool want_hi, bool want_lo, float& lo, float& hi) {
  uint32_t Lh = kmin, Hh = kmax + 1u, Ll = kmin, Hl = kmax + 1u;   // count(>= L) = everything, count(>= H) = 0
  bool done_h = !want_hi, done_l = !want_lo;
  for (int pass = 0; pass < 40 && !(done_h && done_l); ++pass) {
    uint32_t ph = tkg_key(0.5f * tkg_value(Lh) + 0.5f * tkg_value(Hh - 1u));
    if (!(ph > Lh && ph < Hh)) ph = Lh + ((Hh - Lh) >> 1);
    uint32_t pl = tkg_key(0.5f * tkg_value(Ll) + 0.5f * tkg_value(Hl - 1u));
    if (!(pl > Ll && pl < Hl)) pl = Ll + ((Hl - Ll) >> 1);
    const float vh = tkg_value(ph), vl = tkg_value(pl);
    int ch0 = 0, ch1 = 0, cl0 = 0, cl1 = 0;
#pragma unroll
    for (int i = 0; i < 16; i += 2) {
      ch0 += s[i] >= vh;
      ch1 += s[i + 1] >= vh;
      cl0 += s[i] >= vl;
      cl1 += s[i + 1] >= vl;
    }
    const int both = __reduce_add_sync(kFull, ((ch0 + ch1) << 16) | (cl0 + cl1));   // 512 values at most: no carry
    const int ch = both >> 16, cl = both & 0xffff;
    if (!done_h) {
      if (ch > r_hi + slack) Lh = ph;
      else if (ch < r_hi - slack) Hh = ph;
      else hi = vh, done_h = true;
      if (!done_h && Hh - Lh <= 1u) hi = tkg_value(Hh), done_h = true;   // fewer above it: a wider bracket
    }
    if (!done_l) {
      if (cl > r_lo + slack) Ll = pl;
      else if (cl < r_lo - slack) Hl = pl;
      else lo = vl, done_l = true;
      if (!done_l && Hl - Ll <= 1u) lo = tkg_value(Ll), done_l = true;   // more above it: a wider bracket
    }
  }
  if (!done_h) hi = tkg_value(Hh);
  if (!done_l) lo = tkg_value(Ll);
}

// sum of two per-thread counts over the group (every thread gets both sums); one group barrier
__device__ __forceinline__ void tkg_group_sum2(GroupTopk& T, int grp, int gw, int lane, int& a, int& b) {
  a = __reduce_add_sync(kFull, a);
  b = __reduce_add_sync(kFull, b);
  gbar(grp);            // the previous readers of wsum are done
  if (lane == 0) {
    T.wsum[gw][0] = a;
    T.wsum[gw][1] = b;
  }
  gbar(grp);
  a = b = 0;
#pragma unroll
  for (int w = 0; w < GW; ++w) {
    a += T.wsum[w][0];
    b += T.wsum[w][1];
  }
}

// Step 4 of the header comment: the K-th largest by bisection on bit patterns, one pass over the row per step.
// Invariant: count(key >= L) >= K > count(key >= H).  If fewer than K values lie above -inf the answer is
// -inf (nothing is cut).
template <class ZF>
__device__ __forceinline__ float tkg_exact_by_passes(ZF& zchunk, int K, int V, int CH, GroupTopk& T, int grp, int gt) {
  const int gw = gt >> 5, lane = gt & 31;
  const uint32_t KNINF = 0x007fffffu;
  uint32_t L = KNINF, H = 0xff800001u;          // -inf .. just above +inf
  {
    int c = 0, dummy = 0;
    for (int ch = 0; ch < CH; ++ch) {
      const int g = ch * GT + gt;
      if (g * 8 < V) {
        float z[8];
        zchunk(g, z);
#pragma unroll
        for (int e = 0; e < 8; ++e) c += tkg_key(z[e]) > KNINF;
      }
    }
    tkg_group_sum2(T, grp, gw, lane, c, dummy);
    if (c < K) return __int_as_float(0xff800000);
    L = KNINF + 1u;
  }
  for (int pass = 0; pass < 34 && H - L > 1u; ++pass) {
    const uint32_t p = L + ((H - L) >> 1);
    int c = 0, dummy = 0;
    for (int ch = 0; ch < CH; ++ch) {
      const int g = ch * GT + gt;
      if (g * 8 < V) {
        float z[8];
        zchunk(g, z);
#pragma unroll
        for (int e = 0; e < 8; ++e) c += tkg_key(z[e]) >= p;
      }
    }
    tkg_group_sum2(T, grp, gw, lane, c, dummy);
    if (c >= K) L = p;
    else H = p;
  }
  return tkg_value(L);
}

// Step 1 of the header comment, run by one warp (all 32 lanes call it and get the same values): the
// bracket of a row from a 512-value sample.  `zchunk(g, z)` gives the eight processed logits of 16-byte
// group g, from wherever the caller keeps the row.  out = {lo, hi, base, scale}.
template <class ZF>
__device__ __forceinline__ void tkg_warp_bracket(ZF& zchunk, int K, int V, int lane, float (&out)[4]) {
  const float qnan = __int_as_float(0x7fc00000);
  const float pinf = __int_as_float(0x7f800000), ninf = __int_as_float(0xff800000);
  const int groups = V >> 3;
  const int take = groups < 64 ? groups : 64;            // sampled 16-byte groups, spread evenly
  float s[16];
  uint32_t kmin = 0xffffffffu, kmax = 0u;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int j = lane + 32 * h;
    float z[8];
    if (j < take) zchunk(j * groups / take, z);           // j < 64 and groups <= 2048: no overflow
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float v = j < take ? z[e] : qnan;
      s[8 * h + e] = v;
      const uint32_t kk = tkg_key(v);
      if (kk > 0x007fffffu) {                             // above -inf
        kmin = kk < kmin ? kk : kmin;
        kmax = kk > kmax ? kk : kmax;
      }
    }
  }
  kmin = __reduce_min_sync(kFull, kmin);
  kmax = __reduce_max_sync(kFull, kmax);
  float lo = ninf, hi = pinf, base = 0.0f, scale = 0.0f;
  if (kmax >= kmin) {                                     // the sample holds a finite value
    const float ns = static_cast<float>(take * 8);
    const float mean = static_cast<float>(K) * ns / static_cast<float>(V);
    const float sd = sqrtf(mean * (1.0f - static_cast<float>(K) / static_cast<float>(V)));
    const int slack = static_cast<int>(0.25f * sd) + 1;
    const int r_hi = static_cast<int>(mean - 3.0f * sd) - slack - 1;
    const int r_lo = static_cast<int>(mean + 3.0f * sd) + slack + 2;
    tkg_sample_bracket(s, kmin, kmax, r_hi, r_lo, slack, r_hi > slack, r_lo < static_cast<int>(ns) - slack, lo, hi);
    // bins: over [lo, hi) where both are finite, else over the sample's own range (values beyond it are clamped)
    const float b0 = lo > ninf ? lo : tkg_value(kmin), b1 = hi < pinf ? hi : tkg_value(kmax);
    base = b0;
    scale = b1 > b0 ? static_cast<float>(TKG_BINS) / (b1 - b0) : 0.0f;
  }
  out[0] = lo, out[1] = hi, out[2] = base, out[3] = scale;
}

// Steps 2-4: the K-th largest processed logit of the row behind `zchunk` (0 < K < V), given the bracket
// br = {lo, hi, base, scale}; every thread of the group calls it and gets the same value.  CH = 16-byte
// groups per thread.  `which` = 0 for a context's drafter row, 1 for its target row (see GroupTopk).  The
// histogram and the list counter of `which` are zero on entry and left zero on exit.
template <class ZF>
__device__ __forceinline__ float tkg_kth_largest(ZF& zchunk, const float (&br)[4], int K, int V, int CH, GroupTopk& T,
                                                 int which, int grp, int gt, int* slow_count) {
  const int gw = gt >> 5, lane = gt & 31;
  if (gt == 0) T.n_tiny[which] = 0;                       // next touched behind two group barriers
  const float lo = br[0], hi = br[1], base = br[2], scale = br[3];
  auto bin_of = [&](float v) {
    const float x = (v - base) * scale;
    return x < 0.0f ? 0 : (x >= static_cast<float>(TKG_BINS) ? TKG_BINS - 1 : static_cast<int>(x));
  };
  // the value behind a list entry, recomputed from the staged row
  auto value_of = [&](int entry) {
    float z[8];
    zchunk(((entry >> 3) & 7) * GT + (entry >> 8), z);
    const int e = entry & 7;
    const float a0 = (e & 1) ? z[1] : z[0], a1 = (e & 1) ? z[3] : z[2], a2 = (e & 1) ? z[5] : z[4], a3 = (e & 1) ? z[7] : z[6];
    const float b0 = (e & 2) ? a1 : a0, b1 = (e & 2) ? a3 : a2;
    return (e & 4) ? b1 : b0;
  };
  // ---- 2. one pass, thread-local and free of branches: count the values >= hi, note those in [lo, hi) ----
  int c_hi = 0, n_in = 0;
  for (int ch = 0; ch < CH; ++ch) {
    const int g = ch * GT + gt;
    if (g * 8 < V) {
      float z[8];
      zchunk(g, z);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float v = z[e];
        c_hi += v >= hi;
        const bool in = v >= lo && v < hi;
        if (in) T.code[(n_in < TKG_OWN ? n_in : TKG_OWN - 1) * GT + gt] = static_cast<unsigned char>(ch * 8 + e);
        n_in += in;
      }
    }
  }
  // the notes of all threads as one list (one counter update per warp), so that the next steps are balanced
  const int n_own = n_in < TKG_OWN ? n_in : TKG_OWN;
  {
    int incl = n_own;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(kFull, incl, o);
      if (lane >= o) incl += v;
    }
    int start = 0;
    if (lane == 31) start = atomicAdd(&T.n_list[which], incl);
    const int pos = __shfl_sync(kFull, start, 31) + incl - n_own;
    for (int i = 0; i < n_own; ++i)
      if (pos + i < TKG_LIST) T.list[pos + i] = static_cast<unsigned short>((gt << 8) | T.code[i * GT + gt]);
  }
  int c_in = n_in + (n_in > TKG_OWN ? (1 << 20) : 0);     // bit 20 and up: threads whose notes overflowed
  tkg_group_sum2(T, grp, gw, lane, c_hi, c_in);           // its barriers also publish the list
  const bool overflow = (c_in >> 20) != 0 || (c_in & 0xfffff) > TKG_LIST;   // (no overflowing thread: c_in = listed values)
  c_in &= 0xfffff;
  if (gt == 0) T.n_list[which] = 0;                       // everybody has read it (the sum above went through two barriers)
  if (overflow || !(c_hi < K && K <= c_hi + c_in)) {
    if (gt == 0) atomicAdd(slow_count, 1);
    return tkg_exact_by_passes(zchunk, K, V, CH, T, grp, gt);
  }
  // ---- 3. histogram of the bracket values; the bin that holds rank K - c_hi counted from the top ----
  for (int i = gt; i < c_in; i += GT) {
    const int b = bin_of(value_of(T.list[i]));
    T.code[i] = static_cast<unsigned char>(b);            // (the per-thread notes are no longer needed)
    atomicAdd(&T.hist[which][b], 1);
  }
  gbar(grp);
  int bin, rank;
  {                                                       // every warp for itself: no barrier to publish the result
    const int* h = T.hist[which] + lane * (TKG_BINS / 32);
    int mine = 0;
#pragma unroll
    for (int i = 0; i < TKG_BINS / 32; ++i) mine += h[i];
    int suffix = mine;                                    // inclusive suffix sum over the lanes
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_down_sync(kFull, suffix, o);
      if (lane + o < 32) suffix += v;
    }
    const int above = suffix - mine;                      // values in the bins of higher lanes
    const int want = K - c_hi;                            // 1 <= want <= c_in
    const bool here = above < want && want <= above + mine;
    int b = TKG_BINS / 32 - 1, acc = above;
    if (here) {
      for (; b > 0; --b) {
        if (acc + h[b] >= want) break;
        acc += h[b];
      }
    }
    const int src = __ffs(__ballot_sync(kFull, here)) - 1;   // exactly one lane holds the rank
    bin = __shfl_sync(kFull, lane * (TKG_BINS / 32) + b, src);
    rank = __shfl_sync(kFull, want - acc, src);           // rank inside that bin, from its top
  }
  // the values of that bin, for one warp to rank
  for (int i = gt; i < c_in; i += GT) {
    if (T.code[i] == bin) {
      const int pos = atomicAdd(&T.n_tiny[which], 1);
      if (pos < TKG_TINY) T.tiny[which][pos] = value_of(T.list[i]);
    }
  }
  gbar(grp);
  T.hist[which][gt] = 0;                                  // nobody reads the histogram past this barrier
  const int n_tiny = T.n_tiny[which];
  if (n_tiny > TKG_TINY) {                                // a crowded bin (many equal values)
    if (gt == 0) atomicAdd(slow_count, 1);
    return tkg_exact_by_passes(zchunk, K, V, CH, T, grp, gt);
  }
  // lane l holds the bin's l-th value; the wanted one has fewer than `rank` values above it and at least
  // `rank` values not below it (equal values give the same answer)
  const float mine_v = lane < n_tiny ? T.tiny[which][lane] : __int_as_float(0xff800000);
  int gtr = 0, geq = 0;
  for (int j = 0; j < n_tiny; ++j) {                      // (a handful; the bound is the same for every thread)
    const float o = __shfl_sync(kFull, mine_v, j);
    gtr += o > mine_v ? 1 : 0;
    geq += o >= mine_v ? 1 : 0;
  }
  const unsigned hit = __ballot_sync(kFull, lane < n_tiny && gtr < rank && rank <= geq);
  if (hit == 0u) {                                        // cannot happen with a consistent histogram
    if (gt == 0) atomicAdd(slow_count, 1);
    return tkg_exact_by_passes(zchunk, K, V, CH, T, grp, gt);
  }
  return __shfl_sync(kFull, mine_v, __ffs(hit) - 1);
}

}  // namespace lantern
