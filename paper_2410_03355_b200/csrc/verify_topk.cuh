// Top-k logit filter (Appendix B.2: top-k 1000 / 2000 with top-p 1): per context row, the
// value of the top_k-th largest processed logit; included by verify.cu.
//
// The verification kernels then treat every processed logit below that value as -inf (logits
// equal to it are all kept).  One CTA of TKT threads per row job; the raw row(s) arrive in shared
// memory by bulk copy, and as soon as they have been turned into order-preserving 32-bit keys in
// registers (64 per thread at V = 16384) the copy of the CTA's next job is started, so that it runs
// under the selection:
//   1. block statistics: number of keys above -inf, smallest such key, largest key;
//   2. bisection on the key interval [lo, hi) with the invariant
//        count(key >= lo) >= K > count(key >= hi),
//      every pass one compare-and-count over the registers and one block reduction; the split
//      point is the key of the arithmetic mean of the two bounds' values while that lies strictly
//      inside (logit values are spread evenly in value, not in bit pattern), else the integer
//      midpoint, so the search ends after at most 64 passes whatever the data;
//   3. as soon as at most TK_LIST keys remain in [lo, hi) they are gathered into shared memory
//      and the wanted one is found by counting ranks.
// -0 is keyed as +0 (they compare equal as logits); NaN is keyed below -inf (such a row is
// reported by the verification kernels anyway).
#pragma once

namespace lantern {

constexpr int TKT = 256;
constexpr int TKW = TKT / 32;
constexpr int TK_CH = 8;            // 8-token chunks per thread: 8 * 8 * 256 = 16384 tokens at most
constexpr int TK_LIST = 128;
constexpr int TK_CE = 16;           // candidate keys per thread after the pre-filter
constexpr int TK_CAND = TK_CE * 256;
constexpr uint32_t TK_KEY_NINF = 0x007fffffu;

struct TopkShared {
  int cnt[2][TKW];
  unsigned kmin[TKW], kmax[TKW];
  __align__(16) unsigned list[TK_LIST];
  unsigned cand[TK_CAND];           // keys that passed the pre-filter
  int list_n;
  unsigned result;
  unsigned long long bar_full;
};

__device__ __forceinline__ uint32_t topk_key(float z) {
  if (z != z) return 0u;
  if (z == 0.0f) z = 0.0f;          // -0 -> +0
  const uint32_t u = __float_as_uint(z);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float topk_value(uint32_t key) {
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// number of this thread's keys >= t, summed over the block (every thread gets the sum)
template <int NE>
__device__ __forceinline__ int topk_count(const uint32_t (&key)[NE], uint32_t t, TopkShared& S, int& flip) {
  int c0 = 0, c1 = 0;   // two chains: the adds do not wait for one another
#pragma unroll
  for (int i = 0; i < NE; i += 2) {
    c0 += key[i] >= t;
    c1 += key[i + 1] >= t;
  }
  const int c = __reduce_add_sync(kFull, c0 + c1);
  if ((threadIdx.x & 31) == 0) S.cnt[flip][threadIdx.x >> 5] = c;
  __syncthreads();
  int tot = 0;
#pragma unroll
  for (int w = 0; w < TKW; ++w) tot += S.cnt[flip][w];
  flip ^= 1;   // the next call writes the other set: a warp still reading this one is at most one barrier behind
  return tot;
}

// processed logits of one row as keys: base row (+ unconditional row at `branch` elements further on)
template <bool BF16, bool UNC>
__device__ __forceinline__ void topk_load_keys(const void* logits, size_t row_elem, size_t branch_elem, int V, float s,
                                               float T, uint32_t (&key)[TK_CH * 8]) {
  const int tid = threadIdx.x;
#pragma unroll
  for (int c = 0; c < TK_CH; ++c) {
    const int g = c * TKT + tid;
    float lc[8], lu[8];
    if (g * 8 < V) {
      if (BF16) {
        const unsigned short* base = static_cast<const unsigned short*>(logits);
        const uint4 x = __ldg(reinterpret_cast<const uint4*>(base + row_elem) + g);
        const uint32_t xw[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          lc[2 * i] = __uint_as_float(xw[i] << 16);
          lc[2 * i + 1] = __uint_as_float(xw[i] & 0xffff0000u);
        }
        if (UNC) {
          const uint4 y = __ldg(reinterpret_cast<const uint4*>(base + branch_elem + row_elem) + g);
          const uint32_t yw[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            lu[2 * i] = __uint_as_float(yw[i] << 16);
            lu[2 * i + 1] = __uint_as_float(yw[i] & 0xffff0000u);
          }
        }
      } else {
        const float* base = static_cast<const float*>(logits);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float4 x = __ldg(reinterpret_cast<const float4*>(base + row_elem) + 2 * g + h);
          lc[4 * h] = x.x, lc[4 * h + 1] = x.y, lc[4 * h + 2] = x.z, lc[4 * h + 3] = x.w;
          if (UNC) {
            const float4 y = __ldg(reinterpret_cast<const float4*>(base + branch_elem + row_elem) + 2 * g + h);
            lu[4 * h] = y.x, lu[4 * h + 1] = y.y, lu[4 * h + 2] = y.z, lu[4 * h + 3] = y.w;
          }
        }
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        float z = UNC ? __fmaf_rn(s, __fsub_rn(lc[e], lu[e]), lu[e]) : lc[e];
        if (T != 1.0f) z = __fdiv_rn(z, T);
        key[c * 8 + e] = topk_key(z);
      }
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) key[c * 8 + e] = 0u;   // padding: below everything
    }
  }
}

// K-th largest of the block's keys, NE per thread (the key of -inf if fewer than K keys lie above -inf)
template <int NE>
__device__ __forceinline__ uint32_t topk_select_keys(const uint32_t (&key)[NE], int K, TopkShared& S) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float NEG_INF = __int_as_float(0xff800000);
  int flip = 0;
  // block statistics
  uint32_t kmin = 0xffffffffu, kmax = 0u;
#pragma unroll
  for (int i = 0; i < NE; ++i) {
    kmax = key[i] > kmax ? key[i] : kmax;
    kmin = (key[i] > TK_KEY_NINF && key[i] < kmin) ? key[i] : kmin;
  }
  kmin = __reduce_min_sync(kFull, kmin);
  kmax = __reduce_max_sync(kFull, kmax);
  if (lane == 0) {
    S.kmin[warp] = kmin;
    S.kmax[warp] = kmax;
  }
  if (tid == 0) S.list_n = 0;
  if (tid < TK_LIST) S.list[tid] = 0u;   // unused slots: below every listed key
  __syncthreads();
#pragma unroll
  for (int w = 0; w < TKW; ++w) {
    kmin = S.kmin[w] < kmin ? S.kmin[w] : kmin;
    kmax = S.kmax[w] > kmax ? S.kmax[w] : kmax;
  }
  // every exit goes through the barrier at the end: the next row reuses S
  uint32_t answer = TK_KEY_NINF;
  bool open = kmax > TK_KEY_NINF;                              // else: nothing above -inf
  uint32_t lo = kmin, hi = kmax;
  int c_lo = 0, c_hi = 0;
  if (open) {
    c_lo = topk_count(key, lo, S, flip);
    open = c_lo >= K;                                          // else the K-th largest is -inf: nothing to cut
  }
  if (open) {
    c_hi = topk_count(key, hi, S, flip);
    if (c_hi >= K) {
      answer = hi;
      open = false;
    }
  }
  if (open) {
    bool ranked = false;
    for (int pass = 0; pass < 64; ++pass) {
      if (hi - lo <= 1u) break;                                // count(>= lo) >= K > count(>= lo + 1)
      if (c_lo - c_hi <= TK_LIST) {
        ranked = true;
        break;
      }
      uint32_t km = topk_key(0.5f * topk_value(lo) + 0.5f * topk_value(hi));
      if (!(km > lo && km < hi)) km = lo + ((hi - lo) >> 1);
      const int c = topk_count(key, km, S, flip);
      if (c >= K) {
        lo = km;
        c_lo = c;
      } else {
        hi = km;
        c_hi = c;
      }
    }
    uint32_t result = lo;
    if (ranked) {
      // the keys in [lo, hi): at most TK_LIST of them; wanted: the r-th largest, r = K - count(>= hi)
      if (tid == 0) S.result = lo;
      // compaction without a chain of atomics: own count, warp scan, one atomic per warp, then the writes
      int mine = 0;
#pragma unroll
      for (int i = 0; i < NE; ++i) mine += (key[i] >= lo) & (key[i] < hi);
      int incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += v;
      }
      int base = 0;
      if (lane == 31) base = atomicAdd(&S.list_n, incl);
      int pos = __shfl_sync(kFull, base, 31) + incl - mine;
      if (mine) {
#pragma unroll
        for (int i = 0; i < NE; ++i) {
          if (key[i] >= lo && key[i] < hi) {
            if (pos < TK_LIST) S.list[pos] = key[i];
            ++pos;
          }
        }
      }
      __syncthreads();
      const int n = S.list_n < TK_LIST ? S.list_n : TK_LIST;
      const int r = K - c_hi;
      if (tid < n) {
        const uint32_t e = S.list[tid];
        int gt = 0, ge = 0;
#pragma unroll 8
        for (int j = 0; j < TK_LIST / 4; ++j) {                // slots past n hold key 0: below every listed key
          const uint4 o = *reinterpret_cast<const uint4*>(&S.list[4 * j]);
          gt += (o.x > e) + (o.y > e) + (o.z > e) + (o.w > e);
          ge += (o.x >= e) + (o.y >= e) + (o.z >= e) + (o.w >= e);
        }
        if (gt < r && r <= ge) S.result = e;                   // equal keys write the same value
      }
      __syncthreads();
      result = S.result;
    }
    answer = result;
  }
  __syncthreads();
  return answer;
}

// Value of the K-th largest of the row's keys (64 per thread).  Rows of at least 4096 tokens first
// go through a pre-filter: a bisection on a 512-key sample (two keys per thread) finds a bound t0
// that, by the sample's ranks, leaves somewhat more than K keys; one pass over all keys counts
// and compacts those >= t0 into shared memory, and the exact selection then runs on at most
// TK_CE keys per thread instead of 64.  If the bound turns out to keep fewer than K keys or more
// than fit (a sample that misleads, many equal keys), the selection runs on all keys instead.
__device__ __forceinline__ float topk_select(const uint32_t (&key)[TK_CH * 8], int K, int V, TopkShared& S) {
  const int tid = threadIdx.x, lane = tid & 31;
  const float mean = static_cast<float>(K) * 512.0f / static_cast<float>(V);   // expected sample rank of the answer
  const int r_lo = static_cast<int>(mean + 3.5f * sqrtf(mean) + 3.0f);
  const int r_hi = r_lo + (r_lo / 6 > 4 ? r_lo / 6 : 4);
  const bool try_filter = V >= 4096 && static_cast<long long>(r_hi + r_lo / 2) * V / 512 < TK_CAND;
  if (try_filter) {
    int flip = 0;
    const uint32_t smp[2] = {key[0], key[32]};
    // the sample's own range (block minimum above -inf and maximum): the search is on values, so it must
    // start from bounds that are as close together as the data are
    uint32_t lo = 0xffffffffu, hi = 0u, t0 = 0u;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      hi = smp[i] > hi ? smp[i] : hi;
      lo = (smp[i] > TK_KEY_NINF && smp[i] < lo) ? smp[i] : lo;
    }
    lo = __reduce_min_sync(kFull, lo);
    hi = __reduce_max_sync(kFull, hi);
    if (lane == 0) {
      S.kmin[tid >> 5] = lo;
      S.kmax[tid >> 5] = hi;
    }
    __syncthreads();
#pragma unroll
    for (int w = 0; w < TKW; ++w) {
      lo = S.kmin[w] < lo ? S.kmin[w] : lo;
      hi = S.kmax[w] > hi ? S.kmax[w] : hi;
    }
    bool found = false;
    for (int pass = 0; pass < 40 && hi - lo > 1u; ++pass) {
      uint32_t km = topk_key(0.5f * topk_value(lo) + 0.5f * topk_value(hi));
      if (!(km > lo && km < hi)) km = lo + ((hi - lo) >> 1);
      const int c = topk_count<2>(smp, km, S, flip);
      if (c > r_hi) {
        lo = km;
      } else if (c < r_lo) {
        hi = km;
      } else {
        t0 = km;
        found = true;
        break;
      }
    }
    if (!found) t0 = lo;   // many equal sample keys: the bound that keeps more
    // count and compact the keys >= t0
    int mine = 0;
#pragma unroll
    for (int i = 0; i < TK_CH * 8; ++i) mine += key[i] >= t0;
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(kFull, incl, o);
      if (lane >= o) incl += v;
    }
    if (tid == 0) S.list_n = 0;
    __syncthreads();
    int base = 0;
    if (lane == 31) base = atomicAdd(&S.list_n, incl);
    int pos = __shfl_sync(kFull, base, 31) + incl - mine;
    __syncthreads();
    const int total = S.list_n;   // uniform
    if (t0 > 0u && total >= K && total <= TK_CAND) {
#pragma unroll
      for (int i = 0; i < TK_CH * 8; ++i) {
        if (key[i] >= t0) S.cand[pos++] = key[i];
      }
      __syncthreads();
      uint32_t ck[TK_CE];
#pragma unroll
      for (int j = 0; j < TK_CE; ++j) {
        const int idx = tid + j * TKT;
        ck[j] = idx < total ? S.cand[idx] : 0u;
      }
      __syncthreads();   // S.list_n is reused by the selection
      return topk_value(topk_select_keys<TK_CE>(ck, K, S));
    }
    __syncthreads();
  }
  return topk_value(topk_select_keys<TK_CH * 8>(key, K, S));
}

// raw row(s) of one job -> shared memory
template <bool BF16, bool UNC>
__device__ __forceinline__ void topk_issue(const VerifyParams& P, int item, bool drafter, unsigned char* stage,
                                           uint32_t rowbytes, unsigned long long* bar) {
  const size_t esize = BF16 ? 2 : 4;
  const size_t row = static_cast<size_t>(item) * P.V * esize;
  uint64_t* b = reinterpret_cast<uint64_t*>(bar);
  if (drafter) {
    mbar_expect_tx(b, rowbytes);
    bulk_load(stage, static_cast<const unsigned char*>(P.draft) + row, rowbytes, b);
  } else {
    const unsigned char* base = static_cast<const unsigned char*>(P.target);
    const size_t branch = static_cast<size_t>(P.B) * P.R * P.V * esize;
    mbar_expect_tx(b, UNC ? 2 * rowbytes : rowbytes);
    bulk_load(stage, base + row, rowbytes, b);
    if (UNC) bulk_load(stage + rowbytes, base + branch + row, rowbytes, b);
  }
}

// staged raw row(s) -> keys of the processed logits
template <bool BF16>
__device__ __forceinline__ void topk_keys_from_stage(const unsigned char* stage, uint32_t rowbytes, bool unc, int V,
                                                     float s, float T, uint32_t (&key)[TK_CH * 8]) {
  const int tid = threadIdx.x;
#pragma unroll
  for (int c = 0; c < TK_CH; ++c) {
    const int g = c * TKT + tid;
    float lc[8], lu[8];
    if (g * 8 < V) {
      if (BF16) {
        const uint4 x = *reinterpret_cast<const uint4*>(stage + static_cast<size_t>(g) * 16);
        const uint32_t xw[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          lc[2 * i] = __uint_as_float(xw[i] << 16);
          lc[2 * i + 1] = __uint_as_float(xw[i] & 0xffff0000u);
        }
        if (unc) {
          const uint4 y = *reinterpret_cast<const uint4*>(stage + rowbytes + static_cast<size_t>(g) * 16);
          const uint32_t yw[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            lu[2 * i] = __uint_as_float(yw[i] << 16);
            lu[2 * i + 1] = __uint_as_float(yw[i] & 0xffff0000u);
          }
        }
      } else {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float4 x = *reinterpret_cast<const float4*>(stage + static_cast<size_t>(g) * 32 + h * 16);
          lc[4 * h] = x.x, lc[4 * h + 1] = x.y, lc[4 * h + 2] = x.z, lc[4 * h + 3] = x.w;
          if (unc) {
            const float4 y = *reinterpret_cast<const float4*>(stage + rowbytes + static_cast<size_t>(g) * 32 + h * 16);
            lu[4 * h] = y.x, lu[4 * h + 1] = y.y, lu[4 * h + 2] = y.z, lu[4 * h + 3] = y.w;
          }
        }
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        float z = unc ? __fmaf_rn(s, __fsub_rn(lc[e], lu[e]), lu[e]) : lc[e];
        if (T != 1.0f) z = __fdiv_rn(z, T);
        key[c * 8 + e] = topk_key(z);
      }
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) key[c * 8 + e] = 0u;   // padding: below everything
    }
  }
}

// mode 0 (after the plan): per context with children, its target rows and -- in sampling -- its
// drafter row, as separate jobs; mode 1 (after the walk): the target rows of the bonus draws.
template <bool BF16, bool UNC>
__global__ void __launch_bounds__(TKT, 2) lantern_topk_kernel(VerifyParams P, int mode) {
  extern __shared__ __align__(128) unsigned char tsm[];
  __shared__ TopkShared S;
  const int tid = threadIdx.x;
  const int V = P.V, R = P.R, K = P.top_k;
  const float T = P.T == 0.0f ? 1.0f : P.T;   // greedy decoding works at temperature 1
  const uint32_t rowbytes = static_cast<uint32_t>(V) * (BF16 ? 2 : 4);
  const bool sampling = P.T != 0.0f;
  const int n_heavy = P.counters->n_heavy;
  const int cap = P.B * P.N;
  const int per = (mode == 0 && sampling) ? 2 : 1;
  const long long njobs = mode == 0 ? static_cast<long long>(n_heavy + P.counters->n_light) * per : P.counters->n_bonus;
  const long long G = gridDim.x;
  auto job_item = [&](long long j) -> int {
    if (mode == 0) {
      const int w = static_cast<int>(j / per);
      return P.work[P.ctx_slots[w < n_heavy ? w : cap - 1 - (w - n_heavy)]].item;
    }
    return P.bonus_seq[j] * R + P.bonus_ctx[j];
  };
  auto job_is_drafter = [&](long long j) { return per == 2 && (j & 1); };
  uint64_t* bar = reinterpret_cast<uint64_t*>(&S.bar_full);

  long long j = blockIdx.x;
  if (tid == 0) {
    mbar_init(bar, 1);
    fence_mbar_init();
    if (j < njobs) topk_issue<BF16, UNC>(P, job_item(j), job_is_drafter(j), tsm, rowbytes, &S.bar_full);
  }
  __syncthreads();
  if (j >= njobs) return;
  int item = job_item(j);
  uint32_t key[TK_CH * 8];
  for (uint32_t it = 0; j < njobs; j += G, ++it) {
    const long long jn = j + G < njobs ? j + G : j;
    const int item_next = job_item(jn);   // consumed after the keys are out: no select on it before
    const bool drafter = job_is_drafter(j);
    const bool landed = __syncthreads_and(mbar_wait(bar, it & 1, P.wait_tries) ? 1 : 0) != 0;
    if (!landed) {   // the copy did not complete within the wait limit: no filter for this row, reported
      if (tid == 0) {
        (drafter ? P.thr_p : P.thr_q)[item] = __int_as_float(0xff800000);
        if (mode == 0) atomicOr(&P.seq_status[item / R], LANTERN_ST_INTERNAL);
        else if (P.out_status) atomicOr(&P.out_status[item / R], LANTERN_ST_INTERNAL);
      }
      break;
    }
    topk_keys_from_stage<BF16>(tsm, rowbytes, UNC && !drafter, V, P.cfg_scale, T, key);
    __syncthreads();   // the staging area is free
    if (tid == 0 && j + G < njobs)
      topk_issue<BF16, UNC>(P, item_next, job_is_drafter(j + G), tsm, rowbytes, &S.bar_full);
    const float t = topk_select(key, K, V, S);
    if (tid == 0) (drafter ? P.thr_p : P.thr_q)[item] = t;
    item = item_next;
  }
}

}  // namespace lantern
