// Greedy-decoding verification (Section 4.3, last sentence: accept x~ iff it is an arg max of
// q_{k,delta}(.|D = x~)); included by verify.cu.
//
// q is the softmax of the guided target logits at temperature 1.  q_{k,delta}(.|D = x~) puts
// sum_A q on x~, zero on the rest of A and q elsewhere, so x~ is an arg max iff
// sum_A q >= max_x q(x) (the maximum over A's own members can never exceed the sum).  There is no
// drafter distribution, no residual and no random number: children of a context are tried in
// node order against the same q, and wherever the walk stops the next token is arg max q
// (smallest index on ties).  Per context with children: one sweep over the staged target rows
// (maximum, arg max, normaliser), then per child the same gather + double-precision prefix scan
// against the strict bound as in sampling.
#pragma once

namespace lantern {

constexpr int GRT = 256;            // threads per CTA
constexpr int GRW = GRT / 32;

struct GreedyShared {
  double wt[GRW];                   // per-warp totals
  double sbefore[GRW];              // prefix sum just before a warp's first failing slot
  float wm[GRW];                    // per-warp maxima
  int wi[GRW];                      // and their smallest arg max
  int first[GRW];
  int bad;                          // NaN met
  int status;
};

// eight processed target logits (guidance combine, T = 1) of 16-byte group g of context row `item`
template <bool BF16, bool UNC>
__device__ __forceinline__ void greedy_chunk(const VerifyParams& P, size_t item, int g, float (&out)[8]) {
  const size_t row = item * static_cast<size_t>(P.V);
  const size_t branch = static_cast<size_t>(P.B) * P.R * P.V;
  float lc[8], lu[8];
  if (BF16) {
    const unsigned short* base = static_cast<const unsigned short*>(P.target);
    const uint4 x = __ldg(reinterpret_cast<const uint4*>(base + row) + g);
    const uint32_t xw[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      lc[2 * i] = __uint_as_float(xw[i] << 16);
      lc[2 * i + 1] = __uint_as_float(xw[i] & 0xffff0000u);
    }
    if (UNC) {
      const uint4 y = __ldg(reinterpret_cast<const uint4*>(base + branch + row) + g);
      const uint32_t yw[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        lu[2 * i] = __uint_as_float(yw[i] << 16);
        lu[2 * i + 1] = __uint_as_float(yw[i] & 0xffff0000u);
      }
    }
  } else {
    const float* base = static_cast<const float*>(P.target);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const float4 x = __ldg(reinterpret_cast<const float4*>(base + row) + 2 * g + h);
      lc[4 * h] = x.x, lc[4 * h + 1] = x.y, lc[4 * h + 2] = x.z, lc[4 * h + 3] = x.w;
      if (UNC) {
        const float4 y = __ldg(reinterpret_cast<const float4*>(base + branch + row) + 2 * g + h);
        lu[4 * h] = y.x, lu[4 * h + 1] = y.y, lu[4 * h + 2] = y.z, lu[4 * h + 3] = y.w;
      }
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) out[e] = UNC ? __fmaf_rn(P.cfg_scale, __fsub_rn(lc[e], lu[e]), lu[e]) : lc[e];
}

// maximum and smallest arg max of a context's processed logits; returns false on NaN / +inf / no finite logit
template <bool BF16, bool UNC>
__device__ __forceinline__ bool greedy_argmax(const VerifyParams& P, size_t item, GreedyShared& S, float& M, int& arg) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float m = __int_as_float(0xff800000);
  int mi = 0x7fffffff;
  int bad = 0;
  for (int g = tid; g * 8 < P.V; g += GRT) {
    float z[8];
    greedy_chunk<BF16, UNC>(P, item, g, z);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      bad |= (z[e] != z[e]);
      if (z[e] > m) {           // ascending index within a thread: strict > keeps the smallest index
        m = z[e];
        mi = g * 8 + e;
      }
    }
  }
  // warp: maximum, then the smallest index among the lanes that hold it
  const float wm = warp_max(m);
  const int wi = __reduce_min_sync(kFull, (m == wm) ? mi : 0x7fffffff);
  if (tid == 0) S.bad = 0;
  __syncthreads();
  if (lane == 0) {
    S.wm[warp] = wm;
    S.wi[warp] = wi;
  }
  if (bad) atomicOr(&S.bad, 1);
  __syncthreads();
  M = S.wm[0];
  arg = S.wi[0];
#pragma unroll
  for (int w = 1; w < GRW; ++w) {
    const float v = S.wm[w];
    const int i = S.wi[w];
    if (v > M || (v == M && i < arg)) {
      M = v;
      arg = i;
    }
  }
  const bool ok = !S.bad && M > __int_as_float(0xff800000) && M < __int_as_float(0x7f800000);
  __syncthreads();
  return ok;
}

// ---------------------------------------------------------------------------------------
// Context kernel: persistent CTAs of GCT threads, three to an SM where the rows allow it, each
// working through its contexts in order.
//
// Greedy decoding needs, of a context's distribution, only its maximum, its arg max, the
// normaliser Z and the numerators of the ~k tokens the children's neighbour rows name.  So the
// raw target rows are staged in shared memory by bulk copy and never rewritten: one sweep reads
// them once (guidance combine, running maximum / arg max, and a running sum of numerators taken
// against the thread's own running maximum and rescaled whenever that maximum moves), a block
// reduction turns the per-thread (maximum, sum) pairs into (M, arg max, Z), and the gather
// recomputes the numerator 2^((z - M) log2 e) of each token it touches from the staged bytes.
// Because nothing is written back, the staging areas of a CTA form a simple ring (one area for
// 16384 bf16 tokens, more for smaller rows); the copies of one CTA run under the arithmetic of
// the other CTAs of its SM.
// ---------------------------------------------------------------------------------------
constexpr int GCT = 320;
constexpr int GCW = GCT / 32;
constexpr int GGT = 256;            // threads that gather: four neighbour slots each per round
constexpr int GGW = GGT / 32;
constexpr int GRING_MAX = 4;
constexpr int GLOOK = 32;           // slots warp 0 looks at per round trip when it has no candidate left (8 and 16 measured slower)
static_assert(GCW <= 32 && GGT < GCT, "one warp combines the per-warp partials; a thread beyond the gatherers solves the JSD bound");

struct GreedyCtxShared {
  double ws[GCW];                   // per-warp sums of numerators relative to the warp's maximum
  double wt[GGW];
  double sbefore[GGW];
  float wm[GCW];
  int wi[GCW];
  int first[GGW];
  int badslot[GGW];                 // per warp: first neighbour slot with an entry outside [0, V)
  double Z;
  float M;
  int arg;
  int flags[2];                     // bit 0: NaN met, bit 1: a copy did not arrive (by iteration parity)
  int status;
  int done, accept;
  double thr;                       // JSD bound only: the current child's mass bound
  unsigned long long bar_full[GRING_MAX];
  WorkItem item[GRING_MAX];         // the context whose rows are on their way into (or sit in) each staging area
  int cursor;                       // next work slot this CTA looks at
};

// a neighbour entry, by an instruction the compiler neither hoists nor merges into a select
__device__ __forceinline__ int ld_nc_s32(const int32_t* p) {
  int v;
  asm volatile("ld.global.nc.s32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}

__device__ __forceinline__ float greedy_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// four processed logits (guidance combine, T = 1) of quad `qd` from the staged raw rows
template <bool BF16, bool UNC>
__device__ __forceinline__ float4 greedy_quad(const unsigned char* area, uint32_t rowbytes, int qd, float s) {
  float4 c, u;
  if (BF16) {
    const uint2 x = *reinterpret_cast<const uint2*>(area + static_cast<size_t>(qd) * 8);
    c = make_float4(__uint_as_float(x.x << 16), __uint_as_float(x.x & 0xffff0000u), __uint_as_float(x.y << 16),
                    __uint_as_float(x.y & 0xffff0000u));
    if (UNC) {
      const uint2 y = *reinterpret_cast<const uint2*>(area + rowbytes + static_cast<size_t>(qd) * 8);
      u = make_float4(__uint_as_float(y.x << 16), __uint_as_float(y.x & 0xffff0000u), __uint_as_float(y.y << 16),
                      __uint_as_float(y.y & 0xffff0000u));
    }
  } else {
    c = *reinterpret_cast<const float4*>(area + static_cast<size_t>(qd) * 16);
    if (UNC) u = *reinterpret_cast<const float4*>(area + rowbytes + static_cast<size_t>(qd) * 16);
  }
  if (UNC) {   // l_u + s (l_c - l_u) on packed pairs: same roundings as the scalar form, half the instructions
    const uint64_t s2 = pack2(s, s);
    const uint64_t u01 = pack2(u.x, u.y), u23 = pack2(u.z, u.w);
    unpack2(fma2(s2, sub2(pack2(c.x, c.y), u01), u01), c.x, c.y);
    unpack2(fma2(s2, sub2(pack2(c.z, c.w), u23), u23), c.z, c.w);
  }
  return c;
}

// the processed logit of one token, by the same operations as greedy_quad
template <bool BF16, bool UNC>
__device__ __forceinline__ float greedy_one(const unsigned char* area, uint32_t rowbytes, int n, float s) {
  float c, u = 0.0f;
  if (BF16) {
    c = __uint_as_float(static_cast<uint32_t>(*reinterpret_cast<const unsigned short*>(area + 2 * static_cast<size_t>(n))) << 16);
    if (UNC)
      u = __uint_as_float(static_cast<uint32_t>(*reinterpret_cast<const unsigned short*>(area + rowbytes + 2 * static_cast<size_t>(n))) << 16);
  } else {
    c = *reinterpret_cast<const float*>(area + 4 * static_cast<size_t>(n));
    if (UNC) u = *reinterpret_cast<const float*>(area + rowbytes + 4 * static_cast<size_t>(n));
  }
  return UNC ? __fmaf_rn(s, __fsub_rn(c, u), u) : c;
}

template <bool BF16, bool UNC>
__device__ __forceinline__ void greedy_issue_rows(const VerifyParams& P, int item, unsigned char* raw, uint32_t rowbytes,
                                                  unsigned long long* bar) {
  const size_t esize = BF16 ? 2 : 4;
  const unsigned char* base = static_cast<const unsigned char*>(P.target);
  const size_t row = static_cast<size_t>(item) * P.V * esize;
  const size_t branch = static_cast<size_t>(P.B) * P.R * P.V * esize;
  mbar_expect_tx(reinterpret_cast<uint64_t*>(bar), UNC ? 2 * rowbytes : rowbytes);
  bulk_load(raw, base + row, rowbytes, reinterpret_cast<uint64_t*>(bar));
  if (UNC) bulk_load(raw + rowbytes, base + branch + row, rowbytes, reinterpret_cast<uint64_t*>(bar));
}

// TOPK: processed logits below the row's top-k threshold (Appendix B.2; written by lantern_topk_kernel)
// count as -inf: they leave Z and carry no mass in a neighbourhood; maximum and arg max are not affected.
template <bool BF16, bool UNC, bool TOPK>
__global__ void __launch_bounds__(GCT, 3) lantern_greedy_context_kernel(VerifyParams P, int ring) {
  extern __shared__ __align__(128) unsigned char gsm[];
  __shared__ GreedyCtxShared S;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int V = P.V, N = P.N, R = P.R, k = P.k;
  const uint32_t rowbytes = static_cast<uint32_t>(V) * (BF16 ? 2 : 4);
  const uint32_t area_bytes = (UNC ? 2 : 1) * rowbytes;   // a multiple of 16: V % 8 == 0
  const float L_hi = 1.44269502162933349609375f;
  const float NEG_INF = __int_as_float(0xff800000);
  const int total = P.counters->n_rank * P.B;   // occupied part of the slot array (breadth-first order per sequence)
  const int quads = V >> 2;
  const int G = gridDim.x;
  int n_eval = 0, n_skip = 0, n_test = 0;       // thread 0: work accounting
  // Warp 0 keeps the staging areas filled.  The CTA walks the slots blockIdx.x, blockIdx.x + G, ... and, as in
  // the sampling pass, leaves out the empty ones and the contexts known to be unreachable (Algorithm 1 stops at
  // the first rejection); a context whose parent is still undecided is evaluated anyway.  The warp looks at 32
  // slots in one round trip (work item and dead mark of each) and keeps the live ones as candidates, one per
  // lane; when an area falls free, the first candidate's dead mark is read once more -- as late as possible --
  // and the candidate is taken or dropped.
  int q_w = -1, q_mark = 0;      // this lane's candidate: its slot and its dead mark's index
  bool q_live = false;
  auto refill = [&](int area) {  // called by all lanes of warp 0
    for (;;) {
      unsigned m = __ballot_sync(kFull, q_live);
      while (m) {
        const int l = __ffs(m) - 1;
        m &= m - 1u;
        const int w = __shfl_sync(kFull, q_w, l), mk = __shfl_sync(kFull, q_mark, l);
        if (lane == l) q_live = false;
        int4 lo = make_int4(0, 0, 0, 0), hi = make_int4(0, 0, 0, 0);
        int dead = 0;
        if (lane == 0) {           // both round trips at once: the mark, and the item in case it is taken
          dead = *reinterpret_cast<const volatile unsigned char*>(P.dead + mk);
          lo = __ldg(reinterpret_cast<const int4*>(P.work + w));
          hi = __ldg(reinterpret_cast<const int4*>(P.work + w) + 1);
        }
        dead = __shfl_sync(kFull, dead, 0);
        if (dead) {
          if (lane == 0) ++n_skip;
          continue;
        }
        if (lane == 0) {
          WorkItem wi;
          wi.item = lo.x, wi.cbase = lo.y, wi.nchild_node0 = lo.z, wi.span0 = lo.w;
          wi.tok0 = hi.x, wi.r0 = __int_as_float(hi.y), wi.u_final = __int_as_float(hi.z), wi.mark = hi.w;
          S.item[area] = wi;
          greedy_issue_rows<BF16, UNC>(P, wi.item, gsm + static_cast<size_t>(area) * area_bytes, rowbytes, &S.bar_full[area]);
          ++n_eval;
        }
        return;
      }
      // no candidate left: the next 32 slots of this CTA
      const int base = S.cursor;
      if (base >= total) {
        if (lane == 0) S.item[area].item = -1;
        return;
      }
      __syncwarp();
      if (lane == 0) S.cursor = base + GLOOK * G;
      const long long wl = static_cast<long long>(base) + static_cast<long long>(lane) * G;
      const bool valid = lane < GLOOK && wl < total;
      q_w = valid ? static_cast<int>(wl) : -1;
      const int item = valid ? __ldg(&P.work[q_w].item) : -1;
      const bool has = item >= 0;
      q_mark = has ? __ldg(&P.work[q_w].mark) : 0;
      const bool dead = has && *reinterpret_cast<const volatile unsigned char*>(P.dead + q_mark) != 0;
      const unsigned gone = __ballot_sync(kFull, dead);
      if (lane == 0) n_skip += __popc(gone);
      q_live = has && !dead;
      __syncwarp();
    }
  };

  if (tid == 0) {
    for (int r = 0; r < ring; ++r) mbar_init(reinterpret_cast<uint64_t*>(&S.bar_full[r]), 1);
    fence_mbar_init();
    S.status = 0;
    S.flags[0] = S.flags[1] = 0;
    S.cursor = blockIdx.x;
  }
  __syncthreads();
  if (warp == 0)
    for (int r = 0; r < ring; ++r) refill(r);
  __syncthreads();

  uint32_t phase = 0;
  int buf = 0;
  for (uint32_t it = 0;; ++it) {
    const WorkItem cur = S.item[buf];
    if (cur.item < 0) break;                    // the areas are refilled in order: an empty one ends the list
    float tq = 0.0f;
    if (TOPK) tq = __ldg(P.thr_q + cur.item);
    // The first child's neighbour entries are consumed much later: issued without any select on their result
    // (clamped indices instead of predicates), so that no instruction waits for them before their use.
    int nb[4];
    if (tid < GGT) {
      const int32_t* nrow0 = P.nbr + static_cast<size_t>(cur.tok0) * k;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int j = 4 * tid + 1 + i;
        nb[i] = __ldg(nrow0 + (j < k ? j : k - 1));   // slots j >= k are masked where they are used
      }
    }
    unsigned char* raw = gsm + static_cast<size_t>(buf) * area_bytes;
    const bool ok = mbar_wait(reinterpret_cast<uint64_t*>(&S.bar_full[buf]), phase, P.wait_tries);

    // ---- the sweep: maximum, smallest arg max, numerators summed against the running maximum ----
    float m = NEG_INF, ssum = 0.0f;
    float mL = 0.0f;   // m * log2(e) once a finite maximum exists (before that every numerator is 2^-inf = 0)
    int mq = -1;   // the quad that first reached the thread's maximum; the position inside it is found afterwards
    auto quad_of = [&](int qd) {
      float4 z = greedy_quad<BF16, UNC>(raw, rowbytes, qd, P.cfg_scale);
      if (TOPK) {   // a NaN stays, to be reported
        z.x = z.x < tq ? NEG_INF : z.x;
        z.y = z.y < tq ? NEG_INF : z.y;
        z.z = z.z < tq ? NEG_INF : z.z;
        z.w = z.w < tq ? NEG_INF : z.w;
      }
      return z;
    };
#pragma unroll 4
    for (int qd = tid; qd < quads; qd += GCT) {
      const float4 z = quad_of(qd);
      const float old = m;
      const float qm = max3(z.x, z.y, fmaxf(z.z, z.w));
      if (qm > m) {                                // ascending quads: strict > keeps the first one
        m = qm, mq = qd, mL = qm * L_hi;
        ssum *= greedy_ex2((old - m) * L_hi);      // old = -inf: the factor is 0, and so was the sum
      }
      float a0, a1, a2_, a3;
      {
        const uint64_t L2 = pack2(L_hi, L_hi), n2 = pack2(-mL, -mL);
        unpack2(fma2(pack2(z.x, z.y), L2, n2), a0, a1);
        unpack2(fma2(pack2(z.z, z.w), L2, n2), a2_, a3);
      }
      ssum += (greedy_ex2(a0) + greedy_ex2(a1)) + (greedy_ex2(a2_) + greedy_ex2(a3));
    }
    // A NaN logit (or +inf, through inf - inf) makes the thread's sum NaN: no per-element test is needed.
    const int bad = ssum != ssum;
    int mi = 0x7fffffff;   // smallest index at which the thread's maximum sits: one quad read again
    if (mq >= 0) {
      const float4 z = quad_of(mq);
      mi = 4 * mq + (z.x == m ? 0 : (z.y == m ? 1 : (z.z == m ? 2 : 3)));
    }
    {
      const float wmx = warp_max(m);
      const int wix = __reduce_min_sync(kFull, (m == wmx) ? mi : 0x7fffffff);
      float f = ssum > 0.0f ? ssum * greedy_ex2(__fmaf_rn(m, L_hi, -(wmx * L_hi))) : 0.0f;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) f += __shfl_xor_sync(kFull, f, o);
      if (lane == 0) {
        S.wm[warp] = wmx;
        S.wi[warp] = wix;
        S.ws[warp] = static_cast<double>(f);
      }
    }
    if (bad || !ok) atomicOr(&S.flags[it & 1], (bad ? 1 : 0) | (ok ? 0 : 2));
    __syncthreads();   // A
    if (warp == 0) {   // lane v combines warp v
      const float v = lane < GCW ? S.wm[lane] : NEG_INF;
      const int i = lane < GCW ? S.wi[lane] : 0x7fffffff;
      const double sv = lane < GCW ? S.ws[lane] : 0.0;
      const float Mx = warp_max(v);
      const int ax = __reduce_min_sync(kFull, (v == Mx) ? i : 0x7fffffff);
      double c = sv > 0.0 ? sv * static_cast<double>(greedy_ex2(__fmaf_rn(v, L_hi, -(Mx * L_hi)))) : 0.0;
      c = warp_sum(c);
      if (lane == 0) {
        S.M = Mx;
        S.arg = ax;
        S.Z = c;
        S.flags[(it + 1) & 1] = 0;   // last read before A of this iteration, next written after B
      }
    }
    __syncthreads();   // B
    const int flags = S.flags[it & 1];
    const float M = S.M;
    const int arg = S.arg;
    const double Z = S.Z;
    if (flags & 2) {   // a copy did not complete within the wait limit: flag the context and stop
      if (tid == 0) {
        Record rec = {-1, -1, LANTERN_ST_INTERNAL, 0};
        P.records[cur.item] = rec;
        // give the copies still on their way to the other staging areas the same bounded wait
        for (int d = 1; d < ring; ++d) {
          const uint32_t j = it + d;
          if (S.item[j % ring].item >= 0)
            mbar_wait(reinterpret_cast<uint64_t*>(&S.bar_full[j % ring]), (j / ring) & 1, P.wait_tries);
        }
      }
      __syncthreads();
      break;
    }
    const bool finite = !(flags & 1) && M > NEG_INF && M < __int_as_float(0x7f800000);
    int accepted = -1, status = 0;
    if (!finite) {
      status = LANTERN_ST_NONFINITE;
    } else {
      const float mL = M * L_hi;
      auto numer = [&](int n) {   // 2^((z_n - M) log2 e) from the staged bytes
        float zn = greedy_one<BF16, UNC>(raw, rowbytes, n, P.cfg_scale);
        if (TOPK) zn = zn < tq ? NEG_INF : zn;
        return greedy_ex2(__fmaf_rn(zn, L_hi, -mL));
      };
      const double thr_tvd = static_cast<double>(P.delta) * Z;   // the bound in units of the unnormalised sums
      const ChildInfo* kids = P.children + cur.cbase;
      for (int ci = 0; ci < (cur.nchild_node0 >> 16) && accepted < 0; ++ci) {
        ++n_test;
        int node = cur.nchild_node0 & 0xffff, xt = cur.tok0;
        if (ci > 0) {
          const int4 info = __ldg(reinterpret_cast<const int4*>(kids + ci));
          node = info.x, xt = info.y;
        }
        const int32_t* nrow = P.nbr + static_cast<size_t>(xt) * k;
        // A_{k,delta}(x~): gather + prefix scan with the strict bound (Algorithm 2, second block)
        double thr = thr_tvd;
        const bool jsd = P.divergence == LANTERN_DIV_JSD;
        if (jsd && tid == GGT)   // Section 5.3.2: the mass whose JSD is delta, from a thread that does not gather
          S.thr = jsd_mass_bound(static_cast<double>(P.delta), static_cast<double>(numer(xt)) / Z) * Z;
        double carry = 0.0;
        for (int base = 0;; base += 4 * GGT) {
          double pre4[4], run = 0.0, incl = 0.0;
          bool val4[4];
          if (tid < GGT) {
            int nn[4];
            int my_bad = kNone;   // first of this thread's slots whose entry lies outside [0, V)
            if (ci == 0 && base == 0) {   // a real branch: the prefetched entries must not wait for a load
#pragma unroll
              for (int i = 0; i < 4; ++i) nn[i] = nb[i];
            } else {
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const int j = base + 4 * tid + 1 + i;
                nn[i] = ld_nc_s32(nrow + (j < k ? j : k - 1));
              }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int j = base + 4 * tid + 1 + i;
              val4[i] = j < k;
              const int n = nn[i];
              const bool inr = val4[i] && static_cast<unsigned>(n) < static_cast<unsigned>(V);
              if (val4[i] && !inr && my_bad == kNone) my_bad = j;   // carries no mass
              run += inr ? static_cast<double>(numer(n)) : 0.0;
              pre4[i] = run;
            }
            incl = warp_incl_scan(run, lane);
            if (lane == 31) S.wt[warp] = incl;
            const int wbad = __reduce_min_sync(kFull, my_bad);
            if (lane == 0) S.badslot[warp] = wbad;
          }
          __syncthreads();
          if (jsd && base == 0) thr = S.thr;
          double tot = 0.0;
          if (tid < GGT) {
            double pre = 0.0;
#pragma unroll
            for (int v = 0; v < GGW; ++v) {
              const double t = S.wt[v];
              if (v < warp) pre += t;
              tot += t;
            }
            const double before = carry + pre + (incl - run);
            int my_first = kNone;
            double my_before = 0.0;
#pragma unroll
            for (int i = 3; i >= 0; --i) {
              if (val4[i] && !(before + pre4[i] < thr)) {
                my_first = base + 4 * tid + 1 + i;
                my_before = i > 0 ? before + pre4[i > 0 ? i - 1 : 0] : before;
              }
            }
            const int wfirst = __reduce_min_sync(kFull, my_first);
            if (wfirst != kNone && my_first == wfirst) {
              S.first[warp] = wfirst;
              S.sbefore[warp] = my_before;
            } else if (wfirst == kNone && lane == 0) {
              S.first[warp] = kNone;
            }
          }
          __syncthreads();
          if (warp == 0) {
            const int f = lane < GGW ? S.first[lane] : kNone;
            const int gfirst = __reduce_min_sync(kFull, f);
            // a bad entry is reported where Algorithm 2's loop meets it, i.e. ahead of the slot that ends the set
            const int gbad = __reduce_min_sync(kFull, lane < GGW ? S.badslot[lane] : kNone);
            if (lane == 0 && gbad < gfirst) S.status |= LANTERN_ST_BAD_TABLE;
            const bool last = base + 4 * GGT >= k - 1;
            if (gfirst != kNone || last) {
              double sm = carry + tot;
              int mcut = k - 1;
              if (gfirst != kNone) {
                const unsigned who = __ballot_sync(kFull, f == gfirst);   // slot indices are distinct: one lane
                sm = S.sbefore[__ffs(who) - 1];
                mcut = gfirst - 1;
              }
              const double qa_un = static_cast<double>(numer(xt)) + sm;
              const double top = static_cast<double>(numer(arg));   // max_x q(x) in the same units
              if (lane == 0) {
                S.done = 1;
                S.accept = qa_un >= top;   // x~ is an arg max of q_{k,delta}(.|D = x~); ties accept
                const size_t o = static_cast<size_t>(cur.item / R) * N + node;
                if (P.out_qa) P.out_qa[o] = static_cast<float>(qa_un / Z);
                if (P.out_px) P.out_px[o] = 0.0f;   // no drafter probability enters greedy decoding
                if (P.out_m) P.out_m[o] = mcut;
              }
            } else if (lane == 0) {
              S.done = 0;
            }
          }
          carry += tot;
          __syncthreads();
          if (S.done) break;
        }
        if (S.accept) accepted = node;
      }
    }
    // Algorithm 1 goes on from the accepted child only: every context behind another child is dead (one
    // contiguous range of marks per child, see the plan kernel)
    {
      const ChildInfo* kids = P.children + cur.cbase;
      const int nchild = cur.nchild_node0 >> 16;
      unsigned char* marks = P.dead + static_cast<size_t>(cur.item / R) * R;
      for (int j = 0; j < nchild; ++j) {
        int node_j = cur.nchild_node0 & 0xffff, span_j = cur.span0;
        if (j > 0) {
          const int4 kid = __ldg(reinterpret_cast<const int4*>(kids + j));
          node_j = kid.x, span_j = kid.w;
        }
        if (node_j != accepted)
          for (int o = tid; o < (span_j & 0xffff); o += GCT) marks[(span_j >> 16) + o] = 1;
      }
    }
    // every thread's reads of this staging area came before the barrier it passed last
    if (tid == 0) {
      Record rec = {accepted, finite ? arg : -1, status | S.status, 0};
      P.records[cur.item] = rec;
      S.status = 0;
    }
    if (warp == 0) refill(buf);
    __syncthreads();   // the area's next context (or the end of the list) is visible to everybody
    if (++buf == ring) {
      buf = 0;
      phase ^= 1;
    }
  }
  if (tid == 0) {
    if (n_eval) atomicAdd(&P.counters->n_evaluated, n_eval);
    if (n_skip) atomicAdd(&P.counters->n_skipped, n_skip);
    if (n_test) atomicAdd(&P.counters->n_tested, n_test);
  }
}

// next token = arg max of the target at the context where the walk ran out of drafts
template <bool BF16, bool UNC>
__global__ void __launch_bounds__(GRT) lantern_greedy_bonus_kernel(VerifyParams P) {
  __shared__ GreedyShared S;
  const int count = P.counters->n_bonus;
  for (int i = blockIdx.x; i < count; i += gridDim.x) {
    const int b = P.bonus_seq[i], ctx = P.bonus_ctx[i];
    float M;
    int arg;
    const bool finite = greedy_argmax<BF16, UNC>(P, static_cast<size_t>(b) * P.R + ctx, S, M, arg);
    if (threadIdx.x == 0) {
      P.out_tok[b] = finite ? arg : -1;
      if (!finite) {
        if (P.out_status) P.out_status[b] |= LANTERN_ST_NONFINITE;
        atomicOr(&P.counters->status_or, LANTERN_ST_NONFINITE);
      }
    }
  }
}

}  // namespace lantern
