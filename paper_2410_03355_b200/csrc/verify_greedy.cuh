// Greedy-decoding verification (Section 4.3, last sentence: accept x~ iff it is an arg max of
// q_{k,delta}(.|D = x~)); included by verify.cu.
//
// q is the softmax of the guided target logits at temperature 1.  q_{k,delta}(.|D = x~) puts
// sum_A q on x~, zero on the rest of A and q elsewhere, so x~ is an arg max iff
// sum_A q >= max_x q(x) (the maximum over A's own members can never exceed the sum).  There is no
// drafter distribution, no residual and no random number: children of a context are tried in
// node order against the same q, and wherever the walk stops the next token is arg max q
// (smallest index on ties).  One CTA per context with children: two sweeps over the context's
// two target rows (maximum and arg max; numerators into shared memory and their sum), then per
// child the same gather + double-precision prefix scan against the strict bound as in sampling.
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

template <bool BF16, bool UNC>
__global__ void __launch_bounds__(GRT) lantern_greedy_context_kernel(VerifyParams P) {
  extern __shared__ __align__(16) float Eg[];   // numerators 2^((z - M) log2 e), plain token order
  __shared__ GreedyShared S;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int V = P.V, N = P.N, R = P.R, k = P.k;
  const float L_hi = 1.44269502162933349609375f;
  const int n_heavy = P.counters->n_heavy;
  const int total = n_heavy + P.counters->n_light;
  const int cap = P.B * N;

  for (int w = blockIdx.x; w < total; w += gridDim.x) {
    const WorkItem cur = P.work[w < n_heavy ? w : cap - 1 - (w - n_heavy)];
    const size_t item = static_cast<size_t>(cur.item);
    const int b = cur.item / R;
    const ChildInfo* kids = P.children + cur.cbase;
    if (tid == 0) S.status = 0;

    float M;
    int arg;
    const bool finite = greedy_argmax<BF16, UNC>(P, item, S, M, arg);   // barriers inside
    int accepted = -1, status = 0;
    if (!finite) {
      status = LANTERN_ST_NONFINITE;
    } else {
      // numerators and their sum
      const float mL = M * L_hi;
      float part = 0.0f;
      for (int g = tid; g * 8 < V; g += GRT) {
        float z[8];
        greedy_chunk<BF16, UNC>(P, item, g, z);
#pragma unroll
        for (int e = 0; e < 8; ++e) z[e] = ex2_approx(__fmaf_rn(z[e], L_hi, -mL));
        part += sum8(z);
        *reinterpret_cast<float4*>(Eg + g * 8) = make_float4(z[0], z[1], z[2], z[3]);
        *reinterpret_cast<float4*>(Eg + g * 8 + 4) = make_float4(z[4], z[5], z[6], z[7]);
      }
      double Z = warp_sum(static_cast<double>(part));
      if (lane == 0) S.wt[warp] = Z;
      __syncthreads();
      Z = 0.0;
#pragma unroll
      for (int v = 0; v < GRW; ++v) Z += S.wt[v];
      __syncthreads();
      const double thr = static_cast<double>(P.delta) * Z;   // the bound in units of the unnormalised sums
      const double top = static_cast<double>(Eg[arg]);        // max_x q(x) in the same units

      for (int ci = 0; ci < cur.nchild && accepted < 0; ++ci) {
        const int4 info = __ldg(reinterpret_cast<const int4*>(kids + ci));
        const int node = info.x, xt = info.y;
        const int32_t* nrow = P.nbr + static_cast<size_t>(xt) * k;
        // A_{k,delta}(x~): gather + prefix scan with the strict bound (Algorithm 2, second block)
        double carry = 0.0, sm = 0.0;
        int m = k - 1;
        bool cut = false;
        for (int base = 0; base < k - 1 && !cut; base += 4 * GRT) {
          double pre4[4];
          bool val4[4];
          double run = 0.0;
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int j = base + 4 * tid + 1 + i;
            val4[i] = j < k;
            const int n = val4[i] ? __ldg(nrow + j) : -1;
            const bool inr = val4[i] && static_cast<unsigned>(n) < static_cast<unsigned>(V);
            if (val4[i] && !inr) atomicOr(&S.status, LANTERN_ST_BAD_TABLE);   // carries no mass
            run += inr ? static_cast<double>(Eg[n]) : 0.0;
            pre4[i] = run;
          }
          const double incl = warp_incl_scan(run, lane);
          if (lane == 31) S.wt[warp] = incl;
          __syncthreads();
          double pre = 0.0, tot = 0.0;
#pragma unroll
          for (int v = 0; v < GRW; ++v) {
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
          __syncthreads();
          int gfirst = kNone, src = 0;
#pragma unroll
          for (int v = GRW - 1; v >= 0; --v) {
            const int f = S.first[v];
            if (f != kNone && f <= gfirst) {
              gfirst = f;
              src = v;
            }
          }
          if (gfirst != kNone) {
            m = gfirst - 1;
            sm = S.sbefore[src];
            cut = true;
          } else {
            carry += tot;
            sm = carry;
          }
          __syncthreads();   // S.wt / S.first are rewritten by the next round or the next child
        }
        const double qa_un = static_cast<double>(Eg[xt]) + sm;
        const bool accept = qa_un >= top;   // x~ is an arg max of q_{k,delta}(.|D = x~); ties accept
        if (tid == 0) {
          const size_t o = static_cast<size_t>(b) * N + node;
          if (P.out_qa) P.out_qa[o] = static_cast<float>(qa_un / Z);
          if (P.out_px) P.out_px[o] = 0.0f;   // no drafter probability enters greedy decoding
          if (P.out_m) P.out_m[o] = m;
        }
        if (accept) accepted = node;
      }
    }
    __syncthreads();   // every status bit is in; Eg is free for the next context
    if (tid == 0) {
      Record rec = {accepted, finite ? arg : -1, status | S.status, 0};
      P.records[item] = rec;
    }
    __syncthreads();
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
      if (!finite && P.out_status) P.out_status[b] |= LANTERN_ST_NONFINITE;
    }
  }
}

}  // namespace lantern
