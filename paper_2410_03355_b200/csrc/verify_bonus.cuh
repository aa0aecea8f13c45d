// Bonus draw (Algorithm 1, line after the verification loop): where the walk ends on a context
// without children, the next token is drawn from that context's target distribution by inverse
// CDF at the sequence's last uniform.  Included by verify.cu after verify_greedy.cuh, whose row
// staging helpers it shares.
//
// Persistent CTAs of BNT threads, three to an SM; the context's raw target rows are staged in
// shared memory by bulk copy and read twice:
//   sweep 1  guidance combine (+ temperature, + top-k mask), maximum M;
//   sweep 2  numerators exp(z - M); every thread keeps one partial sum per block-wide iteration j
//            (iteration j covers the 4 * BNT consecutive tokens starting at 4 * BNT * j), so that
//            token order is: iteration, then thread, then position in the thread's quad.
// The iteration totals give Z and the iteration in which the cumulative weight first exceeds
// u * Z; a block scan of that iteration's per-thread sums gives the thread, which re-reads its
// four tokens.  All sums beyond four terms are in double precision.
#pragma once

namespace lantern {

constexpr int BNT = 320;
constexpr int BNW = BNT / 32;
constexpr int BN_ITERS = (16384 / 4 + BNT - 1) / BNT;   // 13: iterations of a 16384-token row

struct BonusShared {
  double wj[BNW][BN_ITERS];         // per-warp totals of every iteration
  double wscan[BNW];
  float wm[BNW];
  double Z, base;
  int jstar;
  int tok;
  unsigned long long bar_full;
};

template <bool BF16, bool UNC, bool TOPK>
__global__ void __launch_bounds__(BNT, 3) lantern_bonus_stream_kernel(VerifyParams P) {
  extern __shared__ __align__(128) unsigned char bsm[];
  __shared__ BonusShared S;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int V = P.V, R = P.R, N = P.N;
  const uint32_t rowbytes = static_cast<uint32_t>(V) * (BF16 ? 2 : 4);
  const float NEG_INF = __int_as_float(0xff800000);
  const int quads = V >> 2;
  const int count = P.counters->n_bonus;
  const int G = gridDim.x;
  uint64_t* bar = reinterpret_cast<uint64_t*>(&S.bar_full);
  auto item_of = [&](int i) { return P.bonus_seq[i] * R + P.bonus_ctx[i]; };
  // four processed logits of quad qd of the staged rows
  auto quad = [&](int qd, float tq) {
    float4 z = greedy_quad<BF16, UNC>(bsm, rowbytes, qd, P.cfg_scale);
    if (P.T != 1.0f) {
      z.x = __fdiv_rn(z.x, P.T);
      z.y = __fdiv_rn(z.y, P.T);
      z.z = __fdiv_rn(z.z, P.T);
      z.w = __fdiv_rn(z.w, P.T);
    }
    if (TOPK) {   // below the row's top-k threshold: -inf (a NaN stays, to be reported)
      z.x = z.x < tq ? NEG_INF : z.x;
      z.y = z.y < tq ? NEG_INF : z.y;
      z.z = z.z < tq ? NEG_INF : z.z;
      z.w = z.w < tq ? NEG_INF : z.w;
    }
    return z;
  };

  if (tid == 0) {
    mbar_init(bar, 1);
    fence_mbar_init();
    if (static_cast<int>(blockIdx.x) < count) greedy_issue_rows<BF16, UNC>(P, item_of(blockIdx.x), bsm, rowbytes, &S.bar_full);
  }
  __syncthreads();
  if (static_cast<int>(blockIdx.x) >= count) return;

  uint32_t it = 0;
  for (int i = blockIdx.x; i < count; i += G, ++it) {
    const int b = P.bonus_seq[i];
    const int item = b * R + P.bonus_ctx[i];
    const int i_next = i + G < count ? i + G : i;
    const int item_next = item_of(i_next);   // used when the rows have been read twice: nothing selects on it before
    float tq = 0.0f;
    if (TOPK) tq = __ldg(P.thr_q + item);
    const double u = static_cast<double>(P.uniforms[static_cast<size_t>(b) * R + N]);
    const bool ok = mbar_wait(bar, it & 1, P.wait_tries);

    // ---- sweep 1: maximum ----
    float m = NEG_INF;
    int bad = 0;
    for (int qd = tid; qd < quads; qd += BNT) {
      const float4 z = quad(qd, tq);
      bad |= (z.x != z.x) | (z.y != z.y) | (z.z != z.z) | (z.w != z.w);
      m = fmaxf(fmaxf(m, fmaxf(z.x, z.y)), fmaxf(z.z, z.w));
    }
    m = warp_max(m);
    if (lane == 0) S.wm[warp] = m;
    const bool any_bad = __syncthreads_or(bad) != 0;
    const bool timeout = __syncthreads_or(ok ? 0 : 1) != 0;
    if (timeout) {
      // the copy did not complete within the wait limit: this draw and the CTA's remaining ones are
      // reported instead of made; the late copy gets one more bounded wait before the CTA leaves
      if (tid == 0) {
        for (int j = i; j < count; j += G) {
          const int bj = P.bonus_seq[j];
          P.out_tok[bj] = -1;
          if (P.out_status) P.out_status[bj] |= LANTERN_ST_INTERNAL;
        }
        atomicOr(&P.counters->status_or, LANTERN_ST_INTERNAL);
        mbar_wait(bar, it & 1, P.wait_tries);
      }
      break;
    }
    float M = S.wm[0];
#pragma unroll
    for (int w = 1; w < BNW; ++w) M = fmaxf(M, S.wm[w]);
    const bool finite = !any_bad && M > NEG_INF && M < __int_as_float(0x7f800000);

    int tok = -1, st = 0;
    if (!finite) {
      st = LANTERN_ST_NONFINITE;
      __syncthreads();   // every thread has read S.wm and is done with the rows
    } else {
      // ---- sweep 2: numerators 2^((z - M) log2 e) through the ex2 unit (as in the fused pass), one partial
      // sum per iteration ----
      const float L_hi = 1.44269502162933349609375f;
      const uint64_t L2 = pack2(L_hi, L_hi), nM2 = pack2(-(M * L_hi), -(M * L_hi));
      auto numer4 = [&](const float4& z) {
        float a0, a1, a2_, a3;
        unpack2(fma2(pack2(z.x, z.y), L2, nM2), a0, a1);
        unpack2(fma2(pack2(z.z, z.w), L2, nM2), a2_, a3);
        return make_float4(greedy_ex2(a0), greedy_ex2(a1), greedy_ex2(a2_), greedy_ex2(a3));
      };
      float s[BN_ITERS];
#pragma unroll
      for (int j = 0; j < BN_ITERS; ++j) {
        const int qd = tid + j * BNT;
        s[j] = 0.0f;
        if (qd < quads) {
          const float4 z = quad(qd, tq);
          const float4 e = numer4(z);
          s[j] = (e.x + e.y) + (e.z + e.w);
        }
      }
#pragma unroll
      for (int j = 0; j < BN_ITERS; ++j) {
        const double v = warp_sum(static_cast<double>(s[j]));
        if (lane == 0) S.wj[warp][j] = v;
      }
      __syncthreads();
      if (warp == 0) {   // lane j owns iteration j: its total, the running total, the crossing
        double t = 0.0;
        if (lane < BN_ITERS) {
#pragma unroll
          for (int w = 0; w < BNW; ++w) t += S.wj[w][lane];
        }
        const double incl = warp_incl_scan(t, lane);
        const double Z = __shfl_sync(kFull, incl, 31);
        const double target = u * Z;
        const unsigned over = __ballot_sync(kFull, lane < BN_ITERS && incl > target);
        if (lane == 0) S.Z = Z;
        if (over) {
          const int js = __ffs(over) - 1;
          const double before = __shfl_sync(kFull, incl - t, js);
          if (lane == 0) {
            S.jstar = js;
            S.base = before;
          }
        } else if (lane == 0) {
          S.jstar = -1;
        }
      }
      if (tid == 0) S.tok = -1;
      __syncthreads();
      const double Z = S.Z;
      const int jstar = S.jstar;
      if (!(Z > 0.0 && Z < 1e300)) {
        st = LANTERN_ST_NONFINITE;
      } else if (jstar >= 0) {
        const double target = u * Z;
        float mine = 0.0f;
#pragma unroll
        for (int j = 0; j < BN_ITERS; ++j) mine = j == jstar ? s[j] : mine;
        const double md = static_cast<double>(mine);
        const double incl = warp_incl_scan(md, lane);
        if (lane == 31) S.wscan[warp] = incl;
        __syncthreads();
        double excl = S.base + incl - md;
#pragma unroll
        for (int w = 0; w < BNW; ++w)
          if (w < warp) excl += S.wscan[w];
        if (excl + md > target && !(excl > target)) {   // the first thread whose inclusive sum exceeds the target
          const int qd = tid + jstar * BNT;
          const float4 z = quad(qd, tq);
          const float4 e4 = numer4(z);
          const float e[4] = {e4.x, e4.y, e4.z, e4.w};
          double cum = excl;
          int pick = -1, lastpos = -1;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            cum += static_cast<double>(e[c]);
            if (e[c] > 0.0f) lastpos = c;
            if (pick < 0 && cum > target) pick = c;
          }
          if (pick < 0) pick = lastpos;   // the quad's own rounding: its largest token of positive weight
          S.tok = 4 * qd + pick;
        }
        __syncthreads();
        tok = S.tok;
      }
      if (st == 0 && tok < 0) {
        // rounding left no token above the target: the largest token of positive weight
        int last = -1;
        for (int qd = tid; qd < quads; qd += BNT) {
          const float4 z = quad(qd, tq);
          if (z.x > NEG_INF) last = 4 * qd;
          if (z.y > NEG_INF) last = 4 * qd + 1;
          if (z.z > NEG_INF) last = 4 * qd + 2;
          if (z.w > NEG_INF) last = 4 * qd + 3;
        }
        if (last >= 0) atomicMax(&S.tok, last);
        __syncthreads();
        tok = S.tok;
      }
      __syncthreads();   // S is rewritten by the next row; every thread is done with the staged rows
    }
    if (tid == 0) {
      if (i + G < count) greedy_issue_rows<BF16, UNC>(P, item_next, bsm, rowbytes, &S.bar_full);
      P.out_tok[b] = tok;
      if (st) {
        if (P.out_status) P.out_status[b] |= st;
        atomicOr(&P.counters->status_or, st);
      }
    }
  }
}

}  // namespace lantern
