// Bonus draw (Algorithm 1, line after the verification loop): where the walk ends on a context
// without children, the next token is drawn from that context's target distribution by inverse
// CDF at the sequence's last uniform.  Included by verify.cu after verify_greedy.cuh, whose row
// staging helpers it shares.
//
// Persistent CTAs of BNT threads, three to an SM; the context's raw target rows are staged in
// shared memory by bulk copy.  A thread owns Q consecutive quads of four tokens (Q odd: the stride
// between threads then spreads over all banks), so token order is thread order:
//   sweep 1  guidance combine (+ temperature, + top-k mask), maximum M; the processed logits are
//            written back over the raw logits they came from (16 bytes either way) where there
//            are two rows or fp32 logits, so that sweep 2 does not form them again;
//   sweep 2  numerators exp(z - M), one partial sum per quad, the thread's total.
// One block scan of the totals gives Z and the thread in which the cumulative weight first
// exceeds u * Z; that thread finds the quad among its partial sums and re-forms its four
// numerators.  All sums beyond four terms are in double precision.
#pragma once

namespace lantern {

constexpr int BNT = 320;
constexpr int BNW = BNT / 32;
constexpr int BN_ITERS = (16384 / 4 + BNT - 1) / BNT;   // 13: quads per thread of a 16384-token row
static_assert(BN_ITERS % 2 == 1, "the largest quad count per thread is odd");

struct BonusShared {
  double wscan[BNW];                // per-warp running totals of the block scan
  float wm[BNW];
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

  // quads per thread: the smallest odd number that covers the row
  int Q = (quads + BNT - 1) / BNT;
  Q |= 1;
  constexpr bool IN_PLACE = UNC || !BF16;   // 16 bytes of raw logits per quad: room for its four processed logits
  // the four processed logits of quad qd as sweep 1 left them
  auto stored = [&](int qd, float tq) {
    if (!IN_PLACE) return quad(qd, tq);
    if (BF16) {
      const float2 a = *reinterpret_cast<const float2*>(bsm + static_cast<size_t>(qd) * 8);
      const float2 b = *reinterpret_cast<const float2*>(bsm + rowbytes + static_cast<size_t>(qd) * 8);
      return make_float4(a.x, a.y, b.x, b.y);
    }
    return *reinterpret_cast<const float4*>(bsm + static_cast<size_t>(qd) * 16);
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
    const int q0 = tid * Q;                  // this thread's quads: q0 .. q0 + Q - 1, as far as the row goes

    // ---- sweep 1: processed logits (kept in place), maximum ----
    float m = NEG_INF;
    int bad = 0;
    if (ok) {
#pragma unroll
      for (int j = 0; j < BN_ITERS; ++j) {
        const int qd = q0 + j;
        if (j < Q && qd < quads) {
          const float4 z = quad(qd, tq);
          bad |= (z.x != z.x) | (z.y != z.y) | (z.z != z.z) | (z.w != z.w);
          m = fmaxf(fmaxf(m, fmaxf(z.x, z.y)), fmaxf(z.z, z.w));
          if (IN_PLACE) {
            if (BF16) {
              *reinterpret_cast<float2*>(bsm + static_cast<size_t>(qd) * 8) = make_float2(z.x, z.y);
              *reinterpret_cast<float2*>(bsm + rowbytes + static_cast<size_t>(qd) * 8) = make_float2(z.z, z.w);
            } else {
              *reinterpret_cast<float4*>(bsm + static_cast<size_t>(qd) * 16) = z;
            }
          }
        }
      }
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
      // sum per quad, the thread's total ----
      const float L_hi = 1.44269502162933349609375f;
      const uint64_t L2 = pack2(L_hi, L_hi), nM2 = pack2(-(M * L_hi), -(M * L_hi));
      auto numer4 = [&](const float4& z) {
        float a0, a1, a2_, a3;
        unpack2(fma2(pack2(z.x, z.y), L2, nM2), a0, a1);
        unpack2(fma2(pack2(z.z, z.w), L2, nM2), a2_, a3);
        return make_float4(greedy_ex2(a0), greedy_ex2(a1), greedy_ex2(a2_), greedy_ex2(a3));
      };
      float s[BN_ITERS];
      double mine = 0.0;
#pragma unroll
      for (int j = 0; j < BN_ITERS; ++j) {
        const int qd = q0 + j;
        s[j] = 0.0f;
        if (j < Q && qd < quads) {
          const float4 e = numer4(stored(qd, tq));
          s[j] = (e.x + e.y) + (e.z + e.w);
        }
        mine += static_cast<double>(s[j]);
      }
      const double incl = warp_incl_scan(mine, lane);
      if (lane == 31) S.wscan[warp] = incl;
      if (tid == 0) S.tok = -1;
      __syncthreads();
      double excl = incl - mine, Z = 0.0;
#pragma unroll
      for (int w = 0; w < BNW; ++w) {
        const double t = S.wscan[w];
        if (w < warp) excl += t;
        Z += t;
      }
      if (!(Z > 0.0 && Z < 1e300)) {
        st = LANTERN_ST_NONFINITE;
      } else {
        const double target = u * Z;
        if (excl + mine > target && !(excl > target)) {   // the first thread whose inclusive sum exceeds the target
          double cum = excl;
          int jq = -1, jlast = -1;
#pragma unroll
          for (int j = 0; j < BN_ITERS; ++j) {
            if (s[j] > 0.0f) jlast = j;
            if (jq < 0 && cum + static_cast<double>(s[j]) > target) jq = j;
            if (jq < 0) cum += static_cast<double>(s[j]);
          }
          const bool rounded = jq < 0;   // the thread's own rounding: its largest token of positive weight
          if (rounded) jq = jlast;
          if (jq >= 0) {
            const int qd = q0 + jq;
            const float4 e4 = numer4(stored(qd, tq));
            const float e[4] = {e4.x, e4.y, e4.z, e4.w};
            int pick = -1, lastpos = -1;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              cum += static_cast<double>(e[c]);
              if (e[c] > 0.0f) lastpos = c;
              if (pick < 0 && cum > target) pick = c;
            }
            if (rounded || pick < 0) pick = lastpos;   // (the quad's own rounding likewise)
            if (pick >= 0) S.tok = 4 * qd + pick;
          }
        }
        __syncthreads();
        tok = S.tok;
      }
      if (st == 0 && tok < 0) {
        // rounding left no token above the target: the largest token of positive weight
        int last = -1;
#pragma unroll
        for (int j = 0; j < BN_ITERS; ++j) {
          const int qd = q0 + j;
          if (j < Q && qd < quads) {
            const float4 z = stored(qd, tq);
            if (z.x > NEG_INF) last = 4 * qd;
            if (z.y > NEG_INF) last = 4 * qd + 1;
            if (z.z > NEG_INF) last = 4 * qd + 2;
            if (z.w > NEG_INF) last = 4 * qd + 3;
          }
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
