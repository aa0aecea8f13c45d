// Fused context pass of the LANTERN verification step (included by verify.cu).
//
// Persistent kernel, one CTA per SM: 16 consumer warps and one producer warp, two staging areas
// in shared memory.  The producer hands out contexts and issues bulk asynchronous copies (TMA,
// completion on an mbarrier, no multicast) that bring the NEXT context's rows into one area for
// the whole time the consumers work on the current context in the other, so HBM streams
// continuously and no consumer ever waits on a global round trip of the work queue.  The current context's softmax numerators E are stored over its
// own raw rows once those have been read into registers: every thread overwrites only bytes
// that it alone has read, so this needs no barrier and no third buffer.
//
// Each warp streams its slice of the rows on its own: guidance combine, the warp's own maximum,
// numerators 2^((z - max_w) log2 e) through the hardware ex2 unit, partial sums.  One block
// barrier later every warp has all warps' (maximum, sum) pairs and rescales on the fly: the
// numerators in shared memory stay in their warp's own units and carry a per-warp factor.
// Sums over many numerators average the ex2 unit's ~1e-7 rounding out; the two single
// probabilities that decide a chain position, q(x~) and p(x~), are recomputed by one thread in
// double precision from the raw logits.
//
// Per child (Section 4.3 / Algorithm 2, second block): gather of the neighbour row's
// numerators, double-precision block scan with the strict bound, accept test; on rejection the
// residual [q_{k,delta}(.|D = x~) - p]_+ in one register pass, its total, and either the
// inverse-CDF draw or the write-back for the next sibling.
#pragma once

#define LANTERN_CONTEXT_KERNEL_REVISION 5   // bump on every change to this file

namespace lantern {

constexpr int CNT = 512;        // threads per CTA
constexpr int CNW = CNT / 32;   // warps per CTA
constexpr int LOG_CNT = 9;
constexpr int kNone = 0x7fffffff;

// Thread t owns, for chunk c, the eight consecutive tokens [(c*CNT + t)*8, +8), i.e. 16-byte group
// g = c*CNT + t of a bf16 row.  E is laid over the context's own raw rows: with bf16 logits the low
// four numerators of group g replace group g of the first row and the high four replace group g of
// the second row; with fp32 logits the eight numerators replace the group's own 32 bytes of the
// first row.  Float index of token x inside the staging area:
template <bool BF16>
__device__ __forceinline__ int ephys(int x, int row_floats) {
  if (BF16) return ((x >> 2) & 1) * row_floats + ((x >> 3) << 2) + (x & 3);
  return x;
}
__device__ __forceinline__ int cowner_thread(int x) { return (x >> 3) & (CNT - 1); }

struct CtxShared {
  double sq[CNW], sp[CNW];      // per-warp sums of numerators, in the warp's own units
  double wt[4 * CNW];           // per-(chunk, warp) totals for scans and block sums
  double sbefore[CNW];          // prefix sum just before a warp's first failing neighbour
  double acc_e, acc_p;          // double-precision numerators of the tested x~, global units
  double hist[32];              // drafter/target scale ratio of each earlier rejection round of this context
  int acc_valid;                // acc_e / acc_p are usable for the current child
  float mlq[CNW], mlp[CNW];     // per-warp shift constants fl(max_w * log2 e)
  int first[CNW];               // a warp's first failing neighbour slot
  int cand[CNW];
  int tok;
  int status;                   // OR of status bits seen by single threads
  WorkItem work[2];
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 2^(z log2(e) - shift) for one value, to about 1.5e-7: the exponent is formed in double precision,
// split into an fp32 head for the ex2 unit and a tail that is applied to first order.
__device__ __forceinline__ double exp2_single(float z, float shift) {
  const double x = static_cast<double>(z) * 1.4426950408889634074 - static_cast<double>(shift);
  const float xh = static_cast<float>(x);
  const float xl = static_cast<float>(x - static_cast<double>(xh));
  const float y = ex2_approx(xh);
  return static_cast<double>(__fmaf_rn(y, xl * 0.693147182464599609375f, y));
}

template <bool BF16, bool UNC>
__device__ __forceinline__ void ctx_issue_rows(const VerifyParams& P, int item, unsigned char* stage, int rowbytes,
                                               uint64_t* bar) {
  const int nrows = UNC ? 3 : 2;
  mbar_expect_tx(bar, static_cast<uint32_t>(nrows * rowbytes));
  const size_t row_off = static_cast<size_t>(item) * rowbytes;
  const size_t branch = static_cast<size_t>(P.B) * P.R * rowbytes;
  const unsigned char* src[3];
  src[0] = static_cast<const unsigned char*>(P.target) + row_off;
  src[1] = UNC ? static_cast<const unsigned char*>(P.target) + branch + row_off
               : static_cast<const unsigned char*>(P.draft) + row_off;
  src[2] = static_cast<const unsigned char*>(P.draft) + row_off;
  for (int r = 0; r < nrows; ++r) {
    const int dst_row = (r == nrows - 1) ? 2 : r;   // the drafter row always goes to row slot 2
    for (int off = 0; off < rowbytes; off += 16384) {
      const int n = min(16384, rowbytes - off);
      bulk_load(stage + dst_row * rowbytes + off, src[r] + off, static_cast<uint32_t>(n), bar);
    }
  }
}

// one logit of a row in global memory, widened to fp32
template <bool BF16>
__device__ __forceinline__ float ctx_raw_logit(const void* base, size_t elem) {
  if (BF16) return __uint_as_float(static_cast<uint32_t>(__ldg(static_cast<const unsigned short*>(base) + elem)) << 16);
  return __ldg(static_cast<const float*>(base) + elem);
}

constexpr int CTX_THREADS = CNT + 32;   // 16 consumer warps and one producer warp

// barrier among the 512 consumer threads only (the producer warp never joins it)
__device__ __forceinline__ void cbar() { asm volatile("bar.sync 1, %0;" ::"n"(CNT) : "memory"); }
// the same barrier, returning the AND of every consumer thread's predicate
__device__ __forceinline__ bool cbar_and(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 p, %1, 0;\n\t"
      "bar.red.and.pred q, 1, %2, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r)
      : "r"(static_cast<uint32_t>(pred)), "n"(CNT)
      : "memory");
  return r != 0;
}
// a load that stays where it is written (issued early on purpose; the value is used much later)
__device__ __forceinline__ int ld_nc_here(const int32_t* p) {
  int v;
  asm volatile("ld.global.nc.s32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

template <int CH, bool BF16, bool UNC>
__global__ void __launch_bounds__(CTX_THREADS, 1) lantern_context_kernel(VerifyParams P) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ CtxShared S;
  __shared__ __align__(8) uint64_t bar_full[2], bar_empty[2];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int V = P.V, N = P.N, R = P.R, k = P.k;
  const int rowbytes = V * (BF16 ? 2 : 4);
  const int stage_bytes = (3 * rowbytes + 127) & ~127;   // row slots: conditional, unconditional, drafter
  const int row_floats = rowbytes >> 2;
  auto EI = [&](int x) { return ephys<BF16>(x, row_floats); };
  const float L_hi = 1.44269502162933349609375f;   // fl32(log2 e)
  const float ninf = __int_as_float(0xff800000);

  if (tid == 0) {
    mbar_init(&bar_full[0], 1);
    mbar_init(&bar_full[1], 1);
    mbar_init(&bar_empty[0], CNW);
    mbar_init(&bar_empty[1], CNW);
    fence_mbar_init();
    fence_proxy_async();
    S.status = 0;
  }
  __syncthreads();

  // ======================= producer warp =======================
  // One thread hands out work and keeps the copies going.  Items 0..3G-1 are dealt statically (CTA x
  // takes x, x+G, x+2G); from then on a global counter hands them out.  A three-deep pipeline keeps
  // every global round trip off the critical path: while the consumers process context i, the rows
  // of i+1 are in flight, the descriptor of i+2 is being loaded and the index of i+3 is being fetched.
  if (warp == CNW) {
    if (lane == 0) {
      const int n_heavy = P.counters->n_heavy;
      const int total = n_heavy + P.counters->n_light;
      const int cap = P.B * N;
      const int G = gridDim.x;
      auto load_item = [&](int w) -> WorkItem {
        WorkItem it;
        it.item = -1;
        it.pad = 0;
        if (w < total) {
          const int slot = w < n_heavy ? w : cap - 1 - (w - n_heavy);
          const int4 lo = __ldg(reinterpret_cast<const int4*>(P.work + slot));
          const int4 hi = __ldg(reinterpret_cast<const int4*>(P.work + slot) + 1);
          it.item = lo.x, it.cbase = lo.y, it.nchild = lo.z, it.node0 = lo.w;
          it.tok0 = hi.x, it.r0 = __int_as_float(hi.y), it.u_final = __int_as_float(hi.z);
        }
        return it;
      };
      WorkItem it_cur = load_item(blockIdx.x);
      WorkItem it_next = load_item(blockIdx.x + G);
      int w_next2 = blockIdx.x + 2 * G;
      for (int i = 0;; ++i) {
        const int slot = i & 1;
        // the slot is free once every consumer warp has finished the context that used it
        if (i >= 2 && !mbar_wait(&bar_empty[slot], ((i >> 1) - 1) & 1)) {
          it_cur.item = -1;
          it_cur.pad = LANTERN_ST_INTERNAL;   // a consumer never released the slot: stop handing out work
        }
        S.work[slot] = it_cur;                // published by the mbarrier operation below
        if (it_cur.item < 0) {
          mbar_arrive(&bar_full[slot]);       // wake the consumers; they see the terminator
          break;
        }
        fence_proxy_async();
        ctx_issue_rows<BF16, UNC>(P, it_cur.item, smem + slot * stage_bytes, rowbytes, &bar_full[slot]);
        it_cur = it_next;
        it_next = load_item(w_next2);
        w_next2 = 3 * G + atomicAdd(&P.counters->work_next, 1);
      }
    }
    return;
  }

  // ======================= consumer warps =======================
  for (int iter = 0;; ++iter) {
    const int slot_cur = iter & 1;
    // One warp watches the copy's mbarrier (bounded wait); the consumer barrier then releases everybody
    // at once and tells every thread alike whether the rows have landed.
    bool landed = true;
    if (warp == 0) landed = mbar_wait(&bar_full[slot_cur], (iter >> 1) & 1);
    const bool arrived = cbar_and(landed);
    if (!arrived) break;   // the copy did not land within the limit; the walk reports the missing record
    const WorkItem cur = S.work[slot_cur];
    const int item = cur.item;
    if (item < 0) break;
    unsigned char* stage = smem + slot_cur * stage_bytes;    // this context's rows, later its E
    float* E = reinterpret_cast<float*>(stage);
    const int b = item / R;
    const ChildInfo* kids = P.children + cur.cbase;
    const int nchild = cur.nchild;
    // every consumer is past the previous context (its record included): clear the shared status word;
    // nobody sets it again before the [stats] barrier below
    if (tid == 0) S.status = 0;

    // first child: its neighbour row (two slots per thread) and, for thread 0, its raw logits; issued
    // now, used after the streaming pass
    int node = cur.node0;
    int xt = cur.tok0;
    float r = cur.r0;
    const int j0 = 2 * tid + 1, j1 = 2 * tid + 2;
    int n0 = (j0 < k) ? ld_nc_here(P.nbr + static_cast<size_t>(xt) * k + j0) : -1;
    int n1 = (j1 < k) ? ld_nc_here(P.nbr + static_cast<size_t>(xt) * k + j1) : -1;
    float raw_c = 0.0f, raw_u = 0.0f, raw_d = 0.0f;
    if (tid == 0) {
      const size_t e = static_cast<size_t>(item) * V + xt;
      raw_c = ctx_raw_logit<BF16>(P.target, e);
      if (UNC) raw_u = ctx_raw_logit<BF16>(P.target, static_cast<size_t>(P.B) * R * V + e);
      raw_d = ctx_raw_logit<BF16>(P.draft, e);
    }

    // ---------------- streaming pass, warp-local ----------------
    // staging rows: 0 = conditional target, 1 = unconditional target (if any), 2 = drafter
    const unsigned char* rc = stage;
    const unsigned char* ru = stage + rowbytes;
    unsigned char* rd = stage + 2 * rowbytes;
    const float Tinv_is_one = P.T == 1.0f;
    // eight processed drafter logits of 16-byte group g (z_p = l_d / T)
    auto draft_chunk = [&](int g, float (&out)[8]) {
      if (BF16) {
        const uint4 d = *reinterpret_cast<const uint4*>(rd + g * 16);
        const uint32_t dw[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          out[2 * i] = __uint_as_float(dw[i] << 16);
          out[2 * i + 1] = __uint_as_float(dw[i] & 0xffff0000u);
        }
      } else {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const float4 d = *reinterpret_cast<const float4*>(rd + g * 32 + h * 16);
          out[4 * h] = d.x, out[4 * h + 1] = d.y, out[4 * h + 2] = d.z, out[4 * h + 3] = d.w;
        }
      }
      if (!Tinv_is_one) {
#pragma unroll
        for (int e = 0; e < 8; ++e) out[e] = __fdiv_rn(out[e], P.T);
      }
    };
    float a[CH * 8];
    // --- target: guidance combine, warp maximum, numerators, partial sum; E replaces the raw rows ---
    {
      const float s = P.cfg_scale;
#pragma unroll
      for (int c = 0; c < CH; ++c) {
        const int g = c * CNT + tid;
        if (g * 8 < V) {
          float lc[8], lu[8];
          if (BF16) {
            const uint4 x = *reinterpret_cast<const uint4*>(rc + g * 16);
            const uint32_t xw[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              lc[2 * i] = __uint_as_float(xw[i] << 16);
              lc[2 * i + 1] = __uint_as_float(xw[i] & 0xffff0000u);
            }
            if (UNC) {
              const uint4 y = *reinterpret_cast<const uint4*>(ru + g * 16);
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
              const float4 x = *reinterpret_cast<const float4*>(rc + g * 32 + h * 16);
              lc[4 * h] = x.x, lc[4 * h + 1] = x.y, lc[4 * h + 2] = x.z, lc[4 * h + 3] = x.w;
              if (UNC) {
                const float4 y = *reinterpret_cast<const float4*>(ru + g * 32 + h * 16);
                lu[4 * h] = y.x, lu[4 * h + 1] = y.y, lu[4 * h + 2] = y.z, lu[4 * h + 3] = y.w;
              }
            }
          }
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            float l = lc[e];
            if (UNC) l = __fmaf_rn(s, __fsub_rn(lc[e], lu[e]), lu[e]);   // l_u + s (l_c - l_u)
            if (!Tinv_is_one) l = __fdiv_rn(l, P.T);
            a[c * 8 + e] = l;
          }
        } else {
#pragma unroll
          for (int e = 0; e < 8; ++e) a[c * 8 + e] = ninf;
        }
      }
    }
    float mq = a[0];
#pragma unroll
    for (int i = 1; i < CH * 8; ++i) mq = fmaxf(mq, a[i]);
    // a slice without any finite logit (padding, masked tokens) still needs a finite shift
    mq = fmaxf(warp_max(mq), -1.0e37f);
    const float mlq_w = mq * L_hi;
    float tq = 0.0f;
#pragma unroll
    for (int c = 0; c < CH; ++c) {
#pragma unroll
      for (int e = 0; e < 8; ++e) a[c * 8 + e] = ex2_approx(__fmaf_rn(a[c * 8 + e], L_hi, -mlq_w));
      tq += sum8(&a[c * 8]);
      const int g = c * CNT + tid;
      if (g * 8 < V) {
        *reinterpret_cast<float4*>(E + EI(g * 8)) = make_float4(a[c * 8], a[c * 8 + 1], a[c * 8 + 2], a[c * 8 + 3]);
        *reinterpret_cast<float4*>(E + EI(g * 8 + 4)) =
            make_float4(a[c * 8 + 4], a[c * 8 + 5], a[c * 8 + 6], a[c * 8 + 7]);
      }
    }
    // --- drafter: warp maximum and partial sum of numerators; the raw row stays in shared memory ---
#pragma unroll
    for (int c = 0; c < CH; ++c) {
      const int g = c * CNT + tid;
      float d8[8];
      if (g * 8 < V) {
        draft_chunk(g, d8);
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) d8[e] = ninf;
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) a[c * 8 + e] = d8[e];
    }
    float mp = a[0];
#pragma unroll
    for (int i = 1; i < CH * 8; ++i) mp = fmaxf(mp, a[i]);
    mp = fmaxf(warp_max(mp), -1.0e37f);
    const float mlp_w = mp * L_hi;
    float tp = 0.0f;
#pragma unroll
    for (int c = 0; c < CH; ++c) {
#pragma unroll
      for (int e = 0; e < 8; ++e) a[c * 8 + e] = ex2_approx(__fmaf_rn(a[c * 8 + e], L_hi, -mlp_w));
      tp += sum8(&a[c * 8]);
    }
    {
      const double wq = warp_sum(static_cast<double>(tq));
      const double wp = warp_sum(static_cast<double>(tp));
      if (lane == 0) {
        S.sq[warp] = wq;
        S.sp[warp] = wp;
        S.mlq[warp] = mlq_w;
        S.mlp[warp] = mlp_w;
      }
    }

    cbar();   // [stats] per-warp maxima and sums, and E, are visible

    // ---------------- block statistics, computed by every warp for itself ----------------
    float fq_l, fp_l;            // lane l holds the factor that brings warp l's units to global units
    double Zq, Zp;
    float mlq_g, mlp_g;
    {
      const float mq_l = lane < CNW ? S.mlq[lane] : ninf;
      const float mp_l = lane < CNW ? S.mlp[lane] : ninf;
      mlq_g = warp_max(mq_l);
      mlp_g = warp_max(mp_l);
      fq_l = ex2_approx(mq_l - mlq_g);
      fp_l = ex2_approx(mp_l - mlp_g);
      Zq = warp_sum(lane < CNW ? static_cast<double>(fq_l) * S.sq[lane] : 0.0);
      Zp = warp_sum(lane < CNW ? static_cast<double>(fp_l) * S.sp[lane] : 0.0);
    }
    const float fq_mine = __shfl_sync(kFull, fq_l, warp), fp_mine = __shfl_sync(kFull, fp_l, warp);

    int status = 0;              // bits every thread sets alike
    int accepted = -1;
    bool record_written = false;
    if (!(Zq > 0.0 && Zq < 1e300 && Zp > 0.0 && Zp < 1e300)) {
      status |= LANTERN_ST_NONFINITE;
    } else {
      double qscale = 1.0 / Zq;     // q'(x) = E(x) * fq[warp of x] * qscale
      double pscale = 1.0 / Zp;     // p'(x) = ep(x) * fp[warp of x] * pscale
      const double delta = static_cast<double>(P.delta);
      if (tid == 0) {   // the two single probabilities of the first child, in double precision
        float zq = raw_c;
        if (UNC) zq = __fmaf_rn(P.cfg_scale, __fsub_rn(raw_c, raw_u), raw_u);
        float zp = raw_d;
        if (P.T != 1.0f) {
          zq = __fdiv_rn(zq, P.T);
          zp = __fdiv_rn(zp, P.T);
        }
        S.acc_e = exp2_single(zq, mlq_g);
        S.acc_p = exp2_single(zp, mlp_g);
        S.acc_valid = 1;
      }

      for (int ci = 0; ci < nchild; ++ci) {
        const int32_t* nrow = P.nbr + static_cast<size_t>(xt) * k;
        // the next sibling's description, wanted only after a rejection: in flight meanwhile
        ChildInfo sib = {0, 0, 0.0f, 0};
        if (ci + 1 < nchild) {
          const int4 v = __ldg(reinterpret_cast<const int4*>(kids + ci + 1));
          sib.node = v.x, sib.token = v.y, sib.r = __int_as_float(v.z);
        }
        // drafter numerator of x~ from the raw row (-inf, hence 0, once x~ has been rejected), global units
        float px_bulk;
        {
          float dz = BF16 ? __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const unsigned short*>(rd)[xt]) << 16)
                          : reinterpret_cast<const float*>(rd)[xt];
          if (!Tinv_is_one) dz = __fdiv_rn(dz, P.T);
          const int ow = cowner_thread(xt) >> 5;
          px_bulk = ex2_approx(__fmaf_rn(dz, L_hi, -S.mlp[ow])) * __shfl_sync(kFull, fp_l, ow);
        }
        const float e_xt_bulk = E[EI(xt)] * __shfl_sync(kFull, fq_l, cowner_thread(xt) >> 5);

        // ---- A_{k,delta}(x~): gather + prefix scan with the strict bound ----
        const double thr = delta / qscale;   // the bound in the units of the unnormalised sums
        double carry = 0.0, sm = 0.0;
        int m = k - 1;
        bool cut = false;
        for (int base = 0; base < k - 1 && !cut; base += 2 * CNT) {
          const int ja = base + j0, jb = base + j1;
          const bool va = ja < k, vb = jb < k;
          const int na = base == 0 ? n0 : (va ? __ldg(nrow + ja) : -1);
          const int nb = base == 0 ? n1 : (vb ? __ldg(nrow + jb) : -1);
          const bool ia = va && static_cast<unsigned>(na) < static_cast<unsigned>(V);
          const bool ib = vb && static_cast<unsigned>(nb) < static_cast<unsigned>(V);
          if ((va && !ia) || (vb && !ib)) atomicOr(&S.status, LANTERN_ST_BAD_TABLE);   // carries no mass
          const float fa = __shfl_sync(kFull, fq_l, ia ? cowner_thread(na) >> 5 : 0);
          const float fb = __shfl_sync(kFull, fq_l, ib ? cowner_thread(nb) >> 5 : 0);
          const double da = ia ? static_cast<double>(E[EI(na)] * fa) : 0.0;
          const double db = ib ? static_cast<double>(E[EI(nb)] * fb) : 0.0;
          const double incl = warp_incl_scan(da + db, lane);
          if (lane == 31) S.wt[warp] = incl;
          cbar();   // [scan 1]
          double pre, tot;
          {
            const double t = lane < CNW ? S.wt[lane] : 0.0;
            const double in = warp_incl_scan(t, lane);
            pre = __shfl_sync(kFull, in - t, warp);
            tot = __shfl_sync(kFull, in, CNW - 1);
          }
          const double Sb = carry + pre + incl;          // inclusive prefix at slot jb
          const double Sa = Sb - db;                      // at slot ja
          const bool faila = va && !(Sa < thr);
          const bool failb = vb && !(Sb < thr);
          const int my_first = faila ? ja : (failb ? jb : kNone);
          const int wfirst = __reduce_min_sync(kFull, my_first);
          if (wfirst != kNone && my_first == wfirst) {
            S.first[warp] = wfirst;
            S.sbefore[warp] = faila ? Sa - da : Sa;
          } else if (wfirst == kNone && lane == 0) {
            S.first[warp] = kNone;
          }
          cbar();   // [scan 2]
          const int f_l = lane < CNW ? S.first[lane] : kNone;
          const int gfirst = __reduce_min_sync(kFull, f_l);
          if (gfirst != kNone) {
            const int src = __ffs(__ballot_sync(kFull, f_l == gfirst)) - 1;
            m = gfirst - 1;
            sm = S.sbefore[src];
            cut = true;
          } else {
            carry += tot;
            sm = carry;
          }
        }
        if (k == 1) cbar();   // publish S.acc_* when the scan loop did not run
        // the two single probabilities: thread 0's double-precision values where it has them; a bulk
        // value of exactly zero (token inside an earlier A, or rejected before) stays zero
        const bool acc = S.acc_valid != 0;
        const float pxb = px_bulk;
        const double e_xt = (acc && e_xt_bulk != 0.0f) ? S.acc_e : static_cast<double>(e_xt_bulk);
        const double p_xt = (acc && pxb != 0.0f) ? S.acc_p : static_cast<double>(pxb);
        const double qa = (e_xt + sm) * qscale;
        const double px = p_xt * pscale;
        const bool accept = static_cast<double>(r) * px < qa;   // Section 4.3: min(1, sum_A q / p(x~))
        if (tid == 0) {
          const size_t o = static_cast<size_t>(b) * N + node;
          if (P.out_qa) P.out_qa[o] = static_cast<float>(qa);
          if (P.out_px) P.out_px[o] = static_cast<float>(px);
          if (P.out_m) P.out_m[o] = m;
        }
        if (accept) {
          accepted = node;
          break;
        }
        // ---- rejected: residual [q_{k,delta}(.|D = x~) - p]_+ ----
        // members of A (x~ included) leave no residual mass: flag them with a negative sign
        for (int base = 0; base < m; base += 2 * CNT) {
          const int ja = base + j0, jb = base + j1;
          if (ja <= m) {
            const int n = base == 0 ? n0 : __ldg(nrow + ja);
            if (static_cast<unsigned>(n) < static_cast<unsigned>(V)) E[EI(n)] = -fabsf(E[EI(n)]);
          }
          if (jb <= m) {
            const int n = base == 0 ? n1 : __ldg(nrow + jb);
            if (static_cast<unsigned>(n) < static_cast<unsigned>(V)) E[EI(n)] = -fabsf(E[EI(n)]);
          }
        }
        if (tid == 0) E[EI(xt)] = -fabsf(E[EI(xt)]);
        if (tid == 0) {   // x~ leaves the drafter distribution for the following siblings
          if (BF16) reinterpret_cast<unsigned short*>(rd)[xt] = 0xff80;   // -inf
          else reinterpret_cast<float*>(rd)[xt] = ninf;
        }
        const bool last = (ci + 1 == nchild);
        if (!last) {   // next sibling's neighbour row, in flight during the residual pass
          node = sib.node;
          xt = sib.token;
          r = sib.r;
          n0 = (j0 < k) ? ld_nc_here(P.nbr + static_cast<size_t>(xt) * k + j0) : -1;
          n1 = (j1 < k) ? ld_nc_here(P.nbr + static_cast<size_t>(xt) * k + j1) : -1;
          if (tid == 0) {   // its raw logits, for the double-precision replay below
            const size_t e = static_cast<size_t>(item) * V + xt;
            raw_c = ctx_raw_logit<BF16>(P.target, e);
            if (UNC) raw_u = ctx_raw_logit<BF16>(P.target, static_cast<size_t>(P.B) * R * V + e);
            raw_d = ctx_raw_logit<BF16>(P.draft, e);
          }
        }
        cbar();   // [flags]
        // w = E - (p'/q' scale ratio) * ep, in this warp's own units of E
        const float ratio = static_cast<float>((pscale * static_cast<double>(fp_mine)) /
                                               (qscale * static_cast<double>(fq_mine)));
        float cs[CH];
        float wsum = 0.0f, psum = 0.0f;
#pragma unroll
        for (int c = 0; c < CH; ++c) {
          const int g = c * CNT + tid;
          if (g * 8 < V) {
            const float4 lo = *reinterpret_cast<const float4*>(E + EI(g * 8));
            const float4 hi = *reinterpret_cast<const float4*>(E + EI(g * 8 + 4));
            const float e8[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
            float ep8[8];
            draft_chunk(g, ep8);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              ep8[e] = ex2_approx(__fmaf_rn(ep8[e], L_hi, -mlp_w));
              a[c * 8 + e] = fmaxf(0.0f, __fmaf_rn(-ratio, ep8[e], e8[e]));
            }
            psum += sum8(ep8);
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) a[c * 8 + e] = 0.0f;
          }
          cs[c] = sum8(&a[c * 8]);
          wsum += cs[c];
        }
        const double fqd = static_cast<double>(fq_mine);
        double W, Sp;
        if (!last) {
          // only the totals are needed; the residual becomes the next sibling's target
#pragma unroll
          for (int c = 0; c < CH; ++c) {
            const int g = c * CNT + tid;
            if (g * 8 < V) {
              *reinterpret_cast<float4*>(E + EI(g * 8)) = make_float4(a[c * 8], a[c * 8 + 1], a[c * 8 + 2], a[c * 8 + 3]);
              *reinterpret_cast<float4*>(E + EI(g * 8 + 4)) =
                  make_float4(a[c * 8 + 4], a[c * 8 + 5], a[c * 8 + 6], a[c * 8 + 7]);
            }
          }
          const double ww = warp_sum(static_cast<double>(wsum) * fqd);
          const double wp = warp_sum(static_cast<double>(psum) * static_cast<double>(fp_mine));
          if (lane == 0) {
            S.wt[warp] = ww;
            S.wt[CNW + warp] = wp;
          }
          cbar();   // [totals] also publishes the written-back residual
          W = warp_sum(lane < CNW ? S.wt[lane] : 0.0);
          Sp = warp_sum(lane < CNW ? S.wt[CNW + lane] : 0.0);
          if (!(W > 0.0)) {
            status |= LANTERN_ST_DEGENERATE;
            break;
          }
          if (tid == 0) {
            // The next sibling's own two probabilities in double precision: its numerators from the raw
            // logits, carried through every rejection round so far (E <- max(0, E - ratio_i * ep)); the
            // block totals W, Sp are sums of thousands of terms and do not suffer from cancellation.
            if (ci < 32) {
              S.hist[ci] = pscale / qscale;
              float zq = raw_c;
              if (UNC) zq = __fmaf_rn(P.cfg_scale, __fsub_rn(raw_c, raw_u), raw_u);
              float zp = raw_d;
              if (P.T != 1.0f) {
                zq = __fdiv_rn(zq, P.T);
                zp = __fdiv_rn(zp, P.T);
              }
              double e = exp2_single(zq, mlq_g);
              const double pe = exp2_single(zp, mlp_g);
              for (int i = 0; i <= ci; ++i) e = fmax(0.0, e - S.hist[i] * pe);
              S.acc_e = e;
              S.acc_p = pe;
              S.acc_valid = 1;
            } else {
              S.acc_valid = 0;
            }
          }
          qscale = 1.0 / W;
          pscale = Sp > 0.0 ? 1.0 / Sp : 0.0;
          continue;
        }
        // ---- last child rejected: draw the replacement token from the residual (Algorithm 1) ----
        double csd[CH], incl[CH], excl[CH] = {};
#pragma unroll
        for (int c = 0; c < CH; ++c) {
          csd[c] = static_cast<double>(cs[c]) * fqd;
          incl[c] = warp_incl_scan(csd[c], lane);
          if (lane == 31) S.wt[c * CNW + warp] = incl[c];
        }
        cbar();   // [draw 1]
        {
          // exclusive prefix over (chunk, warp) in chunk-major order; 32 entries per round
          double carry2 = 0.0;
#pragma unroll
          for (int half = 0; half < (CH * CNW + 31) / 32; ++half) {
            const int e = half * 32 + lane;
            const double t = e < CH * CNW ? S.wt[e] : 0.0;
            const double in = warp_incl_scan(t, lane);
            const double ex = carry2 + in - t;
#pragma unroll
            for (int c = 0; c < CH; ++c) {
              const int want = c * CNW + warp;
              const double got = __shfl_sync(kFull, ex, want & 31);
              if ((want >> 5) == half) excl[c] = got + incl[c] - csd[c];
            }
            carry2 += __shfl_sync(kFull, in, 31);
          }
          W = carry2;
        }
        if (!(W > 0.0)) {
          status |= LANTERN_ST_DEGENERATE;
          break;
        }
        const double target = static_cast<double>(cur.u_final) * W;
        int cand = kNone;
#pragma unroll
        for (int c = CH - 1; c >= 0; --c)
          if (excl[c] + csd[c] > target) cand = c * CNT + tid;
        const int wmin = __reduce_min_sync(kFull, cand);
        if (lane == 0) S.cand[warp] = wmin;
        if (tid == 0) S.tok = -1;
        cbar();   // [draw 2]
        const int win = __reduce_min_sync(kFull, lane < CNW ? S.cand[lane] : kNone);
        if (win == kNone) {
          // rounding left no slot above the target: the largest token of positive weight
          int lastp = -1;
#pragma unroll
          for (int c = 0; c < CH; ++c)
#pragma unroll
            for (int e = 0; e < 8; ++e)
              if (a[c * 8 + e] > 0.0f) lastp = (c * CNT + tid) * 8 + e;
          if (lastp >= V) lastp = -1;
          if (lastp >= 0) atomicMax(&S.tok, lastp);
          cbar();
          if (tid == 0) {
            Record rec = {-1, S.tok, status | S.status | (S.tok < 0 ? LANTERN_ST_DEGENERATE : 0), 0};
            P.records[item] = rec;
          }
        } else if ((win & (CNT - 1)) == tid) {
          const int wc = win >> LOG_CNT;
          int tok = -1, lastpos = -1;
#pragma unroll
          for (int c = 0; c < CH; ++c) {
            if (c == wc) {
              double cum = excl[c];
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const float wv = a[c * 8 + e];
                cum += static_cast<double>(wv) * fqd;
                if (wv > 0.0f) lastpos = e;
                if (tok < 0 && cum > target) tok = e;
              }
            }
          }
          if (tok < 0) tok = lastpos;
          Record rec = {-1, win * 8 + tok, status | S.status, 0};
          P.records[item] = rec;
        }
        record_written = true;
      }
    }
    if (!record_written && tid == 0) {
      // S.status was last written before a barrier every thread has passed
      Record rec = {accepted, -1, status | S.status, 0};
      P.records[item] = rec;
    }
    // this context's staging area (rows and E) is no longer needed by this warp
    __syncwarp();
    if (lane == 0) mbar_arrive(&bar_empty[slot_cur]);
  }
}

}  // namespace lantern
