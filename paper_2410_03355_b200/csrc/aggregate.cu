// All-token aggregation: for every token x of a context row, the mass of the row's target
// distribution q over A_{k,delta}(x) -- the V x k gather-sum that building A for EVERY token amounts
// to.  The paper's verification step needs this for the drafted tokens only (verify*.cu*); this
// kernel exists to measure the gather-sum itself and is not used by lantern_verify.
//
// One CTA per row: the row's softmax numerators are built once in shared memory (V floats); then
// each warp takes tokens x = warp, warp + NW, ...: its lanes read B_k(x) four slots each (16-byte
// loads where k is a multiple of 4), gather the numerators from shared memory, and a
// double-precision warp scan finds the first neighbour that no longer fits under the strict bound
// (Algorithm 2, second block).  The table (V * k * 4 bytes) is re-read by every row and lives in L2.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "lantern.h"
#include "lantern_device.cuh"

namespace lantern {

constexpr int AGT = 512;
constexpr int AGW = AGT / 32;

struct AggParams {
  const void* logits;
  const int32_t* nbr;
  float* out_agg;
  int32_t* out_m;
  int32_t* out_status;
  int rows, V, k;
  float cfg_scale, T, delta;
};

struct AggShared {
  double wsum[AGW];
  float wmax[AGW];
  int bad;
};

template <bool BF16, bool UNC>
__device__ __forceinline__ void agg_chunk(const AggParams& P, size_t row, int g, float (&out)[8]) {
  const size_t off = row * static_cast<size_t>(P.V);
  const size_t branch = static_cast<size_t>(P.rows) * P.V;
  float lc[8], lu[8];
  if (BF16) {
    const unsigned short* base = static_cast<const unsigned short*>(P.logits);
    const uint4 x = __ldg(reinterpret_cast<const uint4*>(base + off) + g);
    const uint32_t xw[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      lc[2 * i] = __uint_as_float(xw[i] << 16);
      lc[2 * i + 1] = __uint_as_float(xw[i] & 0xffff0000u);
    }
    if (UNC) {
      const uint4 y = __ldg(reinterpret_cast<const uint4*>(base + branch + off) + g);
      const uint32_t yw[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        lu[2 * i] = __uint_as_float(yw[i] << 16);
        lu[2 * i + 1] = __uint_as_float(yw[i] & 0xffff0000u);
      }
    }
  } else {
    const float* base = static_cast<const float*>(P.logits);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const float4 x = __ldg(reinterpret_cast<const float4*>(base + off) + 2 * g + h);
      lc[4 * h] = x.x, lc[4 * h + 1] = x.y, lc[4 * h + 2] = x.z, lc[4 * h + 3] = x.w;
      if (UNC) {
        const float4 y = __ldg(reinterpret_cast<const float4*>(base + branch + off) + 2 * g + h);
        lu[4 * h] = y.x, lu[4 * h + 1] = y.y, lu[4 * h + 2] = y.z, lu[4 * h + 3] = y.w;
      }
    }
  }
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    float z = UNC ? __fmaf_rn(P.cfg_scale, __fsub_rn(lc[e], lu[e]), lu[e]) : lc[e];
    if (P.T != 1.0f) z = __fdiv_rn(z, P.T);
    out[e] = z;
  }
}

template <bool BF16, bool UNC>
__global__ void __launch_bounds__(AGT) lantern_aggregate_kernel(AggParams P) {
  extern __shared__ __align__(16) float E[];   // numerators 2^((z - M) log2 e), token order
  __shared__ AggShared S;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int V = P.V, k = P.k;
  const float L_hi = 1.44269502162933349609375f;
  const float NEG_INF = __int_as_float(0xff800000);
  const bool vec = (k & 3) == 0;   // rows of the table start on 16-byte boundaries

  for (int row = blockIdx.x; row < P.rows; row += gridDim.x) {
    // ---- the row's numerators ----
    float m = NEG_INF;
    int bad = 0;
    for (int g = tid; g * 8 < V; g += AGT) {
      float z[8];
      agg_chunk<BF16, UNC>(P, row, g, z);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        bad |= (z[e] != z[e]);
        m = fmaxf(m, z[e]);
        E[g * 8 + e] = z[e];
      }
    }
    m = warp_max(m);
    if (tid == 0) S.bad = 0;
    __syncthreads();
    if (lane == 0) S.wmax[warp] = m;
    if (bad) atomicOr(&S.bad, 1);
    __syncthreads();
    float M = S.wmax[0];
#pragma unroll
    for (int w = 1; w < AGW; ++w) M = fmaxf(M, S.wmax[w]);
    const bool finite = !S.bad && M > NEG_INF && M < __int_as_float(0x7f800000);
    if (!finite) {   // uniform
      for (int x = tid; x < V; x += AGT) {
        P.out_agg[static_cast<size_t>(row) * V + x] = __int_as_float(0x7fc00000);
        if (P.out_m) P.out_m[static_cast<size_t>(row) * V + x] = -1;
      }
      if (tid == 0 && P.out_status) P.out_status[row] = LANTERN_ST_NONFINITE;
      __syncthreads();
      continue;
    }
    const float mL = M * L_hi;
    float part = 0.0f;
    for (int g = tid; g * 8 < V; g += AGT) {   // each thread revisits the groups it stored itself
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        float y;
        const float a = __fmaf_rn(E[g * 8 + e], L_hi, -mL);
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(a));
        E[g * 8 + e] = y;
        part += y;
      }
    }
    double Z = warp_sum(static_cast<double>(part));
    if (lane == 0) S.wsum[warp] = Z;
    __syncthreads();   // numerators and per-warp sums are visible
    Z = 0.0;
#pragma unroll
    for (int w = 0; w < AGW; ++w) Z += S.wsum[w];
    const double thr = static_cast<double>(P.delta) * Z;
    const double invZ = 1.0 / Z;

    // ---- every token's neighbourhood ----
    for (int x = warp; x < V; x += AGW) {
      const int32_t* nrow = P.nbr + static_cast<size_t>(x) * k;
      double carry = 0.0, moved = 0.0;
      int mcut = k - 1;
      int bad_entry = 0;
      for (int base = 0; base < k; base += 128) {
        const int j0 = base + 4 * lane;
        int n[4] = {-1, -1, -1, -1};
        if (vec) {
          if (j0 < k) {   // k % 4 == 0: all four slots exist
            const int4 v = __ldg(reinterpret_cast<const int4*>(nrow + j0));
            n[0] = v.x, n[1] = v.y, n[2] = v.z, n[3] = v.w;
          }
        } else {
#pragma unroll
          for (int i = 0; i < 4; ++i)
            if (j0 + i < k) n[i] = __ldg(nrow + j0 + i);
        }
        double pre[4], run = 0.0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int j = j0 + i;
          const bool real = j >= 1 && j < k;   // slot 0 is x itself: it is not moved
          const bool inr = real && static_cast<unsigned>(n[i]) < static_cast<unsigned>(V);
          bad_entry |= real && !inr;
          run += inr ? static_cast<double>(E[n[i]]) : 0.0;
          pre[i] = run;
        }
        const double incl = warp_incl_scan(run, lane);
        const double before = carry + (incl - run);
        int fail = 4;
#pragma unroll
        for (int i = 3; i >= 0; --i) {
          const int j = j0 + i;
          if (j >= 1 && j < k && !(before + pre[i] < thr)) fail = i;
        }
        const unsigned who = __ballot_sync(kFull, fail < 4);
        if (who) {
          const int src = __ffs(who) - 1;
          const double mine = before + (fail > 0 && fail < 4 ? pre[fail > 0 ? fail - 1 : 0] : 0.0);
          moved = __shfl_sync(kFull, mine, src);
          mcut = base + 4 * src + __shfl_sync(kFull, fail, src) - 1;
          break;
        }
        carry += __shfl_sync(kFull, incl, 31);
        moved = carry;
      }
      bad_entry = __any_sync(kFull, bad_entry);
      if (lane == 0) {
        const size_t o = static_cast<size_t>(row) * V + x;
        P.out_agg[o] = static_cast<float>((static_cast<double>(E[x]) + moved) * invZ);
        if (P.out_m) P.out_m[o] = mcut;
        if (bad_entry) atomicOr(&S.bad, 2);
      }
    }
    __syncthreads();   // E is rebuilt for the next row
    if (tid == 0 && P.out_status) P.out_status[row] = (S.bad & 2) ? LANTERN_ST_BAD_TABLE : 0;
    __syncthreads();
  }
}

template <bool BF16, bool UNC>
static cudaError_t launch_aggregate(const AggParams& P, cudaStream_t st) {
  auto kk = lantern_aggregate_kernel<BF16, UNC>;
  const size_t smem = static_cast<size_t>(P.V) * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(kk, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  int dev = 0, sms = 0, per_sm = 0;
  if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kk, AGT, smem)) != cudaSuccess) return e;
  if (per_sm < 1 || sms < 1) return cudaErrorInvalidConfiguration;
  const long long slots = static_cast<long long>(sms) * per_sm;
  const int grid = static_cast<int>(P.rows < slots ? P.rows : slots);
  kk<<<grid, AGT, smem, st>>>(P);
  return cudaGetLastError();
}

}  // namespace lantern

using namespace lantern;

extern "C" lantern_status lantern_aggregate_all(const void* logits, int dtype, float cfg_scale, int has_uncond, float T,
                                                const int32_t* neighbor_idx, int k, float delta, int rows, int V,
                                                float* out_agg, int32_t* out_m, int32_t* out_status,
                                                void* cuda_stream) {
  if (dtype != LANTERN_F32 && dtype != LANTERN_BF16) return LANTERN_E_PARAM;
  if (rows < 0 || V < 8 || V > 16384 || (V % 8) != 0 || k < 1 || k > V) return LANTERN_E_SHAPE;
  if (!(T > 0.0f) || !(delta >= 0.0f) || !isfinite(T) || !isfinite(delta)) return LANTERN_E_PARAM;
  if (has_uncond && !isfinite(cfg_scale)) return LANTERN_E_PARAM;
  if (rows == 0) return LANTERN_OK;
  if (!logits || !neighbor_idx || !out_agg) return LANTERN_E_NULL;
  if ((reinterpret_cast<uintptr_t>(logits) & 15) || (reinterpret_cast<uintptr_t>(neighbor_idx) & 15)) return LANTERN_E_ALIGN;
  AggParams P;
  P.logits = logits;
  P.nbr = neighbor_idx;
  P.out_agg = out_agg;
  P.out_m = out_m;
  P.out_status = out_status;
  P.rows = rows;
  P.V = V;
  P.k = k;
  P.cfg_scale = cfg_scale;
  P.T = T;
  P.delta = delta;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const bool bf = dtype == LANTERN_BF16, un = has_uncond != 0;
  const cudaError_t e = bf ? (un ? launch_aggregate<true, true>(P, st) : launch_aggregate<true, false>(P, st))
                           : (un ? launch_aggregate<false, true>(P, st) : launch_aggregate<false, false>(P, st));
  return e == cudaSuccess ? LANTERN_OK : LANTERN_E_CUDA;
}
