// Neighbour table B_k of a VQ codebook (Algorithm 2, block "Precompute B_k for all tokens").
//
// Key of a pair (i, j): squared l2 distance accumulated in fp32 in dimension order,
// acc = fma(a_d - b_d, a_d - b_d, acc).  That exact operation sequence is kept whatever the
// tiling, so the order of neighbours does not depend on how the work is split.
//
// Small D (<= 32): one CTA per code computes its V keys straight into shared memory.
// Large D: a tiled SIMT kernel writes the keys of a block of rows to global scratch (each
// (i, j) accumulator still runs over d in order), and the per-row CTA reads its row of keys.
// Per row: exclude the code itself, radix-select the (k-1)-th smallest key (ties by smaller
// index), compact the selected (key, index) pairs, bitonic-sort them as 64-bit composites,
// and store the row with the code itself in slot 0.
#include <cuda_runtime.h>
#include <stdint.h>

#include "lantern.h"
#include "lantern_device.cuh"

namespace lantern {

constexpr int BT = 512;          // threads of the per-row kernel
constexpr int BW = BT / 32;
constexpr int SMALL_D = 32;
constexpr int TILE = 64;         // distance tile edge
constexpr int DK = 16;           // dimensions staged per step

struct BuildParams {
  const float* codebook;
  const uint32_t* scratch;       // [rows, V] key bits of rows row0.. (large-D path), else null
  int32_t* idx;
  float* dist;
  int V, D, k, row0;
};

// ---------------------------------------------------------------------------------------
// keys of a block of rows, large D
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) lantern_distance_tile_kernel(const float* __restrict__ cb, uint32_t* out, int V,
                                                                    int D, int row0, int rows) {
  __shared__ float As[TILE][DK + 1];
  __shared__ float Bs[TILE][DK + 1];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int rbase = row0 + blockIdx.y * TILE, cbase = blockIdx.x * TILE;
  float acc[4][4];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[r][c] = 0.0f;
  for (int d0 = 0; d0 < D; d0 += DK) {
#pragma unroll
    for (int l = 0; l < (TILE * DK) / 256; ++l) {
      const int e = l * 256 + tid, rr = e / DK, dd = e % DK;
      const int gr = rbase + rr, gc = cbase + rr, gd = d0 + dd;
      As[rr][dd] = (gr < row0 + rows && gr < V && gd < D) ? cb[static_cast<size_t>(gr) * D + gd] : 0.0f;
      Bs[rr][dd] = (gc < V && gd < D) ? cb[static_cast<size_t>(gc) * D + gd] : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int dd = 0; dd < DK; ++dd) {   // zero padding beyond D adds fma(0,0,acc) = acc exactly
      float a[4], b[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) a[r] = As[ty + 16 * r][dd];
#pragma unroll
      for (int c = 0; c < 4; ++c) b[c] = Bs[tx + 16 * c][dd];
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const float t = __fsub_rn(a[r], b[c]);
          acc[r][c] = __fmaf_rn(t, t, acc[r][c]);
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int gr = rbase + ty + 16 * r;
    if (gr >= row0 + rows || gr >= V) continue;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int gc = cbase + tx + 16 * c;
      if (gc < V) out[static_cast<size_t>(gr - row0) * V + gc] = __float_as_uint(acc[r][c]);
    }
  }
}

// ---------------------------------------------------------------------------------------
// one row: keys -> select -> sort -> store
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(BT) lantern_knn_row_kernel(BuildParams P, int P2 /* pow2 >= k-1 */) {
  extern __shared__ __align__(16) unsigned char dsm[];
  uint32_t* keys = reinterpret_cast<uint32_t*>(dsm);                                  // [V]
  unsigned long long* list =
      reinterpret_cast<unsigned long long*>(dsm + ((static_cast<size_t>(P.V) * 4 + 15) & ~size_t(15)));  // [P2]
  __shared__ int hist[256];
  __shared__ int wcnt[BW];
  __shared__ float ai[SMALL_D];
  __shared__ int s_digit, s_below, s_cnt;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int V = P.V, D = P.D, K = P.k - 1;
  const int i = P.row0 + blockIdx.x;

  // ---- keys ----
  if (P.scratch) {
    const uint32_t* src = P.scratch + static_cast<size_t>(blockIdx.x) * V;
    for (int j = tid; j < V; j += BT) keys[j] = src[j];
  } else {
    if (tid < D) ai[tid] = P.codebook[static_cast<size_t>(i) * D + tid];
    __syncthreads();
    if ((D & 3) == 0) {
      for (int j = tid; j < V; j += BT) {
        const float4* b = reinterpret_cast<const float4*>(P.codebook + static_cast<size_t>(j) * D);
        float acc = 0.0f;
        for (int d = 0; d < D; d += 4) {
          const float4 v = __ldg(b + (d >> 2));
          float t = __fsub_rn(ai[d], v.x);
          acc = __fmaf_rn(t, t, acc);
          t = __fsub_rn(ai[d + 1], v.y);
          acc = __fmaf_rn(t, t, acc);
          t = __fsub_rn(ai[d + 2], v.z);
          acc = __fmaf_rn(t, t, acc);
          t = __fsub_rn(ai[d + 3], v.w);
          acc = __fmaf_rn(t, t, acc);
        }
        keys[j] = __float_as_uint(acc);
      }
    } else {
      for (int j = tid; j < V; j += BT) {
        const float* b = P.codebook + static_cast<size_t>(j) * D;
        float acc = 0.0f;
        for (int d = 0; d < D; ++d) {
          const float t = __fsub_rn(ai[d], __ldg(b + d));
          acc = __fmaf_rn(t, t, acc);
        }
        keys[j] = __float_as_uint(acc);
      }
    }
  }
  __syncthreads();
  const uint32_t self_key = keys[i];
  __syncthreads();
  if (tid == 0) {
    keys[i] = 0xffffffffu;   // the code itself is placed in slot 0, not ranked
    s_cnt = 0;
  }
  __syncthreads();

  if (K > 0) {
    // ---- radix select: tau = K-th smallest key; `need` ties at tau are taken, smallest index first ----
    uint32_t prefix = 0, mask = 0;
    int need = K, ties_total = 0;
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      if (tid < 256) hist[tid] = 0;
      __syncthreads();
      for (int j = tid; j < V; j += BT) {
        const uint32_t key = keys[j];
        if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 0xff], 1);
      }
      __syncthreads();
      if (warp == 0) {
        int loc[8], s = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          loc[q] = hist[lane * 8 + q];
          s += loc[q];
        }
        int incl = s;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_up_sync(kFull, incl, o);
          if (lane >= o) incl += t;
        }
        const int excl = incl - s;
        if (excl < need && need <= incl) {   // exactly one lane
          int run = excl;
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            if (run < need && need <= run + loc[q]) {
              s_digit = lane * 8 + q;
              s_below = run;
            }
            run += loc[q];
          }
        }
      }
      __syncthreads();
      const int digit = s_digit;
      need -= s_below;
      ties_total = hist[digit];
      prefix |= static_cast<uint32_t>(digit) << shift;
      mask |= 0xffu << shift;
      __syncthreads();
    }
    const uint32_t tau = prefix;
    const int n_less = K - need;

    // ---- compaction ----
    const bool all_ties = (ties_total == need);
    for (int j = tid; j < V; j += BT) {
      const uint32_t key = keys[j];
      if (key < tau || (all_ties && key == tau)) {
        const int pos = atomicAdd(&s_cnt, 1);
        list[pos] = (static_cast<unsigned long long>(key) << 32) | static_cast<unsigned>(j);
      }
    }
    if (!all_ties) {   // more ties than places: take them in index order
      int run = 0;
      for (int base = 0; base < V && run < need; base += BT) {
        const int j = base + tid;
        const bool flag = j < V && keys[j] == tau;
        const unsigned bal = __ballot_sync(kFull, flag);
        if (lane == 0) wcnt[warp] = __popc(bal);
        __syncthreads();
        int before = 0, chunk = 0;
#pragma unroll
        for (int w = 0; w < BW; ++w) {
          const int c = wcnt[w];
          if (w < warp) before += c;
          chunk += c;
        }
        const int rank = run + before + __popc(bal & ((1u << lane) - 1u));
        if (flag && rank < need)
          list[n_less + rank] = (static_cast<unsigned long long>(tau) << 32) | static_cast<unsigned>(j);
        run += chunk;
        __syncthreads();
      }
    }
    for (int t = K + tid; t < P2; t += BT) list[t] = ~0ull;
    __syncthreads();

    // ---- bitonic sort of (key, index) composites ----
    for (int size = 2; size <= P2; size <<= 1) {
      for (int stride = size >> 1; stride > 0; stride >>= 1) {
        for (int t = tid; t < (P2 >> 1); t += BT) {
          const int lo = ((t & ~(stride - 1)) << 1) | (t & (stride - 1));
          const int hi = lo | stride;
          const bool up = (lo & size) == 0;
          const unsigned long long x = list[lo], y = list[hi];
          if ((x > y) == up) {
            list[lo] = y;
            list[hi] = x;
          }
        }
        __syncthreads();
      }
    }
  }

  // ---- store ----
  int32_t* irow = P.idx + static_cast<size_t>(i) * P.k;
  float* drow = P.dist ? P.dist + static_cast<size_t>(i) * P.k : nullptr;
  if (tid == 0) {
    irow[0] = i;
    if (drow) drow[0] = __uint_as_float(self_key);
  }
  for (int t = tid; t < K; t += BT) {
    const unsigned long long c = list[t];
    irow[1 + t] = static_cast<int32_t>(c & 0xffffffffu);
    if (drow) drow[1 + t] = __uint_as_float(static_cast<uint32_t>(c >> 32));
  }
}

static int next_pow2(int x) {
  int p = 1;
  while (p < x) p <<= 1;
  return p;
}

static int rows_per_block(int V) {
  int r = V < 1024 ? V : 1024;
  return (r + TILE - 1) / TILE * TILE;
}

}  // namespace lantern

using namespace lantern;

extern "C" size_t lantern_build_workspace_bytes(int V, int D, int k) {
  (void)k;
  if (V < 1 || D < 1) return 0;
  if (D <= SMALL_D) return 0;
  return static_cast<size_t>(rows_per_block(V)) * V * 4;
}

extern "C" lantern_status lantern_build_neighbors(const float* codebook, int V, int D, int k, int32_t* idx,
                                                  float* dist, void* workspace, size_t workspace_bytes,
                                                  void* cuda_stream) {
  if (V < 1 || V > 32768 || D < 1 || D > 4096 || k < 1 || k > V || k > 4097) return LANTERN_E_SHAPE;
  if (!codebook || !idx) return LANTERN_E_NULL;
  if ((reinterpret_cast<uintptr_t>(codebook) & 15)) return LANTERN_E_ALIGN;
  const size_t need_ws = lantern_build_workspace_bytes(V, D, k);
  if (need_ws && (!workspace || workspace_bytes < need_ws || (reinterpret_cast<uintptr_t>(workspace) & 15)))
    return LANTERN_E_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int P2 = k > 1 ? next_pow2(k - 1 < 2 ? 2 : k - 1) : 2;
  const size_t smem = ((static_cast<size_t>(V) * 4 + 15) & ~size_t(15)) + static_cast<size_t>(P2) * 8;
  if (smem > 220 * 1024) return LANTERN_E_SHAPE;
  if (cudaFuncSetAttribute(lantern_knn_row_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) !=
      cudaSuccess)
    return LANTERN_E_CUDA;
  BuildParams P;
  P.codebook = codebook;
  P.idx = idx;
  P.dist = dist;
  P.V = V;
  P.D = D;
  P.k = k;
  if (D <= SMALL_D) {
    P.scratch = nullptr;
    P.row0 = 0;
    lantern_knn_row_kernel<<<V, BT, smem, st>>>(P, P2);
    return cudaGetLastError() == cudaSuccess ? LANTERN_OK : LANTERN_E_CUDA;
  }
  const int rb = rows_per_block(V);
  uint32_t* scratch = static_cast<uint32_t*>(workspace);
  for (int row0 = 0; row0 < V; row0 += rb) {
    const int rows = V - row0 < rb ? V - row0 : rb;
    dim3 grid((V + TILE - 1) / TILE, (rows + TILE - 1) / TILE);
    lantern_distance_tile_kernel<<<grid, 256, 0, st>>>(codebook, scratch, V, D, row0, rows);
    if (cudaGetLastError() != cudaSuccess) return LANTERN_E_CUDA;
    P.scratch = scratch;
    P.row0 = row0;
    lantern_knn_row_kernel<<<rows, BT, smem, st>>>(P, P2);
    if (cudaGetLastError() != cudaSuccess) return LANTERN_E_CUDA;
  }
  return LANTERN_OK;
}

// ---------------------------------------------------------------------------------------
// Cosine variant of the latent proximity (Section 5.3.1): codes scaled to unit length, then the
// same neighbour build -- on unit vectors the squared distance is 2 - 2 cos, so increasing
// distance is decreasing cosine similarity.  One thread per code runs the canonical fp32
// sequence: squared norm by one fused multiply-add per dimension in dimension order, one square
// root, one division per component; a zero code stays zero.
// ---------------------------------------------------------------------------------------
namespace lantern {
__global__ void lantern_normalize_rows_kernel(const float* __restrict__ codebook, float* __restrict__ out, int V,
                                              int D) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= V) return;
  const float* a = codebook + static_cast<size_t>(i) * D;
  float n2 = 0.0f;
  for (int d = 0; d < D; ++d) n2 = __fmaf_rn(a[d], a[d], n2);
  const float n = __fsqrt_rn(n2);
  for (int d = 0; d < D; ++d) out[static_cast<size_t>(i) * D + d] = n > 0.0f ? __fdiv_rn(a[d], n) : 0.0f;
}
}  // namespace lantern

static size_t unit_codes_bytes(int V, int D) { return (static_cast<size_t>(V) * D * 4 + 255) & ~static_cast<size_t>(255); }

extern "C" size_t lantern_build_workspace_bytes_metric(int V, int D, int k, int metric) {
  if (V < 1 || D < 1 || (metric != LANTERN_METRIC_L2 && metric != LANTERN_METRIC_COSINE)) return 0;
  const size_t base = lantern_build_workspace_bytes(V, D, k);
  return metric == LANTERN_METRIC_COSINE ? unit_codes_bytes(V, D) + base : base;
}

extern "C" lantern_status lantern_build_neighbors_metric(const float* codebook, int V, int D, int k, int metric,
                                                         int32_t* idx, float* dist, void* workspace,
                                                         size_t workspace_bytes, void* cuda_stream) {
  if (metric == LANTERN_METRIC_L2)
    return lantern_build_neighbors(codebook, V, D, k, idx, dist, workspace, workspace_bytes, cuda_stream);
  if (metric != LANTERN_METRIC_COSINE) return LANTERN_E_PARAM;
  if (V < 1 || V > 32768 || D < 1 || D > 4096 || k < 1 || k > V || k > 4097) return LANTERN_E_SHAPE;
  if (!codebook || !idx) return LANTERN_E_NULL;
  const size_t unit = unit_codes_bytes(V, D);
  if (!workspace || workspace_bytes < lantern_build_workspace_bytes_metric(V, D, k, metric) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255))
    return LANTERN_E_WORKSPACE;
  float* unit_codes = static_cast<float*>(workspace);
  lantern::lantern_normalize_rows_kernel<<<(V + 127) / 128, 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      codebook, unit_codes, V, D);
  if (cudaGetLastError() != cudaSuccess) return LANTERN_E_CUDA;
  return lantern_build_neighbors(unit_codes, V, D, k, idx, dist, static_cast<unsigned char*>(workspace) + unit,
                                 workspace_bytes - unit, cuda_stream);
}
