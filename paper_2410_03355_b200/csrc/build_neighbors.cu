// Neighbour table B_k of a VQ codebook (Algorithm 2, block "Precompute B_k for all tokens").
//
// Key of a pair (i, j): squared l2 distance accumulated in fp32 in dimension order,
// acc = fma(a_d - b_d, a_d - b_d, acc).  That exact operation sequence is kept whatever the
// tiling, so the order of neighbours does not depend on how the work is split.
//
// Small D (<= 32): one CTA per code computes its V keys straight into shared memory.
// Large D: a tiled SIMT kernel writes the keys of a block of rows to global scratch (each
// (i, j) accumulator still runs over d in order), and the per-row CTA reads its row of keys.
// Per row (the code itself excluded; it goes to slot 0): the keys' range, one 2048-bin histogram of
// the top 11 bits of key - min, the bin that holds the (k-1)-th smallest key and every bin's offset
// by one block scan, then a counting sort -- the index of every key up to that bin is scattered to
// its bin's place, ranked inside its bin by (key, index), and stored at its final position, so that
// ties at the threshold are taken by smaller index.  A row in which one of those bins holds more
// than 256 keys (massive ties, an outlier that stretches the range) takes the general path:
// further histogram passes down to the exact threshold key, compaction of the selected
// (key, index) pairs, bitonic sort of the 64-bit composites.
#include <cuda_runtime.h>
#include <stdint.h>

#include "lantern.h"
#include "lantern_device.cuh"

namespace lantern {

constexpr int BT = 512;          // threads of the per-row kernel
constexpr int BW = BT / 32;
constexpr int SMALL_D = 32;
constexpr int TM = 128;          // distance tile edge (rows and columns of one CTA)
constexpr int DK = 16;           // dimensions staged per step
constexpr int HB = 11;           // radix-select digit: 2048 bins, kept in the (still unused) list area
constexpr int HBINS = 1 << HB;
constexpr int FAST_POP = 256;    // largest bin the counting-sort path ranks by pairwise comparison

struct BuildParams {
  const float* codebook;
  const uint32_t* scratch;       // [rows, V] key bits of rows row0.. (large-D path), else null
  int32_t* idx;
  float* dist;
  int V, D, k, row0;
};

// Two fp32 lanes in one 64-bit register; each lane of the packed operations rounds exactly like the
// scalar instruction, so the key sequence is unchanged.
__device__ __forceinline__ unsigned long long dup2(float a) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %1};" : "=l"(r) : "f"(a));
  return r;
}
__device__ __forceinline__ unsigned long long sub2(unsigned long long a, unsigned long long b) {
  unsigned long long r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}

// ---------------------------------------------------------------------------------------
// keys of a block of rows, large D: a 128 x 128 tile per CTA, 8 x 8 accumulators per thread
// (rows ty*4.. and 64+ty*4.., columns tx*4.. and 64+tx*4.., so that every shared-memory read is
// one conflict-free 16-byte load), the next 16 dimensions fetched into registers while the
// current ones are used.  Every (i, j) accumulator still runs over d in order.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float4 fetch_quad(const float* __restrict__ cb, int row, int row_end, int D, int d, bool vec) {
  float4 v = make_float4(0.0f, 0.0f, 0.0f, 0.0f);   // zero padding adds fma(0, 0, acc) = acc exactly
  if (row < row_end) {
    const float* p = cb + static_cast<size_t>(row) * D + d;
    if (vec && d + 3 < D) {
      v = __ldg(reinterpret_cast<const float4*>(p));
    } else {
      if (d < D) v.x = __ldg(p);
      if (d + 1 < D) v.y = __ldg(p + 1);
      if (d + 2 < D) v.z = __ldg(p + 2);
      if (d + 3 < D) v.w = __ldg(p + 3);
    }
  }
  return v;
}

__global__ void __launch_bounds__(256, 2) lantern_distance_tile_kernel(const float* __restrict__ cb, uint32_t* out, int V,
                                                                       int D, int row0, int rows) {
  __shared__ __align__(16) float As[DK][TM];
  __shared__ __align__(16) float Bs[DK][TM];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int rbase = row0 + blockIdx.y * TM, cbase = blockIdx.x * TM;
  const int row_end = (row0 + rows < V) ? row0 + rows : V;
  const bool vec = (D & 3) == 0;
  unsigned long long acc[8][4];
#pragma unroll
  for (int r = 0; r < 8; ++r)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[r][c] = 0ull;
  // staging: element e = l * 256 + tid of a 128 x 16 tile is (row e & 127, dimensions 4 * (e >> 7) ..+3)
  const int srow = tid & 127, squad = tid >> 7;
  float4 ra[2], rb[2];
#pragma unroll
  for (int l = 0; l < 2; ++l) {
    ra[l] = fetch_quad(cb, rbase + srow, row_end, D, 4 * (squad + 2 * l), vec);
    rb[l] = fetch_quad(cb, cbase + srow, V, D, 4 * (squad + 2 * l), vec);
  }
  for (int d0 = 0; d0 < D; d0 += DK) {
#pragma unroll
    for (int l = 0; l < 2; ++l) {
      const int q = 4 * (squad + 2 * l);
      As[q][srow] = ra[l].x;
      As[q + 1][srow] = ra[l].y;
      As[q + 2][srow] = ra[l].z;
      As[q + 3][srow] = ra[l].w;
      Bs[q][srow] = rb[l].x;
      Bs[q + 1][srow] = rb[l].y;
      Bs[q + 2][srow] = rb[l].z;
      Bs[q + 3][srow] = rb[l].w;
    }
    __syncthreads();
    if (d0 + DK < D) {
#pragma unroll
      for (int l = 0; l < 2; ++l) {
        ra[l] = fetch_quad(cb, rbase + srow, row_end, D, d0 + DK + 4 * (squad + 2 * l), vec);
        rb[l] = fetch_quad(cb, cbase + srow, V, D, d0 + DK + 4 * (squad + 2 * l), vec);
      }
    }
#pragma unroll
    for (int dd = 0; dd < DK; ++dd) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[dd][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[dd][64 + ty * 4]);
      const ulonglong2 b0 = *reinterpret_cast<const ulonglong2*>(&Bs[dd][tx * 4]);
      const ulonglong2 b1 = *reinterpret_cast<const ulonglong2*>(&Bs[dd][64 + tx * 4]);
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const unsigned long long b[4] = {b0.x, b0.y, b1.x, b1.y};
#pragma unroll
      for (int r = 0; r < 8; ++r) {
        const unsigned long long aa = dup2(a[r]);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const unsigned long long t = sub2(aa, b[c]);
          acc[r][c] = fma2(t, t, acc[r][c]);
        }
      }
    }
    __syncthreads();
  }
  const bool vec_out = (V & 3) == 0;
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    const int gr = rbase + (r < 4 ? ty * 4 + r : 64 + ty * 4 + (r - 4));
    if (gr >= row_end) continue;
    uint32_t* orow = out + static_cast<size_t>(gr - row0) * V;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int gc = cbase + 64 * h + tx * 4;
      const unsigned long long p0 = acc[r][2 * h], p1 = acc[r][2 * h + 1];
      const uint32_t w[4] = {static_cast<uint32_t>(p0), static_cast<uint32_t>(p0 >> 32), static_cast<uint32_t>(p1),
                             static_cast<uint32_t>(p1 >> 32)};
      if (vec_out && gc + 3 < V) {
        *reinterpret_cast<uint4*>(orow + gc) = make_uint4(w[0], w[1], w[2], w[3]);
      } else {
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if (gc + c < V) orow[gc + c] = w[c];
      }
    }
  }
}

// ---------------------------------------------------------------------------------------
// one row: keys -> select -> sort -> store
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long shfl_xor_u64(unsigned long long x, int m) {
  const unsigned lo = __shfl_xor_sync(kFull, static_cast<unsigned>(x), m);
  const unsigned hi = __shfl_xor_sync(kFull, static_cast<unsigned>(x >> 32), m);
  return (static_cast<unsigned long long>(hi) << 32) | lo;
}

// Bitonic merge steps of strides 32..1 on one 64-element block held by a warp (elements lane and
// lane + 32), for every merge size from size_lo to size_hi whose strides all lie inside the block.
__device__ __forceinline__ void bitonic_block64(unsigned long long* list, int block, int lane, int size_lo, int size_hi) {
  const int e0 = block * 64 + lane, e1 = e0 + 32;
  unsigned long long x0 = list[e0], x1 = list[e1];
  for (int size = size_lo; size <= size_hi; size <<= 1) {
    if (size >= 64) {
      const bool up = (e0 & size) == 0;
      if ((x0 > x1) == up) {
        const unsigned long long t = x0;
        x0 = x1;
        x1 = t;
      }
    }
    for (int stride = size >= 64 ? 16 : (size >> 1); stride > 0; stride >>= 1) {
      const bool am_lo = (lane & stride) == 0;
      const unsigned long long o0 = shfl_xor_u64(x0, stride), o1 = shfl_xor_u64(x1, stride);
      const bool up0 = (e0 & size) == 0, up1 = (e1 & size) == 0;
      x0 = (am_lo == up0) ? (x0 < o0 ? x0 : o0) : (x0 > o0 ? x0 : o0);
      x1 = (am_lo == up1) ? (x1 < o1 ? x1 : o1) : (x1 > o1 ? x1 : o1);
    }
  }
  list[e0] = x0;
  list[e1] = x1;
}

__global__ void __launch_bounds__(BT) lantern_knn_row_kernel(BuildParams P, int P2 /* pow2 >= max(k-1, 64) */) {
  extern __shared__ __align__(16) unsigned char dsm[];
  uint32_t* keys = reinterpret_cast<uint32_t*>(dsm);                                  // [V]
  unsigned long long* list =
      reinterpret_cast<unsigned long long*>(dsm + ((static_cast<size_t>(P.V) * 4 + 15) & ~size_t(15)));  // [P2]
  // [HBINS] 16-bit counters, two to a word (a row has fewer than 65536 keys); used before the list is filled
  unsigned* hist = reinterpret_cast<unsigned*>(list);
  unsigned short* list16 = reinterpret_cast<unsigned short*>(hist + HBINS / 2);   // [k - 1 + FAST_POP] indices, fast path
  auto bin_count = [hist](int b) { return static_cast<int>((hist[b >> 1] >> ((b & 1) << 4)) & 0xffffu); };
  __shared__ int wcnt[BW];
  __shared__ uint32_t wmin[BW], wmax[BW];
  __shared__ float ai[SMALL_D];
  __shared__ int s_digit, s_below, s_ties, s_cnt;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int V = P.V, D = P.D, K = P.k - 1;
  const int i = P.row0 + blockIdx.x;

  // ---- keys (and their range over j != i) ----
  uint32_t kmin = 0xffffffffu, kmax = 0u;
  if (P.scratch) {
    const uint32_t* src = P.scratch + static_cast<size_t>(blockIdx.x) * V;
    for (int j = tid; j < V; j += BT) {
      const uint32_t key = src[j];
      keys[j] = key;
      if (j != i) {
        kmin = key < kmin ? key : kmin;
        kmax = key > kmax ? key : kmax;
      }
    }
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
        const uint32_t key = __float_as_uint(acc);
        keys[j] = key;
        if (j != i) {
          kmin = key < kmin ? key : kmin;
          kmax = key > kmax ? key : kmax;
        }
      }
    } else {
      for (int j = tid; j < V; j += BT) {
        const float* b = P.codebook + static_cast<size_t>(j) * D;
        float acc = 0.0f;
        for (int d = 0; d < D; ++d) {
          const float t = __fsub_rn(ai[d], __ldg(b + d));
          acc = __fmaf_rn(t, t, acc);
        }
        const uint32_t key = __float_as_uint(acc);
        keys[j] = key;
        if (j != i) {
          kmin = key < kmin ? key : kmin;
          kmax = key > kmax ? key : kmax;
        }
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const uint32_t a = __shfl_xor_sync(kFull, kmin, o), b = __shfl_xor_sync(kFull, kmax, o);
    kmin = a < kmin ? a : kmin;
    kmax = b > kmax ? b : kmax;
  }
  if (lane == 0) {
    wmin[warp] = kmin;
    wmax[warp] = kmax;
  }
  if (tid == 0) s_cnt = 0;
  __syncthreads();
  const uint32_t self_key = keys[i];
#pragma unroll
  for (int w = 0; w < BW; ++w) {
    kmin = wmin[w] < kmin ? wmin[w] : kmin;
    kmax = wmax[w] > kmax ? wmax[w] : kmax;
  }

  if (K > 0) {
    // ---- radix select on rel = key - kmin, 11 bits at a time from the top of the occupied range:
    //      tau = K-th smallest key over j != i; `need` ties at tau are taken, smallest index first ----
    const uint32_t range = kmax - kmin;
    int hi = range ? 32 - __clz(range) : 0;
    uint32_t prefix = 0;
    int need = K, ties_total = V - 1;
    bool first_pass = true;
    while (hi > 0) {
      const int lo = hi > HB ? hi - HB : 0;
      const uint32_t dmask = (1u << (hi - lo)) - 1u;
      for (int t = tid; t < HBINS / 2; t += BT) hist[t] = 0u;
      __syncthreads();
      for (int j = tid; j < V; j += BT) {
        const uint32_t rel = keys[j] - kmin;
        if (j != i && (hi >= 32 || (rel >> hi) == (prefix >> hi))) {
          const uint32_t b = (rel >> lo) & dmask;
          atomicAdd(&hist[b >> 1], 1u << ((b & 1u) << 4));
        }
      }
      __syncthreads();
      int loc[HBINS / BT], s = 0;
#pragma unroll
      for (int q = 0; q < HBINS / BT; ++q) {
        loc[q] = bin_count(tid * (HBINS / BT) + q);
        s += loc[q];
      }
      int incl = s;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += t;
      }
      if (lane == 31) wcnt[warp] = incl;
      __syncthreads();
      int excl = incl - s;
#pragma unroll
      for (int w = 0; w < BW; ++w)
        if (w < warp) excl += wcnt[w];
      if (excl < need && need <= excl + s) {   // exactly one thread
        int run = excl;
#pragma unroll
        for (int q = 0; q < HBINS / BT; ++q) {
          if (run < need && need <= run + loc[q]) {
            s_digit = tid * (HBINS / BT) + q;
            s_below = run;
            s_ties = loc[q];
          }
          run += loc[q];
        }
      }
      __syncthreads();
      if (first_pass) {
        // Common case: no bin up to the one that holds the K-th key is crowded.  The prefix sums of the
        // histogram are then the places of a counting sort by bin: scatter the indices of those keys,
        // rank every key inside its bin by (key, index), and store it at its final place.
        first_pass = false;
        const int digit = s_digit, n_cand = s_below + s_ties;
        bool crowded = false;
#pragma unroll
        for (int q = 0; q < HBINS / BT; ++q) crowded |= (tid * (HBINS / BT) + q <= digit) && loc[q] > FAST_POP;
        if (!__syncthreads_or(crowded)) {
          // own words only: each counter becomes its bin's cursor (offsets stay below 65536; bins past `digit`
          // are never advanced)
          static_assert(HBINS / BT == 4, "a thread owns two words of counters");
          hist[2 * tid] = static_cast<unsigned>(excl) | (static_cast<unsigned>(excl + loc[0]) << 16);
          hist[2 * tid + 1] = static_cast<unsigned>(excl + loc[0] + loc[1]) |
                              (static_cast<unsigned>(excl + loc[0] + loc[1] + loc[2]) << 16);
          __syncthreads();
          for (int j = tid; j < V; j += BT) {
            const int b = static_cast<int>((keys[j] - kmin) >> lo);
            if (j != i && b <= digit) {
              const int sh = (b & 1) << 4;
              const unsigned old = atomicAdd(&hist[b >> 1], 1u << sh);
              list16[(old >> sh) & 0xffffu] = static_cast<unsigned short>(j);
            }
          }
          __syncthreads();   // every cursor now holds the end of its bin = the start of the next
          int32_t* irow = P.idx + static_cast<size_t>(i) * P.k;
          float* drow = P.dist ? P.dist + static_cast<size_t>(i) * P.k : nullptr;
          if (tid == 0) {
            irow[0] = i;
            if (drow) drow[0] = __uint_as_float(self_key);
          }
          for (int t = tid; t < n_cand; t += BT) {
            const unsigned j = list16[t];
            const uint32_t key = keys[j];
            const int b = static_cast<int>((key - kmin) >> lo);
            const int start = b ? bin_count(b - 1) : 0, end = bin_count(b);
            const unsigned long long comp = (static_cast<unsigned long long>(key) << 32) | j;
            int rank = start;
            for (int u = start; u < end; ++u) {
              const unsigned ju = list16[u];
              rank += ((static_cast<unsigned long long>(keys[ju]) << 32) | ju) < comp;
            }
            if (rank < K) {   // in the last bin: the `need` smallest, ties by smaller index
              irow[1 + rank] = static_cast<int32_t>(j);
              if (drow) drow[1 + rank] = __uint_as_float(key);
            }
          }
          return;
        }
      }
      need -= s_below;
      ties_total = s_ties;
      prefix |= static_cast<uint32_t>(s_digit) << lo;
      hi = lo;
    }
    __syncthreads();   // the histogram's storage becomes the list
    const uint32_t tau = kmin + prefix;
    const int n_less = K - need;

    // ---- compaction (one counter update per warp) ----
    const bool all_ties = (ties_total == need);
    for (int base = 0; base < V; base += BT) {
      const int j = base + tid;
      const uint32_t key = j < V ? keys[j] : 0u;
      const bool sel = j < V && j != i && (key < tau || (all_ties && key == tau));
      const unsigned bal = __ballot_sync(kFull, sel);
      if (bal) {
        int pos = 0;
        if (lane == 0) pos = atomicAdd(&s_cnt, __popc(bal));
        pos = __shfl_sync(kFull, pos, 0) + __popc(bal & ((1u << lane) - 1u));
        if (sel) list[pos] = (static_cast<unsigned long long>(key) << 32) | static_cast<unsigned>(j);
      }
    }
    if (!all_ties) {   // more ties than places: take them in index order
      int run = 0;
      for (int base = 0; base < V && run < need; base += BT) {
        const int j = base + tid;
        const bool flag = j < V && j != i && keys[j] == tau;
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

    // ---- bitonic sort of (key, index) composites: strides below 64 in registers by shuffles ----
    const int nblk = P2 >> 6;
    for (int blk = warp; blk < nblk; blk += BW) bitonic_block64(list, blk, lane, 2, 64);
    __syncthreads();
    for (int size = 128; size <= P2; size <<= 1) {
      for (int stride = size >> 1; stride >= 64; stride >>= 1) {
        for (int t = tid; t < (P2 >> 1); t += BT) {
          const int lo = ((t & ~(stride - 1)) << 1) | (t & (stride - 1));
          const int hi2 = lo | stride;
          const bool up = (lo & size) == 0;
          const unsigned long long x = list[lo], y = list[hi2];
          if ((x > y) == up) {
            list[lo] = y;
            list[hi2] = x;
          }
        }
        __syncthreads();
      }
      for (int blk = warp; blk < nblk; blk += BW) bitonic_block64(list, blk, lane, size, size);
      __syncthreads();
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

// Rows whose keys are held in scratch at a time: 64 MB at V = 16384, which the per-row kernel still finds
// in L2 (1152 rows, which would fill the distance kernel's last wave of CTAs, measured slower).
static int rows_per_block(int V) {
  int r = V < 1024 ? V : 1024;
  return (r + TM - 1) / TM * TM;
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
  const int P2 = next_pow2(k - 1 < 64 ? 64 : k - 1);   // the sort works on whole 64-element blocks
  const size_t fast_bytes = HBINS * 2 + ((static_cast<size_t>(k - 1 + FAST_POP) * 2 + 15) & ~size_t(15));
  const size_t list_bytes = static_cast<size_t>(P2) * 8 > fast_bytes ? static_cast<size_t>(P2) * 8 : fast_bytes;
  const size_t smem = ((static_cast<size_t>(V) * 4 + 15) & ~size_t(15)) + list_bytes;
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
    dim3 grid((V + TM - 1) / TM, (rows + TM - 1) / TM);
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
