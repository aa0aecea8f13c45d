// One compile-time variant (TONE, JSD, TOPK) of the fused context kernel for every row layout:
// included by verify_context_v*.cu after defining LANTERN_VARIANT_{TONE,JSD,TOPK,NAME}.
#include "verify_common.cuh"
#include "verify_context.cuh"

namespace lantern {

template <int CHC, bool BF16, bool UNC>
static cudaError_t launch_one(const VerifyParams& P, int grid, size_t smem_bytes, cudaStream_t st) {
  auto kc = lantern_context_kernel<CHC, BF16, UNC, LANTERN_VARIANT_TONE, LANTERN_VARIANT_JSD, LANTERN_VARIANT_TOPK>;
  cudaError_t e = cudaFuncSetAttribute(kc, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_bytes));
  if (e != cudaSuccess) return e;
  kc<<<grid, CTX_THREADS, smem_bytes, st>>>(P);
  return cudaGetLastError();
}

template <int CHC>
static cudaError_t launch_layout(const VerifyParams& P, bool bf, bool un, int grid, size_t smem_bytes, cudaStream_t st) {
  return bf ? (un ? launch_one<CHC, true, true>(P, grid, smem_bytes, st) : launch_one<CHC, true, false>(P, grid, smem_bytes, st))
            : (un ? launch_one<CHC, false, true>(P, grid, smem_bytes, st) : launch_one<CHC, false, false>(P, grid, smem_bytes, st));
}

cudaError_t LANTERN_VARIANT_NAME(const VerifyParams& P, int CH, bool bf, bool un, int grid, size_t smem_bytes,
                                 cudaStream_t st) {
  return CH == 8 ? launch_layout<8>(P, bf, un, grid, smem_bytes, st)
                 : (CH == 4 ? launch_layout<4>(P, bf, un, grid, smem_bytes, st)
                            : (CH == 2 ? launch_layout<2>(P, bf, un, grid, smem_bytes, st)
                                       : launch_layout<1>(P, bf, un, grid, smem_bytes, st)));
}

}  // namespace lantern
