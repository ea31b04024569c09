// Instantiations and host launcher of the tcgen05 grouped GEMM.
#include "gemm_tcgen05.cuh"
#include "kernels.h"

namespace foe {

cudaError_t gemm_configure() {
  cudaError_t e;
  e = cudaFuncSetAttribute(gemm_tcgen05_kernel<kEpiBf16, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kGemmSmemBytes));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(gemm_tcgen05_kernel<kEpiSwiGLU, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kGemmSmemBytes));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(gemm_tcgen05_kernel<kEpiQKV, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kGemmSmemBytes));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(gemm_tcgen05_kernel<kEpiOProj, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kGemmSmemBytes));
  return e;
}

// The box of tmB is gemm_tile_rows_b(epi, N) rows (half a tile: each CTA of a pair loads its half); a ragged problem
// brings the device-built table of 256-row tiles.
void launch_gemm(int epi, const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmArgs& args_in, int n_sms,
                 cudaStream_t st) {
  GemmArgs args = args_in;
  args.bn = 2 * gemm_tile_rows_b(epi, args.N);
  int pairs = n_sms / 2;
  if (args.n_mtiles == nullptr) {
    const int tiles = args.n_groups * ((args.rows_per_group + kPairTileRows - 1) / kPairTileRows) * ((args.N + args.bn - 1) / args.bn);
    if (tiles < pairs) pairs = tiles;
  }
  if (pairs <= 0) return;
  switch (epi) {
    case kEpiBf16: launch_pdl(gemm_tcgen05_kernel<kEpiBf16, false>, dim3(2 * pairs), dim3(kGemmThreads), kGemmSmemBytes, st, tmA, tmB, args); break;
    case kEpiSwiGLU:   // expert GEMM 1: always fed through the dispatch permutation (tmA unused)
      launch_pdl(gemm_tcgen05_kernel<kEpiSwiGLU, true>, dim3(2 * pairs), dim3(kGemmThreads + kGatherThreads), kGemmSmemBytes, st, tmA, tmB, args);
      break;
    case kEpiQKV: launch_pdl(gemm_tcgen05_kernel<kEpiQKV, false>, dim3(2 * pairs), dim3(kGemmThreads), kGemmSmemBytes, st, tmA, tmB, args); break;
    default: launch_pdl(gemm_tcgen05_kernel<kEpiOProj, false>, dim3(2 * pairs), dim3(kGemmThreads), kGemmSmemBytes, st, tmA, tmB, args); break;
  }
}

}  // namespace foe
