// Instantiations and host launcher of the tcgen05 grouped GEMM.
#include "gemm_tcgen05_pair.cuh"
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
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(gemm_tcgen05_pair_kernel<kEpiBf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kPairSmemBytes));
  return e;
}

void launch_gemm(int epi, const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmArgs& args, int n_sms,
                 cudaStream_t st) {
  int grid = n_sms;
  if (args.n_mtiles == nullptr) {
    const int tiles = args.n_groups * ((args.rows_per_group + kBM - 1) / kBM) * ((args.N + kBN - 1) / kBN);
    if (tiles < grid) grid = tiles;
    if (grid <= 0) return;
  }
  switch (epi) {
    case kEpiBf16: gemm_tcgen05_kernel<kEpiBf16, false><<<grid, kGemmThreads, kGemmSmemBytes, st>>>(tmA, tmB, args); break;
    case kEpiSwiGLU:   // expert GEMM 1: always fed through the dispatch permutation
      gemm_tcgen05_kernel<kEpiSwiGLU, true><<<grid, kGemmThreads + kGatherThreads, kGemmSmemBytes, st>>>(tmA, tmB, args);
      break;
    case kEpiQKV: gemm_tcgen05_kernel<kEpiQKV, false><<<grid, kGemmThreads, kGemmSmemBytes, st>>>(tmA, tmB, args); break;
    default: gemm_tcgen05_kernel<kEpiOProj, false><<<grid, kGemmThreads, kGemmSmemBytes, st>>>(tmA, tmB, args); break;
  }
}

// CTA-pair variant (no gathered A): tmB must have 128-row boxes, a ragged problem the table of 256-row tiles.
void launch_gemm_pair(const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmArgs& args, int n_sms,
                      cudaStream_t st) {
  int pairs = n_sms / 2;
  if (args.n_mtiles == nullptr) {
    const int tiles = args.n_groups * ((args.rows_per_group + kPairTileRows - 1) / kPairTileRows) * ((args.N + kBN - 1) / kBN);
    if (tiles < pairs) pairs = tiles;
  }
  if (pairs <= 0) return;
  // only the plain bf16 epilogue is instantiated: the projections are bound by their epilogues, not by the MMA
  gemm_tcgen05_pair_kernel<kEpiBf16><<<2 * pairs, kGemmThreads, kPairSmemBytes, st>>>(tmA, tmB, args);
}

}  // namespace foe
