// Instantiations and host launcher of the tcgen05 grouped GEMM.
#include "gemm_tcgen05.cuh"
#include "kernels.h"

namespace foe {

cudaError_t gemm_configure() {
  cudaError_t e;
  e = cudaFuncSetAttribute(gemm_tcgen05_kernel<kEpiBf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kGemmSmemBytes));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(gemm_tcgen05_kernel<kEpiSwiGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kGemmSmemBytes));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(gemm_tcgen05_kernel<kEpiQKV>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kGemmSmemBytes));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(gemm_tcgen05_kernel<kEpiOProj>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kGemmSmemBytes));
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
    case kEpiBf16: gemm_tcgen05_kernel<kEpiBf16><<<grid, kGemmThreads, kGemmSmemBytes, st>>>(tmA, tmB, args); break;
    case kEpiSwiGLU: gemm_tcgen05_kernel<kEpiSwiGLU><<<grid, kGemmThreads, kGemmSmemBytes, st>>>(tmA, tmB, args); break;
    case kEpiQKV: gemm_tcgen05_kernel<kEpiQKV><<<grid, kGemmThreads, kGemmSmemBytes, st>>>(tmA, tmB, args); break;
    default: gemm_tcgen05_kernel<kEpiOProj><<<grid, kGemmThreads, kGemmSmemBytes, st>>>(tmA, tmB, args); break;
  }
}

}  // namespace foe
