// Instantiations and host launcher of the tcgen05 grouped GEMM.
#include "gemm_tcgen05_pair.cuh"
#include "kernels.h"

namespace foe {

cudaError_t gemm_configure() {
  cudaError_t e;
  e = cudaFuncSetAttribute(gemm_tcgen05_kernel<kEpiSwiGLU, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kGemmSmemBytes));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(gemm_tcgen05_kernel<kEpiOProj, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kGemmSmemBytes));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(gemm_tcgen05_pair_kernel<kEpiBf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kPairSmemBytes));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(gemm_tcgen05_pair_kernel<kEpiQKV>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kPairSmemBytes));
  return e;
}

void launch_gemm(int epi, const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmArgs& args_in, int n_sms,
                 cudaStream_t st) {
  GemmArgs args = args_in;
  args.bn = epi == kEpiSwiGLU ? kBN : gemm_tile_cols(args.N);     // gate and up halves need the full 256-wide tile
  int grid = n_sms;
  if (args.n_mtiles == nullptr) {
    const int tiles = args.n_groups * ((args.rows_per_group + kBM - 1) / kBM) * ((args.N + args.bn - 1) / args.bn);
    if (tiles < grid) grid = tiles;
    if (grid <= 0) return;
  }
  // one CTA per tile: the gathered expert GEMM 1 and the output projection (whose epilogue, not its MMAs, sets
  // its time); the other GEMMs run on CTA pairs
  if (epi == kEpiSwiGLU)   // always fed through the dispatch permutation
    gemm_tcgen05_kernel<kEpiSwiGLU, true><<<grid, kGemmThreads + kGatherThreads, kGemmSmemBytes, st>>>(tmA, tmB, args);
  else
    gemm_tcgen05_kernel<kEpiOProj, false><<<grid, kGemmThreads, kGemmSmemBytes, st>>>(tmA, tmB, args);
}

// CTA-pair variant (no gathered A): the box of tmB is gemm_tile_cols(N) / 2 rows, a ragged problem brings the table
// of 256-row tiles.
void launch_gemm_pair(int epi, const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmArgs& args_in, int n_sms,
                      cudaStream_t st) {
  GemmArgs args = args_in;
  args.bn = gemm_tile_cols(args.N);
  int pairs = n_sms / 2;
  if (args.n_mtiles == nullptr) {
    const int tiles = args.n_groups * ((args.rows_per_group + kPairTileRows - 1) / kPairTileRows) * ((args.N + args.bn - 1) / args.bn);
    if (tiles < pairs) pairs = tiles;
  }
  if (pairs <= 0) return;
  if (epi == kEpiQKV) gemm_tcgen05_pair_kernel<kEpiQKV><<<2 * pairs, kGemmThreads, kPairSmemBytes, st>>>(tmA, tmB, args);
  else gemm_tcgen05_pair_kernel<kEpiBf16><<<2 * pairs, kGemmThreads, kPairSmemBytes, st>>>(tmA, tmB, args);
}

}  // namespace foe
