// The grouped GEMM of gemm_tcgen05.cuh on CTA PAIRS: a cluster of two CTAs (two SMs) computes one 256 x 256 output
// tile with tcgen05.mma.cta_group::2.  Each CTA stages only its own 128 A rows and its own 128 of the 256 B rows, so
// per SM the shared-memory traffic of the tensor core drops from 48 KB to 32 KB per k-block and six stages fit where
// four did.  The leader CTA (cluster rank 0) issues the MMAs for both; accumulators live in each CTA's own tensor
// memory (its 128 rows x 256 columns, two stages) and each CTA's epilogue warps drain their half.
//
// Barrier protocol (every barrier exists in both CTAs at the same shared-memory offset):
//   full[s]      used in the leader: 1 arrival (leader's expect_tx) + the bytes of BOTH CTAs' TMA loads
//   empty[s]     used in each CTA: 1 arrival from the leader's multicast tcgen05.commit
//   acc_full[a]  used in each CTA: 1 arrival from the leader's multicast tcgen05.commit
//   acc_empty[a] used in the leader: 16 arrivals (8 epilogue warps of each CTA; the peer's arrive remotely)
#pragma once

#include "gemm_tcgen05.cuh"

namespace foe {

constexpr int kPairStages = 6;
constexpr int kPairBBytes = (kBN / 2) * kBK * 2;                       // this CTA's half of the B tile: 16 KB
constexpr int kPairStageBytes = kABytes + kPairBBytes;                 // 32 KB
constexpr size_t kPairSmemBytes = size_t(kPairStages) * kPairStageBytes + kEpiWarps * kStgWarpBytes + 1024 + 256;
constexpr int kPairTileRows = 2 * kBM;                                 // 256 rows per pair tile

template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
gemm_tcgen05_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                         const GemmArgs args) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* stg_all = smem + kPairStages * kPairStageBytes;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(stg_all + kEpiWarps * kStgWarpBytes);
  uint64_t* empty_bar = full_bar + kPairStages;
  uint64_t* acc_full = empty_bar + kPairStages;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();               // 0 = leader
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kPairStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], 1);
    }
    for (int s = 0; s < 2; ++s) { mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], 2 * kEpiWarps); }
    mbar_fence_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
  }
  __syncthreads();
  cluster_sync_all();                                    // both CTAs' barriers exist before anything remote touches them
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // tiles: groups are cut into 256-row pair tiles (the device-built table for the ragged experts uses the same size)
  const bool ragged = args.n_mtiles != nullptr;
  const int tiles_per_group = (args.rows_per_group + kPairTileRows - 1) / kPairTileRows;
  const int n_mtiles = ragged ? *args.n_mtiles : args.n_groups * tiles_per_group;
  const int bn = args.bn;                                // tile width; each CTA stages bn / 2 rows of B (= the B map's box)
  const int n_ntiles = (args.N + bn - 1) / bn;
  const int total_tiles = n_mtiles * n_ntiles;
  const int kblocks = (args.K + kBK - 1) / kBK;

  auto tile_coords = [&](int tile, int& group, int& row0, int& row_end, int& group_row0, int& nt) {
    const int mt = tile / n_ntiles;
    nt = tile - mt * n_ntiles;
    if (ragged) {
      group = args.mt_group[mt]; row0 = args.mt_row0[mt]; row_end = args.group_end[group]; group_row0 = 0;
    } else {
      group = mt / tiles_per_group;
      group_row0 = group * args.a_group_stride;
      row0 = group_row0 + (mt - group * tiles_per_group) * kPairTileRows;
      row_end = group_row0 + args.rows_per_group;
    }
    row0 += int(rank) * kBM;                             // this CTA's 128 rows of the pair tile
  };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (one thread per CTA)
    if (elect_one()) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
        int group, row0, row_end, group_row0, nt;
        tile_coords(tile, group, row0, row_end, group_row0, nt);
        const int brow0 = group * args.N + nt * bn + int(rank) * (bn / 2);       // this CTA's half of the B rows
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(&empty_bar[stage], phase ^ 1)) { ok = false; break; }
          uint8_t* sa = smem + stage * kPairStageBytes;
          if (leader) mbar_expect_tx(&full_bar[stage], 2 * (kABytes + (bn / 2) * (kBK * 2)));
          tma_load_2d_pair(sa, &tmA, &full_bar[stage], kb * kBK, row0);
          tma_load_2d_pair(sa + kABytes, &tmB, &full_bar[stage], kb * kBK, brow0);
          if (++stage == kPairStages) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) atomicExch(args.status, kStatusTimeout);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (one thread of the leader CTA)
    if (leader && elect_one()) {
      const uint32_t idesc = umma_idesc_bf16(kPairTileRows, bn);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int tile = pair; tile < total_tiles && ok; tile += n_pairs, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1;
        if (!mbar_wait(&acc_empty[acc], acc_phase ^ 1)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * kBN;
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(&full_bar[stage], phase)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(smem + stage * kPairStageBytes);
          const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) {
            umma_bf16_pair(d_tmem, umma_desc_sw128(a_addr + k * kUmmaK * 2), umma_desc_sw128(b_addr + k * kUmmaK * 2),
                           idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit_pair(&empty_bar[stage], 3);          // both CTAs may refill this stage
          if (++stage == kPairStages) { stage = 0; phase ^= 1; }
        }
        if (ok) umma_commit_pair(&acc_full[acc], 3);       // both CTAs' epilogues may drain their halves
      }
      if (!ok) atomicExch(args.status, kStatusTimeout);
    }
  } else if (warp >= 2 && warp < 2 + kEpiWarps) {
    // ------------------------------------------------------------ epilogue (8 warps per CTA, own 128 rows)
    const int quarter = warp & 3;
    const int half = (warp - 2) >> 2;
    uint8_t* stg = stg_all + (warp - 2) * kStgWarpBytes;
    const uint32_t leader_acc_empty0 = mapa_u32(smem_u32(&acc_empty[0]), 0);
    int it = 0;
    bool ok = true;
    for (int tile = pair; tile < total_tiles && ok; tile += n_pairs, ++it) {
      int group, row0, row_end, group_row0, nt;
      tile_coords(tile, group, row0, row_end, group_row0, nt);
      const int n0 = nt * bn;
      const int acc = it & 1;
      const uint32_t acc_phase = (it >> 1) & 1;
      if (!mbar_wait(&acc_full[acc], acc_phase)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * kBN;
      gemm_epilogue_tile<EPI>(args, taddr, stg, lane, quarter, half, row0, row_end, group, group_row0, n0,
                              min(bn, args.N - n0), [&]() {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(leader_acc_empty0 + acc * 8);
      });
    }
    if (!ok && lane == 0) atomicExch(args.status, kStatusTimeout);
  }

  // ---------------------------------------------------------------- teardown (both CTAs, together)
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

}  // namespace foe
