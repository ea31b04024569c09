// Grouped bf16 GEMM on the 5th-generation tensor cores (tcgen05 + TMEM), operands staged by TMA.
//
//   C_g[m, n] = sum_k A[row_g(m), k] * B_g[n, k]          fp32 accumulation in tensor memory
//
// A cluster of two CTAs (two SMs) computes one 256 x bn output tile (bn <= 256) with tcgen05.mma.cta_group::2 and
// walks a static round-robin list of tiles.  Each CTA stages only its own 128 A rows and its own half of the B rows,
// so the shared-memory traffic per SM and k-block (TMA writes + tensor-core reads) is a third lower than with one
// CTA per tile -- and that traffic, not the MMA rate, is what bounds a one-CTA 128 x 256 tile -- and six stages fit
// where four did.  The leader CTA (cluster rank 0) issues the MMAs for both; accumulators live in each CTA's own
// tensor memory (its 128 rows x 256 columns, two stages, so the epilogue of one tile overlaps the MMAs of the next)
// and each CTA's epilogue warps drain their half.
//
// Warp roles per CTA: warp 0 TMA producer, warp 1 MMA issuer (leader) / gather relay (peer), warps 2..9 epilogue (two
// warps per 32-lane quarter of tensor memory, alternate column passes), warps 10..13 A-gather producers (GATHER only).
// Groups are either uniform (every group has the same row count: the per-cluster QKV projection, the output
// projection) or ragged (the experts: an m-tile table built on the device by the permute step, so no host sync).
//
// Barrier protocol (every barrier exists in both CTAs at the same shared-memory offset):
//   full[s]      used in the leader: 1 arrival (leader's expect_tx) + the bytes of BOTH CTAs' TMA loads; with a
//                gathered A also one arrival per gather thread of the leader (carried by its cp.async copies) and
//                one from the peer's relay thread
//   a_full[s]    gathered A only, used in the peer: one arrival per gather thread of the peer
//   empty[s]     used in each CTA: 1 arrival from the leader's multicast tcgen05.commit
//   acc_full[a]  used in each CTA: 1 arrival from the leader's multicast tcgen05.commit
//   acc_empty[a] used in the leader: 16 arrivals (8 epilogue warps of each CTA; the peer's arrive remotely)
//
// Used for steps of the paper's Table 2: Attn_h's projections ("Attn. residual" row), the sync
// ("Cross-group avg." row, fused into the output-projection epilogue) and FFN_e ("MoE update" row).
#pragma once

#include "common.cuh"
#include "gemm_args.h"

namespace foe {

constexpr int kBK = 64;              // k-block: 64 bf16 = one 128-byte swizzle row
constexpr int kUmmaK = 16;
constexpr int kStages = 6;
constexpr int kABytes = kBM * kBK * 2;                 // this CTA's 128 A rows of a k-block: 16 KB
constexpr int kBHalfBytes = (kBN / 2) * kBK * 2;       // this CTA's half of the widest B tile: 16 KB
constexpr int kStageBytes = kABytes + kBHalfBytes;     // 32 KB
constexpr int kPairTileRows = 2 * kBM;                 // 256 rows per tile
constexpr int kEpiWarps = 8;          // two per tensor-memory lane quarter
constexpr int kGemmThreads = 64 + kEpiWarps * 32;
constexpr int kGatherThreads = 128;   // extra producer warps when the A rows are gathered
constexpr int kTmemCols = 512;
constexpr int kStgPitch = 128;                       // staging row: 128 bytes of output, 16-byte chunks XOR-swizzled by row
constexpr int kStgWarpBytes = 32 * kStgPitch;        // one epilogue warp stages its 32 rows
constexpr size_t kGemmSmemBytes = size_t(kStages) * kStageBytes + kEpiWarps * kStgWarpBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;

// byte offset of 16-byte chunk c of staging row r (conflict-free for row-per-lane writes and 8-lanes-per-row reads)
__device__ __forceinline__ int stg_off(int r, int c) { return r * kStgPitch + ((c ^ (r & 7)) << 4); }

// z * sigmoid(z) with the fast exponential and the fast (two-ulp) division: two special-function operations per value
__device__ __forceinline__ float silu_f(float z) { return __fdividef(z, 1.0f + __expf(-z)); }

// Epilogue of one 128 x tile_cols accumulator tile, run by the eight epilogue warps: the two warps of `quarter` own
// TMEM lanes 32*quarter .. and take the column passes of their `half` (passes half, half + 2, ...).  `row0` is the
// first A row of the CTA's 128 rows; `release` is called once per warp, right after its last tensor-memory read,
// and hands the accumulator stage back to the MMA issuer.
template <int EPI, class ReleaseFn>
__device__ __forceinline__ void gemm_epilogue_tile(const GemmArgs& args, uint32_t taddr, uint8_t* stg, int lane, int quarter,
                                                   int half, int row0, int row_end, int group, int group_row0, int n0,
                                                   int tile_cols, ReleaseFn release) {
  const int row = row0 + quarter * 32 + lane;      // A row of this thread's accumulator lane
  const bool row_ok = row < row_end;
  // Every pass turns 128 bytes of output per row into registers (thread = accumulator row), parks them
  // in the warp's staging tile and writes them out again with 8 lanes per row, so that global stores
  // are whole 128-byte lines instead of 32 scattered 16-byte pieces.
  const int row_local = row - group_row0;
  float scale = 1.0f;
  if constexpr (EPI == kEpiQKV) {
    if (row_ok) scale = args.row_scale[size_t(group) * args.scale_group_stride + row_local];
  }
  constexpr int kPassCols = (EPI == kEpiOProj) ? 32 : 64;          // accumulator columns per pass (SwiGLU: 64 + 64)
  // a head of 96 columns is not a whole number of 64-column passes: its QKV epilogue takes 32 columns at a time
  const bool narrow = (EPI == kEpiQKV) && (args.dh & 63) != 0;
  const int pass_cols = narrow ? 32 : kPassCols;
  const int n_pass = (EPI == kEpiSwiGLU) ? 2 : (tile_cols + pass_cols - 1) / pass_cols;
  const int wr_row = lane >> 3, wr_chunk = lane & 7;                // write-out role: row (+4j), 16-byte chunk
  if (half >= n_pass) { release(); return; }                        // nothing for this warp in a one-pass tile
  // pushed O-proj tiles: elements this warp has written to the current owner since its last counter update
  int push_owner = -1;
  unsigned int push_n = 0;
  auto push_flush = [&]() {
    if (push_n) {
      __threadfence_system();                                       // every lane: its stores before the count
      __syncwarp();
      if (lane == 0) atomicAdd_system(args.push_cnt[push_owner] + row0 / kShardBlockRows, push_n);   // the tile's row block
      push_n = 0;
    }
  };
#pragma unroll 1
  for (int ps = half; ps < n_pass; ps += 2) {
    const int n = (EPI == kEpiSwiGLU) ? (n0 >> 1) + ps * 64 : n0 + ps * pass_cols;   // output column in the group
    uint32_t w[32];                                                // 128 bytes of this row's output
    __syncwarp();
    if constexpr (EPI == kEpiSwiGLU) {
      uint32_t gt[32], up[32];
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        tmem_ld32(taddr + ps * 64 + hf * 32, gt);
        tmem_ld32(taddr + 128 + ps * 64 + hf * 32, up);
        tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          const float h0 = silu_f(__uint_as_float(gt[2 * c])) * __uint_as_float(up[2 * c]);
          const float h1 = silu_f(__uint_as_float(gt[2 * c + 1])) * __uint_as_float(up[2 * c + 1]);
          w[hf * 16 + c] = pack_bf16(h0, h1);
        }
      }
    } else if constexpr (EPI == kEpiOProj) {
      tmem_ld32(taddr + ps * 32, w);
      tmem_ld_wait();
    } else if constexpr (EPI == kEpiQKV) {
      // 64 packed columns = 32 rotation pairs (natural columns i0+m and i0+m+dh/2 of one head).  The first
      // 64 bytes of the staged row are the first-half columns, the second 64 bytes their partners.
      const bool rotate = n < args.q_cols + args.kv_cols;          // q and k heads; v is only de-interleaved
      const int i0 = (n % args.dh) >> 1;
      // the 32 (cos, sin) pairs of this row's position are fetched before the accumulator is read, so their
      // latency overlaps the tensor-memory load
      const float4* tab = reinterpret_cast<const float4*>(
          args.rope_tab + size_t(row_ok ? args.tok_pos[row_local] : 0) * (args.dh >> 1) + i0);
      float4 cs4[16];
#pragma unroll
      for (int m = 0; m < 16; ++m) cs4[m] = (rotate && (m < 8 || !narrow)) ? __ldg(tab + m) : make_float4(1.f, 0.f, 1.f, 0.f);
      uint32_t r[32];
      if (narrow) {
        // 32 packed columns = 16 pairs: the first 32 bytes of the staged row are the first-half columns, the next 32
        // bytes their partners; the rest of the row is unused
        tmem_ld32(taddr + ps * 32, r);
        tmem_ld_wait();
        float lo[16], hi[16];
#pragma unroll
        for (int m = 0; m < 16; ++m) {
          const float a = __uint_as_float(r[2 * m]) * scale, b = __uint_as_float(r[2 * m + 1]) * scale;
          const float4 c4 = cs4[m >> 1];
          const float cx = (m & 1) ? c4.z : c4.x, cy = (m & 1) ? c4.w : c4.y;
          lo[m] = a * cx - b * cy;
          hi[m] = b * cx + a * cy;
        }
#pragma unroll
        for (int m = 0; m < 8; ++m) {
          w[m] = pack_bf16(lo[2 * m], lo[2 * m + 1]);
          w[8 + m] = pack_bf16(hi[2 * m], hi[2 * m + 1]);
          w[16 + m] = 0u;
          w[24 + m] = 0u;
        }
      } else
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        tmem_ld32(taddr + ps * 64 + hf * 32, r);
        tmem_ld_wait();
        float lo[16], hi[16];
#pragma unroll
        for (int m = 0; m < 16; ++m) {
          const float a = __uint_as_float(r[2 * m]) * scale, b = __uint_as_float(r[2 * m + 1]) * scale;
          const float4 c4 = cs4[hf * 8 + (m >> 1)];
          const float cx = (m & 1) ? c4.z : c4.x, cy = (m & 1) ? c4.w : c4.y;
          lo[m] = a * cx - b * cy;
          hi[m] = b * cx + a * cy;
        }
#pragma unroll
        for (int m = 0; m < 8; ++m) {
          w[hf * 8 + m] = pack_bf16(lo[2 * m], lo[2 * m + 1]);
          w[16 + hf * 8 + m] = pack_bf16(hi[2 * m], hi[2 * m + 1]);
        }
      }
    } else {
      uint32_t r[32];
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        tmem_ld32(taddr + ps * 64 + hf * 32, r);
        tmem_ld_wait();
#pragma unroll
        for (int c = 0; c < 16; ++c)
          w[hf * 16 + c] = pack_bf16(__uint_as_float(r[2 * c]), __uint_as_float(r[2 * c + 1]));
      }
    }
    if (ps + 2 >= n_pass) release();                               // this warp's last TMEM read of the tile
#pragma unroll
    for (int c = 0; c < 8; ++c)
      *reinterpret_cast<uint4*>(stg + stg_off(lane, c)) = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
    __syncwarp();
    if constexpr (EPI == kEpiOProj) {
      // r_full = scale * (C + sum_h x[h]); all loads of the pass are issued before the first use.
      const int or_row = lane >> 2, or_cg = lane & 3;           // row (+8j) and group of 8 columns
      // what is added to C: the fp32 sum of the residual streams already sitting in `out` (two float4 per row), or
      // one bf16 stream (a first layer's shared x, a rank's own x[h]), or nothing
      float4 xf[4][2];
      uint4 xq[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int grow = row0 + quarter * 32 + or_row + 8 * j;
        const size_t off = size_t(grow) * args.ldo + n + or_cg * 8;
        xf[j][0] = xf[j][1] = make_float4(0.f, 0.f, 0.f, 0.f);
        xq[j] = make_uint4(0u, 0u, 0u, 0u);
        if (grow < row_end) {
          if (args.x_in_out) {
            xf[j][0] = *reinterpret_cast<const float4*>(static_cast<const float*>(args.out) + off);
            xf[j][1] = *reinterpret_cast<const float4*>(static_cast<const float*>(args.out) + off + 4);
          } else if (args.x_count > 0) {
            xq[j] = __ldg(reinterpret_cast<const uint4*>(args.xsum + off));
          }
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int rr = or_row + 8 * j;
        const int grow = row0 + quarter * 32 + rr;
        if (grow >= row_end) continue;
        const float4 c0 = *reinterpret_cast<const float4*>(stg + stg_off(rr, 2 * or_cg));
        const float4 c1 = *reinterpret_cast<const float4*>(stg + stg_off(rr, 2 * or_cg + 1));
        float a8[8] = {c0.x + xf[j][0].x, c0.y + xf[j][0].y, c0.z + xf[j][0].z, c0.w + xf[j][0].w,
                       c1.x + xf[j][1].x, c1.y + xf[j][1].y, c1.z + xf[j][1].z, c1.w + xf[j][1].w};
        {
          const uint32_t w4[4] = {xq[j].x, xq[j].y, xq[j].z, xq[j].w};
#pragma unroll
          for (int q = 0; q < 4; ++q) { a8[2 * q] += bf16_lo(w4[q]); a8[2 * q + 1] += bf16_hi(w4[q]); }
        }
        const float sc = args.out_scale;
        if (args.push_span) {
          // the 32 columns of a pass lie inside one owner's span (a multiple of 32)
          const int owner = n / args.push_span;
          __nv_bfloat16* dst = args.push_base[owner] + args.push_slot_off + size_t(grow) * args.push_span +
                               (n - owner * args.push_span) + or_cg * 8;
          *reinterpret_cast<uint4*>(dst) = make_uint4(pack_bf16(a8[0] * sc, a8[1] * sc), pack_bf16(a8[2] * sc, a8[3] * sc),
                                                      pack_bf16(a8[4] * sc, a8[5] * sc), pack_bf16(a8[6] * sc, a8[7] * sc));
        } else {
          float* dst = static_cast<float*>(args.out) + size_t(grow) * args.ldo + n + or_cg * 8;
          *reinterpret_cast<float4*>(dst) = make_float4(a8[0] * sc, a8[1] * sc, a8[2] * sc, a8[3] * sc);
          *reinterpret_cast<float4*>(dst + 4) = make_float4(a8[4] * sc, a8[5] * sc, a8[6] * sc, a8[7] * sc);
        }
      }
      if (args.push_span) {
        const int owner = n / args.push_span;
        if (owner != push_owner) { push_flush(); push_owner = owner; }
        const int rows_here = min(32, max(0, row_end - (row0 + quarter * 32)));
        push_n += unsigned(rows_here) * 32u;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int rr = wr_row + 4 * j;                              // row inside the warp's 32
        const int grow = row0 + quarter * 32 + rr;
        if (grow >= row_end) continue;
        const uint4 v = *reinterpret_cast<const uint4*>(stg + stg_off(rr, wr_chunk));
        if constexpr (EPI == kEpiQKV) {
          const int tok = grow - group_row0;
          // natural column inside the head of this lane's 8 values: chunks 0-3 first half, 4-7 second half
          // (32-column passes: chunks 0-1 first half, 2-3 second half, 4-7 nothing)
          if (narrow && wr_chunk >= 4) continue;
          const int hcol = narrow ? ((n % args.dh) >> 1) + (wr_chunk & 1) * 8 + (wr_chunk >> 1) * (args.dh >> 1)
                                  : ((n % args.dh) >> 1) + (wr_chunk & 3) * 8 + (wr_chunk >> 2) * (args.dh >> 1);
          if (n < args.q_cols) {
            const int head = group * (args.q_cols / args.dh) + n / args.dh;
            *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(args.out) + size_t(tok) * args.ldo + head * args.q_head_stride + hcol) = v;
          } else {
            const bool is_k = n < args.q_cols + args.kv_cols;
            const int nn = n - args.q_cols - (is_k ? 0 : args.kv_cols);
            const int kvh = group * (args.kv_cols / args.dh) + nn / args.dh;
            const int slot = args.tok_slot[tok];
            if (slot >= 0) {
              const int page = slot >> 6, off = slot & 63;
              __nv_bfloat16* base = is_k ? args.k_pages : args.v_pages;
              *reinterpret_cast<uint4*>(base + ((size_t(page) * args.n_kv + kvh) * 64 + off) * args.dh + hcol) = v;
            }
          }
        } else {
          *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(args.out) + size_t(grow) * args.ldo + n + wr_chunk * 8) = v;
        }
      }
    }
  }
  if constexpr (EPI == kEpiOProj) push_flush();
}

template <int EPI, bool GATHER>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads + (GATHER ? kGatherThreads : 0), 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                         const GemmArgs args) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* stg_all = smem + kStages * kStageBytes;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(stg_all + kEpiWarps * kStgWarpBytes);
  uint64_t* empty_bar = full_bar + kStages;
  uint64_t* acc_full = empty_bar + kStages;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* a_full = acc_empty + 2;                      // gathered A only (peer CTA)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(a_full + kStages);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();               // 0 = leader
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full_bar[s], GATHER ? 1 + kGatherThreads + 1 : 1);
      mbar_init(&empty_bar[s], 1);
      mbar_init(&a_full[s], kGatherThreads);
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
  pdl_wait();                                            // (barriers, tensor memory and descriptors were set up meanwhile)
  pdl_launch_dependents();

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
          uint8_t* sa = smem + stage * kStageBytes;
          if (leader) mbar_expect_tx(&full_bar[stage], 2 * ((GATHER ? 0 : kABytes) + (bn / 2) * (kBK * 2)));
          if constexpr (!GATHER) tma_load_2d_pair(sa, &tmA, &full_bar[stage], kb * kBK, row0);
          tma_load_2d_pair(sa + kABytes, &tmB, &full_bar[stage], kb * kBK, brow0);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
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
          if constexpr (GATHER) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the leader's cp.async-written rows
          const uint32_t a_addr = smem_u32(smem + stage * kStageBytes);
          const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) {
            umma_bf16_pair(d_tmem, umma_desc_sw128(a_addr + k * kUmmaK * 2), umma_desc_sw128(b_addr + k * kUmmaK * 2),
                           idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit_pair(&empty_bar[stage], 3);          // both CTAs may refill this stage
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (ok) umma_commit_pair(&acc_full[acc], 3);       // both CTAs' epilogues may drain their halves
      }
      if (!ok) atomicExch(args.status, kStatusTimeout);
    } else if (GATHER && !leader && elect_one()) {
      // relay (the peer's otherwise idle warp 1): the peer's gathered A rows of a stage have landed -> make them
      // visible to the tensor core's reads and tell the leader's MMA thread.  The arrival is relaxed: a releasing
      // remote arrival costs about a microsecond each, more than two k-blocks, and orders nothing that matters
      // here: the rows are in shared memory once the copies have arrived on a_full, the proxy fence below comes
      // before the arrival in program order, and the reader is the tensor core, which starts after the leader has
      // seen this arrival.
      const uint32_t leader_full0 = mapa_u32(smem_u32(&full_bar[0]), 0);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
        for (int kb = 0; kb < kblocks; ++kb) {
          if (!mbar_wait(&a_full[stage], phase)) { ok = false; break; }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          mbar_arrive_cluster_relaxed(leader_full0 + stage * 8);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) atomicExch(args.status, kStatusTimeout);
    }
  } else if (GATHER && warp >= 2 + kEpiWarps) {
    // ------------------------------------------------------------ A-gather producers (4 warps in each CTA, own 128 rows)
    // Row r of the tile is row a_row_index[row0 + r] of a_gather.  Each thread copies one 16-byte chunk of eight
    // rows per k-block with cp.async into the swizzled operand layout; the copies themselves arrive on a barrier of
    // their own CTA (cp.async.mbarrier.arrive.noinc): the leader's on full[s], the peer's on a_full[s].  One lane
    // per warp polls the stage's empty barrier: it receives its arrivals from the other SM, and a crowd of
    // pollers slows those down.
    const int gt = threadIdx.x - kGemmThreads;
    const int gc = gt & 7, gr = gt >> 3;
    uint64_t* my_full = leader ? full_bar : a_full;
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    auto tile_rows = [&](int tile, int (&rows)[8]) {
      if (tile < total_tiles) {
        int group, row0, row_end, group_row0, nt;
        tile_coords(tile, group, row0, row_end, group_row0, nt);
#pragma unroll
        for (int j = 0; j < 8; ++j) rows[j] = args.a_row_index[min(row0 + gr + 16 * j, row_end - 1)];
      }
    };
    int next_rows[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    tile_rows(pair, next_rows);
    for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
      const uint8_t* src[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        src[j] = reinterpret_cast<const uint8_t*>(args.a_gather) + size_t(next_rows[j]) * args.K * 2 + gc * 16;
      tile_rows(tile + n_pairs, next_rows);
      for (int kb = 0; kb < kblocks; ++kb) {
        if (lane == 0) ok = mbar_wait(&empty_bar[stage], phase ^ 1);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        const uint32_t dst = smem_u32(smem + stage * kStageBytes);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int r = gr + 16 * j;
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + r * 128 + ((gc ^ (r & 7)) << 4)),
                       "l"(src[j] + size_t(kb) * 128) : "memory");
        }
        asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(&my_full[stage])) : "memory");
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    if (!ok && lane == 0) atomicExch(args.status, kStatusTimeout);
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
        if (lane == 0) mbar_arrive_cluster_relaxed(leader_acc_empty0 + acc * 8);   // tensor memory is not ordered by a release anyway
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
