// Router scores on the 5th-generation tensor cores at fp32 accuracy, for calls with thousands of tokens
// (Section 3.1 "Routing": one fp32 score per token and expert).
//
//   score[i, e] = inv_rms[i] * sum_k r[i, k] * (gain[k] * W[e, k])
//
// The decision taken from these scores (which experts) must agree with a float32 reference, so a plain bf16 product
// is not enough.  Both operands are split into three bf16 terms, x = x1 + x2 + x3, which together hold all 24
// significant bits of a float; the six products of weight 1, 2^-8 and 2^-16 (x1 w1, x1 w2, x2 w1, x2 w2, x1 w3,
// x3 w1) are issued as bf16 MMAs with fp32 accumulation -- every product of two bf16 values is exact in fp32 -- and
// the three dropped ones are below 2^-24.  Eight (64 experts per CTA) or four (128) accumulators take the k-blocks in
// turn and are summed in fp32 by the epilogue, which keeps the tensor-core accumulation chains short (96 steps for a
// hidden size of 2048 with eight accumulators).
//
// The weights are split when the layer is created (gain folded in); the residual r is split on the fly: sixteen
// converter warps read a 128 x 64 fp32 tile per k-block straight from global memory (coalesced, 512 bytes per warp
// instruction), split it in registers and store the three bf16 tiles in the 128-byte-swizzled operand layout, then
// cross to the async proxy and arrive on the stage's barrier.  The kernel runs at the rate of this conversion.  One CTA
// per 128 tokens x 64 experts, or x 128 experts when the (padded) expert count is a multiple of 128: every token tile
// is then converted once per 128 experts.
//
// Warp roles: 0 TMA producer (weight planes), 1 MMA issuer, 2-5 epilogue, 6-21 converters.  All waits are bounded.
#include "common.cuh"
#include "kernels.h"

namespace foe {

constexpr int kRtRows = 128, kRtBK = 64;
constexpr int kRtATile = kRtRows * kRtBK * 2;       // 16 KB: one bf16 term of the A tile
// A CTA takes CHUNK = 64 or 128 experts.  The kernel runs at the rate its converters split the residual, so a layer
// with 128 experts or more converts every token tile once per 128 experts instead of once per 64;
// the price is a ring of two stages instead of three and accumulation chains twice as long.
template <int CHUNK> struct RtCfg {
  static constexpr int kBTile = CHUNK * kRtBK * 2;                 // 8 or 16 KB: one bf16 term of the B tile
  static constexpr int kStageBytes = 3 * kRtATile + 3 * kBTile;    // 72 or 96 KB
  static constexpr int kStages = CHUNK == 64 ? 3 : 2;
  static constexpr int kAccs = 512 / CHUNK;                        // accumulators of CHUNK columns: all 512 TMEM columns
  static constexpr size_t kSmemBytes = size_t(kStages) * kStageBytes + 1024 + 256;
};
constexpr int kRtConvWarps = 16;
constexpr int kRtThreads = (6 + kRtConvWarps) * 32;
constexpr int kRtRowsPerLane = kRtRows / (2 * kRtConvWarps);   // tile rows one converter lane handles per k-block

// split two floats into three packed bf16 pairs (x = hi + mid + lo up to 2^-24 |x|)
__device__ __forceinline__ void split3(float x, float y, uint32_t& hi, uint32_t& mid, uint32_t& lo) {
  hi = pack_bf16(x, y);
  const float rx = x - bf16_lo(hi), ry = y - bf16_hi(hi);
  mid = pack_bf16(rx, ry);
  lo = pack_bf16(rx - bf16_lo(mid), ry - bf16_hi(mid));
}

// planes[(p * E_pad + e) * d + k] = term p of gain[k] * W[e, k]; rows e >= E are zero.
__global__ void split_router_weights_kernel(const float* __restrict__ wr, const bf16* __restrict__ gain,
                                            bf16* __restrict__ planes, int E, int E_pad, int d) {
  const size_t idx = size_t(blockIdx.x) * blockDim.x + threadIdx.x;    // one pair of columns
  const size_t total = size_t(E_pad) * d / 2;
  if (idx >= total) return;
  const int e = int(idx / (d / 2)), k = int(idx % (d / 2)) * 2;
  float x = 0.f, y = 0.f;
  if (e < E) {
    x = wr[size_t(e) * d + k] * __bfloat162float(gain[k]);
    y = wr[size_t(e) * d + k + 1] * __bfloat162float(gain[k + 1]);
  }
  uint32_t hi, mid, lo;
  split3(x, y, hi, mid, lo);
  uint32_t* out = reinterpret_cast<uint32_t*>(planes);
  const size_t plane = size_t(E_pad) * d / 2;
  out[idx] = hi;
  out[plane + idx] = mid;
  out[2 * plane + idx] = lo;
}

template <int CHUNK>
__global__ void __launch_bounds__(kRtThreads, 1)
router_tc_kernel(const __grid_constant__ CUtensorMap tmW, const void* __restrict__ r_in, int r_is_bf16,
                 const float* __restrict__ inv_rms, float* __restrict__ part, int n_tokens, int d, int E, int E_pad,
                 int* __restrict__ status) {
  pdl_wait();
  pdl_launch_dependents();
  using Cfg = RtCfg<CHUNK>;
  constexpr int kRtChunk = CHUNK, kRtBTile = Cfg::kBTile, kRtStageBytes = Cfg::kStageBytes, kRtStages = Cfg::kStages,
                kRtAccs = Cfg::kAccs;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + kRtStages * kRtStageBytes);
  uint64_t* empty_bar = full_bar + kRtStages;
  uint64_t* acc_full = empty_bar + kRtStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row0 = blockIdx.x * kRtRows, chunk = blockIdx.y;
  const int kblocks = d / kRtBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kRtStages; ++s) { mbar_init(&full_bar[s], 1 + kRtConvWarps); mbar_init(&empty_bar[s], 1); }
    mbar_init(acc_full, 1);
    mbar_fence_init();
    tma_prefetch_desc(&tmW);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ weight planes by TMA
    if (elect_one()) {
      bool ok = true;
      for (int kb = 0; kb < kblocks; ++kb) {
        const int s = kb % kRtStages;
        if (!mbar_wait(&empty_bar[s], ((kb / kRtStages) & 1) ^ 1)) { ok = false; break; }
        uint8_t* sb = smem + s * kRtStageBytes + 3 * kRtATile;
        mbar_expect_tx(&full_bar[s], 3 * kRtBTile);
        for (int p = 0; p < 3; ++p)
#pragma unroll
          for (int hb = 0; hb < kRtChunk / kRouterChunk; ++hb)          // the tensor map's box is 64 rows
            tma_load_2d(sb + p * kRtBTile + hb * (kRouterChunk * kRtBK * 2), &tmW, &full_bar[s], kb * kRtBK,
                        p * E_pad + chunk * kRtChunk + hb * kRouterChunk);
      }
      if (!ok) atomicExch(status, kStatusTimeout);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (elect_one()) {
      constexpr uint32_t idesc = umma_idesc_bf16(kRtRows, kRtChunk);
      bool ok = true;
      for (int kb = 0; kb < kblocks; ++kb) {
        const int s = kb % kRtStages;
        if (!mbar_wait(&full_bar[s], (kb / kRtStages) & 1)) { ok = false; break; }
        tc_fence_after();
        const uint32_t a0 = smem_u32(smem + s * kRtStageBytes), b0 = a0 + 3 * kRtATile;
        const uint32_t d_tmem = tmem_base + (kb % kRtAccs) * kRtChunk;
        // term pairs (A term, B term), smallest products first
        constexpr int pa[6] = {2, 0, 1, 1, 0, 0}, pb[6] = {0, 2, 1, 0, 1, 0};
#pragma unroll
        for (int k = 0; k < kRtBK / 16; ++k) {
#pragma unroll
          for (int q = 0; q < 6; ++q) {
            umma_bf16(d_tmem, umma_desc_sw128(a0 + pa[q] * kRtATile + k * 32), umma_desc_sw128(b0 + pb[q] * kRtBTile + k * 32),
                      idesc, (kb >= kRtAccs || k != 0 || q != 0) ? 1u : 0u);
          }
        }
        umma_commit(&empty_bar[s]);
      }
      if (ok) umma_commit(acc_full);
      else atomicExch(status, kStatusTimeout);
    }
  } else if (warp >= 6) {
    // ------------------------------------------------------------ converters: fp32 tile -> three bf16 operand tiles
    // lane = (row parity, 16 float4 columns): one warp instruction reads two whole 256-byte tile rows
    const int cw = warp - 6;
    const int sub = lane >> 4, c4 = lane & 15;             // row inside the pair; float4 column (4 k values)
    const int chunk16 = c4 >> 1, half8 = (c4 & 1) * 8;      // 16-byte chunk of the bf16 row and offset inside it
    constexpr int NR = kRtRowsPerLane;
    size_t src[NR];                                         // element offset of this lane's four values in k-block 0
    int trow[NR];
#pragma unroll
    for (int i = 0; i < NR; ++i) {
      trow[i] = cw * (2 * NR) + 2 * i + sub;                // row of the tile
      src[i] = size_t(min(row0 + trow[i], n_tokens - 1)) * d + c4 * 4;          // rows past the end repeat the last one
    }
    // the residual comes as fp32 (inside a block) or as bf16 (routing call on a caller's tensor)
    auto load4 = [&](size_t off) {
      if (r_is_bf16) {
        const uint2 q = __ldg(reinterpret_cast<const uint2*>(static_cast<const bf16*>(r_in) + off));
        return make_float4(bf16_lo(q.x), bf16_hi(q.x), bf16_lo(q.y), bf16_hi(q.y));
      }
      return __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(r_in) + off));
    };
    // two k-blocks of loads stay in flight per lane while a third is converted
    bool ok = true;
    float4 cur[NR], nxt[NR], nx2[NR];
#pragma unroll
    for (int i = 0; i < NR; ++i) cur[i] = load4(src[i]);
    if (kblocks > 1) {
#pragma unroll
      for (int i = 0; i < NR; ++i) nxt[i] = load4(src[i] + size_t(kRtBK));
    }
    for (int kb = 0; kb < kblocks; ++kb) {
      if (kb + 2 < kblocks) {
#pragma unroll
        for (int i = 0; i < NR; ++i) nx2[i] = load4(src[i] + size_t(kb + 2) * kRtBK);
      }
      const int s = kb % kRtStages;
      if (lane == 0) ok = mbar_wait(&empty_bar[s], ((kb / kRtStages) & 1) ^ 1);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      uint8_t* sa = smem + s * kRtStageBytes;
#pragma unroll
      for (int i = 0; i < NR; ++i) {
        uint32_t h0, m0, l0, h1, m1, l1;
        split3(cur[i].x, cur[i].y, h0, m0, l0);
        split3(cur[i].z, cur[i].w, h1, m1, l1);
        const int off = trow[i] * 128 + ((chunk16 ^ (trow[i] & 7)) << 4) + half8;
        *reinterpret_cast<uint2*>(sa + off) = make_uint2(h0, h1);
        *reinterpret_cast<uint2*>(sa + kRtATile + off) = make_uint2(m0, m1);
        *reinterpret_cast<uint2*>(sa + 2 * kRtATile + off) = make_uint2(l0, l1);
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy stores -> tensor-core reads
      __syncwarp();
      if (lane == 0) mbar_arrive(&full_bar[s]);
#pragma unroll
      for (int i = 0; i < NR; ++i) { cur[i] = nxt[i]; nxt[i] = nx2[i]; }
    }
    if (!ok && lane == 0) atomicExch(status, kStatusTimeout);
  } else {
    // ------------------------------------------------------------ epilogue: sum the accumulators, scale, store
    const int quarter = warp & 3;
    const int row = row0 + quarter * 32 + lane;
    if (mbar_wait(acc_full, 0)) {
      tc_fence_after();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
      const int n_acc = kblocks < kRtAccs ? kblocks : kRtAccs;
      const float inv = row < n_tokens ? inv_rms[row] : 0.f;
#pragma unroll
      for (int hf = 0; hf < kRtChunk / 32; ++hf) {
        float sum[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) sum[c] = 0.f;
        for (int a = 0; a < n_acc; ++a) {
          uint32_t v[32];
          tmem_ld32(taddr + a * kRtChunk + hf * 32, v);
          tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 32; ++c) sum[c] += __uint_as_float(v[c]);
        }
        if (row < n_tokens) {
          const int e0 = chunk * kRtChunk + hf * 32;
          float* dst = part + size_t(row) * E + e0;
          if ((E & 3) == 0 && e0 + 32 <= E) {
#pragma unroll
            for (int c = 0; c < 32; c += 4)
              *reinterpret_cast<float4*>(dst + c) = make_float4(sum[c] * inv, sum[c + 1] * inv, sum[c + 2] * inv, sum[c + 3] * inv);
          } else {
#pragma unroll
            for (int c = 0; c < 32; ++c)
              if (e0 + c < E) dst[c] = sum[c] * inv;
          }
        }
      }
    } else if (lane == 0) {
      atomicExch(status, kStatusTimeout);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

void launch_split_router_weights(const float* wr, const bf16* gain, bf16* planes, int E, int d, cudaStream_t st) {
  const int E_pad = router_padded_experts(E);
  const size_t total = size_t(E_pad) * d / 2;
  split_router_weights_kernel<<<unsigned((total + 255) / 256), 256, 0, st>>>(wr, gain, planes, E, E_pad, d);
}

cudaError_t router_tc_configure() {
  cudaError_t e = cudaFuncSetAttribute(router_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(RtCfg<64>::kSmemBytes));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(router_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(RtCfg<128>::kSmemBytes));
}

void launch_router_tc(const CUtensorMap& tmW, const void* r, int r_is_bf16, const float* inv_rms, float* part,
                      int n_tokens, int d, int E, int* status, cudaStream_t st) {
  const int E_pad = router_padded_experts(E);
  const int tiles = (n_tokens + kRtRows - 1) / kRtRows;
  if (E_pad % 128 == 0) {
    launch_pdl(router_tc_kernel<128>, dim3(tiles, E_pad / 128), dim3(kRtThreads), RtCfg<128>::kSmemBytes, st, tmW, r, r_is_bf16, inv_rms,
               part, n_tokens, d, E, E_pad, status);
  } else {
    launch_pdl(router_tc_kernel<64>, dim3(tiles, E_pad / 64), dim3(kRtThreads), RtCfg<64>::kSmemBytes, st, tmW, r, r_is_bf16, inv_rms,
               part, n_tokens, d, E, E_pad, status);
  }
}

}  // namespace foe
