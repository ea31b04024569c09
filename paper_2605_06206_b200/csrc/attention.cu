// Attention core of the FoE block ("Attn_h" of Table 2): causal softmax(q k^T / sqrt(d_h)) v per sequence,
// every query head reading the KV head of its cluster from the paged cache (the paper's KV cache is split
// across the expert groups; on one GPU that is the head index of the page layout).
//
// This file holds the decode kernel (one new token per sequence; the prefill kernel on the tcgen05 tensor
// cores is in attention_tc.cu).  Decode is bound by reading the KV cache once from HBM: K and V are staged
// through shared memory with TMA -- one cache page of one KV head ([64 tokens][d_h] bf16, contiguous) is one or
// two 64 x 64 boxes written with the 128-byte swizzle, the bank-conflict-free layout ldmatrix wants.  One CTA
// per (sequence, KV head, split of the context); the g query heads of the KV head are the rows of mma.sync
// m16n8k16 tiles (fp32 accumulate, online softmax in the exp2 domain); each of 4 warps takes 16 keys of every
// page; partial (m, l, o) per split are merged by whichever CTA of the (sequence, KV head) finishes last.
#include <math.h>

#include "common.cuh"
#include "kernels.h"

namespace foe {

// byte offset of element (r, c) inside a [rows][DH] bf16 tile stored as 64-column halves, each half
// rows x 128 bytes with the 16-byte chunk index XOR-ed by (r & 7)  (= TMA SWIZZLE_128B).
template <int ROWS>
__device__ __forceinline__ uint32_t tile_off(int r, int c) {
  return uint32_t((c >> 6) * (ROWS * 128) + r * 128 + ((((c & 63) >> 3) ^ (r & 7)) << 4) + (c & 7) * 2);
}

template <int DH>
__device__ __forceinline__ void tma_load_page(uint8_t* k_dst, uint8_t* v_dst, const CUtensorMap* tmK,
                                              const CUtensorMap* tmV, uint64_t* bar, int row0) {
  mbar_expect_tx(bar, 2 * 64 * DH * 2);
#pragma unroll
  for (int h = 0; h < DH / 64; ++h) {
    tma_load_2d(k_dst + h * 64 * 128, tmK, bar, h * 64, row0);
    tma_load_2d(v_dst + h * 64 * 128, tmV, bar, h * 64, row0);
  }
}

// ======================================================================================= decode
constexpr int kDcThreads = 128;
constexpr int kDcStages = 3;

template <int DH>
__global__ void __launch_bounds__(kDcThreads, 2)
attn_decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const AttnArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr int kTileBytes = 64 * DH * 2;
  constexpr int kQBytes = 16 * DH * 2;
  uint8_t* kv_s = smem;                                            // [stage][K | V]; reused for the merge
  uint8_t* q_s = smem + kDcStages * 2 * kTileBytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(q_s + kQBytes);
  int* abort_s = reinterpret_cast<int*>(full + kDcStages);         // [2]: a wait ran out in an (even, odd) iteration

  // Until pdl_wait() nothing is read that the previous kernel writes: this grid may start while the QKV projection of
  // the same step is still running, and that kernel writes q and the new token's K / V (into the sequence's last
  // page).  Everything older is complete (a kernel lets its successor start only after its own wait).
  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int ctx = min(max(a.context_lens[b], 0), a.max_pages_per_seq * 64 - 1);     // (out-of-range values are reported by the QKV step)
  const int kv_len = ctx + 1;                                      // cached tokens + the new one
  const int n_pages = (kv_len + 63) >> 6;
  const int p_begin = split * a.pages_per_split;
  if (p_begin >= n_pages) return;
  const int p_end = min(n_pages, p_begin + a.pages_per_split);
  const int n_tiles = p_end - p_begin;
  const int G = a.n_q / a.n_kv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ld_q = a.n_q * DH;

  auto page_row0 = [&](int lp) -> int {
    int page = a.block_table[size_t(b) * a.max_pages_per_seq + min(lp, a.max_pages_per_seq - 1)];
    if (page < 0 || page >= a.num_pages) { atomicExch(a.status, kStatusBounds); page = 0; }
    return (page * a.n_kv + kvh) * 64;
  };
  if (threadIdx.x == 0) {
    for (int s = 0; s < kDcStages; ++s) mbar_init(&full[s], 1);
    abort_s[0] = abort_s[1] = 0;
    mbar_fence_init();
    for (int s = 0; s < kDcStages && s < n_tiles; ++s)             // the ring's first tiles, except the page being written
      if (p_begin + s != n_pages - 1)
        tma_load_page<DH>(kv_s + s * 2 * kTileBytes, kv_s + s * 2 * kTileBytes + kTileBytes, &tmK, &tmV, &full[s],
                          page_row0(p_begin + s));
  }
  pdl_wait();
  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int s = 0; s < kDcStages && s < n_tiles; ++s)
      if (p_begin + s == n_pages - 1)
        tma_load_page<DH>(kv_s + s * 2 * kTileBytes, kv_s + s * 2 * kTileBytes + kTileBytes, &tmK, &tmV, &full[s],
                          page_row0(p_begin + s));
  }
  const int tok = a.cu_q ? a.cu_q[b] : b;
  for (int q = threadIdx.x; q < 16 * (DH / 8); q += kDcThreads) {
    const int r = q / (DH / 8), ch = q - r * (DH / 8);
    uint4 v = make_uint4(0, 0, 0, 0);
    if (r < G) v = __ldg(reinterpret_cast<const uint4*>(a.q + size_t(tok) * ld_q + (kvh * G + r) * DH + ch * 8));
    *reinterpret_cast<uint4*>(q_s + tile_off<16>(r, ch * 8)) = v;
  }
  __syncthreads();

  float o[DH / 8][4];
#pragma unroll
  for (int n = 0; n < DH / 8; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  const int g = lane >> 2, t4 = lane & 3;
  const uint32_t q_base = smem_u32(q_s);
  bool ok = true;

  for (int j = 0; j < n_tiles; ++j) {
    const int st = j % kDcStages;
    // A wait that runs out is announced through shared memory and the whole CTA leaves the loop together after the
    // barrier below (the flag alternates with the iteration's parity, so a thread that is already one iteration ahead
    // cannot change what a slower one reads).
    const bool landed = mbar_wait(&full[st], (j / kDcStages) & 1);
    if (!landed) abort_s[j & 1] = 1;
    const uint32_t k_base = smem_u32(kv_s + st * 2 * kTileBytes);
    const uint32_t v_base = k_base + kTileBytes;
    const int key0 = (p_begin + j) * 64 + warp * 16;               // this warp's 16 keys of the page
    if (landed && key0 < kv_len) {
      float s[2][4];
      s[0][0] = s[0][1] = s[0][2] = s[0][3] = s[1][0] = s[1][1] = s[1][2] = s[1][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < DH / 16; ++ks) {
        uint32_t qa[4], kb[4];
        ldmatrix_x4(qa, q_base + tile_off<16>((lane & 7) + ((lane >> 3) & 1) * 8, ks * 16 + (lane >> 4) * 8));
        ldmatrix_x4(kb, k_base + tile_off<64>(warp * 16 + (lane & 7) + (lane >> 4) * 8, ks * 16 + ((lane >> 3) & 1) * 8));
        mma_bf16_16816(s[0], qa, kb[0], kb[1]);
        mma_bf16_16816(s[1], qa, kb[2], kb[3]);
      }
      float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
      for (int n = 0; n < 2; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float v = s[n][e] * a.scale_log2;
          if (key0 + n * 8 + t4 * 2 + (e & 1) >= kv_len) v = -INFINITY;
          s[n][e] = v;
          mx[e >> 1] = fmaxf(mx[e >> 1], v);
        }
      float alpha[2], m_use[2];
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
        mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
        const float m_new = fmaxf(m_run[r], mx[r]);
        m_use[r] = (m_new == -INFINITY) ? 0.f : m_new;
        alpha[r] = fast_exp2(m_run[r] - m_use[r]);
        m_run[r] = m_new;
      }
      float rs[2] = {0.f, 0.f};
#pragma unroll
      for (int n = 0; n < 2; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float p = fast_exp2(s[n][e] - m_use[e >> 1]);
          s[n][e] = p;
          rs[e >> 1] += p;
        }
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        rs[r] += __shfl_xor_sync(0xffffffffu, rs[r], 1);
        rs[r] += __shfl_xor_sync(0xffffffffu, rs[r], 2);
        l_run[r] = l_run[r] * alpha[r] + rs[r];
      }
      uint32_t pa[4];
      pa[0] = pack_bf16(s[0][0], s[0][1]);
      pa[1] = pack_bf16(s[0][2], s[0][3]);
      pa[2] = pack_bf16(s[1][0], s[1][1]);
      pa[3] = pack_bf16(s[1][2], s[1][3]);
#pragma unroll
      for (int dp = 0; dp < DH / 16; ++dp) {
        uint32_t vb[4];
        ldmatrix_x4_trans(vb, v_base + tile_off<64>(warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, dp * 16 + (lane >> 4) * 8));
        o[2 * dp][0] *= alpha[0]; o[2 * dp][1] *= alpha[0]; o[2 * dp][2] *= alpha[1]; o[2 * dp][3] *= alpha[1];
        o[2 * dp + 1][0] *= alpha[0]; o[2 * dp + 1][1] *= alpha[0]; o[2 * dp + 1][2] *= alpha[1]; o[2 * dp + 1][3] *= alpha[1];
        mma_bf16_16816(o[2 * dp], pa, vb[0], vb[1]);
        mma_bf16_16816(o[2 * dp + 1], pa, vb[2], vb[3]);
      }
    }
    __syncthreads();
    if (abort_s[j & 1]) { ok = false; break; }
    if (threadIdx.x == 0 && j + kDcStages < n_tiles)
      tma_load_page<DH>(kv_s + st * 2 * kTileBytes, kv_s + st * 2 * kTileBytes + kTileBytes, &tmK, &tmV, &full[st],
                        page_row0(p_begin + j + kDcStages));
  }
  // A split whose wait ran out records the timeout and writes no partial state, but still takes its ticket below: the
  // counter of its (sequence, KV head) returns to zero and the handle stays usable (this call's output is not).
  if (!ok && threadIdx.x == 0) atomicExch(a.status, kStatusTimeout);

  // merge the four warps' partial states (each saw a different quarter of every page)
  float* mo = reinterpret_cast<float*>(kv_s);                      // [4][16][DH]
  float* mm = mo + 4 * 16 * DH;                                    // [4][16] running max
  float* ml = mm + 64;                                             // [4][16] running sum
#pragma unroll
  for (int n = 0; n < DH / 8; ++n) {
    *reinterpret_cast<float2*>(mo + (warp * 16 + g) * DH + n * 8 + t4 * 2) = make_float2(o[n][0], o[n][1]);
    *reinterpret_cast<float2*>(mo + (warp * 16 + g + 8) * DH + n * 8 + t4 * 2) = make_float2(o[n][2], o[n][3]);
  }
  if (t4 == 0) {
    mm[warp * 16 + g] = m_run[0]; mm[warp * 16 + g + 8] = m_run[1];
    ml[warp * 16 + g] = l_run[0]; ml[warp * 16 + g + 8] = l_run[1];
  }
  __syncthreads();
  for (int q = threadIdx.x; ok && q < G * DH; q += kDcThreads) {
    const int r = q / DH, c = q - r * DH;
    float m = -INFINITY;
#pragma unroll
    for (int w = 0; w < 4; ++w) m = fmaxf(m, mm[w * 16 + r]);
    float acc = 0.f, l = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float f = fast_exp2(mm[w * 16 + r] - m);                   // 0 for a warp that saw no valid key
      acc += f * mo[(w * 16 + r) * DH + c];
      l += f * ml[w * 16 + r];
    }
    const size_t pidx = (size_t(b) * a.n_q + kvh * G + r) * a.max_splits + split;
    a.part_o[pidx * DH + c] = acc;
    if (c == 0) { a.part_ml[pidx * 2] = m; a.part_ml[pidx * 2 + 1] = l; }
  }

  // The CTA that finishes last among the splits of this (sequence, KV head) combines them (always in split order, so
  // the result does not depend on which one that is) and re-arms the counter for the next call: no merge launch.
  const int n_splits = min(a.max_splits, (n_pages + a.pages_per_split - 1) / a.pages_per_split);
  int* ticket_s = reinterpret_cast<int*>(ml + 64);
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) *ticket_s = atomicAdd(&a.split_done[b * a.n_kv + kvh], 1);
  __syncthreads();
  if (*ticket_s != n_splits - 1) return;
  if (threadIdx.x == 0) a.split_done[b * a.n_kv + kvh] = 0;
  __threadfence();
  for (int r = warp; r < G; r += kDcThreads / 32) {                 // one warp per query head of the group
    const int head = kvh * G + r;
    const size_t base = (size_t(b) * a.n_q + head) * a.max_splits;
    float m = -INFINITY;
    for (int s = 0; s < n_splits; ++s) m = fmaxf(m, __ldcg(a.part_ml + (base + s) * 2));
    float acc[DH / 32];
#pragma unroll
    for (int q = 0; q < DH / 32; ++q) acc[q] = 0.f;
    float l = 0.f;
    for (int s = 0; s < n_splits; ++s) {
      const float f = fast_exp2(__ldcg(a.part_ml + (base + s) * 2) - m);
      l += f * __ldcg(a.part_ml + (base + s) * 2 + 1);
#pragma unroll
      for (int q = 0; q < DH / 32; ++q) acc[q] += f * __ldcg(a.part_o + (base + s) * DH + q * 32 + lane);
    }
    const float inv = 1.f / l;
    bf16* dst = a.out + size_t(tok) * (a.n_q * a.dh) + head * a.dh;       // (a 96-wide head is computed zero-padded to 128)
#pragma unroll
    for (int q = 0; q < DH / 32; ++q)
      if (q * 32 + lane < a.dh) dst[q * 32 + lane] = __float2bfloat16_rn(acc[q] * inv);
  }
}

template <int DH>
constexpr size_t decode_smem_bytes() { return kDcStages * 2 * 64 * DH * 2 + 16 * DH * 2 + 1024 + 64; }   // ... + barriers and abort flags

// opt in to the dynamic shared memory of the decode kernels on the current device (every layer creation calls this)
cudaError_t attn_decode_configure() {
  cudaError_t e = cudaFuncSetAttribute(attn_decode_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(decode_smem_bytes<64>()));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(attn_decode_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(decode_smem_bytes<128>()));
}

template <int DH>
static void launch_decode_t(const CUtensorMap& tmK, const CUtensorMap& tmV, const AttnArgs& a, cudaStream_t st) {
  constexpr size_t smem = decode_smem_bytes<DH>();
  static_assert(kDcStages * 2 * 64 * DH * 2 >= (4 * 16 * DH + 128 + 4) * 4, "merge buffer must fit in the stages");
  dim3 grid(a.max_splits, a.n_kv, a.n_seqs);
  launch_pdl(attn_decode_kernel<DH>, grid, dim3(kDcThreads), smem, st, tmK, tmV, a);
}

void launch_attn_decode(const CUtensorMap& tmK, const CUtensorMap& tmV, const AttnArgs& a, cudaStream_t st) {
  if (a.n_seqs <= 0) return;
  if (a.dh > 64) launch_decode_t<128>(tmK, tmV, a, st);
  else launch_decode_t<64>(tmK, tmV, a, st);
}

}  // namespace foe
