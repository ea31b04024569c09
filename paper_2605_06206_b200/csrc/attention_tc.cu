// Prefill attention on the 5th-generation tensor cores: causal softmax(q k^T / sqrt(d_h)) v for the new
// tokens of every sequence against the paged cache ("Attn_h" of the paper's Table 2; cluster h's query heads
// read cluster h's KV heads).
//
// One CTA owns 128 query rows of TWO query heads that share a KV head (GQA), so both tiles walk the same K/V
// pages with the same causal extent.  Per page of 64 keys:
//     S_t = Q_t K^T        tcgen05.mma  M128 N64  K16 x (d_h/16)   accumulator in tensor memory
//     P_t = softmax step   one thread per query row: tcgen05.ld, exp2, row max/sum without any shuffle,
//                          P written back into tensor memory as bf16 pairs over the scores it came from (tcgen05.st)
//     O_t += P_t V         tcgen05.mma  M128 N d_h K16 x 4 with the A operand read from tensor memory, V used straight
//                          from its page ([key][d_h], i.e. an MN-major B operand); O stays in tensor memory for the
//                          whole row block
// The running maximum used for the exponentials is only moved when the true maximum has grown by more than
// 2^8 since it was last moved (the result is mathematically the same, probabilities stay below 256); only
// then is O rescaled in tensor memory (tcgen05.ld / tcgen05.st), which after the first pages is rare.
// Warp roles: warp 0 TMA producer (Q once, K/V pages through a 5-stage ring), warp 1 MMA issuer (warps 2-3
// idle), warps 4-7 softmax of tile 0, warps 8-11
// softmax of tile 1.  While one tile's softmax runs, the tensor core works on
// the other tile.  All waits are bounded; on expiry the role records a timeout in the status word and the
// CTA still reaches its teardown (tensor memory is released).
#include <math.h>

#include "common.cuh"
#include "kernels.h"

namespace foe {

constexpr int kAtRows = 128;          // query rows per tile
constexpr int kAtKeys = 64;           // keys per step = one cache page
constexpr int kAtStages = 5;
constexpr int kAtThreads = 384;        // warpgroup 0: producer + MMA issuer (+2 idle warps); warpgroups 1, 2: softmax

// two fp32 values in one 64-bit register and the packed instructions on them
__device__ __forceinline__ uint64_t pack_b32x2(uint32_t lo, uint32_t hi) {
  uint64_t v;
  asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "r"(lo), "r"(hi));
  return v;
}
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) { return pack_b32x2(__float_as_uint(lo), __float_as_uint(hi)); }
__device__ __forceinline__ void unpack_f32x2(uint64_t v, float& lo, float& hi) {
  uint32_t a, b;
  asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(v));
  lo = __uint_as_float(a);
  hi = __uint_as_float(b);
}
__device__ __forceinline__ uint64_t fma_f32x2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add_f32x2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// K-major operand, 128-byte swizzle (rows of 128 bytes, 8-row groups 1024 bytes apart)
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t addr) { return umma_desc_sw128(addr); }
// MN-major operand, 128-byte swizzle: 64 contiguous elements of the M/N dimension per 128-byte row, one row
// per k; 8-k groups `sbo` bytes apart, successive 64-element blocks of M/N `lbo` bytes apart.
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr >> 4) & 0x3fff);
  d |= static_cast<uint64_t>((lbo >> 4) & 0x3fff) << 16;
  d |= static_cast<uint64_t>((sbo >> 4) & 0x3fff) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}

template <int DH>
struct AtSmem {
  static constexpr int kHalves = DH / 64;
  static constexpr int kQTile = kAtRows * DH * 2;              // one query tile
  static constexpr int kKVTile = kAtKeys * DH * 2;             // one K or V page of one head
  static constexpr int kQOff = 0;
  static constexpr int kKVOff = 2 * kQTile;
  static constexpr int kBarOff = kKVOff + kAtStages * 2 * kKVTile;
  static constexpr size_t kBytes = kBarOff + 256 + 1024;
};

template <int DH>
__global__ void __launch_bounds__(kAtThreads, 1)
attn_prefill_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                       const __grid_constant__ CUtensorMap tmV, const AttnArgs a) {
  pdl_wait();
  pdl_launch_dependents();
  using L = AtSmem<DH>;
  constexpr int HN = DH / 64;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOff);
  uint64_t* q_full = bars;                 // 1
  uint64_t* kv_full = bars + 1;            // kAtStages
  uint64_t* kv_empty = kv_full + kAtStages;
  uint64_t* s_full = kv_empty + kAtStages; // 2 tiles x 2 score buffers
  uint64_t* p_ready = s_full + 4;          // 2
  uint64_t* o_full = p_ready + 2;          // 2
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_full + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Blocks start in the order of their linear index.  The work of a block grows with its query block (causal
  // extent), so the index runs over (sequence, head pair) fastest and over the query block slowest, late query
  // blocks first: every long block of the whole call starts before any short one, and the short ones fill the tail.
  const int lin = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
  const int per_qb = gridDim.y * gridDim.z;
  const int qb = gridDim.x - 1 - lin / per_qb;
  const int pair = (lin % per_qb) % gridDim.y;
  const int b = (lin % per_qb) / gridDim.y;
  const int G = a.n_q / a.n_kv;
  const int n_tiles_q = (G % 2 == 0) ? 2 : 1;              // heads per CTA
  const int head0 = pair * n_tiles_q;
  const int q_len = a.q_lens ? a.q_lens[b] : 1;
  const int q0 = qb * kAtRows;
  if (q0 >= q_len) return;
  const int tok0 = a.cu_q[b] + q0;
  if (tok0 < 0 || tok0 >= a.n_tokens) return;              // q_lens that disagree with the call's token count (reported by the token map)
  const int kvh = head0 / G;
  const int rows_here = min(min(kAtRows, q_len - q0), a.n_tokens - tok0);
  // a context length outside what the block table can describe is reported by the token map; here it is only kept
  // from driving the loop bounds
  const int ctx = min(max(a.context_lens[b], 0), max(a.max_pages_per_seq * kAtKeys - (q0 + rows_here), 0));
  const int kv_len = ctx + q0 + rows_here;
  const int n_tiles = (kv_len + kAtKeys - 1) / kAtKeys;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < kAtStages; ++s) { mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1); }
    for (int t = 0; t < 2; ++t) {
      mbar_init(&s_full[2 * t], 1); mbar_init(&s_full[2 * t + 1], 1); mbar_init(&p_ready[t], 4); mbar_init(&o_full[t], 1);
    }
    mbar_fence_init();
    tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // tensor-memory columns: scores of tile t, step parity b at 128 t + 64 b (double-buffered so that the next
  // step's Q K^T runs while this step's softmax is still reading); O of tile t at 256 + DH t
  const uint32_t q_u32 = smem_u32(smem + L::kQOff), kv_u32 = smem_u32(smem + L::kKVOff);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (elect_one()) {
      bool ok = true;
      mbar_expect_tx(q_full, n_tiles_q * L::kQTile);
      for (int t = 0; t < n_tiles_q; ++t)
        for (int h = 0; h < HN; ++h)
          tma_load_2d(smem + L::kQOff + t * L::kQTile + h * (kAtRows * 128), &tmQ, q_full, (head0 + t) * DH + h * 64, tok0);
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int s = j % kAtStages;
        if (!mbar_wait(&kv_empty[s], ((j / kAtStages) & 1) ^ 1)) { ok = false; break; }
        int page = a.block_table[size_t(b) * a.max_pages_per_seq + min(j, a.max_pages_per_seq - 1)];
        if (page < 0 || page >= a.num_pages) { atomicExch(a.status, kStatusBounds); page = 0; }
        const int row0 = (page * a.n_kv + kvh) * kAtKeys;
        uint8_t* kd = smem + L::kKVOff + s * 2 * L::kKVTile;
        mbar_expect_tx(&kv_full[s], 2 * L::kKVTile);
        for (int h = 0; h < HN; ++h) {
          tma_load_2d(kd + h * (kAtKeys * 128), &tmK, &kv_full[s], h * 64, row0);
          tma_load_2d(kd + L::kKVTile + h * (kAtKeys * 128), &tmV, &kv_full[s], h * 64, row0);
        }
      }
      if (!ok) atomicExch(a.status, kStatusTimeout);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (elect_one()) {
      constexpr uint32_t idesc_s = umma_idesc_bf16(kAtRows, kAtKeys);
      constexpr uint32_t idesc_o = umma_idesc_bf16(kAtRows, DH) | (1u << 16);      // B operand (V) is MN-major
      bool ok = mbar_wait(q_full, 0);
      auto issue_s = [&](int t, int j) {                      // S_t = Q_t K_j^T
        const int s = j % kAtStages;
        const uint32_t qb_ = q_u32 + t * L::kQTile, kb_ = kv_u32 + s * 2 * L::kKVTile;
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks) {
          const uint32_t off_q = (ks >> 2) * (kAtRows * 128) + (ks & 3) * 32;
          const uint32_t off_k = (ks >> 2) * (kAtKeys * 128) + (ks & 3) * 32;
          umma_bf16(tmem_base + t * 128 + (j & 1) * 64, desc_kmajor(qb_ + off_q), desc_kmajor(kb_ + off_k), idesc_s, ks != 0);
        }
        umma_commit(&s_full[2 * t + (j & 1)]);
      };
      auto issue_o = [&](int t, int j) {                      // O_t = P_t V_j
        const int s = j % kAtStages;
        // P_t(j) sits in tensor memory, over the first 32 columns of the score buffer it was computed from
        // (two bf16 per column, 8 columns per K = 16)
        const uint32_t p_tmem = tmem_base + t * 128 + (j & 1) * 64, vb_ = kv_u32 + s * 2 * L::kKVTile + L::kKVTile;
#pragma unroll
        for (int kk = 0; kk < kAtKeys / 16; ++kk)
          umma_bf16_ts(tmem_base + 256 + t * DH, p_tmem + kk * 8,
                       desc_mnmajor(vb_ + kk * (16 * 128), kAtKeys * 128, 1024), idesc_o, (j | kk) != 0);
        umma_commit(&o_full[t]);
      };
      if (ok && n_tiles > 0) {
        ok = mbar_wait(&kv_full[0], 0);
        if (ok) {
          tc_fence_after();
          for (int t = 0; t < n_tiles_q; ++t) issue_s(t, 0);
        }
      }
      for (int j = 0; j < n_tiles && ok; ++j) {
        const uint32_t ph = j & 1;
        // scores of the next step first: their buffer was released by p_ready(j-1), waited for one iteration ago
        if (j + 1 < n_tiles) {
          if (!mbar_wait(&kv_full[(j + 1) % kAtStages], ((j + 1) / kAtStages) & 1)) { ok = false; break; }
          tc_fence_after();
          for (int t = 0; t < n_tiles_q; ++t) issue_s(t, j + 1);
        }
        for (int t = 0; t < n_tiles_q && ok; ++t) {
          if (!mbar_wait(&p_ready[t], ph)) { ok = false; break; }       // P_t(j) is in tensor memory
          tc_fence_after();
          issue_o(t, j);
        }
        if (ok) umma_commit(&kv_empty[j % kAtStages]);                  // stage j reusable once those MMAs retire
      }
      if (!ok) atomicExch(a.status, kStatusTimeout);
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ softmax, one thread per query row
    const int t = (warp - 4) >> 2;                           // tile of this warp group
    if (t < n_tiles_q) {
      const int quarter = warp & 3;
      const int row = quarter * 32 + lane;                   // row of the tile = TMEM lane
      const uint32_t lane_sel = static_cast<uint32_t>(quarter * 32) << 16;
      const uint32_t s_base = tmem_base + lane_sel + t * 128;
      const uint32_t o_addr = tmem_base + lane_sel + 256 + t * DH;
      const int qpos = ctx + q0 + row;
      const int first_mask_tile = (ctx + q0) / kAtKeys;
      float m_ref = -INFINITY, l_run = 0.f;                  // m_ref: the (possibly stale) maximum the exponentials use
      bool ok = true;
      uint32_t r0[32], r1[32];                               // the 64 scores of this row
      bool preloaded = false;                                // the loads of step j were issued at the end of step j-1
      for (int j = 0; j < n_tiles; ++j) {
        const uint32_t ph = j & 1;
        const bool masked = j >= first_mask_tile;
        if (!preloaded) {
          if (!mbar_wait(&s_full[2 * t + (j & 1)], (j >> 1) & 1)) { ok = false; break; }
          tc_fence_after();
          tmem_ld32(s_base + (j & 1) * 64, r0);              // two loads in flight, one wait
          tmem_ld32(s_base + (j & 1) * 64 + 32, r1);
        }
        tmem_ld_wait();
        float mx = -INFINITY;
        if (masked) {
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            if (j * kAtKeys + c > qpos) r0[c] = 0xff800000u;          // -inf: key after the query
            if (j * kAtKeys + 32 + c > qpos) r1[c] = 0xff800000u;
          }
        }
        {                                                    // four independent chains, then a short tree
          float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int c = 0; c < 32; c += 4) {
#pragma unroll
            for (int q = 0; q < 4; ++q)
              m4[q] = fmax3(m4[q], __uint_as_float(r0[c + q]), __uint_as_float(r1[c + q]));
          }
          mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        }
        const float m_new = fmaxf(m_ref, mx * a.scale_log2);
        // move the reference maximum (and rescale O) only when it is off by more than 2^8; warp-uniform so that
        // the tensor-memory accesses stay aligned
        const bool move = __any_sync(0xffffffffu, m_new > m_ref + 8.0f);
        // A parity wait only tells phases apart if the waiter is at most one phase behind the barrier, so every step
        // observes the completion of the previous step's P V product exactly once: here when O has to be rescaled,
        // otherwise at the end of the step, when it has long landed.
        bool o_seen = (j == 0);
        if (move) {
          const float alpha = (m_ref == -INFINITY) ? 0.f : fast_exp2(m_ref - m_new);
          if (j > 0) {
            if (!mbar_wait(&o_full[t], ph ^ 1)) { ok = false; break; }      // every P V product so far has landed
            o_seen = true;
            tc_fence_after();
#pragma unroll
            for (int ch = 0; ch < DH / 32; ++ch) {
              uint32_t r[32];
              tmem_ld32(o_addr + ch * 32, r);
              tmem_ld_wait();
#pragma unroll
              for (int c = 0; c < 32; ++c) r[c] = __float_as_uint(__uint_as_float(r[c]) * alpha);
              tmem_st32(o_addr + ch * 32, r);
            }
            tmem_st_wait();
          }
          l_run *= alpha;
          m_ref = m_new;
        }
        const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
        // probabilities, written as the bf16 A operand of the PV product (exp2(-inf) = 0 handles the mask)
        const uint32_t p_addr = s_base + (j & 1) * 64;
        // Written in stages over 32 values: all scalings, then all exponentials back to back, then sums and packing.
        // Packed fp32 arithmetic (two values per instruction) for the scaling and the row sums: the step is bound by
        // the softmax warps' instruction stream, not by any one unit.
        uint64_t rs2[4] = {0ull, 0ull, 0ull, 0ull};           // four independent chains of (even, odd) partial sums
        const uint64_t sc2 = pack_f32x2(a.scale_log2, a.scale_log2), nm2 = pack_f32x2(-m_use, -m_use);
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          uint32_t (&rr)[32] = hf ? r1 : r0;
          float e[32];
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            const uint64_t v = fma_f32x2(pack_b32x2(rr[2 * c], rr[2 * c + 1]), sc2, nm2);
            unpack_f32x2(v, e[2 * c], e[2 * c + 1]);
          }
#pragma unroll
          for (int c = 0; c < 32; ++c) asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(e[c]) : "f"(e[c]));
          uint32_t pk[16];
#pragma unroll
          for (int c = 0; c < 16; ++c) {
            rs2[c & 3] = add_f32x2(rs2[c & 3], pack_f32x2(e[2 * c], e[2 * c + 1]));
            pk[c] = pack_bf16(e[2 * c], e[2 * c + 1]);
          }
          tmem_st16(p_addr + hf * 16, pk);                  // (the scores of this buffer are all in registers by now)
        }
        float rs4[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) { float lo, hi; unpack_f32x2(rs2[q], lo, hi); rs4[q] = lo + hi; }
        l_run += (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]);
        // The scores are used up: if the next step's are already there (they usually are, the issuer runs a step
        // ahead), start loading them now, so that the load's latency passes behind the stores and arrivals below.
        preloaded = false;
        if (j + 1 < n_tiles) {
          const int jn = j + 1;
          bool ready = false;
          if (lane == 0) ready = mbar_test(&s_full[2 * t + (jn & 1)], (jn >> 1) & 1);
          preloaded = __shfl_sync(0xffffffffu, ready, 0);
          if (preloaded) {
            tc_fence_after();
            tmem_ld32(s_base + (jn & 1) * 64, r0);
            tmem_ld32(s_base + (jn & 1) * 64 + 32, r1);
          }
        }
        // (before this warp's arrival below: P V of step j cannot have been issued yet, so the barrier is at most one
        // phase ahead of what is waited for)
        if (!o_seen && !mbar_wait(&o_full[t], ph ^ 1)) { ok = false; break; }
        tmem_st_wait();                                      // P is in tensor memory
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_ready[t]);
      }
      if (ok && n_tiles > 0) ok = mbar_wait(&o_full[t], (n_tiles - 1) & 1);
      tc_fence_after();
      if (!ok) {
        if (lane == 0) atomicExch(a.status, kStatusTimeout);
      } else {
        // normalise; stage the warp's 32 rows in its slice of the (no longer needed) query tile; store rows whole
        const float inv_l = 1.f / l_run;
        uint8_t* stg = smem + L::kQOff + t * L::kQTile + quarter * 32 * (DH * 2);
        constexpr int CH = DH / 8;                           // 16-byte chunks per row
#pragma unroll
        for (int ch = 0; ch < DH / 32; ++ch) {
          uint32_t r[32];
          tmem_ld32(o_addr + ch * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int c = ch * 4 + q;
            uint4 v = make_uint4(pack_bf16(__uint_as_float(r[8 * q]) * inv_l, __uint_as_float(r[8 * q + 1]) * inv_l),
                                 pack_bf16(__uint_as_float(r[8 * q + 2]) * inv_l, __uint_as_float(r[8 * q + 3]) * inv_l),
                                 pack_bf16(__uint_as_float(r[8 * q + 4]) * inv_l, __uint_as_float(r[8 * q + 5]) * inv_l),
                                 pack_bf16(__uint_as_float(r[8 * q + 6]) * inv_l, __uint_as_float(r[8 * q + 7]) * inv_l));
            *reinterpret_cast<uint4*>(stg + lane * (DH * 2) + ((c ^ (lane & 7)) << 4)) = v;
          }
        }
        __syncwarp();
        constexpr int RPI = 32 / CH;                         // rows per store instruction
        for (int r0 = 0; r0 < 32; r0 += RPI) {
          const int rr = r0 + lane / CH, c = lane % CH;
          const int grow = quarter * 32 + rr;
          if (grow < rows_here && c * 8 < a.dh)            // (a 96-wide head is computed zero-padded to 128)
            *reinterpret_cast<uint4*>(a.out + size_t(tok0 + grow) * (a.n_q * a.dh) + (head0 + t) * a.dh + c * 8) =
                *reinterpret_cast<const uint4*>(stg + rr * (DH * 2) + ((c ^ (rr & 7)) << 4));
        }
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

cudaError_t attn_prefill_configure() {
  cudaError_t e = cudaFuncSetAttribute(attn_prefill_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(AtSmem<64>::kBytes));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(attn_prefill_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(AtSmem<128>::kBytes));
}

template <int DH>
static void launch_tc(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const AttnArgs& a,
                      cudaStream_t st) {
  const int G = a.n_q / a.n_kv;
  const int heads_per_cta = (G % 2 == 0) ? 2 : 1;
  dim3 grid((a.max_q_len + kAtRows - 1) / kAtRows, a.n_q / heads_per_cta, a.n_seqs);
  launch_pdl(attn_prefill_tc_kernel<DH>, grid, dim3(kAtThreads), size_t(AtSmem<DH>::kBytes), st, tmQ, tmK, tmV, a);
}

void launch_attn_prefill_tc(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const AttnArgs& a,
                            cudaStream_t st) {
  if (a.n_seqs <= 0 || a.max_q_len <= 0) return;
  if (a.dh > 64) launch_tc<128>(tmQ, tmK, tmV, a, st);
  else launch_tc<64>(tmQ, tmK, tmV, a, st);
}

}  // namespace foe
