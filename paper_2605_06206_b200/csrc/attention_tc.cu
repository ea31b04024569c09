// Prefill attention on the 5th-generation tensor cores: causal softmax(q k^T / sqrt(d_h)) v for the new
// tokens of every sequence against the paged cache ("Attn_h" of the paper's Table 2; cluster h's query heads
// read cluster h's KV heads).
//
// One CTA owns 128 query rows of TWO query heads that share a KV head (GQA), so both tiles walk the same K/V
// pages with the same causal extent.  Per page of 64 keys:
//     S_t = Q_t K^T        tcgen05.mma  M128 N64  K16 x (d_h/16)   accumulator in tensor memory
//     P_t = softmax step   TWO threads per query row (in two warps that own the same tensor-memory lanes) take the
//                          64-key steps in turn: one the even steps, the other the odd ones.  A step's thread loads the
//                          row's 64 scores (tcgen05.ld), takes their maximum, receives the running reference maximum
//                          from the other thread (published early in ITS step, long before its exponentials are done),
//                          publishes its own, and then has two step times for exponentials, row sum and packing; so the
//                          softmax of step j+1 overlaps that of step j.  P goes into tensor memory as bf16 pairs
//                          (tcgen05.st), in one of two 32-column buffers beside the scores
//     O_t += P_t V         tcgen05.mma  M128 N d_h K16 x 4 with the A operand read from tensor memory, V used straight
//                          from its page ([key][d_h], i.e. an MN-major B operand); O stays in tensor memory for the
//                          whole row block
// The running maximum used for the exponentials is only moved when the true maximum has grown by more than
// 2^8 since it was last moved (the result is mathematically the same, probabilities stay below 256); only
// then is O rescaled in tensor memory (tcgen05.ld / tcgen05.st), which after the first pages is rare.
// Warp roles: warp 0 TMA producer (Q once, K/V pages through a 5-stage ring), warps 1 and 2 MMA issuers (one per tile), warps 4-19 softmax:
// four groups of four warps (tile 0 even steps, tile 0 odd steps, tile 1 even, tile 1 odd), a warp's lane quarter of
// tensor memory being warp % 4 as the hardware fixes it.  One thread per row and step (the whole dependent chain of a
// step in one thread) left the tensor core and the special-function unit idle half of the time, because a tile's next
// step could not start before the previous one had finished; with the steps alternating between two threads that
// chain is two steps long.  While one tile's softmax runs, the tensor core works on the other tile.  All waits are
// bounded; on expiry the role records a timeout in the status word and the CTA still reaches its teardown (tensor
// memory is released).
#include <math.h>

#include "common.cuh"
#include "kernels.h"

namespace foe {

constexpr int kAtRows = 128;          // query rows per tile
constexpr int kAtKeys = 64;           // keys per step = one cache page
constexpr int kAtStages = 5;
constexpr int kAtThreads = 640;        // warpgroup 0: producer, MMA issuer (+2 idle warps); warpgroups 1-4: softmax
// Registers: 640 threads start with kAtRegsLaunch = 96 each (the most a block of this size can have).  Warpgroup 0
// needs few and hands its share back (setmaxnreg.dec), the four softmax warpgroups take 112 (setmaxnreg.inc): with 96
// the softmax loop spills, and a spilled value in its chain of dependent instructions costs a round trip to L1 each
// time (measured: a quarter of all executed instructions were local loads and stores, the kernel 3.4 times slower).
// setmaxnreg.inc WAITS, without a limit, until the block's own pool holds the registers it asks for, and that pool is
// only what the block was launched with: what the four softmax warpgroups take must not exceed what warpgroup 0 gives
// back.  The launcher checks the kernel's actual register count against this before the first launch.
constexpr int kAtRegsLaunch = 96, kAtRegsLow = 32, kAtRegsHigh = 112;
static_assert(4 * (kAtRegsHigh - kAtRegsLaunch) <= kAtRegsLaunch - kAtRegsLow, "softmax warpgroups would wait for registers forever");

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
// barrier among `count` threads (whole warps) that name the same id; ids 1..15 (0 is __syncthreads)
__device__ __forceinline__ void named_barrier(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
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
  static constexpr int kHandOff = kBarOff + 256;               // [2 tiles][128 rows] reference maximum handed between a row's threads
  static constexpr size_t kBytes = kHandOff + 2 * kAtRows * 4 + 1024;
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
  uint64_t* s_full = kv_empty + kAtStages; // 2 tiles: the tile's scores are in tensor memory
  uint64_t* s_free = s_full + 2;           // 2 tiles: the step's four softmax warps hold the scores in registers
  uint64_t* p_ready = s_free + 2;          // 2
  uint64_t* o_full = p_ready + 2;          // 2 tiles x 2 step parities: phase i of [t][b] = the P V product of step 2 i + b has completed
  uint64_t* o_done = o_full + 4;           // 2 tiles: every product of the block has completed (one phase)
  uint64_t* hand = o_done + 2;             // 2 tiles x 4 lane quarters: phase j = step j's reference maximum is published
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(hand + 8);

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
    for (int s = 0; s < kAtStages; ++s) { mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], n_tiles_q); }
    for (int t = 0; t < 2; ++t) {
      mbar_init(&s_full[t], 1); mbar_init(&s_free[t], 4); mbar_init(&p_ready[t], 4);
      mbar_init(&o_full[2 * t], 1); mbar_init(&o_full[2 * t + 1], 1);
      mbar_init(&o_done[t], 1);
      for (int q = 0; q < 4; ++q) mbar_init(&hand[4 * t + q], 1);
    }
    mbar_fence_init();
    tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // tensor-memory columns of tile t: scores at 128 t (64 columns, rewritten by the next step's Q K^T as soon as every
  // softmax warp of the tile has them in registers), P of step parity b at 128 t + 64 + 32 b; O at 256 + DH t
  const uint32_t q_u32 = smem_u32(smem + L::kQOff), kv_u32 = smem_u32(smem + L::kKVOff);

  if (warp < 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kAtRegsLow));
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
  } else if (warp == 1 || warp == 2) {
    // ------------------------------------------------------------------ MMA issuers, one per tile: a tile's products are
    // issued as soon as ITS scores have been read or ITS probabilities are in place, whatever the other tile is waiting for
    const int t = warp - 1;
    if (t < n_tiles_q && elect_one()) {
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
          umma_bf16(tmem_base + t * 128, desc_kmajor(qb_ + off_q), desc_kmajor(kb_ + off_k), idesc_s, ks != 0);
        }
        umma_commit(&s_full[t]);
      };
      auto issue_o = [&](int t, int j) {                      // O_t = P_t V_j
        const int s = j % kAtStages;
        // P_t(j) sits in tensor memory beside the scores (two bf16 per column, 8 columns per K = 16)
        const uint32_t p_tmem = tmem_base + t * 128 + 64 + (j & 1) * 32, vb_ = kv_u32 + s * 2 * L::kKVTile + L::kKVTile;
#pragma unroll
        for (int kk = 0; kk < kAtKeys / 16; ++kk)
          umma_bf16_ts(tmem_base + 256 + t * DH, p_tmem + kk * 8,
                       desc_mnmajor(vb_ + kk * (16 * 128), kAtKeys * 128, 1024), idesc_o, (j | kk) != 0);
        umma_commit(&o_full[2 * t + (j & 1)]);
      };
      if (ok && n_tiles > 0) {
        ok = mbar_wait(&kv_full[0], 0);
        if (ok) {
          tc_fence_after();
          issue_s(t, 0);
        }
      }
      // Two streams of work, each in its own order: Q K^T of step q as soon as its K/V page has landed and the scores of
      // step q-1 have been read out of the buffer; P V of step p as soon as its probabilities are in place.  Whichever is
      // ready is issued (the scores of step j+2 are not held back by the probabilities of step j: the thread that
      // will need them is the one that is finishing step j).
      int q = 1, p = 0;                                                 // next Q K^T, next P V
      unsigned long long t0 = 0;
      for (uint32_t spin = 0; p < n_tiles && ok;) {
        bool did = false;
        if (q < n_tiles && mbar_test(&kv_full[q % kAtStages], (q / kAtStages) & 1) && mbar_test(&s_free[t], (q - 1) & 1)) {
          tc_fence_after();
          issue_s(t, q);
          ++q;
          did = true;
        }
        if (mbar_test(&p_ready[t], p & 1)) {                            // P_t(p) is in tensor memory
          tc_fence_after();
          issue_o(t, p);
          umma_commit(&kv_empty[p % kAtStages]);                        // stage p reusable once both tiles' products retire
          ++p;
          did = true;
        }
        if (did) { spin = 0; t0 = 0; continue; }
        if ((++spin & 0x3ff) == 0) {                                    // bounded like every other wait
          const unsigned long long now = globaltimer_ns();
          if (t0 == 0) t0 = now;
          else if (now - t0 > kWaitLimitNs) ok = false;
        }
      }
      umma_commit(&o_done[t]);                                          // (also after a timeout: nobody waits in vain)
      if (!ok) atomicExch(a.status, kStatusTimeout);
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kAtRegsHigh));
    // ------------------------------------------------------------------ softmax, two threads per query row
    const int grp = (warp - 4) >> 2;                         // four consecutive warps cover the four lane quarters
    const int t = grp >> 1;                                  // tile of this warp group
    const int g = grp & 1;                                   // this thread takes the steps j with j % 2 == g
    if (t < n_tiles_q) {
      const int quarter = warp & 3;
      const int row = quarter * 32 + lane;                   // row of the tile = TMEM lane
      const uint32_t lane_sel = static_cast<uint32_t>(quarter * 32) << 16;
      const uint32_t s_base = tmem_base + lane_sel + t * 128;
      const uint32_t p_base = s_base + 64;
      const uint32_t o_addr = tmem_base + lane_sel + 256 + t * DH;
      const int qpos = ctx + q0 + row;
      const int first_mask_tile = (ctx + q0) / kAtKeys;
      float* m_hand = reinterpret_cast<float*>(smem + L::kHandOff) + t * kAtRows + row;
      uint64_t* hand_bar = &hand[4 * t + quarter];
      // m_ref: the (possibly stale) maximum the exponentials of the row use, the same in both of its threads at every
      // step; l_run: sum of the probabilities of THIS thread's steps, kept relative to m_ref
      float m_ref = -INFINITY, l_run = 0.f;
      bool ok = true;
      for (int j = g; j < n_tiles; j += 2) {
        const uint32_t ph = j & 1;
        const bool masked = j >= first_mask_tile;
        // The reference the row's other thread used in step j-1 (it may have moved it); this thread's sum follows.
        // Waiting for it FIRST also keeps the parity wait on the scores sound: a thread sees only every other phase of
        // that barrier, and a parity wait must not start before the phase preceding the awaited one has completed
        // (the other thread publishes its reference after it has read the scores of step j-1).  It costs nothing: the
        // scores of step j cannot be there before the other thread has released the buffer, just before it publishes.
        if (j > 0) {
          if (!mbar_wait(hand_bar, ph ^ 1)) { ok = false; break; }
          const float m_prev = *m_hand;
          if (m_prev != m_ref) {
            l_run *= (m_ref == -INFINITY) ? 0.f : fast_exp2(m_ref - m_prev);
            m_ref = m_prev;
          }
        }
        uint32_t r0[32], r1[32];                             // the 64 scores of this row
        if (!mbar_wait(&s_full[t], ph)) { ok = false; break; }
        tc_fence_after();
        tmem_ld32(s_base, r0);                               // two loads in flight, one wait
        tmem_ld32(s_base + 32, r1);
        tmem_ld_wait();
        tc_fence_before();                                   // the scores are in registers: the buffer may take step j+1
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_free[t]);
        if (masked) {
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            if (j * kAtKeys + c > qpos) r0[c] = 0xff800000u;          // -inf: key after the query
            if (j * kAtKeys + 32 + c > qpos) r1[c] = 0xff800000u;
          }
        }
        float mx;
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
        // publish this step's reference at once: the other thread needs nothing else to start its exponentials
        *m_hand = move ? m_new : m_ref;
        __syncwarp();
        if (lane == 0) mbar_arrive(hand_bar);
        // The completion of the previous step's P V product is observed exactly once per step (a parity wait only tells
        // phases apart if the waiter is at most one phase behind; the scores of step j being there means that every
        // product up to step j-2 has completed, the tensor core finishing its work in the order of issue): here when O
        // has to be rescaled, otherwise at the end of the step.
        bool o_seen = (j == 0);
        if (move) {
          const float alpha = (m_ref == -INFINITY) ? 0.f : fast_exp2(m_ref - m_new);
          if (j > 0) {
            if (!mbar_wait(&o_full[2 * t + (ph ^ 1)], ((j - 1) >> 1) & 1)) { ok = false; break; }   // every P V product so far has landed
            o_seen = true;
            tc_fence_after();
            // eight columns at a time: this path is rare, and a wider chunk here would raise the register demand of
            // the whole loop (the scores stay live across it)
#pragma unroll 1
            for (int c8 = 0; c8 < DH / 8; ++c8) {
              uint32_t r[8];
              tmem_ld8(o_addr + c8 * 8, r);
              tmem_ld_wait();
#pragma unroll
              for (int c = 0; c < 8; ++c) r[c] = __float_as_uint(__uint_as_float(r[c]) * alpha);
              tmem_st8(o_addr + c8 * 8, r);
            }
            tmem_st_wait();
          }
          l_run *= alpha;
          m_ref = m_new;
        }
        const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
        // probabilities, written as the bf16 A operand of the PV product (exp2(-inf) = 0 handles the mask), sixteen
        // scores at a time: scalings (packed, two values per instruction), exponentials back to back, sums and packing.
        // P of step j-2 sat in this buffer; its product has completed (see above).
        const uint32_t p_addr = p_base + (j & 1) * 32;
        if (j >= 2 && !mbar_wait(&o_full[2 * t + ph], ((j - 2) >> 1) & 1)) { ok = false; break; }   // P V of step j-2 has read this buffer
        uint64_t rs2[4] = {0ull, 0ull, 0ull, 0ull};           // four independent chains of (even, odd) partial sums
        const uint64_t sc2 = pack_f32x2(a.scale_log2, a.scale_log2), nm2 = pack_f32x2(-m_use, -m_use);
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          uint32_t (&rr)[32] = (q4 < 2) ? r0 : r1;
          const int c0 = (q4 & 1) * 16;
          float e[16];
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            const uint64_t v = fma_f32x2(pack_b32x2(rr[c0 + 2 * c], rr[c0 + 2 * c + 1]), sc2, nm2);
            unpack_f32x2(v, e[2 * c], e[2 * c + 1]);
          }
#pragma unroll
          for (int c = 0; c < 16; ++c) asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(e[c]) : "f"(e[c]));
          uint32_t pk[8];
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            rs2[c & 3] = add_f32x2(rs2[c & 3], pack_f32x2(e[2 * c], e[2 * c + 1]));
            pk[c] = pack_bf16(e[2 * c], e[2 * c + 1]);
          }
          tmem_st8(p_addr + q4 * 8, pk);
        }
        float rs4[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) { float lo, hi; unpack_f32x2(rs2[q], lo, hi); rs4[q] = lo + hi; }
        l_run += (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]);
        // (before this warp's arrival below: P V of step j cannot have been issued yet, so the barrier is at most one
        // phase ahead of what is waited for)
        if (!o_seen && !mbar_wait(&o_full[2 * t + (ph ^ 1)], ((j - 1) >> 1) & 1)) { ok = false; break; }
        tmem_st_wait();                                      // P is in tensor memory
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_ready[t]);
      }
      if (ok) ok = mbar_wait(&o_done[t], 0);                 // every product of the block has completed
      tc_fence_after();
      if (!ok && lane == 0) atomicExch(a.status, kStatusTimeout);
      // The row's two threads meet here, once per block, through four columns of the tile's score buffer in tensor
      // memory (free by now): each leaves the reference it last knew and its partial sum.  Both warps of a row reach
      // this barrier whatever happened before (every wait above is bounded), so it cannot hang.
      tmem_st1(s_base + 2 * g, __float_as_uint(m_ref));
      tmem_st1(s_base + 2 * g + 1, __float_as_uint(l_run));
      tmem_st_wait();
      tc_fence_before();
      const int pair_bar = 1 + t * 4 + quarter;              // the two warps that own these 32 rows
      named_barrier(pair_bar, 64);
      tc_fence_after();
      if (ok) {
        // The reference only ever grows and O is scaled to its last value, the larger of the two; each sum is brought to
        // it.  Then normalise: the pair stages its 32 rows in its slice of the (no longer needed) query tile, each
        // thread half of the row's columns; after a second barrier each warp stores 16 of the rows whole.
        const float m_o = __uint_as_float(tmem_ld1(s_base + 2 * (g ^ 1)));
        const float l_o = __uint_as_float(tmem_ld1(s_base + 2 * (g ^ 1) + 1));
        const float m_fin = fmaxf(m_ref, m_o);
        const float l_mine = (m_ref == -INFINITY) ? 0.f : l_run * fast_exp2(m_ref - m_fin);
        const float l_oth = (m_o == -INFINITY) ? 0.f : l_o * fast_exp2(m_o - m_fin);
        const float inv_l = 1.f / (g ? l_oth + l_mine : l_mine + l_oth);      // same order in both threads
        uint8_t* stg = smem + L::kQOff + t * L::kQTile + quarter * 32 * (DH * 2);
#pragma unroll
        for (int cq = 0; cq < DH / 64; ++cq) {
          const int ch = g * (DH / 64) + cq;
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
      }
      named_barrier(pair_bar, 64);
      if (ok) {
        const uint8_t* stg = smem + L::kQOff + t * L::kQTile + quarter * 32 * (DH * 2);
        constexpr int CH = DH / 8;                           // 16-byte chunks per row
        constexpr int RPI = 32 / CH;                         // rows per store instruction
        for (int r0 = g * 16; r0 < g * 16 + 16; r0 += RPI) {
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

// The register hand-over inside the kernel assumes it was compiled to kAtRegsLaunch registers per thread; anything else
// (another compiler, other flags) would make setmaxnreg.inc wait forever, so it is refused here instead.
template <int DH>
static cudaError_t check_registers() {
  cudaFuncAttributes fa;
  const cudaError_t e = cudaFuncGetAttributes(&fa, attn_prefill_tc_kernel<DH>);
  if (e != cudaSuccess) return e;
  return fa.numRegs == kAtRegsLaunch ? cudaSuccess : cudaErrorInvalidConfiguration;
}

cudaError_t attn_prefill_configure() {
  cudaError_t e = check_registers<64>();
  if (e == cudaSuccess) e = check_registers<128>();
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attn_prefill_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(AtSmem<64>::kBytes));
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
