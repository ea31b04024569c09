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
// page.  The CTAs are persistent and split the call's pages evenly (see the kernel).
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
// Persistent CTAs (two per SM), warp-specialised: warp 4 streams pages through a ring of shared-memory stages that
// keeps running across the CTA's pieces of work; warps 0..3 each take 16 keys of every page.
//
// Work is cut by PAGES, not by sequences: the pages of all (sequence, KV head) pairs form one list (sequence-major,
// then KV head, then page) of T entries and CTA c takes entries [c * per, (c + 1) * per), per = max(kDcMinTiles,
// ceil(T / grid)).  The part of a pair inside one CTA's range is a segment; a pair is covered by the segments of
// consecutive CTAs, numbered in CTA order.  Every segment leaves a partial (m, l, o) in global memory and takes a ticket
// on its pair; whichever CTA takes the last ticket merges the pair's segments in segment order (so the result does not
// depend on which one that is).  A pair that lies inside one segment is finished without either.  The partition is a
// function of the call's context lengths and the grid only: the same call gives the same bits.  Where a sequence's pages
// are cut depends on the other sequences of the call, so its output can differ in the last bits (the rounding of the
// merge) between two batches it is part of.
constexpr int kDcConsumers = 4;
constexpr int kDcThreads = (kDcConsumers + 1) * 32;
constexpr int kDcStages = 3;
constexpr int kDcMinTiles = 16;                  // fewest pages per CTA: bounds the segments of a pair by pages / 16 + 2
                                                 // (a short call is bound by the GPU's memory rate whether 150 or 296 CTAs
                                                 // stream it; fewer, longer ranges mean fewer segments to merge)

template <int DH>
struct DcSmem {
  static constexpr int kTileBytes = 64 * DH * 2;
  static constexpr int kRingBytes = kDcStages * 2 * kTileBytes;
  static constexpr int kQBytes = 16 * DH * 2;
  static constexpr int kMoPitch = DH + 8;        // floats per row of the merge buffer (rows 8 apart hit different banks)
  static constexpr int kMoBytes = 16 * kMoPitch * 4;
  static constexpr int kQOff = kRingBytes;
  static constexpr int kMoOff = kQOff + kQBytes;
  static constexpr int kMmOff = kMoOff + kMoBytes;               // [4][16] running maxima, then [4][16] running sums
  static constexpr int kBarOff = kMmOff + 2 * 4 * 16 * 4;        // full[stages], empty[stages]
  static constexpr int kMiscOff = kBarOff + 2 * kDcStages * 8;   // ticket
  static constexpr size_t kBytes = size_t(kMiscOff) + 16 + 1024; // + alignment slack
};

// position inside the list of pages
struct DcWalk {
  int b, kvh, page;      // current entry
  int np, kv_len;        // pages and keys (cached + the new token) of sequence b
  int seq_first;         // list index of the first page of sequence b
  int t, t_end;          // current list index, end of this CTA's range
  int per;
};

__device__ __forceinline__ int dc_pages(const AttnArgs& a, int b, int* kv_len) {
  const int ctx = min(max(a.context_lens[b], 0), a.max_kv_pages * 64 - 1);   // (out-of-range values are reported by the QKV step)
  *kv_len = ctx + 1;                                                          // cached tokens + the new one
  return (ctx + 64) >> 6;
}

// Every warp works this out for itself (all 32 lanes): the CTA's range and where it starts.  False: nothing to do.
__device__ __forceinline__ bool dc_begin(const AttnArgs& a, DcWalk& w) {
  const int lane = threadIdx.x & 31;
  int sum = 0, np_first = 0, kl_first = 0;        // (the first 32 sequences' values are kept for the search below)
  for (int b0 = 0; b0 < a.n_seqs; b0 += 32) {
    int kl = 0;
    const int np = b0 + lane < a.n_seqs ? dc_pages(a, b0 + lane, &kl) : 0;
    if (b0 == 0) { np_first = np; kl_first = kl; }
    sum += np;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const int T = sum * a.n_kv;
  w.per = max(kDcMinTiles, (T + int(gridDim.x) - 1) / int(gridDim.x));
  const long long t0 = (long long)blockIdx.x * w.per;
  if (t0 >= T) return false;
  w.t = int(t0);
  w.t_end = min(T, w.t + w.per);
  int base = 0;                                  // pages of the sequences before this chunk of 32
  for (int b0 = 0; b0 < a.n_seqs; b0 += 32) {
    int kl = kl_first;
    const int np = b0 == 0 ? np_first : (b0 + lane < a.n_seqs ? dc_pages(a, b0 + lane, &kl) : 0);
    int incl = np;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    const int first = a.n_kv * (base + incl - np);
    const bool hit = np > 0 && w.t >= first && w.t < first + a.n_kv * np;
    const uint32_t m = __ballot_sync(0xffffffffu, hit);
    if (m) {
      const int src = __ffs(m) - 1;
      w.b = b0 + src;
      w.seq_first = __shfl_sync(0xffffffffu, first, src);
      w.np = __shfl_sync(0xffffffffu, np, src);
      w.kv_len = __shfl_sync(0xffffffffu, kl, src);
      const int rem = w.t - w.seq_first;
      w.kvh = rem / w.np;
      w.page = rem - w.kvh * w.np;
      return true;
    }
    base += __shfl_sync(0xffffffffu, incl, 31);
  }
  return false;                                  // (not reached: t0 < T)
}

// pages of the segment that starts at the current entry
__device__ __forceinline__ int dc_segment_len(const DcWalk& w) { return min(w.np - w.page, w.t_end - w.t); }

__device__ __forceinline__ void dc_advance(const AttnArgs& a, DcWalk& w, int len) {
  w.t += len;
  w.page += len;
  if (w.page >= w.np) {
    w.page = 0;
    w.kvh += 1;
    if (w.kvh == a.n_kv) {
      w.kvh = 0;
      w.seq_first += a.n_kv * w.np;
      w.b += 1;
      if (w.t < w.t_end) w.np = dc_pages(a, w.b, &w.kv_len);
    }
  }
}

__device__ __forceinline__ void dc_consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kDcConsumers * 32) : "memory"); }

template <int DH>
__global__ void __launch_bounds__(kDcThreads, 2)
attn_decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const AttnArgs a) {
  using SM = DcSmem<DH>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr int kTileBytes = SM::kTileBytes;
  uint8_t* kv_s = smem;                                            // [stage][K | V]
  uint8_t* q_s = smem + SM::kQOff;
  float* mo = reinterpret_cast<float*>(smem + SM::kMoOff);         // [16][kMoPitch]
  float* mm = reinterpret_cast<float*>(smem + SM::kMmOff);         // [4][16]
  float* ml = mm + 64;                                             // [4][16]
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + SM::kBarOff);
  uint64_t* empty = full + kDcStages;
  int* ticket_s = reinterpret_cast<int*>(smem + SM::kMiscOff);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kDcStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kDcConsumers); }
    mbar_fence_init();
  }
  __syncthreads();

  // Until pdl_wait() nothing is read that the previous kernel writes.  That kernel is the QKV projection of the same
  // step: it writes q and the new token's K / V, into the last page of every sequence.  Context lengths, the block
  // table and all other pages are older and complete (a kernel lets its successor start only after its own wait).
  DcWalk w;
  const bool any = dc_begin(a, w);                                 // (warp-uniform, and the same in every warp)

  if (warp == kDcConsumers) {
    // ------------------------------------------------------------------ producer
    bool waited = false, ok = true;
    int it = 0;
    while (any && ok && w.t < w.t_end) {
      const int len = dc_segment_len(w);
      for (int j0 = 0; j0 < len && ok; j0 += 32) {
        const int n = min(32, len - j0);
        int row0 = 0;
        if (lane < n) {
          const int lp = w.page + j0 + lane;
          int page = a.block_table[size_t(w.b) * a.max_pages_per_seq + min(lp, a.max_pages_per_seq - 1)];
          if (page < 0 || page >= a.num_pages) { atomicExch(a.status, kStatusBounds); page = 0; }
          row0 = (page * a.n_kv + w.kvh) * 64;
        }
        for (int j = 0; j < n && ok; ++j, ++it) {
          const int st = it % kDcStages;
          const uint32_t ph = (it / kDcStages) & 1;
          const int r0 = __shfl_sync(0xffffffffu, row0, j);
          if (!waited && w.page + j0 + j == w.np - 1) {            // the page the previous kernel writes into
            pdl_wait();
            pdl_launch_dependents();
            waited = true;
          }
          if (lane == 0) {
            ok = mbar_wait(&empty[st], ph ^ 1);
            if (ok) tma_load_page<DH>(kv_s + st * 2 * kTileBytes, kv_s + st * 2 * kTileBytes + kTileBytes, &tmK, &tmV, &full[st], r0);
          }
          ok = __shfl_sync(0xffffffffu, ok, 0);
        }
      }
      dc_advance(a, w, len);
    }
    if (!waited) { pdl_wait(); pdl_launch_dependents(); }
    if (!ok && lane == 0) atomicExch(a.status, kStatusTimeout);
    return;
  }

  // -------------------------------------------------------------------- consumers
  pdl_wait();
  pdl_launch_dependents();
  if (!any) return;
  const int G = a.n_q / a.n_kv;
  const int ld_q = a.n_q * DH;
  const int g = lane >> 2, t4 = lane & 3;
  const uint32_t q_base = smem_u32(q_s);
  const int ctid = threadIdx.x;                                    // 0..127
  bool ok = true;
  int it = 0;

  while (w.t < w.t_end) {
    const int len = dc_segment_len(w);
    const int b = w.b, kvh = w.kvh, kv_len = w.kv_len;
    const int pair_first = w.seq_first + kvh * w.np;
    const int c_first = pair_first / w.per;
    const int n_segs = (pair_first + w.np - 1) / w.per - c_first + 1;
    const int seg = int(blockIdx.x) - c_first;
    const int tok = a.cu_q ? a.cu_q[b] : b;

    dc_consumer_bar();                                             // the previous segment is done with q_s, mo, mm, ticket_s
    for (int q = ctid; q < 16 * (DH / 8); q += kDcConsumers * 32) {
      const int r = q / (DH / 8), ch = q - r * (DH / 8);
      uint4 v = make_uint4(0, 0, 0, 0);
      if (r < G) v = __ldg(reinterpret_cast<const uint4*>(a.q + size_t(tok) * ld_q + (kvh * G + r) * DH + ch * 8));
      *reinterpret_cast<uint4*>(q_s + tile_off<16>(r, ch * 8)) = v;
    }
    dc_consumer_bar();

    float o[DH / 8][4];
#pragma unroll
    for (int n = 0; n < DH / 8; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

    for (int j = 0; j < len; ++j, ++it) {
      const int st = it % kDcStages;
      // A wait that runs out ends this warp's work: it keeps walking the segments (so that it still meets the other
      // warps at every barrier and the tickets are taken) but waits for and computes nothing more.
      if (ok && !mbar_wait(&full[st], (it / kDcStages) & 1)) ok = false;
      if (!ok) continue;
      const uint32_t k_base = smem_u32(kv_s + st * 2 * kTileBytes);
      const uint32_t v_base = k_base + kTileBytes;
      const int key0 = (w.page + j) * 64 + warp * 16;              // this warp's 16 keys of the page
      if (key0 < kv_len) {
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
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[st]);                      // this warp is done with the stage
    }

    // ---- the four warps' states (each saw a different quarter of every page) become one: common maximum, then the
    // warps add their rescaled sums into the buffer in four rounds (fixed order)
    if (t4 == 0) {
      mm[warp * 16 + g] = m_run[0]; mm[warp * 16 + g + 8] = m_run[1];
      ml[warp * 16 + g] = l_run[0]; ml[warp * 16 + g + 8] = l_run[1];
    }
    dc_consumer_bar();
    float f[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      const int row = g + 8 * r;
      const float m_all = fmaxf(fmaxf(mm[row], mm[16 + row]), fmaxf(mm[32 + row], mm[48 + row]));
      f[r] = fast_exp2(m_run[r] - m_all);                          // 0 for a warp that saw no valid key
    }
    // (round k: warp w adds its share of column quarter (w + k) % 4 -- every warp is busy in every round and no two
    //  touch the same columns; quarter c is summed in the order of warps c, c - 1, c - 2, c - 3)
#pragma unroll
    for (int k = 0; k < kDcConsumers; ++k) {
      const int qtr = (warp + k) & 3;
#pragma unroll
      for (int n = 0; n < DH / 8; ++n) {
        if (n / (DH / 32) != qtr) continue;                        // (o[] stays in registers: n is a compile-time index)
        float2* p0 = reinterpret_cast<float2*>(mo + g * SM::kMoPitch + n * 8 + t4 * 2);
        float2* p1 = reinterpret_cast<float2*>(mo + (g + 8) * SM::kMoPitch + n * 8 + t4 * 2);
        float2 a0 = make_float2(0.f, 0.f), a1 = make_float2(0.f, 0.f);
        if (k) { a0 = *p0; a1 = *p1; }
        a0.x += f[0] * o[n][0]; a0.y += f[0] * o[n][1];
        a1.x += f[1] * o[n][2]; a1.y += f[1] * o[n][3];
        *p0 = a0;
        *p1 = a1;
      }
      dc_consumer_bar();
    }
    // row r of the segment: maximum m, sum l, unnormalised output mo[r][.]
    auto row_ml = [&](int r, float& m, float& l) {
      m = fmaxf(fmaxf(mm[r], mm[16 + r]), fmaxf(mm[32 + r], mm[48 + r]));
      l = 0.f;
#pragma unroll
      for (int wq = 0; wq < 4; ++wq) l += fast_exp2(mm[wq * 16 + r] - m) * ml[wq * 16 + r];
    };
    if (n_segs == 1) {
      // the whole pair was this segment: normalise and store
      for (int q = ctid; ok && q < G * DH; q += kDcConsumers * 32) {
        const int r = q / DH, c = q - r * DH;
        float m, l;
        row_ml(r, m, l);
        if (c < a.dh)                                              // (a 96-wide head is computed zero-padded to 128)
          a.out[size_t(tok) * (a.n_q * a.dh) + (kvh * G + r) * a.dh + c] = __float2bfloat16_rn(mo[r * SM::kMoPitch + c] / l);
      }
    } else {
      // A segment whose wait ran out writes no partial state but still takes its ticket: the counter of its pair
      // returns to zero and the handle stays usable (this call's output is not; the status word says so).
      for (int q = ctid; ok && q < G * DH; q += kDcConsumers * 32) {
        const int r = q / DH, c = q - r * DH;
        const size_t pidx = (size_t(b) * a.n_q + kvh * G + r) * a.max_splits + seg;
        a.part_o[pidx * DH + c] = mo[r * SM::kMoPitch + c];
        if (c == 0) {
          float m, l;
          row_ml(r, m, l);
          a.part_ml[pidx * 2] = m;
          a.part_ml[pidx * 2 + 1] = l;
        }
      }
      // (Taking the tickets only when the CTA has finished its range -- one fence and one round trip instead of two --
      //  was slower: a pair's merge then always falls at the very end of the kernel, where nothing overlaps it.)
      __threadfence();
      dc_consumer_bar();
      if (ctid == 0) *ticket_s = atomicAdd(&a.split_done[b * a.n_kv + kvh], 1);
      dc_consumer_bar();
      if (*ticket_s == n_segs - 1) {
        if (ctid == 0) a.split_done[b * a.n_kv + kvh] = 0;         // re-armed for the next call
        __threadfence();
        // One warp per query head of the group.  The segments' (m, l) are read one per lane and their outputs eight
        // segments at a time, so that the merge costs a few round trips to L2 whatever the number of segments.  The
        // sums run in segment order.
        for (int r = warp; r < G; r += kDcConsumers) {
          const int head = kvh * G + r;
          const size_t base = (size_t(b) * a.n_q + head) * a.max_splits;
          float m = -INFINITY;
          for (int s = lane; s < n_segs; s += 32) m = fmaxf(m, __ldcg(a.part_ml + (base + s) * 2));
#pragma unroll
          for (int o2 = 16; o2 > 0; o2 >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o2));
          float acc[DH / 32];
#pragma unroll
          for (int q = 0; q < DH / 32; ++q) acc[q] = 0.f;
          float l = 0.f;
          for (int c0 = 0; c0 < n_segs; c0 += 32) {
            const int n = min(32, n_segs - c0);
            float fs = 0.f, ls = 0.f;                              // lane s: factor and row sum of segment c0 + s
            if (lane < n) {
              fs = fast_exp2(__ldcg(a.part_ml + (base + c0 + lane) * 2) - m);
              ls = __ldcg(a.part_ml + (base + c0 + lane) * 2 + 1);
            }
            for (int u0 = 0; u0 < n; u0 += 8) {
              float v[8][DH / 32];
#pragma unroll
              for (int u = 0; u < 8; ++u)
#pragma unroll
                for (int q = 0; q < DH / 32; ++q)
                  v[u][q] = u0 + u < n ? __ldcg(a.part_o + (base + c0 + u0 + u) * DH + q * 32 + lane) : 0.f;
#pragma unroll
              for (int u = 0; u < 8; ++u) {
                const float fu = __shfl_sync(0xffffffffu, fs, (u0 + u) & 31);   // (0 past the last segment)
                const float lu = __shfl_sync(0xffffffffu, ls, (u0 + u) & 31);
                l += fu * lu;
#pragma unroll
                for (int q = 0; q < DH / 32; ++q) acc[q] += fu * v[u][q];
              }
            }
          }
          const float inv = 1.f / l;
          bf16* dst = a.out + size_t(tok) * (a.n_q * a.dh) + head * a.dh;
#pragma unroll
          for (int q = 0; q < DH / 32; ++q)
            if (q * 32 + lane < a.dh) dst[q * 32 + lane] = __float2bfloat16_rn(acc[q] * inv);
        }
      }
    }
    dc_advance(a, w, len);
  }
  if (!ok && lane == 0) atomicExch(a.status, kStatusTimeout);
}

template <int DH>
constexpr size_t decode_smem_bytes() { return DcSmem<DH>::kBytes; }

// opt in to the dynamic shared memory of the decode kernels on the current device (every layer creation calls this)
cudaError_t attn_decode_configure() {
  cudaError_t e = cudaFuncSetAttribute(attn_decode_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(decode_smem_bytes<64>()));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(attn_decode_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(decode_smem_bytes<128>()));
}

// segments a (sequence, KV head) pair can have: what part_o / part_ml must hold per query head
int attn_decode_max_segments(int max_pages_per_seq) { return max_pages_per_seq / kDcMinTiles + 2; }

template <int DH>
static void launch_decode_t(const CUtensorMap& tmK, const CUtensorMap& tmV, const AttnArgs& a, int n_sms, cudaStream_t st) {
  constexpr size_t smem = decode_smem_bytes<DH>();
  static_assert(2 * (smem + 1024) <= 228 * 1024, "two CTAs per SM");
  // no more CTAs than the longest possible list of pages can occupy
  const long long most = ((long long)a.n_seqs * a.n_kv * a.max_kv_pages + kDcMinTiles - 1) / kDcMinTiles;
  const int grid = int(most < 2LL * n_sms ? (most < 1 ? 1 : most) : 2LL * n_sms);
  launch_pdl(attn_decode_kernel<DH>, dim3(grid), dim3(kDcThreads), smem, st, tmK, tmV, a);
}

void launch_attn_decode(const CUtensorMap& tmK, const CUtensorMap& tmV, const AttnArgs& a, int n_sms, cudaStream_t st) {
  if (a.n_seqs <= 0) return;
  if (a.dh > 64) launch_decode_t<128>(tmK, tmV, a, n_sms, st);
  else launch_decode_t<64>(tmK, tmV, a, n_sms, st);
}

}  // namespace foe
