// Dispatch maps of the FoE block: the local form of the token -> expert all-to-all.  Integer work:
// per-expert counts, an exclusive scan, and a stable scatter (inside an expert, tokens ascend), so
// the maps are a pure function of the routing decision -- no atomics decide an order.
//
//   counts[e]  = number of (token, cluster, j) selections of expert e
//   offsets    = exclusive scan of counts over the global expert id
//   perm[slot] = token of the slot,  inv[token, cluster, j] = slot
//
// The activation rows themselves are not moved here: expert GEMM 1 gathers them through perm while it stages
// its A operand.  Three launches: (1) every block of 256 tokens builds a token-bitmap per expert in shared memory,
// from which each selection reads its rank inside the block; (2) one block scans block counts and
// expert totals and writes the m-tile table the grouped GEMMs walk; (3) every selection computes its
// slot.
#include <climits>
#include "common.cuh"
#include "kernels.h"

namespace foe {

constexpr int kPB = kPermuteBlockTokens;      // 256 tokens per block = 8 bitmap words per expert

__global__ void __launch_bounds__(kPB)
permute_count_kernel(const int* __restrict__ idx, int* __restrict__ rank, int* __restrict__ blk_counts, int n_tokens,
                     int sel, int E, int* __restrict__ status) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ uint32_t bm[];            // [E][8]
  for (int q = threadIdx.x; q < E * 8; q += kPB) bm[q] = 0u;
  __syncthreads();
  const int t = threadIdx.x;
  const int i = blockIdx.x * kPB + t;
  if (i < n_tokens) {
    for (int s = 0; s < sel; ++s) {
      const int e = idx[size_t(i) * sel + s];
      if (e < 0 || e >= E) { atomicExch(status, kStatusBounds); continue; }
      atomicOr(&bm[e * 8 + (t >> 5)], 1u << (t & 31));
    }
  }
  __syncthreads();
  if (i < n_tokens) {
    for (int s = 0; s < sel; ++s) {
      const int e = idx[size_t(i) * sel + s];
      int r = 0;
      if (e >= 0 && e < E) {
        const uint32_t* w = bm + e * 8;
        for (int k = 0; k < (t >> 5); ++k) r += __popc(w[k]);
        r += __popc(w[t >> 5] & ((1u << (t & 31)) - 1u));
      }
      rank[size_t(i) * sel + s] = r;
    }
  }
  for (int e = threadIdx.x; e < E; e += kPB) {
    int c = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) c += __popc(bm[e * 8 + k]);
    blk_counts[size_t(blockIdx.x) * E + e] = c;
  }
}

// Tile table the grouped GEMMs walk: expert and first row of every 256-row tile of every non-empty expert.  Expert e
// owns `tiles` entries from tile0 on; the last expert also writes the table length.
constexpr int kTileRows = 256;
__device__ __forceinline__ void write_tile_table(const PermuteBuffers& pb, int e, int E, int row0, int tiles, int tile0,
                                                 int n_tiles_all) {
  if (e == E - 1) *pb.n_mtiles = n_tiles_all;
  for (int j = 0; j < tiles; ++j) { pb.mt_group[tile0 + j] = e; pb.mt_row0[tile0 + j] = row0 + j * kTileRows; }
}

// Single block.  blk_counts[b][e] becomes the exclusive prefix over b; counts/offsets and the tile table are written.
__global__ void __launch_bounds__(1024)
permute_scan_kernel(int* __restrict__ blk_counts, int n_blocks, int E, const PermuteBuffers pb) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ int s_a[1024], s_b[1024];
  int* counts = pb.counts;
  int* offsets = pb.offsets;
  const int e = threadIdx.x;
  int total = 0;
  if (e < E) {
    for (int b0 = 0; b0 < n_blocks; b0 += 16) {          // 16 independent loads in flight, then their prefix
      int c[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) c[j] = b0 + j < n_blocks ? blk_counts[size_t(b0 + j) * E + e] : 0;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        if (b0 + j < n_blocks) blk_counts[size_t(b0 + j) * E + e] = total;
        total += c[j];
      }
    }
    counts[e] = total;
  }
  const int tiles = (total + kTileRows - 1) / kTileRows;
  // two inclusive Hillis-Steele scans over the expert id (rows and tiles)
  s_a[e] = total;
  s_b[e] = tiles;
  __syncthreads();
  for (int o = 1; o < E; o <<= 1) {                 // (entries from E on are zero)
    const int va = e >= o ? s_a[e - o] : 0;
    const int vb = e >= o ? s_b[e - o] : 0;
    __syncthreads();
    s_a[e] += va;
    s_b[e] += vb;
    __syncthreads();
  }
  if (e < E) {
    const int row0 = s_a[e] - total;
    offsets[e] = row0;
    if (e == E - 1) offsets[E] = s_a[e];
    write_tile_table(pb, e, E, row0, tiles, s_b[e] - tiles, s_b[e]);
  }
}

__global__ void permute_scatter_kernel(const int* __restrict__ idx, const int* __restrict__ rank,
                                       const int* __restrict__ blk_prefix, const int* __restrict__ offsets,
                                       int* __restrict__ perm, int* __restrict__ inv, int n_tokens, int sel, int E) {
  pdl_wait();
  pdl_launch_dependents();
  const int q = blockIdx.x * blockDim.x + threadIdx.x;
  if (q >= n_tokens * sel) return;
  const int i = q / sel;
  const int e = idx[q];
  if (e < 0 || e >= E) { inv[q] = 0; return; }
  const int slot = offsets[e] + blk_prefix[size_t(i / kPB) * E + e] + rank[q];
  inv[q] = slot;
  perm[slot] = i;
}

// All three steps in one block, for calls of at most 256 tokens (a decode step): bitmap, scan over the
// experts, slots.  Same results as the three-kernel path, two launches fewer.
// With `scores` given, the block first takes the routing decision itself (so that a decode step needs one launch for
// top-k, gates and maps): one thread per (token, cluster) adds the bias, writes the scores, selects the k_c largest of
// the cluster's E_c (larger score first, equal scores: lower expert id first) and their softmax gates.
struct TopkSmall {
  const float* scores;    // [k_splits][n_tokens][E] partial router scores, or nullptr: idx is an input
  int k_splits;
  const float* bias;      // [E] or nullptr
  float* logits_out;      // [n_tokens][E]
  int* idx_out;           // [n_tokens][H][kc]
  float* w_out;
  int H, Ec, kc;
};

// Top-k and gates of one (token, cluster) with the cluster's E_c scores in registers (E_c a power of two up to 32):
// all loads at once, then k_c selection passes without touching memory.  Order and ties as in the generic loop of
// the kernel below: score descending, expert id ascending.
template <int EC>
__device__ __forceinline__ void topk_small_regs(const TopkSmall& tk, int task) {
  const int H = tk.H, kc = tk.kc;
  const int i = task / H, h = task - i * H;
  const float* src = tk.logits_out + (size_t(i) * H + h) * EC;
  float v[EC];
#pragma unroll
  for (int e = 0; e < EC; e += 4) {
    const float4 a = *reinterpret_cast<const float4*>(src + e);
    v[e] = a.x; v[e + 1] = a.y; v[e + 2] = a.z; v[e + 3] = a.w;
  }
  uint32_t taken = 0u;
  float m = 0.f, sum = 0.f;
  const size_t oo = size_t(task) * kc;
  for (int j = 0; j < kc; ++j) {
    float bv = 0.f;
    int bi = -1;
#pragma unroll
    for (int e = 0; e < EC; ++e)
      if (!((taken >> e) & 1u) && (bi < 0 || v[e] > bv)) { bv = v[e]; bi = e; }
    taken |= 1u << bi;
    if (j == 0) m = bv;
    const float x = expf(bv - m);
    sum += x;
    tk.idx_out[oo + j] = h * EC + bi;
    tk.w_out[oo + j] = x;
  }
  for (int j = 0; j < kc; ++j) tk.w_out[oo + j] = tk.w_out[oo + j] / sum;
}

__global__ void __launch_bounds__(1024)
permute_small_kernel(const int* idx, int n_tokens, int sel, int E, const PermuteBuffers pb,
                     int* __restrict__ status, const TopkSmall tk, int idx_in_smem) {
  pdl_wait();
  pdl_launch_dependents();
  extern __shared__ uint32_t bm[];            // [E][8], then (idx_in_smem) a copy of idx: [n_tokens][sel]
  int* s_idx = reinterpret_cast<int*>(bm + E * 8);
  __shared__ int s_a[1024], s_b[1024], s_off[1024];
  int* counts = pb.counts;
  int* offsets = pb.offsets;
  int* perm = pb.perm;
  int* inv = pb.inv;
  const int t = threadIdx.x;
  if (tk.scores) {
    const int H = tk.H, Ec = tk.Ec, kc = tk.kc;
    // scores = partial sums in fixed order + bias, all threads; then one thread per (token, cluster)
    // (sixteen loads in flight per element: the partials sit in L2, and one round trip per split would cost more
    // than everything else in this kernel)
    for (int q = t; q < n_tokens * E; q += 1024) {
      float v = 0.f;
      for (int z0 = 0; z0 < tk.k_splits; z0 += 16) {
        float p[16];
#pragma unroll
        for (int u = 0; u < 16; ++u)
          p[u] = (z0 + u < tk.k_splits) ? __ldcg(tk.scores + size_t(z0 + u) * n_tokens * E + q) : 0.f;
#pragma unroll
        for (int u = 0; u < 16; ++u) v += p[u];             // split order; the zeros of absent splits change nothing
      }
      tk.logits_out[q] = v + (tk.bias ? tk.bias[q % E] : 0.f);
    }
    __threadfence_block();
    __syncthreads();
    const bool in_regs = Ec == 4 || Ec == 8 || Ec == 16 || Ec == 32;
    if (in_regs) {
      for (int task = t; task < n_tokens * H; task += 1024) {
        switch (Ec) {
          case 4: topk_small_regs<4>(tk, task); break;
          case 8: topk_small_regs<8>(tk, task); break;
          case 16: topk_small_regs<16>(tk, task); break;
          default: topk_small_regs<32>(tk, task); break;
        }
      }
    }
    // any other E_c (up to 128): one warp per (token, cluster), the scores in registers (lane l holds experts l, l + 32,
    // ...), one shuffle arg-max per selection; selection j is kept by lane j % 32 and written once
    for (int task = in_regs ? n_tokens * H : (t >> 5); task < n_tokens * H; task += 32) {
      const int lane = t & 31;
      const int i = task / H, h = task - i * H;
      const size_t o = size_t(i) * E + size_t(h) * Ec;
      float cand[4];
      bool taken[4];
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        const int e = lane + 32 * s;
        taken[s] = e >= Ec;
        cand[s] = taken[s] ? 0.f : tk.logits_out[o + e];
      }
      float m = 0.f, sum = 0.f;
      const size_t oo = size_t(task) * kc;
      for (int j = 0; j < kc; ++j) {
        float bv = 0.f;
        int bi = INT_MAX;                                   // INT_MAX: nothing left in this lane
#pragma unroll
        for (int s = 0; s < 4; ++s)
          if (!taken[s] && (bi == INT_MAX || cand[s] > bv)) { bv = cand[s]; bi = lane + 32 * s; }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) {
          const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
          const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
          if (oi != INT_MAX && (bi == INT_MAX || ov > bv || (ov == bv && oi < bi))) { bv = ov; bi = oi; }
        }
        if ((bi & 31) == lane) {
#pragma unroll
          for (int s = 0; s < 4; ++s) taken[s] = taken[s] || (bi >> 5) == s;
        }
        if (j == 0) m = bv;
        const float ex = expf(bv - m);                      // the same value in every lane
        sum += ex;
        if ((j & 31) == lane) {
          tk.idx_out[oo + j] = h * Ec + bi;
          tk.w_out[oo + j] = ex;
        }
      }
      for (int j = lane; j < kc; j += 32) tk.w_out[oo + j] = tk.w_out[oo + j] / sum;   // lane j % 32 wrote entry j
    }
    __threadfence_block();
    __syncthreads();                            // idx (== tk.idx_out) is read below by other threads of this block
  }
  for (int q = t; q < E * 8; q += 1024) bm[q] = 0u;
  // the selections are read twice below, token by token; one coalesced pass brings them next to the bitmap when they fit
  // (a thread walking its token's list in global memory pays one round trip to L2 per selection)
  if (idx_in_smem) {
    for (int q = t; q < n_tokens * sel; q += 1024) s_idx[q] = idx[q];
    idx = s_idx;
  }
  __syncthreads();
  if (t < n_tokens) {
    for (int s = 0; s < sel; ++s) {
      const int e = idx[size_t(t) * sel + s];
      if (e < 0 || e >= E) { atomicExch(status, kStatusBounds); continue; }
      atomicOr(&bm[e * 8 + (t >> 5)], 1u << (t & 31));
    }
  }
  __syncthreads();
  int total = 0;
  if (t < E) {
#pragma unroll
    for (int k = 0; k < 8; ++k) total += __popc(bm[t * 8 + k]);
    counts[t] = total;
  }
  const int tiles = (total + kTileRows - 1) / kTileRows;
  s_a[t] = total;
  s_b[t] = tiles;
  __syncthreads();
  for (int o = 1; o < E; o <<= 1) {                 // (entries from E on are zero)
    const int va = t >= o ? s_a[t - o] : 0;
    const int vb = t >= o ? s_b[t - o] : 0;
    __syncthreads();
    s_a[t] += va;
    s_b[t] += vb;
    __syncthreads();
  }
  if (t < E) {
    const int row0 = s_a[t] - total;
    offsets[t] = row0;
    s_off[t] = row0;
    if (t == E - 1) offsets[E] = s_a[t];
    write_tile_table(pb, t, E, row0, tiles, s_b[t] - tiles, s_b[t]);
  }
  __syncthreads();
  for (int q = t; q < n_tokens * sel; q += 1024) {
    const int i = q / sel;
    const int e = idx[q];
    if (e < 0 || e >= E) { inv[q] = 0; continue; }
    const uint32_t* w = bm + e * 8;
    int r = 0;
    for (int k = 0; k < (i >> 5); ++k) r += __popc(w[k]);
    r += __popc(w[i >> 5] & ((1u << (i & 31)) - 1u));
    const int slot = s_off[e] + r;
    inv[q] = slot;
    perm[slot] = i;
  }
}

// Bytes of the selections' copy in shared memory, or 0 when it does not fit beside the bitmap and the 12 KB of static
// arrays within the 48 KB a kernel gets without opting in.
static size_t small_idx_bytes(int n_tokens, int sel, int E) {
  const size_t want = size_t(n_tokens) * sel * sizeof(int);
  return size_t(E) * 32 + want <= 34 * 1024 ? want : 0;
}

int launch_permute(const int* idx, const PermuteBuffers& pb, int n_tokens, int sel, int E, int* status,
                   cudaStream_t st) {
  if (n_tokens <= 0) return 0;
  if (n_tokens <= kPB) {
    TopkSmall none;
    none.scores = nullptr;
    const size_t copy = small_idx_bytes(n_tokens, sel, E);
    launch_pdl(permute_small_kernel, dim3(1), dim3(1024), size_t(E) * 32 + copy, st, idx, n_tokens, sel, E, pb, status, none,
               copy ? 1 : 0);
    return 1;
  }
  const int n_blocks = (n_tokens + kPB - 1) / kPB;
  launch_pdl(permute_count_kernel, dim3(n_blocks), dim3(kPB), size_t(E) * 32, st, idx, pb.rank, pb.blk_counts, n_tokens, sel, E, status);
  launch_pdl(permute_scan_kernel, dim3(1), dim3(1024), 0, st, pb.blk_counts, n_blocks, E, pb);
  const int total = n_tokens * sel;
  launch_pdl(permute_scatter_kernel, dim3((total + 255) / 256), dim3(256), 0, st, idx, pb.rank, pb.blk_counts, pb.offsets, pb.perm, pb.inv,
                                                            n_tokens, sel, E);
  return 3;
}

// top-k + gates + dispatch maps of a call of at most 256 tokens in one launch (scores: [k_splits][n_tokens][E])
int launch_topk_permute_small(const float* scores, int k_splits, const float* bias, float* logits, int* idx, float* w,
                              const PermuteBuffers& pb, int n_tokens, int H, int Ec, int kc, int* status, cudaStream_t st) {
  if (n_tokens <= 0) return 0;
  TopkSmall tk;
  tk.scores = scores; tk.k_splits = k_splits; tk.bias = bias; tk.logits_out = logits; tk.idx_out = idx; tk.w_out = w; tk.H = H; tk.Ec = Ec; tk.kc = kc;
  const int E = H * Ec;
  const size_t copy = small_idx_bytes(n_tokens, H * kc, E);
  launch_pdl(permute_small_kernel, dim3(1), dim3(1024), size_t(E) * 32 + copy, st, idx, n_tokens, H * kc, E, pb, status, tk,
             copy ? 1 : 0);
  return 1;
}

}  // namespace foe
