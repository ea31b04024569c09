// Dense projections of a decode step (QKV and output projection; Table 2, row "attention") on tcgen05 with the
// operands swapped: a CTA multiplies a slab of 128 WEIGHT rows (the MMA's M) by up to 64 TOKEN rows (its N), so that
// a handful of tokens still fills the tensor core's 128 accumulator lanes.  With 16 to 256 tokens per step these two
// GEMMs are far too small to be bound by HBM and far too narrow for the 256-row tiles of the prefill GEMM; on the
// legacy warp-level MMA path they were bound by its issue rate.
//
//   warp 0        TMA: per 64-wide k-block one 128 x 64 box of W and one 64 x 64 box of the activations (both K-major,
//                 128-byte swizzle), 8 stages -- a CTA's whole k-range is usually in flight at once
//   warp 1        one thread issues tcgen05.mma (M 128, N 64, K 16) into a 64-column TMEM accumulator
//   warps 2..17   QKV: sum of squares of the staged activation rows during the main loop (the RMSNorm statistics);
//                 then the epilogue: thread = accumulator lane = one output column, 16 of the 64 token values each
//
// The K dimension is split over the CTAs of a thread-block cluster (1, 2, 4 or 8; a 2048 x 2048 projection has only
// 16 slabs, and ~one CTA per SM should stream weights).  Every split leaves its fp32 partial tile in its own shared
// memory; after a cluster barrier CTA r adds up -- in rank order, so the sum does not depend on timing -- the tokens
// [r * 64/ks, (r+1) * 64/ks) of all partials straight out of the peers' shared memory and finishes them:
//   QKV    1/rms of the token, RoPE on q and k (a rotation pair is two adjacent packed columns: heads are stored with
//          their halves interleaved), q -> out[token][head][.], k / v -> their cache pages
//   OProj  r_full = scale * (C + sum_h x[h])  as fp32
// No scratch in global memory, no tickets, and the epilogue work is spread over all CTAs.
// All waits are bounded; a wait that runs out records kStatusTimeout and the CTA still reaches its teardown.
#include <string.h>

#include "common.cuh"
#include "kernels.h"

namespace foe {

namespace {

constexpr int kDpSlab = 128;                    // weight rows per CTA (UMMA M)
constexpr int kDpTok = 64;                      // token rows per CTA (UMMA N)
constexpr int kDpBK = 64;                       // k per stage (one 128-byte swizzle row)
constexpr int kDpStages = 8;
constexpr int kDpWBytes = kDpSlab * kDpBK * 2;  // 16 KB
constexpr int kDpXBytes = kDpTok * kDpBK * 2;   // 8 KB
constexpr int kDpStageBytes = kDpWBytes + kDpXBytes;
constexpr int kDpEpiWarps = 16;                 // four per TMEM lane quarter, 16 tokens each
constexpr int kDpEpiThreads = kDpEpiWarps * 32;
constexpr int kDpTokPerWarp = kDpTok / (kDpEpiWarps / 4);
constexpr int kDpThreads = 64 + kDpEpiThreads;
constexpr size_t kDpSmemBytes = size_t(kDpStages) * kDpStageBytes + 1024 + 1024;

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kDpEpiThreads) : "memory"); }

__device__ __forceinline__ float ld_cluster_f1(uint32_t addr) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ float2 ld_cluster_f2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}


}  // namespace

template <int EPI>
__global__ void __launch_bounds__(kDpThreads, 1)
decode_proj_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                   const DecodeProjArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + kDpStages * kDpStageBytes);
  uint64_t* empty_bar = full_bar + kDpStages;
  uint64_t* acc_full = empty_bar + kDpStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 1);
  float* s_ssq = reinterpret_cast<float*>(tmem_slot + 2);        // [64] sum of squares, then 1/rms, per token
  constexpr bool kStats = (EPI == kEpiQKV);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int slabs = a.N / kDpSlab;
  const int chunks = (a.rows_per_group + kDpTok - 1) / kDpTok;
  const int ks = a.k_splits;
  const int task = blockIdx.x;
  const int z = task % ks, tnz = task / ks;                       // split, tile
  const int chunk = tnz % chunks, t2 = tnz / chunks;
  const int slab = t2 % slabs, group = t2 / slabs;
  const int kblocks = a.K / kDpBK;
  const int kb0 = int((long long)z * kblocks / ks), kb1 = int((long long)(z + 1) * kblocks / ks);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kDpStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], kStats ? 1 + kDpEpiWarps : 1); }
    mbar_init(acc_full, 1);
    mbar_fence_init();
    tma_prefetch_desc(&tmW);
    tma_prefetch_desc(&tmX);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 64); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (elect_one()) {
      bool ok = true;
      const int w_row = group * a.N + slab * kDpSlab;
      const int x_row = group * a.x_group_stride + chunk * kDpTok;
      // The weights do not depend on anything an earlier kernel wrote: the first ring of weight tiles is requested
      // before this grid waits for its predecessor (whose tail it overlaps); the activations follow after the wait.
      const int n_first = min(kb1 - kb0, kDpStages);
      for (int i = 0; i < n_first; ++i) {
        mbar_expect_tx(&full_bar[i], kDpStageBytes);
        tma_load_2d(smem + i * kDpStageBytes, &tmW, &full_bar[i], (kb0 + i) * kDpBK, w_row);
      }
      pdl_wait();
      pdl_launch_dependents();
      for (int i = 0; i < n_first; ++i)
        tma_load_2d(smem + i * kDpStageBytes + kDpWBytes, &tmX, &full_bar[i], (kb0 + i) * kDpBK, x_row);
      for (int kb = kb0 + n_first; kb < kb1; ++kb) {
        const int i = kb - kb0, s = i % kDpStages;
        if (!mbar_wait(&empty_bar[s], ((i / kDpStages) & 1) ^ 1)) { ok = false; break; }
        uint8_t* dst = smem + s * kDpStageBytes;
        mbar_expect_tx(&full_bar[s], kDpStageBytes);
        tma_load_2d(dst, &tmW, &full_bar[s], kb * kDpBK, w_row);
        tma_load_2d(dst + kDpWBytes, &tmX, &full_bar[s], kb * kDpBK, x_row);
      }
      if (!ok) atomicExch(a.status, kStatusTimeout);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (elect_one()) {
      constexpr uint32_t idesc = umma_idesc_bf16(kDpSlab, kDpTok);
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb) {
        const int i = kb - kb0, s = i % kDpStages;
        if (!mbar_wait(&full_bar[s], (i / kDpStages) & 1)) { ok = false; break; }
        tc_fence_after();
        const uint32_t w0 = smem_u32(smem + s * kDpStageBytes), x0 = w0 + kDpWBytes;
#pragma unroll
        for (int k = 0; k < kDpBK / 16; ++k)
          umma_bf16(tmem_base, umma_desc_sw128(w0 + k * 32), umma_desc_sw128(x0 + k * 32), idesc, (i > 0 || k > 0) ? 1u : 0u);
        umma_commit(&empty_bar[s]);
      }
      if (ok) umma_commit(acc_full);
      else atomicExch(a.status, kStatusTimeout);
    }
  } else {
    // ------------------------------------------------------------ statistics (QKV) and epilogue
    // 16 warps: warp (quarter, tg) reads TMEM lanes 32*quarter.. (the hardware ties a warp to the lane quarter
    // warp % 4) and the 16 accumulator columns (tokens) 16*tg..; four warps per scheduler hide each other's latency.
    pdl_wait();                                           // everything these warps read or write depends on earlier kernels
    const int quarter = warp & 3, tg = (warp - 2) >> 2;
    const int col = quarter * 32 + lane;                  // 0..127 = accumulator lane = weight row of the slab
    const int etid = tg * 128 + col;                      // 0..511
    bool ok = true;
    if constexpr (kStats) {
      // thread = (token, 16-byte piece of the 64-wide k-block)
      const int tok = etid >> 3, c = etid & 7;
      float ssq = 0.f;
      for (int kb = kb0; kb < kb1 && ok; ++kb) {
        const int i = kb - kb0, s = i % kDpStages;
        if (!mbar_wait(&full_bar[s], (i / kDpStages) & 1)) { ok = false; break; }
        const uint4 q = *reinterpret_cast<const uint4*>(smem + s * kDpStageBytes + kDpWBytes + tok * 128 + ((c ^ (tok & 7)) << 4));
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float lo = bf16_lo(w[e]), hi = bf16_hi(w[e]);
          ssq = fmaf(lo, lo, fmaf(hi, hi, ssq));
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[s]);
      }
      ssq += __shfl_xor_sync(0xffffffffu, ssq, 1);
      ssq += __shfl_xor_sync(0xffffffffu, ssq, 2);
      ssq += __shfl_xor_sync(0xffffffffu, ssq, 4);
      if (c == 0) s_ssq[tok] = ssq;
    }
    ok = ok && mbar_wait(acc_full, 0);
    if (!ok && lane == 0) atomicExch(a.status, kStatusTimeout);
    // (after a timed-out wait the values below are meaningless, but every thread still walks the same barriers)
    tc_fence_after();
    float v[kDpTokPerWarp];
    {
      uint32_t r[kDpTokPerWarp];
      tmem_ld16(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + tg * kDpTokPerWarp, r);
      tmem_ld_wait();
#pragma unroll
      for (int t = 0; t < kDpTokPerWarp; ++t) v[t] = __uint_as_float(r[t]);
    }
    epi_bar();                                            // every statistics warp is done with the staged rows
    // this split's partial tile: [token][column] fp32 over the (by now idle) pipeline stages; s_ssq holds its
    // partial sums of squares
    float* s_part = reinterpret_cast<float*>(smem);
#pragma unroll
    for (int t = 0; t < kDpTokPerWarp; ++t) s_part[(tg * kDpTokPerWarp + t) * kDpSlab + col] = v[t];
  }

  // ---- the CTAs of a cluster hold the k-splits of one tile: after the cluster barrier CTA r adds up, in rank order
  //      and straight out of the peers' shared memory, the tokens [r * 64/ks, (r+1) * 64/ks) and finishes them
  tc_fence_before();
  cluster_sync_all();
  if (warp >= 2) {
    const int etid = threadIdx.x - 64;
    const int share = kDpTok / ks;                          // ks is 1, 2, 4 or 8
    const int t_lo = z * share;
    const int tok0 = chunk * kDpTok;
    const int n_tok = min(kDpTok, a.rows_per_group - tok0);
    uint32_t part_addr[8], ssq_addr[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      part_addr[r] = mapa_u32(smem_u32(smem), r < ks ? r : 0);
      ssq_addr[r] = mapa_u32(smem_u32(s_ssq), r < ks ? r : 0);
    }
    if constexpr (EPI == kEpiQKV) {
      // item = (token, rotation pair): packed columns 2p and 2p+1 of a head are its natural columns i and i + dh/2
      const int half = a.dh >> 1;
      for (int q = etid; q < share * (kDpSlab / 2); q += kDpEpiThreads) {
        const int t = t_lo + (q >> 6), p = q & 63;
        if (t >= n_tok) continue;
        const int tok = tok0 + t;
        int pos, slot;
        if (a.tok_pos) {
          pos = a.tok_pos[tok];
          slot = a.tok_slot[tok];
        } else {                                          // decode step: position and cache slot of sequence `tok`
          pos = a.context_lens[tok];
          const int lp = pos >> 6;
          slot = -1;
          if (pos >= 0 && lp < a.max_pages_per_seq && pos < a.max_context) {
            const int page = a.block_table[size_t(tok) * a.max_pages_per_seq + lp];
            if (page >= 0 && page < a.num_pages) slot = page * 64 + (pos & 63);
          }
          if (slot < 0) { atomicExch(a.status, kStatusBounds); pos = min(max(pos, 0), a.max_context - 1); }
        }
        float2 pv[8];
        float sq[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) {
          pv[r] = make_float2(0.f, 0.f);
          sq[r] = 0.f;
          if (r < ks) {
            pv[r] = ld_cluster_f2(part_addr[r] + (t * kDpSlab + 2 * p) * 4);
            sq[r] = ld_cluster_f1(ssq_addr[r] + t * 4);
          }
        }
        float x = 0.f, y = 0.f, ssq = 0.f;
#pragma unroll
        for (int r = 0; r < 8; ++r) { x += pv[r].x; y += pv[r].y; ssq += sq[r]; }        // rank order
        const float scale = rsqrtf(ssq / float(a.K) + a.rms_eps);
        const int n = slab * kDpSlab + 2 * p;             // packed column inside the group
        const int i = (n % a.dh) >> 1;
        float lo = x * scale, hi = y * scale;
        const bool is_q = n < a.q_cols, is_k = !is_q && n < a.q_cols + a.kv_cols;
        if (is_q || is_k) {
          const float2 cs = __ldg(a.rope_tab + size_t(pos) * half + i);
          const float x0 = lo, x1 = hi;
          lo = x0 * cs.x - x1 * cs.y;
          hi = x1 * cs.x + x0 * cs.y;
        }
        if (is_q) {
          const int head = group * (a.q_cols / a.dh) + n / a.dh;
          bf16* o = static_cast<bf16*>(a.out) + size_t(tok) * a.ldo + head * a.q_head_stride;
          o[i] = __float2bfloat16_rn(lo);
          o[i + half] = __float2bfloat16_rn(hi);
        } else {
          const int nn = n - a.q_cols - (is_k ? 0 : a.kv_cols);
          const int kvh = group * (a.kv_cols / a.dh) + nn / a.dh;
          if (slot >= 0) {
            bf16* o = (is_k ? a.k_pages : a.v_pages) + ((size_t(slot >> 6) * a.n_kv + kvh) * 64 + (slot & 63)) * a.dh;
            o[i] = __float2bfloat16_rn(lo);
            o[i + half] = __float2bfloat16_rn(hi);
          }
        }
      }
    } else {
      // r_full = scale * (C + sum_h x[h]); item = (token, four columns)
      const int n0 = slab * kDpSlab;
      for (int q = etid; q < share * (kDpSlab / 4); q += kDpEpiThreads) {
        const int t = t_lo + (q >> 5), c4 = q & 31;
        if (t >= n_tok) continue;
        const size_t off = size_t(tok0 + t) * a.ldo + n0 + c4 * 4;
        uint2 xr[8];
        float4 pv[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) {
          xr[r] = make_uint2(0u, 0u);
          pv[r] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (r < a.x_count) xr[r] = __ldg(reinterpret_cast<const uint2*>(a.xsum + r * a.x_stride + off));
          if (r < ks) pv[r] = ld_cluster_f4(part_addr[r] + (t * kDpSlab + c4 * 4) * 4);
        }
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int r = 0; r < 8; ++r) { sum.x += pv[r].x; sum.y += pv[r].y; sum.z += pv[r].z; sum.w += pv[r].w; }   // rank order
#pragma unroll
        for (int r = 0; r < 8; ++r) {
          sum.x += bf16_lo(xr[r].x); sum.y += bf16_hi(xr[r].x); sum.z += bf16_lo(xr[r].y); sum.w += bf16_hi(xr[r].y);
        }
        const float sc = a.out_scale;
        if (a.push_span) {
          // one rank of a cluster-per-GPU group: the slab's 128 columns lie inside one owner's span; bf16 to its slot
          const int col = n0 + c4 * 4, owner = col / a.push_span;
          bf16* dst = a.push_base[owner] + a.push_slot_off + size_t(tok0 + t) * a.push_span + (col - owner * a.push_span);
          *reinterpret_cast<uint2*>(dst) = make_uint2(pack_bf16(sum.x * sc, sum.y * sc), pack_bf16(sum.z * sc, sum.w * sc));
        } else {
          *reinterpret_cast<float4*>(static_cast<float*>(a.out) + off) = make_float4(sum.x * sc, sum.y * sc, sum.z * sc, sum.w * sc);
        }
      }
      if (a.push_span) __threadfence_system();               // every storing thread: its stores before the count below
    }
  }
  cluster_sync_all();                                       // nobody leaves while a peer may still read its tile
  if constexpr (EPI == kEpiOProj) {
    if (a.push_span && threadIdx.x == 64) {
      // this CTA finished the tokens [t_lo, t_lo + share) of the tile: their element count goes to the owner's counter
      // of the tile's row block (a tile's 64 tokens lie inside one block of 256)
      const int share = kDpTok / ks, tok0 = chunk * kDpTok;
      const int n_tok = min(kDpTok, a.rows_per_group - tok0);
      const int mine = max(0, min(share, n_tok - z * share));
      if (mine > 0) {
        const int owner = slab * kDpSlab / a.push_span;
        atomicAdd_system(a.push_cnt[owner] + tok0 / kShardBlockRows, unsigned(mine) * unsigned(kDpSlab));
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 64);
  }
}

namespace {

// clusters of 1, 2, 4, 8 CTAs of each kernel the device holds at once (a property of the GPU model, refreshed by
// every decode_proj_configure)
template <int EPI>
struct DpOccupancy { static int max_active[4]; };
template <int EPI>
int DpOccupancy<EPI>::max_active[4] = {0, 0, 0, 0};

template <int EPI>
cudaError_t configure_one() {
  const cudaError_t e = cudaFuncSetAttribute(decode_proj_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kDpSmemBytes));
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.blockDim = dim3(kDpThreads, 1, 1);
  cfg.dynamicSmemBytes = kDpSmemBytes;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  for (int i = 0; i < 4; ++i) {
    int n = 0;
    attr.val.clusterDim.x = 1 << i;
    cfg.gridDim = dim3(1 << i, 1, 1);
    if (cudaOccupancyMaxActiveClusters(&n, decode_proj_kernel<EPI>, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
    DpOccupancy<EPI>::max_active[i] = n;
  }
  return cudaSuccess;
}

template <int EPI>
void launch_one(const CUtensorMap& tmW, const CUtensorMap& tmX, DecodeProjArgs a, int tiles, cudaStream_t st) {
  const int* max_active = DpOccupancy<EPI>::max_active;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.blockDim = dim3(kDpThreads, 1, 1);
  cfg.dynamicSmemBytes = kDpSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attrs[2];
  cudaLaunchAttribute& attr = attrs[0];
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  attrs[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attrs[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attrs;
  cfg.numAttrs = g_overlap_launches ? 2 : 1;
  // all clusters of a launch should be resident together: a cluster that has to wait for a free group of SMs
  // doubles the kernel's time
  while (a.k_splits > 1) {
    int i = 0;
    while ((1 << i) < a.k_splits) ++i;
    if (tiles <= max_active[i]) break;
    a.k_splits >>= 1;
  }
  attr.val.clusterDim.x = a.k_splits;
  cfg.gridDim = dim3(tiles * a.k_splits, 1, 1);
  cudaLaunchKernelEx(&cfg, decode_proj_kernel<EPI>, tmW, tmX, a);
}

}  // namespace

cudaError_t decode_proj_configure() {
  const cudaError_t e = configure_one<kEpiQKV>();
  return e != cudaSuccess ? e : configure_one<kEpiOProj>();
}

bool decode_proj_supported(int epi, int N, int K, int dh) {
  if (N <= 0 || N % kDpSlab || K <= 0 || K % kDpBK) return false;
  if (epi == kEpiQKV) return dh == 64 || dh == 128;       // a slab must hold whole heads
  return epi == kEpiOProj;
}

// K is split (by 1, 2, 4 or 8 = the cluster size) so that about one CTA per SM streams weights, every split keeping
// at least two k-blocks
int decode_proj_splits(int tiles, int K, int n_sms) {
  const int kblocks = K / kDpBK;
  int ks = 1;
  while (ks < 8 && tiles * ks * 2 <= n_sms && ks * 2 * 2 <= kblocks) ks *= 2;
  return ks;
}

void launch_decode_proj(const CUtensorMap& tmW, const CUtensorMap& tmX, DecodeProjArgs a, int n_sms, cudaStream_t st) {
  const int tiles = a.n_groups * (a.N / kDpSlab) * ((a.rows_per_group + kDpTok - 1) / kDpTok);
  if (tiles <= 0) return;
  a.k_splits = decode_proj_splits(tiles, a.K, n_sms);
  if (a.epi == kEpiQKV) launch_one<kEpiQKV>(tmW, tmX, a, tiles, st);
  else launch_one<kEpiOProj>(tmW, tmX, a, tiles, st);
}

}  // namespace foe
