// Cross-cluster sync of a cluster-per-GPU group (Section 3.2: one all-reduce of the attention residual per layer is
// the only traffic between clusters; Table 2, row "sync").
//
// Each rank h holds one cluster.  r_full = sum_h partial[h] is formed as a two-step exchange over peer memory,
// with the columns of the [S][d] tensor split evenly between the ranks (rank o owns columns [o*span, (o+1)*span)):
//   push    every rank writes its partial of owner o's columns into slot h of o's receive buffer (the O-projections
//           do this from their epilogues, tile by tile; shard_push_kernel does it for a tensor that already sits in
//           memory), then adds the element count to o's arrival counter for (source h, block of 256 rows);
//   reduce  owner o: every block of 16 rows waits until the H counters of ITS 256-row block hold the block's element
//           count -- so the reduction of the first rows runs while later tiles are still being pushed --, adds the H
//           slots in rank order in fp32, rounds to bf16 and writes the result into the gather buffer of every rank,
//           then adds to their counters for owner o;
//   gather  every rank waits for the H owners' counters and reads its own gather buffer; it also zeroes its own slot
//           counters of this exchange (its reduction is over, and a peer's next push with the same parity comes two
//           exchanges later, after that peer has gathered the exchange in between, which this rank's reduction of
//           that exchange -- queued behind this kernel -- feeds).
// The gather counters only ever grow (the expected totals are kept by the host), buffers and slot counters alternate
// between two halves by the parity of the exchange number, and all waits are bounded by a wall-clock limit after which the kernel records
// kStatusTimeout and returns.  A rank never waits for something that needs one of its own later kernels, so the
// three kernels of one rank can be queued back to back on a stream; ranks emulated on ONE device must run all
// pushes before the first reduce and all reduces before the first gather, so that no wait ever spins.
#include "common.cuh"
#include "kernels.h"

namespace foe {

namespace {

constexpr int kShardThreads = 256;
constexpr int kShardRows = 16;       // rows of one block's share (divides kShardBlockRows)

__device__ __forceinline__ unsigned int ld_acquire_sys(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// true once *cnt has reached `expect` (wrap-safe), false if limit_ns went by first
__device__ __forceinline__ bool wait_count(const unsigned int* cnt, unsigned int expect, unsigned long long limit_ns) {
  if (int(ld_acquire_sys(cnt) - expect) >= 0) return true;
  const unsigned long long t0 = global_timer_ns();
  while (true) {
    __nanosleep(200);
    if (int(ld_acquire_sys(cnt) - expect) >= 0) return true;
    if (global_timer_ns() - t0 > limit_ns) return false;
  }
}

// block (rb, o): rows [rb*16, +16) of owner o's columns, read from src ([S][d] bf16 or fp32), scaled, written as
// bf16 into slot `rank` of o's receive buffer
__global__ void __launch_bounds__(kShardThreads)
shard_push_kernel(const void* __restrict__ src, int src_is_f32, float scale, int S, int d, int span, ShardPeerTable t,
                  long long slot_off, int cnt_off) {
  const int o = blockIdx.y;
  const int r0 = blockIdx.x * kShardRows;
  const int rows = min(kShardRows, S - r0);
  const int c8 = span >> 3;                       // 16-byte pieces per row
  bf16* dst = t.slots[o] + slot_off;
  for (int i = threadIdx.x; i < rows * c8; i += kShardThreads) {
    const int r = r0 + i / c8, c = (i % c8) * 8;
    const size_t s_off = size_t(r) * d + size_t(o) * span + c;
    float v[8];
    if (src_is_f32) {
      const float4 a = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(src) + s_off));
      const float4 b = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(src) + s_off + 4));
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
      const uint4 a = __ldg(reinterpret_cast<const uint4*>(static_cast<const bf16*>(src) + s_off));
      const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) { v[2 * q] = bf16_lo(w[q]); v[2 * q + 1] = bf16_hi(w[q]); }
    }
    *reinterpret_cast<uint4*>(dst + size_t(r) * span + c) =
        make_uint4(pack_bf16(v[0] * scale, v[1] * scale), pack_bf16(v[2] * scale, v[3] * scale),
                   pack_bf16(v[4] * scale, v[5] * scale), pack_bf16(v[6] * scale, v[7] * scale));
  }
  __threadfence_system();
  __syncthreads();
  if (threadIdx.x == 0) atomicAdd_system(t.slot_cnt[o] + cnt_off + r0 / kShardBlockRows, unsigned(rows) * unsigned(span));
}

// owner side: block rb reduces rows [rb*16, +16) of this rank's columns over the H slots and hands the result to
// every rank's gather buffer
__global__ void __launch_bounds__(kShardThreads)
shard_reduce_kernel(const bf16* __restrict__ my_slots, const unsigned int* my_slot_cnt, int n_blocks, int S,
                    size_t S_cap, int d, int span, int H, int rank, ShardPeerTable t, long long gather_off,
                    unsigned long long limit_ns, int* status) {
  __shared__ int s_ok;
  if (threadIdx.x == 0) s_ok = 1;
  __syncthreads();
  {
    // only the partials of this block's rows have to be there
    const int blk = blockIdx.x * kShardRows / kShardBlockRows;
    const unsigned int expect = unsigned(min(kShardBlockRows, S - blk * kShardBlockRows)) * unsigned(span);
    if (threadIdx.x < H) {
      if (!wait_count(my_slot_cnt + threadIdx.x * n_blocks + blk, expect, limit_ns)) s_ok = 0;
    }
  }
  __syncthreads();
  if (!s_ok) {
    if (threadIdx.x == 0) atomicExch(status, kStatusTimeout);
    return;
  }
  const int r0 = blockIdx.x * kShardRows;
  const int rows = min(kShardRows, S - r0);
  const int c8 = span >> 3;
  for (int i = threadIdx.x; i < rows * c8; i += kShardThreads) {
    const int r = r0 + i / c8, c = (i % c8) * 8;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int h = 0; h < H; ++h) {                                 // rank order: the sum does not depend on timing
      const uint4 a = __ldcg(reinterpret_cast<const uint4*>(my_slots + (size_t(h) * S_cap + r) * span + c));
      const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) { acc[2 * q] += bf16_lo(w[q]); acc[2 * q + 1] += bf16_hi(w[q]); }
    }
    const uint4 v = make_uint4(pack_bf16(acc[0], acc[1]), pack_bf16(acc[2], acc[3]), pack_bf16(acc[4], acc[5]),
                               pack_bf16(acc[6], acc[7]));
    for (int p = 0; p < H; ++p)
      *reinterpret_cast<uint4*>(t.gather[p] + gather_off + size_t(r) * d + size_t(rank) * span + c) = v;
  }
  __threadfence_system();
  __syncthreads();
  if (threadIdx.x < H) atomicAdd_system(t.gather_cnt[threadIdx.x] + rank, unsigned(rows) * unsigned(span));
}

// block (rb, o): waits for owner o's share of the gathered tensor and copies rows [rb*16, +16) of it out of the
// gather buffer (to fp32 and / or bf16)
__global__ void __launch_bounds__(kShardThreads)
shard_gather_kernel(const bf16* __restrict__ my_gather, const unsigned int* my_gather_cnt, unsigned int expect, int S,
                    int d, int span, float* dst_f32, bf16* dst_bf16, unsigned int* zero_cnt, int zero_n,
                    unsigned long long limit_ns, int* status) {
  __shared__ int s_ok;
  const int o = blockIdx.y;
  if (blockIdx.x == 0 && o == 0)
    for (int i = threadIdx.x; i < zero_n; i += kShardThreads) zero_cnt[i] = 0u;
  if (threadIdx.x == 0) s_ok = wait_count(my_gather_cnt + o, expect, limit_ns) ? 1 : 0;
  __syncthreads();
  if (!s_ok) {
    if (threadIdx.x == 0) atomicExch(status, kStatusTimeout);
    return;
  }
  const int r0 = blockIdx.x * kShardRows;
  const int rows = min(kShardRows, S - r0);
  const int c8 = span >> 3;
  for (int i = threadIdx.x; i < rows * c8; i += kShardThreads) {
    const int r = r0 + i / c8, c = (i % c8) * 8;
    const size_t off = size_t(r) * d + size_t(o) * span + c;
    const uint4 a = __ldcg(reinterpret_cast<const uint4*>(my_gather + off));
    if (dst_bf16) *reinterpret_cast<uint4*>(dst_bf16 + off) = a;
    if (dst_f32) {
      const uint32_t w[4] = {a.x, a.y, a.z, a.w};
      *reinterpret_cast<float4*>(dst_f32 + off) = make_float4(bf16_lo(w[0]), bf16_hi(w[0]), bf16_lo(w[1]), bf16_hi(w[1]));
      *reinterpret_cast<float4*>(dst_f32 + off + 4) = make_float4(bf16_lo(w[2]), bf16_hi(w[2]), bf16_lo(w[3]), bf16_hi(w[3]));
    }
  }
}

}  // namespace

void launch_shard_push(const void* src, int src_is_f32, float scale, int S, int d, int H, const ShardPeerTable& t,
                       long long slot_off, int cnt_off, cudaStream_t st) {
  const dim3 grid((S + kShardRows - 1) / kShardRows, H);
  shard_push_kernel<<<grid, kShardThreads, 0, st>>>(src, src_is_f32, scale, S, d, d / H, t, slot_off, cnt_off);
}

void launch_shard_reduce(const bf16* my_slots, const unsigned int* my_slot_cnt, int n_blocks, int S, size_t S_cap,
                         int d, int H, int rank, const ShardPeerTable& t, long long gather_off,
                         unsigned long long limit_ns, int* status, cudaStream_t st) {
  shard_reduce_kernel<<<(S + kShardRows - 1) / kShardRows, kShardThreads, 0, st>>>(
      my_slots, my_slot_cnt, n_blocks, S, S_cap, d, d / H, H, rank, t, gather_off, limit_ns, status);
}

void launch_shard_gather(const bf16* my_gather, const unsigned int* my_gather_cnt, unsigned int expect, int S, int d,
                         int H, float* dst_f32, bf16* dst_bf16, unsigned int* zero_cnt, int zero_n,
                         unsigned long long limit_ns, int* status, cudaStream_t st) {
  const dim3 grid((S + kShardRows - 1) / kShardRows, H);
  shard_gather_kernel<<<grid, kShardThreads, 0, st>>>(my_gather, my_gather_cnt, expect, S, d, d / H, dst_f32, dst_bf16,
                                                      zero_cnt, zero_n, limit_ns, status);
}

}  // namespace foe
