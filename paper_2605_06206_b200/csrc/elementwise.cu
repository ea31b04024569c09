// Streaming (HBM-bound) steps of the FoE block and the create-time weight repacks.
#include "common.cuh"
#include "kernels.h"

namespace foe {

// ------------------------------------------------------------------ RMS statistics (pre-attention norm)
// One warp per row: inv_rms = rsqrt(mean(x^2) + eps).  The gain is folded into the projection weights
// and the scale is applied in the GEMM epilogue, so the normalised tensor is never written.
__global__ void row_inv_rms_kernel(const bf16* __restrict__ x, float* __restrict__ inv_rms, int n_rows, int d,
                                   float eps) {
  pdl_wait();
  pdl_launch_dependents();
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (warp >= n_rows) return;
  const uint4* row = reinterpret_cast<const uint4*>(x + size_t(warp) * d);
  float ss = 0.f;
  for (int c = lane; c < d / 8; c += 32) {
    const uint4 q = __ldg(row + c);
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float a = bf16_lo(w[j]), b = bf16_hi(w[j]);
      ss += a * a + b * b;
    }
  }
  ss = warp_sum(ss);
  if (lane == 0) inv_rms[warp] = rsqrtf(ss / float(d) + eps);
}

// The same statistics for the H residual streams x[h] of a middle or last layer, plus their sum: one warp per token
// reads its H rows once, writes inv_rms[h * S + s] and xsum[s][:] = sum_h x[h][s][:] (fp32, h ascending).  The output
// projection then adds ONE fp32 tensor in its epilogue instead of reading the H streams again.
template <int H>
__global__ void row_inv_rms_xsum_kernel(const bf16* __restrict__ x, float* __restrict__ inv_rms, float* __restrict__ xsum,
                                        int S, int d, float eps) {
  pdl_wait();
  pdl_launch_dependents();
  const int s = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (s >= S) return;
  float ss[H];
#pragma unroll
  for (int h = 0; h < H; ++h) ss[h] = 0.f;
  for (int c = lane; c < d / 8; c += 32) {
    uint4 q[H];
#pragma unroll
    for (int h = 0; h < H; ++h) q[h] = __ldg(reinterpret_cast<const uint4*>(x + (size_t(h) * S + s) * d) + c);
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int h = 0; h < H; ++h) {
      const uint32_t w[4] = {q[h].x, q[h].y, q[h].z, q[h].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float a = bf16_lo(w[j]), b = bf16_hi(w[j]);
        ss[h] += a * a + b * b;
        acc[2 * j] += a;
        acc[2 * j + 1] += b;
      }
    }
    float4* o = reinterpret_cast<float4*>(xsum + size_t(s) * d + c * 8);
    o[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
    o[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
  }
#pragma unroll
  for (int h = 0; h < H; ++h) {
    const float t = warp_sum(ss[h]);
    if (lane == 0) inv_rms[size_t(h) * S + s] = rsqrtf(t / float(d) + eps);
  }
}

bool launch_row_inv_rms_xsum(const bf16* x, float* inv_rms, float* xsum, int S, int d, int H, float eps, cudaStream_t st) {
  if (S <= 0) return true;
  const int threads = 256;
  const int blocks = (S * 32 + threads - 1) / threads;
  switch (H) {
    case 2: launch_pdl(row_inv_rms_xsum_kernel<2>, dim3(blocks), dim3(threads), 0, st, x, inv_rms, xsum, S, d, eps); return true;
    case 3: launch_pdl(row_inv_rms_xsum_kernel<3>, dim3(blocks), dim3(threads), 0, st, x, inv_rms, xsum, S, d, eps); return true;
    case 4: launch_pdl(row_inv_rms_xsum_kernel<4>, dim3(blocks), dim3(threads), 0, st, x, inv_rms, xsum, S, d, eps); return true;
    case 5: launch_pdl(row_inv_rms_xsum_kernel<5>, dim3(blocks), dim3(threads), 0, st, x, inv_rms, xsum, S, d, eps); return true;
    case 6: launch_pdl(row_inv_rms_xsum_kernel<6>, dim3(blocks), dim3(threads), 0, st, x, inv_rms, xsum, S, d, eps); return true;
    case 7: launch_pdl(row_inv_rms_xsum_kernel<7>, dim3(blocks), dim3(threads), 0, st, x, inv_rms, xsum, S, d, eps); return true;
    case 8: launch_pdl(row_inv_rms_xsum_kernel<8>, dim3(blocks), dim3(threads), 0, st, x, inv_rms, xsum, S, d, eps); return true;
    default: return false;
  }
}

void launch_row_inv_rms(const bf16* x, float* inv_rms, int n_rows, int d, float eps, cudaStream_t st) {
  if (n_rows <= 0) return;
  const int threads = 256;
  const int blocks = (n_rows * 32 + threads - 1) / threads;
  launch_pdl(row_inv_rms_kernel, dim3(blocks), dim3(threads), 0, st, x, inv_rms, n_rows, d, eps);
}

// ------------------------------------------------------------------ token -> (sequence, position, cache slot)
__global__ void cu_q_kernel(const int* __restrict__ q_lens, int n_seqs, int* __restrict__ cu_q) {
  pdl_wait();
  pdl_launch_dependents();
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    int acc = 0;
    cu_q[0] = 0;
    for (int b = 0; b < n_seqs; ++b) { acc += q_lens ? q_lens[b] : 1; cu_q[b + 1] = acc; }
  }
}

// With `q_lens` given (at most kMapScanSeqs sequences) every block first builds the prefix sums of the sequences'
// new-token counts in shared memory -- one warp, 32 consecutive sequences per lane -- and block 0 also writes them to
// cu_q_out for the attention kernel: no separate one-thread prefix kernel in front of this one.
constexpr int kMapScanSeqs = 1024;

__global__ void token_map_kernel(const int* cu_q_in, int* cu_q_out, int has_q_lens,
                                 const int* __restrict__ q_lens, const int* __restrict__ context_lens,
                                 const int* __restrict__ block_table, int n_seqs, int max_pages_per_seq,
                                 int num_pages, int page_size, int n_tokens, int max_context, int max_q_len,
                                 int* __restrict__ tok_seq, int* __restrict__ tok_pos, int* __restrict__ tok_slot,
                                 int* __restrict__ status) {
  __shared__ int s_cu[kMapScanSeqs + 1];
  pdl_wait();
  pdl_launch_dependents();
  const int* cu_q = cu_q_in;
  if (q_lens) {                               // (n_seqs <= kMapScanSeqs: the launcher's choice)
    for (int b = threadIdx.x; b < n_seqs; b += blockDim.x) s_cu[b + 1] = q_lens[b];
    if (threadIdx.x == 0) s_cu[0] = 0;
    __syncthreads();
    if (threadIdx.x < 32) {
      const int lane = threadIdx.x;
      const int b0 = lane * 32;               // this lane's sequences: b0 .. b0 + 31
      int sum = 0;
      for (int k = 0; k < 32; ++k)
        if (b0 + k < n_seqs) sum += s_cu[b0 + k + 1];
      int incl = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      int run = incl - sum;                   // tokens of the sequences before b0
      for (int k = 0; k < 32; ++k)
        if (b0 + k < n_seqs) { run += s_cu[b0 + k + 1]; s_cu[b0 + k + 1] = run; }
    }
    __syncthreads();
    if (blockIdx.x == 0)
      for (int b = threadIdx.x; b <= n_seqs; b += blockDim.x) cu_q_out[b] = s_cu[b];
    cu_q = s_cu;
  }
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_tokens) return;
  int b;
  if (!has_q_lens) {                         // one token per sequence: the prefix is the identity, written here
    b = i;
    cu_q_out[i] = i;
    if (i == n_tokens - 1) cu_q_out[n_tokens] = n_tokens;
  } else {
    int lo = 0, hi = n_seqs;                 // largest b with cu_q[b] <= i
    while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (cu_q[mid] <= i) lo = mid; else hi = mid; }
    b = lo;
  }
  const int local = has_q_lens ? i - cu_q[b] : 0;
  const int q_len = has_q_lens ? cu_q[b + 1] - cu_q[b] : 1;
  const int pos = context_lens[b] + local;
  int slot = -1;
  // a position outside [0, max_context) never reaches the block table; a sequence longer than the call's stated
  // bound, or a prefix sum that disagrees with the call's token count, is an error of the whole call
  bool ok = pos >= 0 && pos < max_context && q_len <= max_q_len;
  if (has_q_lens && i == n_tokens - 1 && cu_q[n_seqs] != n_tokens) ok = false;
  if (ok) {
    const int lp = pos / page_size;
    if (lp < max_pages_per_seq) {
      const int page = block_table[size_t(b) * max_pages_per_seq + lp];
      if (page >= 0 && page < num_pages) slot = page * page_size + (pos - lp * page_size);
    }
  }
  if (slot < 0) atomicExch(status, kStatusBounds);
  tok_seq[i] = b;
  // consumers index the rotary table with this: keep it inside the table whatever the caller passed
  tok_pos[i] = min(max(pos, 0), max_context - 1);
  tok_slot[i] = slot;
}

int launch_token_map(const int* q_lens, const int* context_lens, const int* block_table, int n_seqs,
                      int max_pages_per_seq, int num_pages, int page_size, int n_tokens, int max_context, int max_q_len,
                      int* cu_q, int* tok_seq, int* tok_pos, int* tok_slot, int* status, cudaStream_t st) {
  int launches = 0;
  const bool scan_in_block = q_lens && n_seqs <= kMapScanSeqs && n_tokens > 0;
  if (q_lens && !scan_in_block) { launch_pdl(cu_q_kernel, dim3(1), dim3(32), 0, st, q_lens, n_seqs, cu_q); ++launches; }
  if (n_tokens <= 0) return launches;
  launch_pdl(token_map_kernel, dim3((n_tokens + 255) / 256), dim3(256), 0, st, cu_q, cu_q, q_lens != nullptr,
             scan_in_block ? q_lens : static_cast<const int*>(nullptr), context_lens, block_table, n_seqs,
             max_pages_per_seq, num_pages, page_size, n_tokens, max_context, max_q_len, tok_seq, tok_pos, tok_slot, status);
  return launches + 1;
}

// v[i] += by: the caller's context lengths after a step, bumped on the device so that a decode loop never touches them
// from the host.  An ordinary launch (no early start): it follows kernels that still read the old values.
__global__ void add_to_ints_kernel(int* __restrict__ v, int n, int by) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) v[i] += by;
}

void launch_add_to_ints(int* v, int n, int by, cudaStream_t st) {
  if (n <= 0) return;
  add_to_ints_kernel<<<(n + 255) / 256, 256, 0, st>>>(v, n, by);
}

// ------------------------------------------------------------------ combine (+ residual, + last-layer mean)
// Block per token; each thread owns 8 consecutive columns.  x'[h,i] = r_full[i] + sum_j w[i,h,j] y[inv[i,h,j]].
// The token's slots and gates are brought into shared memory with one coalesced load, and for the usual numbers of
// experts per cluster (KC = 1, 2, 4, 8; 0 = any) the k_c row loads of a cluster are written out, so that they are all
// in flight before the first is used: with one 16-byte load in flight per thread (a slot looked up in global memory,
// then its row) the kernel sat at 5 TB/s whatever the clock.  The sums run in the order of j, as everywhere else.
template <int KC>
__global__ void __launch_bounds__(256)
combine_kernel(const float* __restrict__ r_full, const bf16* __restrict__ y, const float* __restrict__ w,
               const int* __restrict__ inv, bf16* __restrict__ out, int n_tokens, int d, int H, int kc_rt, int last_mean) {
  __shared__ int s_slot[256];                 // H <= 8, k_c <= 32
  __shared__ float s_gate[256];
  pdl_wait();
  pdl_launch_dependents();
  const int i = blockIdx.x;
  const int kc = KC ? KC : kc_rt;
  const int n_sel = H * kc;
  for (int t = threadIdx.x; t < n_sel; t += blockDim.x) {
    s_slot[t] = __ldg(inv + size_t(i) * n_sel + t);
    s_gate[t] = __ldg(w + size_t(i) * n_sel + t);
  }
  __syncthreads();
  const float inv_h = 1.0f / float(H);
  for (int c = threadIdx.x * 8; c < d; c += blockDim.x * 8) {
    float r[8];
    {
      const float4 r0 = *reinterpret_cast<const float4*>(r_full + size_t(i) * d + c);
      const float4 r1 = *reinterpret_cast<const float4*>(r_full + size_t(i) * d + c + 4);
      r[0] = r0.x; r[1] = r0.y; r[2] = r0.z; r[3] = r0.w; r[4] = r1.x; r[5] = r1.y; r[6] = r1.z; r[7] = r1.w;
    }
    float mean[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) mean[t] = 0.f;
#pragma unroll 2
    for (int h = 0; h < H; ++h) {
      float acc[8];
#pragma unroll
      for (int t = 0; t < 8; ++t) acc[t] = r[t];
      if (KC) {
        uint4 q[KC ? KC : 1];
#pragma unroll
        for (int j = 0; j < KC; ++j)
          q[j] = __ldg(reinterpret_cast<const uint4*>(y + size_t(s_slot[h * KC + j]) * d + c));
#pragma unroll
        for (int j = 0; j < KC; ++j) {
          const float g = s_gate[h * KC + j];
          const uint32_t v[4] = {q[j].x, q[j].y, q[j].z, q[j].w};
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            acc[2 * t] += g * bf16_lo(v[t]);
            acc[2 * t + 1] += g * bf16_hi(v[t]);
          }
        }
      } else {
        for (int j = 0; j < kc; ++j) {
          const float g = s_gate[h * kc + j];
          const uint4 q = __ldg(reinterpret_cast<const uint4*>(y + size_t(s_slot[h * kc + j]) * d + c));
          const uint32_t v[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
          for (int t = 0; t < 4; ++t) {
            acc[2 * t] += g * bf16_lo(v[t]);
            acc[2 * t + 1] += g * bf16_hi(v[t]);
          }
        }
      }
      if (last_mean) {
#pragma unroll
        for (int t = 0; t < 8; ++t) mean[t] += acc[t];
      } else {
        *reinterpret_cast<uint4*>(out + (size_t(h) * n_tokens + i) * d + c) =
            make_uint4(pack_bf16(acc[0], acc[1]), pack_bf16(acc[2], acc[3]), pack_bf16(acc[4], acc[5]),
                       pack_bf16(acc[6], acc[7]));
      }
    }
    if (last_mean) {
      *reinterpret_cast<uint4*>(out + size_t(i) * d + c) =
          make_uint4(pack_bf16(mean[0] * inv_h, mean[1] * inv_h), pack_bf16(mean[2] * inv_h, mean[3] * inv_h),
                     pack_bf16(mean[4] * inv_h, mean[5] * inv_h), pack_bf16(mean[6] * inv_h, mean[7] * inv_h));
    }
  }
}

// The same for calls of a few hundred tokens, where the kernel is a chain of dependent loads rather than a stream: the
// token's slots and gates (and the residual) are fetched before the wait for the expert GEMM -- they are older than
// that kernel -- and the expert rows are requested eight at a time instead of one after the other.  Same sums in the
// same order as combine_kernel.
__global__ void combine_small_kernel(const float* __restrict__ r_full, const bf16* __restrict__ y, const float* __restrict__ w,
                                     const int* __restrict__ inv, bf16* __restrict__ out, int n_tokens, int d, int H, int kc,
                                     int last_mean) {
  __shared__ int s_slot[256];                 // H <= 8, k_c <= 32
  __shared__ float s_gate[256];
  const int i = blockIdx.x;
  const int n_sel = H * kc;
  for (int t = threadIdx.x; t < n_sel; t += blockDim.x) {
    s_slot[t] = __ldg(inv + size_t(i) * n_sel + t);
    s_gate[t] = __ldg(w + size_t(i) * n_sel + t);
  }
  const int c0 = threadIdx.x * 8;
  float r0[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (c0 < d) {
    const float4 a = *reinterpret_cast<const float4*>(r_full + size_t(i) * d + c0);
    const float4 b = *reinterpret_cast<const float4*>(r_full + size_t(i) * d + c0 + 4);
    r0[0] = a.x; r0[1] = a.y; r0[2] = a.z; r0[3] = a.w; r0[4] = b.x; r0[5] = b.y; r0[6] = b.z; r0[7] = b.w;
  }
  pdl_wait();                                 // the expert rows come from the kernel before this one
  pdl_launch_dependents();
  __syncthreads();
  const float inv_h = 1.0f / float(H);
  for (int c = c0; c < d; c += blockDim.x * 8) {
    float r[8];
    if (c == c0) {
#pragma unroll
      for (int t = 0; t < 8; ++t) r[t] = r0[t];
    } else {
      const float4 a = *reinterpret_cast<const float4*>(r_full + size_t(i) * d + c);
      const float4 b = *reinterpret_cast<const float4*>(r_full + size_t(i) * d + c + 4);
      r[0] = a.x; r[1] = a.y; r[2] = a.z; r[3] = a.w; r[4] = b.x; r[5] = b.y; r[6] = b.z; r[7] = b.w;
    }
    float mean[8], acc[8];
#pragma unroll
    for (int t = 0; t < 8; ++t) { mean[t] = 0.f; acc[t] = r[t]; }
    int j = 0, h = 0;                         // position of the next selection inside its cluster
    for (int s0 = 0; s0 < n_sel; s0 += 8) {
      uint4 q[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        q[u] = make_uint4(0u, 0u, 0u, 0u);
        if (s0 + u < n_sel) q[u] = __ldcg(reinterpret_cast<const uint4*>(y + size_t(s_slot[s0 + u]) * d + c));
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        if (s0 + u >= n_sel) break;
        const float g = s_gate[s0 + u];
        const uint32_t v[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
          acc[2 * t] += g * bf16_lo(v[t]);
          acc[2 * t + 1] += g * bf16_hi(v[t]);
        }
        if (++j == kc) {                      // cluster h is complete
          if (last_mean) {
#pragma unroll
            for (int t = 0; t < 8; ++t) mean[t] += acc[t];
          } else {
            *reinterpret_cast<uint4*>(out + (size_t(h) * n_tokens + i) * d + c) =
                make_uint4(pack_bf16(acc[0], acc[1]), pack_bf16(acc[2], acc[3]), pack_bf16(acc[4], acc[5]),
                           pack_bf16(acc[6], acc[7]));
          }
#pragma unroll
          for (int t = 0; t < 8; ++t) acc[t] = r[t];
          j = 0;
          ++h;
        }
      }
    }
    if (last_mean) {
      *reinterpret_cast<uint4*>(out + size_t(i) * d + c) =
          make_uint4(pack_bf16(mean[0] * inv_h, mean[1] * inv_h), pack_bf16(mean[2] * inv_h, mean[3] * inv_h),
                     pack_bf16(mean[4] * inv_h, mean[5] * inv_h), pack_bf16(mean[6] * inv_h, mean[7] * inv_h));
    }
  }
}

void launch_combine(const float* r_full, const bf16* y, const float* w, const int* inv, bf16* out, int n_tokens, int d,
                    int H, int kc, int last_mean, cudaStream_t st) {
  if (n_tokens <= 0) return;
  int threads = d / 8;
  if (threads > 256) threads = 256;
  if (threads < 32) threads = 32;
  if (n_tokens <= 1024) {
    if (d / 8 >= 512) threads = 512;          // one pass over the row: the kernel is a chain of round trips, not a stream
    launch_pdl(combine_small_kernel, dim3(n_tokens), dim3(threads), 0, st, r_full, y, w, inv, out, n_tokens, d, H, kc, last_mean);
    return;
  }
  switch (kc) {
    case 1: launch_pdl(combine_kernel<1>, dim3(n_tokens), dim3(threads), 0, st, r_full, y, w, inv, out, n_tokens, d, H, kc, last_mean); break;
    case 2: launch_pdl(combine_kernel<2>, dim3(n_tokens), dim3(threads), 0, st, r_full, y, w, inv, out, n_tokens, d, H, kc, last_mean); break;
    case 4: launch_pdl(combine_kernel<4>, dim3(n_tokens), dim3(threads), 0, st, r_full, y, w, inv, out, n_tokens, d, H, kc, last_mean); break;
    case 8: launch_pdl(combine_kernel<8>, dim3(n_tokens), dim3(threads), 0, st, r_full, y, w, inv, out, n_tokens, d, H, kc, last_mean); break;
    default: launch_pdl(combine_kernel<0>, dim3(n_tokens), dim3(threads), 0, st, r_full, y, w, inv, out, n_tokens, d, H, kc, last_mean); break;
  }
}

// ------------------------------------------------------------------ create-time repacks
// dst[b][n'][k] = src[b][k][n] * gain[k]   (gain optional): makes the projection weights K-major.  With
// interleave_dh > 0 the rows of every head of interleave_dh columns are stored as 0, dh/2, 1, dh/2+1, ... so that
// the two members of a rotary pair are neighbours in the GEMM's accumulator.
__global__ void transpose_batched_kernel(const bf16* __restrict__ src, size_t src_batch, int src_ld,
                                         bf16* __restrict__ dst, size_t dst_batch, int dst_ld, int K, int N,
                                         const bf16* __restrict__ gain, int interleave_dh) {
  __shared__ float tile[32][33];
  const bf16* s = src + blockIdx.z * src_batch;
  bf16* d = dst + blockIdx.z * dst_batch;
  const int k0 = blockIdx.y * 32, n0 = blockIdx.x * 32;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int k = k0 + r, n = n0 + threadIdx.x;
    float v = 0.f;
    if (k < K && n < N) {
      v = __bfloat162float(s[size_t(k) * src_ld + n]);
      if (gain) v *= __bfloat162float(gain[k]);
    }
    tile[r][threadIdx.x] = v;
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int n = n0 + r, k = k0 + threadIdx.x;
    int nd = n;                                // destination row; heads may be stored with their halves interleaved
    if (interleave_dh > 0) {
      const int j = n % interleave_dh, half = interleave_dh >> 1;
      nd = n - j + (j < half ? 2 * j : 2 * (j - half) + 1);
    }
    if (k < K && n < N) d[size_t(nd) * dst_ld + k] = __float2bfloat16_rn(tile[threadIdx.x][r]);
  }
}

void launch_transpose_batched(const bf16* src, size_t src_batch, int src_ld, bf16* dst, size_t dst_batch, int dst_ld,
                              int K, int N, int batch, const bf16* gain, int interleave_dh, cudaStream_t st) {
  if (batch <= 0) return;
  dim3 grid((N + 31) / 32, (K + 31) / 32, batch), block(32, 8);
  transpose_batched_kernel<<<grid, block, 0, st>>>(src, src_batch, src_ld, dst, dst_batch, dst_ld, K, N, gain, interleave_dh);
}

// dst[e][b*256 + half*128 + j][k] = (half ? w_up : w_gate)[e][k][b*128 + j]: gate and up columns of one
// 128-wide block share one 256-wide GEMM tile, so SwiGLU is an epilogue.
__global__ void pack_gate_up_kernel(const bf16* __restrict__ wg, const bf16* __restrict__ wu, bf16* __restrict__ dst,
                                    int d, int I) {
  __shared__ bf16 tile[32][34];
  const int e = blockIdx.z;
  const int k0 = blockIdx.y * 32, np0 = blockIdx.x * 32;      // np = packed row index in [0, 2I)
  const int blk = np0 / 256, half = (np0 % 256) / 128, j0 = np0 % 128;
  const bf16* src = (half ? wu : wg) + size_t(e) * d * I;
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int k = k0 + r;
    tile[r][threadIdx.x] = (k < d) ? src[size_t(k) * I + blk * 128 + j0 + threadIdx.x] : __float2bfloat16_rn(0.f);
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += blockDim.y) {
    const int k = k0 + threadIdx.x;
    if (k < d) dst[(size_t(e) * 2 * I + np0 + r) * d + k] = tile[threadIdx.x][r];
  }
}

void launch_pack_gate_up(const bf16* wg, const bf16* wu, bf16* dst, int E, int d, int I, cudaStream_t st) {
  dim3 grid(2 * I / 32, (d + 31) / 32, E), block(32, 8);
  pack_gate_up_kernel<<<grid, block, 0, st>>>(wg, wu, dst, d, I);
}

}  // namespace foe
