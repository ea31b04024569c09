// Router of the FoE block (Section 3.1 "Routing"): FFN RMSNorm, one fp32 score vector per token,
// per-cluster top-k inside the cluster's contiguous expert block, gates = softmax over the selected
// scores.  Everything on this path is fp32 on the plain ALUs: the decision it takes (which experts)
// is an integer result that must agree with a float32 reference, so no reduced-precision tensor path.
//
// Three kernels (for calls of kRouterTcMinTokens tokens or more, the tensor-core kernel of router_tc.cu replaces 2):
//  1. ffn_norm:     one warp per token: inv_rms and the bf16 expert input u = r * inv_rms * gain.
//  2. router_gemm:  SIMT fp32 GEMM, 64 tokens x 64 experts per CTA, 8 x 4 register tiles, k-major shared
//                   tiles, register-staged double buffering; the normalisation is applied while the token
//                   tile is loaded (u is never rounded to bf16 on this path).  For a handful of tokens the
//                   reduction dimension is split over gridDim.z so that the grid still fills the GPU; the
//                   partial scores are summed in a fixed order by kernel 3.
//  3. topk_gates:   8, 16 or 32 lanes per (token, cluster): bias, top-k by (score descending, expert id ascending),
//                   softmax over the selected scores.
#include <float.h>

#include <atomic>

#include "common.cuh"
#include "kernels.h"

namespace foe {

// ------------------------------------------------------------------------------------------------ 1
// The same for an fp32 input whose row fits in registers (d = 128 * NV, NV float4 per lane): the row is read once.
// Same arithmetic in the same order as ffn_norm_kernel.
template <int NV>
__global__ void ffn_norm_f32_kernel(const float* __restrict__ r_in, const bf16* __restrict__ gain, bf16* __restrict__ u_out,
                                    float* __restrict__ inv_out, int n_tokens, float eps) {
  pdl_wait();
  pdl_launch_dependents();
  constexpr int d = NV * 128;
  const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (i >= n_tokens) return;
  const float4* row = reinterpret_cast<const float4*>(r_in + size_t(i) * d);
  float4 q[NV];
#pragma unroll
  for (int j = 0; j < NV; ++j) q[j] = __ldg(row + lane + 32 * j);
  float ss = 0.f;
#pragma unroll
  for (int j = 0; j < NV; ++j) ss += q[j].x * q[j].x + q[j].y * q[j].y + q[j].z * q[j].z + q[j].w * q[j].w;
  ss = warp_sum(ss);
  const float inv = rsqrtf(ss / float(d) + eps);
  if (lane == 0) inv_out[i] = inv;
  // lane's float4 j covers columns 4 * (lane + 32 j) ..: written as 8-byte bf16 quadruples
#pragma unroll
  for (int j = 0; j < NV; ++j) {
    const int c4 = lane + 32 * j;
    const uint2 gq = __ldg(reinterpret_cast<const uint2*>(gain) + c4);
    const float v0 = q[j].x * inv * bf16_lo(gq.x), v1 = q[j].y * inv * bf16_hi(gq.x);
    const float v2 = q[j].z * inv * bf16_lo(gq.y), v3 = q[j].w * inv * bf16_hi(gq.y);
    *reinterpret_cast<uint2*>(u_out + size_t(i) * d + c4 * 4) = make_uint2(pack_bf16(v0, v1), pack_bf16(v2, v3));
  }
}

__global__ void ffn_norm_kernel(const void* __restrict__ r_in, int r_is_bf16, const bf16* __restrict__ gain,
                                bf16* __restrict__ u_out, float* __restrict__ inv_out, int n_tokens, int d,
                                float eps) {
  pdl_wait();
  pdl_launch_dependents();
  const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (i >= n_tokens) return;
  float ss = 0.f;
  if (r_is_bf16) {
    const uint4* row = reinterpret_cast<const uint4*>(static_cast<const bf16*>(r_in) + size_t(i) * d);
    for (int c = lane; c < d / 8; c += 32) {
      const uint4 q = __ldg(row + c);
      const uint32_t v[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) { const float a = bf16_lo(v[j]), b = bf16_hi(v[j]); ss += a * a + b * b; }
    }
  } else {
    const float4* row = reinterpret_cast<const float4*>(static_cast<const float*>(r_in) + size_t(i) * d);
    for (int c = lane; c < d / 4; c += 32) {
      const float4 q = __ldg(row + c);
      ss += q.x * q.x + q.y * q.y + q.z * q.z + q.w * q.w;
    }
  }
  ss = warp_sum(ss);
  const float inv = rsqrtf(ss / float(d) + eps);
  if (lane == 0) inv_out[i] = inv;
  for (int c = lane; c < d / 8; c += 32) {
    float v[8];
    if (r_is_bf16) {
      const uint4 q = __ldg(reinterpret_cast<const uint4*>(static_cast<const bf16*>(r_in) + size_t(i) * d) + c);
      const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) { v[2 * j] = bf16_lo(w[j]); v[2 * j + 1] = bf16_hi(w[j]); }
    } else {
      const float4* row = reinterpret_cast<const float4*>(static_cast<const float*>(r_in) + size_t(i) * d);
      const float4 a = __ldg(row + 2 * c), b = __ldg(row + 2 * c + 1);
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    }
    const uint4 gq = __ldg(reinterpret_cast<const uint4*>(gain) + c);
    const uint32_t g[4] = {gq.x, gq.y, gq.z, gq.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) { v[2 * j] = v[2 * j] * inv * bf16_lo(g[j]); v[2 * j + 1] = v[2 * j + 1] * inv * bf16_hi(g[j]); }
    *reinterpret_cast<uint4*>(u_out + size_t(i) * d + c * 8) =
        make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
  }
}

// ------------------------------------------------------------------------------------------------ 2
constexpr int kRgTM = 64, kRgTN = 64, kRgKC = 32, kRgThreads = 128;
constexpr int kRgPA = kRgTM + 4, kRgPB = kRgTN + 4;      // padded pitches (floats), multiples of 4

__global__ void __launch_bounds__(kRgThreads, 4)
router_gemm_kernel(const void* __restrict__ r_in, int r_is_bf16, const float* __restrict__ inv_rms,
                   const bf16* __restrict__ gain, const float* __restrict__ wr, float* __restrict__ part,
                   int n_tokens, int d, int E, int k_per_split) {
  pdl_wait();
  pdl_launch_dependents();
  __shared__ __align__(16) float As[2][kRgKC][kRgPA];     // [k][token]
  __shared__ __align__(16) float Bs[2][kRgKC][kRgPB];     // [k][expert]
  const int tid = threadIdx.x;
  const int tok0 = blockIdx.x * kRgTM, exp0 = blockIdx.y * kRgTN;
  const int kbeg = blockIdx.z * k_per_split, kend = min(d, kbeg + k_per_split);
  const int ty = tid >> 4, tx = tid & 15;                 // 8 x 16 threads, 8 tokens x 4 experts each

  // loader roles: a tile is 64 rows x 8 float4; thread loads float4 (row = tid/8 + 16 j, k4 = tid%8), j < 4
  const int l_k4 = tid & 7, l_r = tid >> 3;
  float inv_t[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int t = tok0 + l_r + 16 * j;
    inv_t[j] = t < n_tokens ? inv_rms[t] : 0.f;
  }
  float4 ra[4], rb[4];

  auto load_chunk = [&](int k0) {
    const int k = k0 + l_k4 * 4;
    float g4[4];
    {
      const uint2 gq = __ldg(reinterpret_cast<const uint2*>(gain + k));
      g4[0] = bf16_lo(gq.x); g4[1] = bf16_hi(gq.x); g4[2] = bf16_lo(gq.y); g4[3] = bf16_hi(gq.y);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int t = tok0 + l_r + 16 * j;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (t < n_tokens) {
        if (r_is_bf16) {
          const uint2 q = __ldg(reinterpret_cast<const uint2*>(static_cast<const bf16*>(r_in) + size_t(t) * d + k));
          v = make_float4(bf16_lo(q.x), bf16_hi(q.x), bf16_lo(q.y), bf16_hi(q.y));
        } else {
          v = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(r_in) + size_t(t) * d + k));
        }
      }
      ra[j] = make_float4(v.x * inv_t[j] * g4[0], v.y * inv_t[j] * g4[1], v.z * inv_t[j] * g4[2], v.w * inv_t[j] * g4[3]);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int e = min(exp0 + l_r + 16 * j, E - 1);
      rb[j] = __ldg(reinterpret_cast<const float4*>(wr + size_t(e) * d + k));
    }
  };
  auto store_chunk = [&](int buf) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int r = l_r + 16 * j;
      As[buf][l_k4 * 4 + 0][r] = ra[j].x; As[buf][l_k4 * 4 + 1][r] = ra[j].y;
      As[buf][l_k4 * 4 + 2][r] = ra[j].z; As[buf][l_k4 * 4 + 3][r] = ra[j].w;
      Bs[buf][l_k4 * 4 + 0][r] = rb[j].x; Bs[buf][l_k4 * 4 + 1][r] = rb[j].y;
      Bs[buf][l_k4 * 4 + 2][r] = rb[j].z; Bs[buf][l_k4 * 4 + 3][r] = rb[j].w;
    }
  };

  float acc[8][4];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

  load_chunk(kbeg);
  store_chunk(0);
  __syncthreads();
  int buf = 0;
  for (int k0 = kbeg; k0 < kend; k0 += kRgKC) {
    const bool more = k0 + kRgKC < kend;
    if (more) load_chunk(k0 + kRgKC);
#pragma unroll 8
    for (int k = 0; k < kRgKC; ++k) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[buf][k][ty * 8]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[buf][k][ty * 8 + 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[buf][k][tx * 4]);
      const float a8[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float b4[4] = {b0.x, b0.y, b0.z, b0.w};
#pragma unroll
      for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(a8[a], b4[b], acc[a][b]);
    }
    if (more) store_chunk(buf ^ 1);
    __syncthreads();
    buf ^= 1;
  }
  float* dst = part + size_t(blockIdx.z) * n_tokens * E;
#pragma unroll
  for (int a = 0; a < 8; ++a) {
    const int t = tok0 + ty * 8 + a;
    if (t >= n_tokens) continue;
    const int e = exp0 + tx * 4;
    if (e + 3 < E && (E & 3) == 0) {
      *reinterpret_cast<float4*>(dst + size_t(t) * E + e) = make_float4(acc[a][0], acc[a][1], acc[a][2], acc[a][3]);
    } else {
#pragma unroll
      for (int b = 0; b < 4; ++b)
        if (e + b < E) dst[size_t(t) * E + e + b] = acc[a][b];
    }
  }
}

// ------------------------------------------------------------------------------------------------ 3
__global__ void topk_gates_kernel(const float* __restrict__ part, int k_splits, const float* __restrict__ br,
                                  float* __restrict__ logits_out, int* __restrict__ idx_out, float* __restrict__ w_out,
                                  int n_tokens, int H, int Ec, int kc) {
  pdl_wait();
  pdl_launch_dependents();
  // a (token, cluster) task is handled by a group of W lanes (W = 8, 16 or 32), several tasks per warp
  const int W = Ec <= 8 ? 8 : (Ec <= 16 ? 16 : 32);
  const int per_warp = 32 / W;
  const int lane = threadIdx.x & 31, li = lane & (W - 1);
  const int warp_id = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int task = warp_id * per_warp + lane / W;
  const bool live = task < n_tokens * H;
  const int i = live ? task / H : 0, h = live ? task - i * H : 0;
  const int E = H * Ec;
  float cand[4];
  bool taken[4];
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    const int e = li + W * s;
    float v = -FLT_MAX;
    if (live && e < Ec && (W == 32 || s == 0)) {
      const size_t o = size_t(i) * E + h * Ec + e;
      v = 0.f;
      for (int z = 0; z < k_splits; ++z) v += part[size_t(z) * n_tokens * E + o];
      if (br) v += __ldg(br + h * Ec + e);
      logits_out[o] = v;
      taken[s] = false;
    } else {
      taken[s] = true;
    }
    cand[s] = v;
  }
  float my_sel = -FLT_MAX;      // lane j of the group keeps the j-th selected score
  int my_idx = 0;
  for (int j = 0; j < kc; ++j) {
    float bv = -FLT_MAX;
    int bi = 0x7fffffff;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const int e = li + W * s;
      if (!taken[s] && (bi == 0x7fffffff || cand[s] > bv)) { bv = cand[s]; bi = e; }   // ascending e: first wins ties
    }
    for (int o = W >> 1; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (oi != 0x7fffffff && (bi == 0x7fffffff || ov > bv || (ov == bv && oi < bi))) { bv = ov; bi = oi; }
    }
    if (bi != 0x7fffffff && (bi & (W - 1)) == li) {
#pragma unroll
      for (int s = 0; s < 4; ++s)
        if (bi / W == s) taken[s] = true;
    }
    if (li == j) { my_sel = bv; my_idx = bi; }
  }
  const float m = __shfl_sync(0xffffffffu, my_sel, 0, W);
  float ex = li < kc ? expf(my_sel - m) : 0.f;
  float sum = ex;
  for (int o = W >> 1; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (live && li < kc) {
    const size_t o = (size_t(i) * H + h) * kc + li;
    idx_out[o] = h * Ec + my_idx;
    w_out[o] = ex / sum;
  }
}

// ------------------------------------------------------------------------------------------------ 1+2, small calls
// FFN norm and router scores of a call of at most 256 tokens (a decode step) in one launch: a CTA owns 4 tokens and
// 64 experts.  It first reduces its tokens' rows to 1/rms, then walks K in tiles of 64: the normalised activations
// (fp32, never rounded on this path) and a 64 x 64 tile of router weights go through shared memory, every thread
// accumulates one (token, expert) score in four interleaved fp32 chains.  K is also split over gridDim.z (partial
// scores, summed in a fixed order by the top-k kernel).  The CTAs of the first expert chunk also write the bf16
// expert input u for their slice of K.
constexpr int kRsTok = 4, kRsExp = 64, kRsK = 64, kRsThreads = kRsTok * kRsExp;

__global__ void __launch_bounds__(kRsThreads)
route_scores_small_kernel(const void* __restrict__ r_in, int r_is_bf16, const bf16* __restrict__ gain,
                          const float* __restrict__ wr, bf16* __restrict__ u_out, float* __restrict__ scores,
                          int n_tokens, int d, int E, float eps, int k_per_split) {
  __shared__ float w_s[kRsK][kRsExp + 1];
  __shared__ float u_s[kRsTok][kRsK];
  __shared__ float red[kRsTok][2];
  const int tid = threadIdx.x, el = tid & 63, tq = tid >> 6;
  const int tok = min(blockIdx.x * kRsTok + tq, n_tokens - 1);          // rows past the end repeat the last one
  const int e0 = blockIdx.y * kRsExp;
  const int kbeg = blockIdx.z * k_per_split, kend = min(d, kbeg + k_per_split);   // this CTA's slice of K
  // loader roles for the weight tile: float4 (row = i >> 4, column group = i & 15), i = tid + 256 j
  float4 wq[4];
  float uq;
  auto fetch_w = [&](int k0) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = tid + kRsThreads * j;
      const int e = min(e0 + (i >> 4), E - 1);
      wq[j] = __ldg(reinterpret_cast<const float4*>(wr + size_t(e) * d + k0 + (i & 15) * 4));
    }
  };
  // The router weights are older than the kernel before this one: the first tile is requested before the wait for it.
  fetch_w(kbeg);
  pdl_wait();
  pdl_launch_dependents();
  auto load_r = [&](int k) -> float {
    return r_is_bf16 ? __bfloat162float(static_cast<const bf16*>(r_in)[size_t(tok) * d + k])
                     : static_cast<const float*>(r_in)[size_t(tok) * d + k];
  };
  // 1/rms of this thread's token: 64 threads per token, eight 16-byte loads in flight per thread (the row sits in L2;
  // one element per load made this pass a chain of d / 256 round trips)
  float ss = 0.f;
  if (!r_is_bf16) {
    const float4* row = reinterpret_cast<const float4*>(static_cast<const float*>(r_in) + size_t(tok) * d);
    const int n4 = d >> 2;
    for (int k4 = el; k4 < n4; k4 += 64 * 8) {
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = k4 + 64 * u < n4 ? row[k4 + 64 * u] : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int u = 0; u < 8; ++u) ss += (v[u].x * v[u].x + v[u].y * v[u].y) + (v[u].z * v[u].z + v[u].w * v[u].w);
    }
  } else {
    const uint2* row = reinterpret_cast<const uint2*>(static_cast<const bf16*>(r_in) + size_t(tok) * d);
    const int n4 = d >> 2;
    for (int k4 = el; k4 < n4; k4 += 64 * 8) {
      uint2 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = k4 + 64 * u < n4 ? row[k4 + 64 * u] : make_uint2(0u, 0u);
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float a = bf16_lo(v[u].x), b = bf16_hi(v[u].x), c = bf16_lo(v[u].y), e = bf16_hi(v[u].y);
        ss += (a * a + b * b) + (c * c + e * e);
      }
    }
  }
  ss = warp_sum(ss);
  if ((tid & 31) == 0) red[tq][(tid >> 5) & 1] = ss;
  __syncthreads();
  const float inv = rsqrtf((red[tq][0] + red[tq][1]) / float(d) + eps);

  auto fetch = [&](int k0) {
    fetch_w(k0);
    uq = load_r(k0 + el) * inv * __bfloat162float(gain[k0 + el]);
  };
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  uq = load_r(kbeg + el) * inv * __bfloat162float(gain[kbeg + el]);
  for (int k0 = kbeg; k0 < kend; k0 += kRsK) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = tid + kRsThreads * j, row = i >> 4, c = (i & 15) * 4;
      w_s[c][row] = wq[j].x; w_s[c + 1][row] = wq[j].y; w_s[c + 2][row] = wq[j].z; w_s[c + 3][row] = wq[j].w;
    }
    u_s[tq][el] = uq;
    if (blockIdx.y == 0 && blockIdx.x * kRsTok + tq < n_tokens) u_out[size_t(tok) * d + k0 + el] = __float2bfloat16_rn(uq);
    __syncthreads();
    if (k0 + kRsK < kend) fetch(k0 + kRsK);            // in flight during the products below
#pragma unroll
    for (int k = 0; k < kRsK; ++k) acc[k & 3] = fmaf(u_s[tq][k], w_s[k][el], acc[k & 3]);
    __syncthreads();
  }
  if (blockIdx.x * kRsTok + tq < n_tokens && e0 + el < E)
    scores[(size_t(blockIdx.z) * n_tokens + tok) * E + e0 + el] = (acc[0] + acc[1]) + (acc[2] + acc[3]);
}

int route_small_k_splits(int d) {
  int ks = 1;
  while (ks < 16 && (d / (ks * 2)) % kRsK == 0 && d / (ks * 2) >= 2 * kRsK) ks *= 2;
  return ks;
}

int launch_route_small(const void* r_in, int r_is_bf16, const bf16* gain, const float* wr, const float* br, bf16* u_out,
                       float* scores, size_t scores_cap, float* logits, int* idx, float* w, const PermuteBuffers& pb,
                       int n_tokens, int d, int H, int Ec, int kc, float eps, int* status, cudaStream_t st) {
  if (n_tokens <= 0) return 0;
  const int E = H * Ec;
  // K is cut into slices so that a few dozen tokens still spread over the GPU; the partial scores are summed in a
  // fixed order by the second kernel
  const int ks = clamp_k_splits(route_small_k_splits(d), n_tokens, E, scores_cap);
  dim3 grid((n_tokens + kRsTok - 1) / kRsTok, (E + kRsExp - 1) / kRsExp, ks);
  launch_pdl(route_scores_small_kernel, grid, dim3(kRsThreads), 0, st, r_in, r_is_bf16, gain, wr, u_out, scores, n_tokens, d, E, eps, d / ks);
  return 1 + launch_topk_permute_small(scores, ks, br, logits, idx, w, pb, n_tokens, H, Ec, kc, status, st);
}

// The same selection with one thread per (token, cluster) and the cluster's scores in registers: for the common
// cluster sizes (a power of two up to 32) there is nothing to exchange between lanes.  Ties and order exactly as in
// topk_gates_kernel: score descending, expert id ascending.
template <int EC>
__global__ void topk_gates_thread_kernel(const float* __restrict__ part, int k_splits, const float* __restrict__ br,
                                         float* __restrict__ logits_out, int* __restrict__ idx_out,
                                         float* __restrict__ w_out, int n_tokens, int H, int kc) {
  pdl_wait();
  pdl_launch_dependents();
  const int task = blockIdx.x * blockDim.x + threadIdx.x;
  if (task >= n_tokens * H) return;
  const int i = task / H, h = task - i * H;
  const size_t o = size_t(i) * H * EC + size_t(h) * EC;
  const size_t split_stride = size_t(n_tokens) * H * EC;
  float v[EC];
#pragma unroll
  for (int e = 0; e < EC; e += 4) {
    float4 a = *reinterpret_cast<const float4*>(part + o + e);
    for (int z = 1; z < k_splits; ++z) {
      const float4 b = *reinterpret_cast<const float4*>(part + z * split_stride + o + e);
      a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
    }
    if (br) { a.x += __ldg(br + h * EC + e); a.y += __ldg(br + h * EC + e + 1); a.z += __ldg(br + h * EC + e + 2); a.w += __ldg(br + h * EC + e + 3); }
    v[e] = a.x; v[e + 1] = a.y; v[e + 2] = a.z; v[e + 3] = a.w;
    *reinterpret_cast<float4*>(logits_out + o + e) = a;
  }
  uint32_t taken = 0u;
  float m = 0.f, sum = 0.f;
  const size_t oo = size_t(task) * kc;
  for (int j = 0; j < kc; ++j) {
    float bv = -FLT_MAX;
    int bi = -1;
#pragma unroll
    for (int e = 0; e < EC; ++e)
      if (!((taken >> e) & 1u) && (bi < 0 || v[e] > bv)) { bv = v[e]; bi = e; }      // ascending e: first wins ties
    taken |= 1u << bi;
    if (j == 0) m = bv;
    const float ex = expf(bv - m);
    sum += ex;
    idx_out[oo + j] = h * EC + bi;
    w_out[oo + j] = ex;                 // normalised below
  }
  for (int j = 0; j < kc; ++j) w_out[oo + j] = w_out[oo + j] / sum;
}

static void launch_topk_gates(const float* part, int ks, const float* br, float* logits, int* idx, float* w,
                              int n_tokens, int H, int Ec, int kc, cudaStream_t st) {
  const int tasks = n_tokens * H;
  const int tb = (tasks + 127) / 128;
  switch (Ec) {
    case 4: launch_pdl(topk_gates_thread_kernel<4>, dim3(tb), dim3(128), 0, st, part, ks, br, logits, idx, w, n_tokens, H, kc); return;
    case 8: launch_pdl(topk_gates_thread_kernel<8>, dim3(tb), dim3(128), 0, st, part, ks, br, logits, idx, w, n_tokens, H, kc); return;
    case 16: launch_pdl(topk_gates_thread_kernel<16>, dim3(tb), dim3(128), 0, st, part, ks, br, logits, idx, w, n_tokens, H, kc); return;
    case 32: launch_pdl(topk_gates_thread_kernel<32>, dim3(tb), dim3(128), 0, st, part, ks, br, logits, idx, w, n_tokens, H, kc); return;
    default: break;
  }
  const int per_warp = Ec <= 8 ? 4 : (Ec <= 16 ? 2 : 1);
  const int warps = (tasks + per_warp - 1) / per_warp;
  launch_pdl(topk_gates_kernel, dim3((warps * 32 + 255) / 256), dim3(256), 0, st, part, ks, br, logits, idx, w, n_tokens, H, Ec, kc);
}

// the partial scores of all splits ([ks][n_tokens][E] floats) must fit the buffer they go to
int clamp_k_splits(int ks, int n_tokens, int E, size_t part_cap) {
  while (ks > 1 && size_t(ks) * size_t(n_tokens) * size_t(E) > part_cap) ks >>= 1;
  return ks;
}

int route_k_splits(int n_tokens, int d, int E, int n_sms) {
  const int ctas = ((n_tokens + kRgTM - 1) / kRgTM) * ((E + kRgTN - 1) / kRgTN);
  int ks = 1;
  while (ctas * ks < 2 * n_sms && ks < 16 && (d / (ks * 2)) % kRgKC == 0 && d / (ks * 2) >= 64) ks *= 2;
  return ks;
}

int launch_route(const void* r_in, int r_is_bf16, const bf16* gain, const float* wr, const CUtensorMap* tm_wr_split,
                 const float* br, bf16* u_out, float* inv_rms, float* part, size_t part_cap, float* logits, int* idx,
                 float* w, int n_tokens, int d, int H, int Ec, int kc, float eps, int n_sms, int* status, cudaStream_t st) {
  if (n_tokens <= 0) return 0;
  const int E = H * Ec;
  const dim3 ngrid((n_tokens * 32 + 255) / 256);
  const float* rf = static_cast<const float*>(r_in);
  if (!r_is_bf16 && d == 1024) launch_pdl(ffn_norm_f32_kernel<8>, ngrid, dim3(256), 0, st, rf, gain, u_out, inv_rms, n_tokens, eps);
  else if (!r_is_bf16 && d == 2048) launch_pdl(ffn_norm_f32_kernel<16>, ngrid, dim3(256), 0, st, rf, gain, u_out, inv_rms, n_tokens, eps);
  else launch_pdl(ffn_norm_kernel, ngrid, dim3(256), 0, st, r_in, r_is_bf16, gain, u_out, inv_rms, n_tokens, d, eps);
  int ks = 1;
  if (tm_wr_split && n_tokens >= kRouterTcMinTokens) {
    launch_router_tc(*tm_wr_split, r_in, r_is_bf16, inv_rms, part, n_tokens, d, E, status, st);
  } else {
    ks = clamp_k_splits(route_k_splits(n_tokens, d, E, n_sms), n_tokens, E, part_cap);
    dim3 grid((n_tokens + kRgTM - 1) / kRgTM, (E + kRgTN - 1) / kRgTN, ks);
    launch_pdl(router_gemm_kernel, grid, dim3(kRgThreads), 0, st, r_in, r_is_bf16, inv_rms, gain, wr, part, n_tokens, d, E, d / ks);
  }
  launch_topk_gates(part, ks, br, logits, idx, w, n_tokens, H, Ec, kc, st);
  return 3;
}


// ================================================================================================
// Routing without any allocation.
//
// Some callers of this library cannot allocate device memory at all: a serving process that handed the whole
// GPU to its own memory pool when it started (cudaMalloc would fail or steal from that pool), or a thread on a
// latency-critical path that must not take the driver's allocation lock nor run into the device-wide
// synchronisation that freeing memory implies.  foe_layer_create allocates, so those callers cannot even own a
// handle.  For them the routing step is offered on a fixed scratch area that lives inside the library image:
// the array below is part of every GPU's copy of the module from load until the process exits (about 6 MB).
// The array's name is only a host-side stand-in; the device address is looked up once per device with
// cudaGetSymbolAddress and handed to the same kernels the handle-based path runs.
// ================================================================================================
constexpr size_t kNaMaxTokens = 8192;                 // inv_rms entries
constexpr size_t kNaMaxScores = size_t(1) << 19;      // n_tokens * n_experts of one call
constexpr size_t kNaMaxPartial = size_t(1) << 20;     // split-K partial scores
constexpr int kNaMaxDevices = 64;

static __device__ __align__(256) float g_route_scratch[kNaMaxTokens + kNaMaxScores + kNaMaxPartial];

// Device address of the array and SM count, per device.  Host threads may make their first calls at the same time:
// each resolves the same two values, stores the SM count first and then publishes the address with release order, so a
// thread that sees a non-null address also sees the SM count.
static std::atomic<float*> g_route_scratch_dev[kNaMaxDevices];
static std::atomic<int> g_route_sms[kNaMaxDevices];

// inv_rms only: the expert input u is not produced on this path (the caller asked for routing, nothing else)
__global__ void ffn_inv_rms_bf16_kernel(const bf16* __restrict__ r_in, float* __restrict__ inv_out, int n_tokens, int d,
                                        float eps) {
  pdl_wait();
  pdl_launch_dependents();
  const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (i >= n_tokens) return;
  const uint4* row = reinterpret_cast<const uint4*>(r_in + size_t(i) * d);
  float ss = 0.f;
  for (int c = lane; c < d / 8; c += 32) {
    const uint4 q = __ldg(row + c);
    const uint32_t v[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) { const float a = bf16_lo(v[j]), b = bf16_hi(v[j]); ss += a * a + b * b; }
  }
  ss = warp_sum(ss);
  if (lane == 0) inv_out[i] = rsqrtf(ss / float(d) + eps);
}

// Returns 0 on success, -3 when the sizes exceed the fixed scratch, -6 on a CUDA error.  Calls nothing that
// allocates.  The first call on a device resolves the scratch address (and reads the SM count).
int launch_route_noalloc(const bf16* h, const bf16* gain, const float* wr, const float* br, int* idx, float* w,
                         int n_tokens, int d, int H, int Ec, int kc, float eps, cudaStream_t st) {
  const int E = H * Ec;
  if (size_t(n_tokens) > kNaMaxTokens || size_t(n_tokens) * E > kNaMaxScores) return -3;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNaMaxDevices) return -6;
  float* inv = g_route_scratch_dev[dev].load(std::memory_order_acquire);
  if (!inv) {
    float* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_route_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return -6;
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return -6;
    g_route_sms[dev].store(sms, std::memory_order_relaxed);
    g_route_scratch_dev[dev].store(p, std::memory_order_release);
    inv = p;
  }
  float* logits = inv + kNaMaxTokens;
  float* part = logits + kNaMaxScores;
  if (n_tokens <= 0) return 0;
  // Nothing in the scratch has to start at zero: every entry that is read below is written first by this call.
  ffn_inv_rms_bf16_kernel<<<(n_tokens * 32 + 255) / 256, 256, 0, st>>>(h, inv, n_tokens, d, eps);
  const int ks = clamp_k_splits(route_k_splits(n_tokens, d, E, g_route_sms[dev].load(std::memory_order_relaxed)), n_tokens, E, kNaMaxPartial);
  dim3 grid((n_tokens + kRgTM - 1) / kRgTM, (E + kRgTN - 1) / kRgTN, ks);
  router_gemm_kernel<<<grid, kRgThreads, 0, st>>>(h, 1, inv, gain, wr, part, n_tokens, d, E, d / ks);
  launch_topk_gates(part, ks, br, logits, idx, w, n_tokens, H, Ec, kc, st);
  return cudaGetLastError() == cudaSuccess ? 0 : -6;
}

}  // namespace foe
