// Router of the FoE block (Section 3.1 "Routing"): FFN RMSNorm, one fp32 score vector per token,
// per-cluster top-k inside the cluster's contiguous expert block, gates = softmax over the selected
// scores.  Everything on this path is fp32 on the plain ALUs: the decision it takes (which experts)
// is an integer result that must agree with a float32 reference, so no reduced-precision tensor path.
#include <float.h>

#include "common.cuh"
#include "kernels.h"

namespace foe {

constexpr int kRouteThreads = 256;

template <int TOK>
__global__ void __launch_bounds__(kRouteThreads)
route_kernel(const void* __restrict__ r_in, int r_is_bf16, const bf16* __restrict__ gain,
             const float* __restrict__ wr, const float* __restrict__ br, bf16* __restrict__ u_out,
             float* __restrict__ logits_out, int* __restrict__ idx_out, float* __restrict__ w_out, int n_tokens,
             int d, int H, int Ec, int kc, float eps) {
  extern __shared__ float smem_f[];
  float* u_s = smem_f;                       // [TOK][d]
  float* lg_s = u_s + size_t(TOK) * d;       // [TOK][E]
  const int E = H * Ec;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_warps = kRouteThreads / 32;
  const int tok0 = blockIdx.x * TOK;

  // ---- 1. FFN norm: u = r * rsqrt(mean r^2 + eps) * gain   (fp32, kept in shared memory)
  for (int t = warp; t < TOK; t += n_warps) {
    const int i = tok0 + t;
    float* urow = u_s + size_t(t) * d;
    if (i >= n_tokens) {
      for (int c = lane; c < d; c += 32) urow[c] = 0.f;
      continue;
    }
    float ss = 0.f;
    if (r_is_bf16) {
      const uint4* row = reinterpret_cast<const uint4*>(static_cast<const bf16*>(r_in) + size_t(i) * d);
      for (int c = lane; c < d / 8; c += 32) {
        const uint4 q = __ldg(row + c);
        const uint32_t v[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float a = bf16_lo(v[j]), b = bf16_hi(v[j]);
          urow[c * 8 + 2 * j] = a;
          urow[c * 8 + 2 * j + 1] = b;
          ss += a * a + b * b;
        }
      }
    } else {
      const float4* row = reinterpret_cast<const float4*>(static_cast<const float*>(r_in) + size_t(i) * d);
      for (int c = lane; c < d / 4; c += 32) {
        const float4 q = __ldg(row + c);
        *reinterpret_cast<float4*>(urow + c * 4) = q;
        ss += q.x * q.x + q.y * q.y + q.z * q.z + q.w * q.w;
      }
    }
    ss = warp_sum(ss);
    const float inv = rsqrtf(ss / float(d) + eps);
    __syncwarp();
    for (int c = lane; c < d / 8; c += 32) {
      const uint4 gq = __ldg(reinterpret_cast<const uint4*>(gain) + c);
      const uint32_t g[4] = {gq.x, gq.y, gq.z, gq.w};
      float v[8];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        v[2 * j] = urow[c * 8 + 2 * j] * inv * bf16_lo(g[j]);
        v[2 * j + 1] = urow[c * 8 + 2 * j + 1] * inv * bf16_hi(g[j]);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) urow[c * 8 + j] = v[j];
      if (u_out)
        *reinterpret_cast<uint4*>(u_out + size_t(i) * d + c * 8) =
            make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
    }
  }
  __syncthreads();

  // ---- 2. scores: register tile of 4 experts x 4 tokens per warp task, K split over the lanes
  const int e_groups = (E + 3) / 4, t_groups = TOK / 4;
  for (int task = warp; task < e_groups * t_groups; task += n_warps) {
    const int eg = task / t_groups, tg = task - eg * t_groups;
    const float* wrow[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) wrow[a] = wr + size_t(min(eg * 4 + a, E - 1)) * d;
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
    for (int k = lane * 4; k < d; k += 128) {
      float4 wv[4], uv[4];
#pragma unroll
      for (int a = 0; a < 4; ++a) wv[a] = __ldg(reinterpret_cast<const float4*>(wrow[a] + k));
#pragma unroll
      for (int b = 0; b < 4; ++b) uv[b] = *reinterpret_cast<const float4*>(u_s + size_t(tg * 4 + b) * d + k);
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          acc[a][b] = fmaf(wv[a].x, uv[b].x, acc[a][b]);
          acc[a][b] = fmaf(wv[a].y, uv[b].y, acc[a][b]);
          acc[a][b] = fmaf(wv[a].z, uv[b].z, acc[a][b]);
          acc[a][b] = fmaf(wv[a].w, uv[b].w, acc[a][b]);
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
      for (int b = 0; b < 4; ++b) acc[a][b] = warp_sum(acc[a][b]);
    if (lane < 16) {
      const int a = lane >> 2, b = lane & 3;
      const int e = eg * 4 + a, t = tg * 4 + b;
      float v = 0.f;
#pragma unroll
      for (int aa = 0; aa < 4; ++aa)
#pragma unroll
        for (int bb = 0; bb < 4; ++bb)
          if (aa == a && bb == b) v = acc[aa][bb];
      if (e < E) {
        if (br) v += __ldg(br + e);
        lg_s[t * E + e] = v;
        if (logits_out && tok0 + t < n_tokens) logits_out[size_t(tok0 + t) * E + e] = v;
      }
    }
  }
  __syncthreads();

  // ---- 3. per (token, cluster): top-k_c by (score descending, expert id ascending), then gates
  for (int task = warp; task < TOK * H; task += n_warps) {
    const int t = task / H, h = task - t * H;
    const int i = tok0 + t;
    if (i >= n_tokens) continue;
    const float* lg = lg_s + t * E + h * Ec;
    float cand[4];
    bool taken[4];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const int e = lane + 32 * s;
      cand[s] = e < Ec ? lg[e] : -FLT_MAX;
      taken[s] = e >= Ec;
    }
    float my_sel = -FLT_MAX;      // lane j keeps the j-th selected score
    int my_idx = 0;
    for (int j = 0; j < kc; ++j) {
      float bv = -FLT_MAX;
      int bi = 0x7fffffff;
#pragma unroll
      for (int s = 0; s < 4; ++s) {
        const int e = lane + 32 * s;
        if (!taken[s] && (bi == 0x7fffffff || cand[s] > bv)) { bv = cand[s]; bi = e; }   // ascending e: first wins ties
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (oi != 0x7fffffff && (bi == 0x7fffffff || ov > bv || (ov == bv && oi < bi))) { bv = ov; bi = oi; }
      }
      if ((bi & 31) == lane) {
#pragma unroll
        for (int s = 0; s < 4; ++s)
          if ((bi >> 5) == s) taken[s] = true;
      }
      if (lane == j) { my_sel = bv; my_idx = bi; }
    }
    const float m = __shfl_sync(0xffffffffu, my_sel, 0);
    const float ex = lane < kc ? expf(my_sel - m) : 0.f;
    const float sum = warp_sum(ex);
    if (lane < kc) {
      const size_t o = (size_t(i) * H + h) * kc + lane;
      idx_out[o] = h * Ec + my_idx;
      w_out[o] = ex / sum;
    }
  }
}

void launch_route(const void* r_in, int r_is_bf16, const bf16* gain, const float* wr, const float* br, bf16* u_out,
                  float* logits, int* idx, float* w, int n_tokens, int d, int H, int Ec, int kc, float eps,
                  cudaStream_t st) {
  if (n_tokens <= 0) return;
  const int E = H * Ec;
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(route_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    cudaFuncSetAttribute(route_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    cudaFuncSetAttribute(route_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    configured = true;
  }
  int tok = 16;
  while (tok > 4 && size_t(tok) * (d + E) * 4 > 160 * 1024) tok >>= 1;
  const size_t smem = size_t(tok) * (d + E) * 4;
  const int blocks = (n_tokens + tok - 1) / tok;
  if (tok == 16)
    route_kernel<16><<<blocks, kRouteThreads, smem, st>>>(r_in, r_is_bf16, gain, wr, br, u_out, logits, idx, w,
                                                         n_tokens, d, H, Ec, kc, eps);
  else if (tok == 8)
    route_kernel<8><<<blocks, kRouteThreads, smem, st>>>(r_in, r_is_bf16, gain, wr, br, u_out, logits, idx, w,
                                                        n_tokens, d, H, Ec, kc, eps);
  else
    route_kernel<4><<<blocks, kRouteThreads, smem, st>>>(r_in, r_is_bf16, gain, wr, br, u_out, logits, idx, w,
                                                        n_tokens, d, H, Ec, kc, eps);
}

}  // namespace foe
