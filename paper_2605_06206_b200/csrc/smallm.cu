// Weight-streaming grouped GEMM for a handful of activation rows per group (the decode regime).
//
//   C_g[m, n] = sum_k X[row_g(m), k] * W_g[n, k]
//
// Here every weight byte is used by ~8 rows, so the step is bound by HBM bandwidth, not by the tensor
// cores: the job is to read each touched weight exactly once with full-width, fully used memory
// transactions and to keep enough loads in flight.  One warp owns 16 weight rows of one group and walks
// K; weights go HBM -> registers with 16-byte loads (two 64-byte runs per row per step, so every 128-byte
// line is consumed whole), activations come from L1/L2.  The multiply itself uses mma.sync m16n8k16 with
// the weight rows as the M side and 8 tokens as the N side; both operands use the same permutation of k
// inside each 16-wide step so that a thread's 16-byte load feeds its fragments directly.  Groups with no
// rows are never read ("touched experts only").
#include "common.cuh"
#include "kernels.h"

namespace foe {

constexpr int kSmWarps = 8;

template <int NT, int EPI>
__global__ void __launch_bounds__(kSmWarps * 32)
smallm_kernel(const SmallMArgs a) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t4 = lane & 3;
  const int tasks_per_group = a.N / 16;
  const long long task = (long long)blockIdx.x * kSmWarps + warp;
  if (task >= (long long)a.n_groups * tasks_per_group) return;
  const int group = int(task / tasks_per_group);
  const int tt = int(task - (long long)group * tasks_per_group);

  int row_begin, rows;
  if (a.group_offsets) { row_begin = a.group_offsets[group]; rows = a.group_offsets[group + 1] - row_begin; }
  else { row_begin = group * a.x_group_stride; rows = a.rows_per_group; }
  if (rows <= 0) return;

  // the two weight rows this thread feeds (MMA rows g and g+8)
  int n_a, n_b;
  if (EPI == kEpiSwiGLU) {
    const int i0 = tt * 8;                                   // 8 intermediate indices: gate rows + their up rows
    n_a = (i0 >> 7) * 256 + (i0 & 127) + g;
    n_b = n_a + 128;
  } else {
    n_a = tt * 16 + g;
    n_b = n_a + 8;
  }
  const uint4* wa = reinterpret_cast<const uint4*>(a.W + (size_t(group) * a.N + n_a) * a.K) + t4;
  const uint4* wb = reinterpret_cast<const uint4*>(a.W + (size_t(group) * a.N + n_b) * a.K) + t4;

  for (int m0 = 0; m0 < rows; m0 += NT * 8) {
    const uint4* xr[NT];
    bool xok[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int r = m0 + nt * 8 + g;
      xok[nt] = r < rows;
      int xrow = row_begin + (xok[nt] ? r : 0);
      if (a.row_index) xrow = a.row_index[xrow];
      xr[nt] = reinterpret_cast<const uint4*>(a.X + size_t(xrow) * a.ldx) + t4;
    }
    float c[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f; }

#pragma unroll 4
    for (int k8 = 0; k8 < a.K / 8; k8 += 8) {                // 64 k per step; index in 16-byte units
      const uint4 a0 = __ldg(wa + k8), a1 = __ldg(wa + k8 + 4);
      const uint4 b0 = __ldg(wb + k8), b1 = __ldg(wb + k8 + 4);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        if (m0 + nt * 8 < rows) {                            // warp-uniform
          uint4 x0 = make_uint4(0, 0, 0, 0), x1 = make_uint4(0, 0, 0, 0);
          if (xok[nt]) { x0 = __ldg(xr[nt] + k8); x1 = __ldg(xr[nt] + k8 + 4); }
          { const uint32_t f[4] = {a0.x, b0.x, a0.y, b0.y}; mma_bf16_16816(c[nt], f, x0.x, x0.y); }
          { const uint32_t f[4] = {a0.z, b0.z, a0.w, b0.w}; mma_bf16_16816(c[nt], f, x0.z, x0.w); }
          { const uint32_t f[4] = {a1.x, b1.x, a1.y, b1.y}; mma_bf16_16816(c[nt], f, x1.x, x1.y); }
          { const uint32_t f[4] = {a1.z, b1.z, a1.w, b1.w}; mma_bf16_16816(c[nt], f, x1.z, x1.w); }
        }
      }
    }

    // epilogue: c[nt][0..1] = (weight row g, tokens 2*t4, 2*t4+1), c[nt][2..3] = (weight row g+8, same tokens)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int r = m0 + nt * 8 + t4 * 2 + e;              // logical row inside the group
        if (r >= rows) continue;
        const float va = c[nt][e], vb = c[nt][2 + e];
        if (EPI == kEpiSwiGLU) {
          const float h = va / (1.0f + __expf(-va)) * vb;
          static_cast<bf16*>(a.out)[size_t(row_begin + r) * a.ldo + tt * 8 + g] = __float2bfloat16_rn(h);
        } else if (EPI == kEpiBf16) {
          bf16* o = static_cast<bf16*>(a.out) + size_t(row_begin + r) * a.ldo;
          o[n_a] = __float2bfloat16_rn(va);
          o[n_b] = __float2bfloat16_rn(vb);
        } else if (EPI == kEpiQKV) {
          const float sc = a.row_scale[size_t(group) * a.scale_group_stride + r];
          bf16* o = static_cast<bf16*>(a.out) + size_t(r) * a.ldo;
#pragma unroll
          for (int w = 0; w < 2; ++w) {
            const int n = w ? n_b : n_a;
            int col;
            if (n < a.q_cols) col = group * a.q_cols + n;
            else if (n < a.q_cols + a.kv_cols) col = a.q_total + group * a.kv_cols + (n - a.q_cols);
            else col = a.q_total + a.kv_total + group * a.kv_cols + (n - a.q_cols - a.kv_cols);
            o[col] = __float2bfloat16_rn((w ? vb : va) * sc);
          }
        } else {  // kEpiOProj: r_full = scale * (C + sum_h x[h])
          float sa = va, sb = vb;
          for (int h = 0; h < a.x_count; ++h) {
            const bf16* xs = a.xsum + h * a.x_stride + size_t(r) * a.ldo;
            sa += __bfloat162float(xs[n_a]);
            sb += __bfloat162float(xs[n_b]);
          }
          float* o = static_cast<float*>(a.out) + size_t(r) * a.ldo;
          o[n_a] = sa * a.out_scale;
          o[n_b] = sb * a.out_scale;
        }
      }
    }
  }
}

template <int NT>
static void launch_nt(const SmallMArgs& a, cudaStream_t st) {
  const long long tasks = (long long)a.n_groups * (a.N / 16);
  if (tasks <= 0) return;
  const unsigned blocks = unsigned((tasks + kSmWarps - 1) / kSmWarps);
  switch (a.epi) {
    case kEpiBf16: smallm_kernel<NT, kEpiBf16><<<blocks, kSmWarps * 32, 0, st>>>(a); break;
    case kEpiSwiGLU: smallm_kernel<NT, kEpiSwiGLU><<<blocks, kSmWarps * 32, 0, st>>>(a); break;
    case kEpiQKV: smallm_kernel<NT, kEpiQKV><<<blocks, kSmWarps * 32, 0, st>>>(a); break;
    default: smallm_kernel<NT, kEpiOProj><<<blocks, kSmWarps * 32, 0, st>>>(a); break;
  }
}

void launch_smallm(const SmallMArgs& a, cudaStream_t st) {
  // ragged groups (experts) see a handful of rows each: 4 n-tiles = 32 rows per pass; uniform groups
  // (projections over all sequences) use 8 n-tiles = 64 rows per pass.
  if (a.group_offsets) launch_nt<4>(a, st);
  else launch_nt<8>(a, st);
}

}  // namespace foe
