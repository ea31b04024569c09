// Weight-streaming grouped GEMM for a handful of activation rows per group (the decode regime).
//
//   C_g[m, n] = sum_k X[row_g(m), k] * W_g[n, k]
//
// Every weight byte is used by ~8 rows, so the step is bound by HBM bandwidth, not by the tensor cores:
// the job is to read each touched weight exactly once and to keep enough bytes in flight.  One CTA owns a
// slab of 64 weight rows of one group and walks K in steps of 128.  A producer warp streams the slab
// through a ring of shared-memory stages with TMA (64- or 32-row boxes of 64 bf16, 128-byte swizzle,
// completion on an mbarrier), so the depth of the memory pipeline does not cost registers; next to every
// weight tile its lanes bulk-copy the matching 256-byte slice of each activation row (gathered through
// the dispatch map), so the consumers never wait on a global load.  Four consumer warps own 16 weight
// rows each; the weight rows are the M side of mma.sync m16n8k16 and 8 tokens the N side.  Both operands
// use the same permutation of k inside a 16-wide step, so that one 16-byte shared-memory load per operand
// feeds two MMAs directly.  Groups with no rows exit at once: only touched experts are read.
#include "common.cuh"
#include "kernels.h"

namespace foe {

constexpr int kSmConsumers = 4;
constexpr int kSmThreads = (kSmConsumers + 1) * 32;
constexpr int kSmSlab = 64;                     // weight rows per CTA
constexpr int kSmKStep = 128;                   // k per stage
constexpr int kSmNT = 2;                        // 8-token MMA tiles per pass
constexpr int kSmRows = kSmNT * 8;              // activation rows per pass
constexpr int kSmWBytes = kSmSlab * kSmKStep * 2;        // 16 KB of weights per stage
constexpr int kSmXPitch = kSmKStep * 2 + 16;             // padded activation row (bank spread)
constexpr int kSmStageBytes = ((kSmWBytes + kSmRows * kSmXPitch + 1023) / 1024) * 1024;
constexpr int kSmStages = 5;
constexpr size_t kSmSmemBytes = size_t(kSmStages) * kSmStageBytes + 1024 + 128;

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(gsrc)), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

template <int EPI>
__global__ void __launch_bounds__(kSmThreads)
smallm_kernel(const __grid_constant__ CUtensorMap tmW, const SmallMArgs a) {
  constexpr int NT = kSmNT;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kSmStages * kSmStageBytes);
  uint64_t* empty = full + kSmStages;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int slabs_per_group = a.N / kSmSlab;
  const int group = blockIdx.x / slabs_per_group;
  const int slab = blockIdx.x - group * slabs_per_group;

  // rows of this CTA: a ragged group takes all its rows (in passes of 16); a uniform group is cut into
  // 16-row chunks over blockIdx.y so that the few CTAs of a small projection still spread over the GPU
  int row_begin, rows, out_row0;
  if (a.group_offsets) {
    row_begin = a.group_offsets[group];
    rows = a.group_offsets[group + 1] - row_begin;
    out_row0 = row_begin;
  } else {
    const int r0 = blockIdx.y * kSmRows;
    row_begin = group * a.x_group_stride + r0;
    rows = min(kSmRows, a.rows_per_group - r0);
    out_row0 = r0;
  }
  if (rows <= 0) return;                                      // untouched group: its weights are never read

  if (threadIdx.x == 0) {
    for (int s = 0; s < kSmStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kSmConsumers); }
    mbar_fence_init();
  }
  __syncthreads();

  const int k_steps = a.K / kSmKStep;
  const int passes = (rows + kSmRows - 1) / kSmRows;
  const int total = passes * k_steps;

  // first weight row of the slab inside the [n_groups * N][K] matrix.  SwiGLU slabs are 32 gate rows and
  // their 32 up rows (128 rows further in the packed layout), everything else 64 consecutive rows.
  int wrow0;
  if (EPI == kEpiSwiGLU) {
    const int i0 = slab * 32;
    wrow0 = group * a.N + (i0 >> 7) * 256 + (i0 & 127);
  } else {
    wrow0 = group * a.N + slab * kSmSlab;
  }

  if (warp == kSmConsumers) {
    // ---------------------------------------------------------------- producer warp
    // lane 0 arms the barrier and issues the weight boxes; lane r copies the 256-byte k-slice of activation
    // row r (gathered through row_index) next to them.
    bool ok = true;
    const bf16* xsrc = nullptr;
    int cur_pass = -1, rows_pass = 0;
    for (int it = 0; it < total; ++it) {
      const int s = it % kSmStages;
      const uint32_t ph = (it / kSmStages) & 1;
      const int pass = it / k_steps, ks = it - pass * k_steps;
      if (pass != cur_pass) {
        cur_pass = pass;
        rows_pass = min(kSmRows, rows - pass * kSmRows);
        if (lane < rows_pass) {
          int xrow = row_begin + pass * kSmRows + lane;
          if (a.row_index) xrow = a.row_index[xrow];
          xsrc = a.X + size_t(xrow) * a.ldx;
        }
      }
      if (lane == 0) ok = mbar_wait(&empty[s], ph ^ 1);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      uint8_t* dst = smem + s * kSmStageBytes;
      if (lane == 0) {
        mbar_expect_tx(&full[s], kSmWBytes + rows_pass * (kSmKStep * 2));
        const int k0 = ks * kSmKStep;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (EPI == kEpiSwiGLU) {
            tma_load_2d(dst + h * 8192, &tmW, &full[s], k0 + h * 64, wrow0);
            tma_load_2d(dst + h * 8192 + 4096, &tmW, &full[s], k0 + h * 64, wrow0 + 128);
          } else {
            tma_load_2d(dst + h * 8192, &tmW, &full[s], k0 + h * 64, wrow0);
          }
        }
      }
      __syncwarp();
      if (lane < rows_pass) bulk_load(dst + kSmWBytes + lane * kSmXPitch, xsrc + ks * kSmKStep, kSmKStep * 2, &full[s]);
    }
    if (!ok && lane == 0) atomicExch(a.status, kStatusTimeout);
    return;
  }

  // ------------------------------------------------------------------ consumers
  const int g = lane >> 2, t4 = lane & 3;
  // shared-memory rows of the two weight rows this thread feeds (MMA rows g and g+8)
  const int sr_a = (EPI == kEpiSwiGLU) ? warp * 8 + g : warp * 16 + g;
  const int sr_b = (EPI == kEpiSwiGLU) ? 32 + warp * 8 + g : warp * 16 + g + 8;
  // global output columns of those rows
  const int n_a = (EPI == kEpiSwiGLU) ? slab * 32 + warp * 8 + g : slab * kSmSlab + warp * 16 + g;
  const int n_b = (EPI == kEpiSwiGLU) ? n_a : n_a + 8;
  const uint32_t sw_a = uint32_t(sr_a * 128), sx_a = uint32_t(sr_a & 7);
  const uint32_t sw_b = uint32_t(sr_b * 128), sx_b = uint32_t(sr_b & 7);
  const uint32_t smem_base = smem_u32(smem);
  bool ok = true;
  int it = 0;

  auto lds128 = [](uint32_t addr) -> uint4 {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
  };

  for (int pass = 0; pass < passes && ok; ++pass) {
    const int m0 = pass * kSmRows;
    float c[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f; }

    for (int ks = 0; ks < k_steps; ++ks, ++it) {
      const int s = it % kSmStages;
      const uint32_t ph = (it / kSmStages) & 1;
      const uint32_t st_base = smem_base + s * kSmStageBytes;
      if (!mbar_wait(&full[s], ph)) { ok = false; break; }
#pragma unroll
      for (int h = 0; h < 2; ++h) {                          // two 64-wide halves of the k step
        const uint32_t hb = st_base + h * 8192;
        const uint4 wa0 = lds128(hb + sw_a + ((uint32_t(t4) ^ sx_a) << 4));      // chunks t4 and t4+4
        const uint4 wa1 = lds128(hb + sw_a + ((uint32_t(t4 + 4) ^ sx_a) << 4));
        const uint4 wb0 = lds128(hb + sw_b + ((uint32_t(t4) ^ sx_b) << 4));
        const uint4 wb1 = lds128(hb + sw_b + ((uint32_t(t4 + 4) ^ sx_b) << 4));
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          if (m0 + nt * 8 < rows) {                          // warp-uniform
            const uint32_t xb = st_base + kSmWBytes + (nt * 8 + g) * kSmXPitch + h * 128 + t4 * 16;
            const uint4 x0 = lds128(xb), x1 = lds128(xb + 64);
            { const uint32_t f[4] = {wa0.x, wb0.x, wa0.y, wb0.y}; mma_bf16_16816(c[nt], f, x0.x, x0.y); }
            { const uint32_t f[4] = {wa0.z, wb0.z, wa0.w, wb0.w}; mma_bf16_16816(c[nt], f, x0.z, x0.w); }
            { const uint32_t f[4] = {wa1.x, wb1.x, wa1.y, wb1.y}; mma_bf16_16816(c[nt], f, x1.x, x1.y); }
            { const uint32_t f[4] = {wa1.z, wb1.z, wa1.w, wb1.w}; mma_bf16_16816(c[nt], f, x1.z, x1.w); }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);
    }
    if (!ok) break;

    // epilogue: c[nt][0..1] = (weight row A, tokens 2*t4, 2*t4+1), c[nt][2..3] = (weight row B, same tokens)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int r = m0 + nt * 8 + t4 * 2 + e;              // logical row inside the group
        if (r >= rows) continue;
        const float va = c[nt][e], vb = c[nt][2 + e];
        if (EPI == kEpiSwiGLU) {
          const float h = va / (1.0f + __expf(-va)) * vb;
          static_cast<bf16*>(a.out)[size_t(out_row0 + r) * a.ldo + n_a] = __float2bfloat16_rn(h);
        } else if (EPI == kEpiBf16) {
          bf16* o = static_cast<bf16*>(a.out) + size_t(out_row0 + r) * a.ldo;
          o[n_a] = __float2bfloat16_rn(va);
          o[n_b] = __float2bfloat16_rn(vb);
        } else if (EPI == kEpiQKV) {
          const float sc = a.row_scale[size_t(group) * a.scale_group_stride + out_row0 + r];
          bf16* o = static_cast<bf16*>(a.out) + size_t(out_row0 + r) * a.ldo;
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
            const bf16* xs = a.xsum + h * a.x_stride + size_t(out_row0 + r) * a.ldo;
            sa += __bfloat162float(xs[n_a]);
            sb += __bfloat162float(xs[n_b]);
          }
          float* o = static_cast<float*>(a.out) + size_t(out_row0 + r) * a.ldo;
          o[n_a] = sa * a.out_scale;
          o[n_b] = sb * a.out_scale;
        }
      }
    }
  }
  if (!ok && lane == 0) atomicExch(a.status, kStatusTimeout);
}

template <int EPI>
static void launch_one(const CUtensorMap& tmW, const SmallMArgs& a, cudaStream_t st) {
  static bool configured = false;
  if (!configured) {
    cudaFuncSetAttribute(smallm_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kSmSmemBytes));
    configured = true;
  }
  const int blocks = a.n_groups * (a.N / kSmSlab);
  if (blocks <= 0) return;
  const int chunks = a.group_offsets ? 1 : (a.rows_per_group + kSmRows - 1) / kSmRows;
  if (chunks <= 0) return;
  smallm_kernel<EPI><<<dim3(blocks, chunks), kSmThreads, kSmSmemBytes, st>>>(tmW, a);
}

void launch_smallm(const CUtensorMap& tmW, const SmallMArgs& a, cudaStream_t st) {
  switch (a.epi) {
    case kEpiSwiGLU: launch_one<kEpiSwiGLU>(tmW, a, st); break;
    case kEpiBf16: launch_one<kEpiBf16>(tmW, a, st); break;
    case kEpiQKV: launch_one<kEpiQKV>(tmW, a, st); break;
    default: launch_one<kEpiOProj>(tmW, a, st); break;
  }
}

}  // namespace foe
