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
// ring depth: 5 stages of 21 KB, two CTAs per SM
template <int EPI> __host__ __device__ constexpr int sm_stages() { return 5; }
constexpr int kSmMaxGroups = 1024;              // ragged problems: experts of a layer
// stages | barriers + statistics scratch (512 B) | list of the groups that have rows (2 KB) ; + alignment slack
template <int EPI> constexpr size_t sm_smem_bytes() { return size_t(sm_stages<EPI>()) * kSmStageBytes + 1024 + 512 + kSmMaxGroups * 2; }

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(gsrc)), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

struct SmTask {
  int group, slab, row_begin, rows, out_row0;
};

// task t of the persistent loop -> (group, slab, rows).  A ragged group takes all its rows (in passes of 16);
// a uniform group is cut into 16-row chunks so that the few slabs of a small projection still spread out.
// Ragged problems number their tasks over the groups that HAVE rows only (`live`, built by every CTA when it starts):
// with a quarter of the experts touched, tasks numbered over all groups leave some CTAs with twice the work of others.
__device__ __forceinline__ SmTask sm_task(const SmallMArgs& a, int t, int slabs_per_group, int chunks, const uint16_t* live) {
  SmTask k;
  const int sc = slabs_per_group * chunks;
  k.group = t / sc;
  const int r = t - k.group * sc;
  if (a.group_offsets) k.group = live[k.group];
  k.slab = r / chunks;
  const int chunk = r - k.slab * chunks;
  if (a.group_offsets) {
    k.row_begin = a.group_offsets[k.group];
    k.rows = a.group_offsets[k.group + 1] - k.row_begin;
    k.out_row0 = k.row_begin;
  } else {
    const int r0 = chunk * kSmRows;
    k.row_begin = k.group * a.x_group_stride + r0;
    k.rows = min(kSmRows, a.rows_per_group - r0);
    k.out_row0 = r0;
  }
  return k;
}

template <int EPI>
__global__ void __launch_bounds__(kSmThreads)
smallm_kernel(const __grid_constant__ CUtensorMap tmW, const SmallMArgs a) {
  // (expert GEMM 2 of a step waits later: its producer first requests the weights of its first ring, see below)
  const bool early_weights = EPI == kEpiBf16 && a.early_weights != 0;
  if (!early_weights) {
    pdl_wait();
    pdl_launch_dependents();
  }
  constexpr int NT = kSmNT;
  constexpr int kSmStages = sm_stages<EPI>();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + kSmStages * kSmStageBytes);
  uint64_t* empty = full + kSmStages;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int slabs_per_group = (a.N + kSmSlab - 1) / kSmSlab;    // the last slab of a group may be partly past its rows
  const int chunks = a.group_offsets ? 1 : (a.rows_per_group + kSmRows - 1) / kSmRows;
  const int k_steps = a.K / kSmKStep;
  uint16_t* live = reinterpret_cast<uint16_t*>(smem + kSmStages * kSmStageBytes + 512);
  int* n_live_s = reinterpret_cast<int*>(smem + kSmStages * kSmStageBytes + 512 - 16);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kSmStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kSmConsumers); }
    mbar_fence_init();
  }
  if (a.group_offsets && warp == 0) {
    // the groups with rows, in ascending order (the offsets are complete: they are older than this kernel's
    // predecessor when it starts before its wait, see early_weights)
    int n = 0;
    for (int g0 = 0; g0 < a.n_groups; g0 += 32) {
      const int g = g0 + lane;
      const bool has = g < a.n_groups && a.group_offsets[g + 1] > a.group_offsets[g];
      const uint32_t m = __ballot_sync(0xffffffffu, has);
      if (has) live[n + __popc(m & ((1u << lane) - 1u))] = uint16_t(g);
      n += __popc(m);
    }
    if (lane == 0) *n_live_s = n;
  }
  __syncthreads();
  const int n_tasks = (a.group_offsets ? *n_live_s : a.n_groups) * slabs_per_group * chunks;

  // The CTA is persistent: it walks tasks blockIdx.x, blockIdx.x + gridDim.x, ... and the stage ring keeps
  // running across task boundaries, so the producer is already streaming the next slab while the consumers
  // finish the current one.  Tasks of groups without rows are skipped by both roles: untouched experts are
  // never read.
  if (warp == kSmConsumers) {
    // ---------------------------------------------------------------- producer warp
    // lane 0 arms the barrier and issues the weight boxes; lane r copies the 256-byte k-slice of activation
    // row r (gathered through row_index) next to them.
    bool ok = true;
    int it = 0;
    int pre = 0;                       // leading iterations whose barrier is armed and whose weights are on their way
    if (early_weights) {
      // The previous kernel (expert GEMM 1) writes this kernel's activations, nothing else it needs: the dispatch maps
      // are older and complete.  So the weight tiles of the first ring can be requested while that kernel drains.
      for (int t = blockIdx.x; t < n_tasks; t += gridDim.x) {
        const SmTask k = sm_task(a, t, slabs_per_group, chunks, live);
        if (k.rows <= 0) continue;
        if (lane == 0) {
          const int wrow0 = k.group * a.N + k.slab * kSmSlab;
          const int rows_pass = min(kSmRows, k.rows);
          pre = min(kSmStages, k_steps);
          for (int i = 0; i < pre; ++i) {
            mbar_expect_tx(&full[i], kSmWBytes + rows_pass * (kSmKStep * 2));
            tma_load_2d(smem + i * kSmStageBytes, &tmW, &full[i], i * kSmKStep, wrow0);
            tma_load_2d(smem + i * kSmStageBytes + 8192, &tmW, &full[i], i * kSmKStep + 64, wrow0);
          }
        }
        break;
      }
      pre = __shfl_sync(0xffffffffu, pre, 0);
      pdl_wait();
      pdl_launch_dependents();
    }
    for (int t = blockIdx.x; t < n_tasks && ok; t += gridDim.x) {
      const SmTask k = sm_task(a, t, slabs_per_group, chunks, live);
      if (k.rows <= 0) continue;
      // first weight row of the slab inside the [n_groups * N][K] matrix.  SwiGLU slabs are 32 gate rows and
      // their 32 up rows (128 rows further in the packed layout), everything else 64 consecutive rows.
      int wrow0;
      if (EPI == kEpiSwiGLU) {
        const int i0 = k.slab * 32;
        wrow0 = k.group * a.N + (i0 >> 7) * 256 + (i0 & 127);
      } else {
        wrow0 = k.group * a.N + k.slab * kSmSlab;
      }
      const int passes = (k.rows + kSmRows - 1) / kSmRows;
      for (int pass = 0; pass < passes && ok; ++pass) {
        const int rows_pass = min(kSmRows, k.rows - pass * kSmRows);
        const bf16* xsrc = nullptr;
        if (lane < rows_pass) {
          int xrow = k.row_begin + pass * kSmRows + lane;
          if (a.row_index) xrow = a.row_index[xrow];
          xsrc = a.X + size_t(xrow) * a.ldx;
        }
        for (int ks = 0; ks < k_steps; ++ks, ++it) {
          const int s = it % kSmStages;
          const uint32_t ph = (it / kSmStages) & 1;
          uint8_t* dst = smem + s * kSmStageBytes;
          if (it < pre) {              // armed and weights requested before the wait: only the activations are missing
            __syncwarp();
            if (lane < rows_pass) bulk_load(dst + kSmWBytes + lane * kSmXPitch, xsrc + ks * kSmKStep, kSmKStep * 2, &full[s]);
            continue;
          }
          if (lane == 0) ok = mbar_wait(&empty[s], ph ^ 1);
          ok = __shfl_sync(0xffffffffu, ok, 0);
          if (!ok) break;
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
      }
    }
    if (!ok && lane == 0) atomicExch(a.status, kStatusTimeout);
    return;
  }

  // ------------------------------------------------------------------ consumers
  if (early_weights) pdl_wait();
  const int g = lane >> 2, t4 = lane & 3;
  // shared-memory rows of the two weight rows this thread feeds (MMA rows g and g+8)
  // (QKV: heads are stored with their halves interleaved, so rows 2g and 2g+1 are the two members of a rotary pair)
  const int sr_a = (EPI == kEpiSwiGLU) ? warp * 8 + g : (EPI == kEpiQKV ? warp * 16 + 2 * g : warp * 16 + g);
  const int sr_b = (EPI == kEpiSwiGLU) ? 32 + warp * 8 + g : (EPI == kEpiQKV ? warp * 16 + 2 * g + 1 : warp * 16 + g + 8);
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

  for (int t = blockIdx.x; t < n_tasks && ok; t += gridDim.x) {
    const SmTask k = sm_task(a, t, slabs_per_group, chunks, live);
    if (k.rows <= 0) continue;
    const int group = k.group, rows = k.rows, out_row0 = k.out_row0;
    // global output columns of this thread's two weight rows
    const int n_a = (EPI == kEpiSwiGLU) ? k.slab * 32 + warp * 8 + g
                                        : (EPI == kEpiQKV ? k.slab * kSmSlab + warp * 16 + 2 * g : k.slab * kSmSlab + warp * 16 + g);
    const int n_b = (EPI == kEpiSwiGLU) ? n_a : (EPI == kEpiQKV ? n_a + 1 : n_a + 8);
    const int passes = (rows + kSmRows - 1) / kSmRows;

  for (int pass = 0; pass < passes && ok; ++pass) {
    const int m0 = pass * kSmRows;
    float c[NT][4];
    float ssq[NT];                        // sum of squares of activation row nt*8+g (QKV: fused RMS statistics)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f; ssq[nt] = 0.f; }

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
            if (EPI == kEpiQKV && (ks & 3) == warp) {        // each consumer warp covers a quarter of the k steps
              const uint32_t xs[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
              float s0 = 0.f, s1 = 0.f;
#pragma unroll
              for (int q = 0; q < 8; q += 2) {
                const float a0 = bf16_lo(xs[q]), a1 = bf16_hi(xs[q]), b0 = bf16_lo(xs[q + 1]), b1 = bf16_hi(xs[q + 1]);
                s0 = fmaf(a0, a0, fmaf(a1, a1, s0));
                s1 = fmaf(b0, b0, fmaf(b1, b1, s1));
              }
              ssq[nt] += s0 + s1;
            }
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
    if (EPI == kEpiQKV) {   // (also reached after a timed-out wait, so that the warps never miss each other at bar.sync)
      // the four lanes of a quad saw disjoint quarters of row nt*8+g and the four warps disjoint k steps: finish
      // the sum (quad shuffle, then across the consumer warps through shared memory) and turn it into 1/rms.
      // (rows past the end hold stale shared memory; their value is never used)
      float* red = reinterpret_cast<float*>(empty + kSmStages);          // [4 warps][NT * 8 rows]
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        float v = ssq[nt];
        v += __shfl_xor_sync(0xffffffffu, v, 1);
        v += __shfl_xor_sync(0xffffffffu, v, 2);
        if (t4 == 0) red[warp * (NT * 8) + nt * 8 + g] = v;
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");                       // the four consumer warps only
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const int r = nt * 8 + g;
        const float v = red[r] + red[NT * 8 + r] + red[2 * NT * 8 + r] + red[3 * NT * 8 + r];
        ssq[nt] = rsqrtf(v / float(a.K) + a.rms_eps);
      }
      asm volatile("bar.sync 1, 128;" ::: "memory");                       // red is reused by the next pass
    }
    if (!ok) break;

    // epilogue: c[nt][0..1] = (weight row A, tokens 2*t4, 2*t4+1), c[nt][2..3] = (weight row B, same tokens)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      // QKV: 1/rms of token row nt*8 + 2*t4 + e sits in the quad whose g equals that row index.  Fetched here by ALL
      // lanes: below, lanes whose row lies past the end of a ragged chunk skip the row, and a full-mask shuffle that
      // some lanes never reach leaves the others waiting for them -- forever once the skipping lanes have run on into
      // the next task's __syncwarp (a CTA with a second task and a last chunk of fewer than 16 tokens hung).
      float sc_e[2] = {1.f, 1.f};
      if (EPI == kEpiQKV) {
#pragma unroll
        for (int e = 0; e < 2; ++e) sc_e[e] = __shfl_sync(0xffffffffu, ssq[nt], (t4 * 2 + e) * 4);
      }
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int r = m0 + nt * 8 + t4 * 2 + e;              // logical row inside the group
        if (r >= rows) continue;
        const float va = c[nt][e], vb = c[nt][2 + e];
        if (EPI != kEpiSwiGLU && n_a >= a.N) continue;       // (both columns of a thread lie on the same side of the end)
        if (EPI == kEpiSwiGLU) {
          const float h = __fdividef(va, 1.0f + __expf(-va)) * vb;
          static_cast<bf16*>(a.out)[size_t(out_row0 + r) * a.ldo + n_a] = __float2bfloat16_rn(h);
        } else if (EPI == kEpiBf16) {
          bf16* o = static_cast<bf16*>(a.out) + size_t(out_row0 + r) * a.ldo;
          o[n_a] = __float2bfloat16_rn(va);
          o[n_b] = __float2bfloat16_rn(vb);
        } else if (EPI == kEpiQKV) {
          const float sc = sc_e[e];
          const int tok = out_row0 + r;
          // packed columns n_a = 2i and n_a + 1 of a head are its natural columns i and i + dh/2: one rotary pair
          const int i = (n_a % a.dh) >> 1, half = a.dh >> 1;
          float lo = va * sc, hi = vb * sc;
          const bool is_q = n_a < a.q_cols, is_k = !is_q && n_a < a.q_cols + a.kv_cols;
          if (is_q || is_k) {
            const float2 cs = __ldg(a.rope_tab + size_t(a.tok_pos[tok]) * half + i);
            const float x0 = lo, x1 = hi;
            lo = x0 * cs.x - x1 * cs.y;
            hi = x1 * cs.x + x0 * cs.y;
          }
          if (is_q) {
            const int head = group * (a.q_cols / a.dh) + n_a / a.dh;
            bf16* o = static_cast<bf16*>(a.out) + size_t(tok) * a.ldo + head * a.q_head_stride;
            o[i] = __float2bfloat16_rn(lo);
            o[i + half] = __float2bfloat16_rn(hi);
          } else {
            const int nn = n_a - a.q_cols - (is_k ? 0 : a.kv_cols);
            const int kvh = group * (a.kv_cols / a.dh) + nn / a.dh;
            const int slot = a.tok_slot[tok];
            if (slot >= 0) {
              bf16* o = (is_k ? a.k_pages : a.v_pages) + ((size_t(slot >> 6) * a.n_kv + kvh) * 64 + (slot & 63)) * a.dh;
              o[i] = __float2bfloat16_rn(lo);
              o[i + half] = __float2bfloat16_rn(hi);
            }
          }
        } else {  // kEpiOProj: r_full = scale * (C + sum_h x[h])
          float sa = va, sb = vb;
          bf16 xa[8], xb[8];
#pragma unroll
          for (int h = 0; h < 8; ++h) {                       // all loads first (up to 8 residual streams)
            xa[h] = __float2bfloat16_rn(0.f);
            xb[h] = xa[h];
            if (h < a.x_count) {
              const bf16* xs = a.xsum + h * a.x_stride + size_t(out_row0 + r) * a.ldo;
              xa[h] = xs[n_a];
              xb[h] = xs[n_b];
            }
          }
#pragma unroll
          for (int h = 0; h < 8; ++h) { sa += __bfloat162float(xa[h]); sb += __bfloat162float(xb[h]); }
          float* o = static_cast<float*>(a.out) + size_t(out_row0 + r) * a.ldo;
          o[n_a] = sa * a.out_scale;
          o[n_b] = sb * a.out_scale;
        }
      }
    }
  }
  }
  if (!ok && lane == 0) atomicExch(a.status, kStatusTimeout);
}


template <int EPI>
static void launch_one(const CUtensorMap& tmW, const SmallMArgs& a, int n_sms, cudaStream_t st) {
  const int chunks = a.group_offsets ? 1 : (a.rows_per_group + kSmRows - 1) / kSmRows;
  const long long tasks = (long long)a.n_groups * ((a.N + kSmSlab - 1) / kSmSlab) * chunks;
  if (tasks <= 0) return;
  const int grid = int(tasks < 2LL * n_sms ? tasks : 2LL * n_sms);          // two resident CTAs per SM
  launch_pdl(smallm_kernel<EPI>, dim3(grid), dim3(kSmThreads), sm_smem_bytes<EPI>(), st, tmW, a);
}

template <int EPI>
static cudaError_t configure_one() {
  return cudaFuncSetAttribute(smallm_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sm_smem_bytes<EPI>()));
}

cudaError_t smallm_configure() {
  cudaError_t e = configure_one<kEpiSwiGLU>();
  if (e == cudaSuccess) e = configure_one<kEpiBf16>();
  if (e == cudaSuccess) e = configure_one<kEpiQKV>();
  if (e == cudaSuccess) e = configure_one<kEpiOProj>();
  return e;
}

void launch_smallm(const CUtensorMap& tmW, const SmallMArgs& a, int n_sms, cudaStream_t st) {
  switch (a.epi) {
    case kEpiSwiGLU: launch_one<kEpiSwiGLU>(tmW, a, n_sms, st); break;
    case kEpiBf16: launch_one<kEpiBf16>(tmW, a, n_sms, st); break;
    case kEpiQKV: launch_one<kEpiQKV>(tmW, a, n_sms, st); break;
    default: launch_one<kEpiOProj>(tmW, a, n_sms, st); break;
  }
}

}  // namespace foe
