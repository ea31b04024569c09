// Host-callable launchers of the FoE kernels (internal to the library).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gemm_args.h"

namespace foe {

typedef __nv_bfloat16 bf16;

// Launch with programmatic stream serialization: the kernel may be scheduled while its predecessor in the stream is
// still running and must call pdl_wait() before it touches anything the predecessor wrote (everything older is complete
// by then, because every kernel of the library triggers its successor only after its own wait).
// It pays for calls made of short kernels (a decode step: -6 % of the step, a 1024-token block: -8 %) and costs a
// little when a kernel's CTAs sit resident beside a predecessor that runs for hundreds of microseconds (a 16k-token
// prefill with the attribute on every launch: +0.7 %), so the API layer switches it per call and, inside large calls,
// per launch (this flag, per host thread).
inline thread_local bool g_overlap_launches = true;
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = g_overlap_launches ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- elementwise.cu
// inv_rms[r] = rsqrt(mean(x[r,:]^2) + eps) for n_rows rows of d bf16 values
void launch_row_inv_rms(const bf16* x, float* inv_rms, int n_rows, int d, float eps, cudaStream_t st);
// the same for x = [H][S][d], plus xsum[s][:] = sum_h x[h][s][:] in fp32; false (nothing launched) unless 2 <= H <= 8
bool launch_row_inv_rms_xsum(const bf16* x, float* inv_rms, float* xsum, int S, int d, int H, float eps, cudaStream_t st);
// per-token position / sequence / cache slot from q_lens and context_lens (device arrays); positions outside
// [0, max_context), a q_len above max_q_len or sum(q_lens) != n_tokens set the bounds status (slot -1, position clamped)
// returns the number of kernels launched
int launch_token_map(const int* q_lens, const int* context_lens, const int* block_table, int n_seqs,
                      int max_pages_per_seq, int num_pages, int page_size, int n_tokens, int max_context, int max_q_len,
                      int* cu_q, int* tok_seq, int* tok_pos, int* tok_slot, int* status, cudaStream_t st);
void launch_add_to_ints(int* v, int n, int by, cudaStream_t st);
// combine: out = r_full + sum_j w * y[inv]  (per cluster), optional mean over clusters
void launch_combine(const float* r_full, const bf16* y, const float* w, const int* inv, bf16* out, int n_tokens,
                    int d, int H, int kc, int last_mean, cudaStream_t st);
// weight repacks (create time)
void launch_transpose_batched(const bf16* src, size_t src_batch, int src_ld, bf16* dst, size_t dst_batch, int dst_ld,
                              int K, int N, int batch, const bf16* gain, int interleave_dh, cudaStream_t st);
void launch_pack_gate_up(const bf16* wg, const bf16* wu, bf16* dst, int E, int d, int I, cudaStream_t st);

// ---- route.cu
// FFN norm + fp32 router + per-cluster top-k + gates.  r_in is fp32 or bf16 [S][d].
// Returns the number of kernels launched.  inv_rms: [S] scratch; part: scratch of part_cap floats (at least S*E) for the
// split-K partial scores [k_splits][S][E]; the number of splits is reduced until they fit.
// tm_wr_split: map of the split router weights (launch_split_router_weights; box 64 x 64), or null: plain-ALU scores
// at every size.
constexpr int kRouterTcMinTokens = 2048;
constexpr int kRouterChunk = 64;              // experts per CTA of the tensor-core score kernel
inline int router_padded_experts(int E) { return (E + kRouterChunk - 1) / kRouterChunk * kRouterChunk; }
int launch_route(const void* r_in, int r_is_bf16, const bf16* gain, const float* wr, const CUtensorMap* tm_wr_split,
                 const float* br, bf16* u_out, float* inv_rms, float* part, size_t part_cap, float* logits, int* idx,
                 float* w, int n_tokens, int d, int H, int Ec, int kc, float eps, int n_sms, int* status, cudaStream_t st);
// split-K factors the two score kernels would like for a call (before the clamp to the partial-score buffer) and the clamp
int route_k_splits(int n_tokens, int d, int E, int n_sms);
int route_small_k_splits(int d);
int clamp_k_splits(int ks, int n_tokens, int E, size_t part_cap);
// planes: [3][router_padded_experts(E)][d] bf16 terms of gain * W
void launch_split_router_weights(const float* wr, const bf16* gain, bf16* planes, int E, int d, cudaStream_t st);
void launch_router_tc(const CUtensorMap& tmW, const void* r, int r_is_bf16, const float* inv_rms, float* part,
                      int n_tokens, int d, int E, int* status, cudaStream_t st);

// Calls of at most kRouteSmallMaxTokens tokens: FFN norm + scores in one launch, top-k + gates + dispatch maps in a
// second one (launch_route followed by launch_permute give the same results in up to six).
constexpr int kRouteSmallMaxTokens = 256;
struct PermuteBuffers;
int launch_route_small(const void* r_in, int r_is_bf16, const bf16* gain, const float* wr, const float* br, bf16* u_out,
                       float* scores, size_t scores_cap, float* logits, int* idx, float* w, const PermuteBuffers& pb,
                       int n_tokens, int d, int H, int Ec, int kc, float eps, int* status, cudaStream_t st);
int launch_topk_permute_small(const float* scores, int k_splits, const float* bias, float* logits, int* idx, float* w,
                              const PermuteBuffers& pb, int n_tokens, int H, int Ec, int kc, int* status, cudaStream_t st);

// routing on the library's built-in scratch area (no allocation); 0, -3 (too large) or -6 (CUDA error)
int launch_route_noalloc(const bf16* h, const bf16* gain, const float* wr, const float* br, int* idx, float* w,
                         int n_tokens, int d, int H, int Ec, int kc, float eps, cudaStream_t st);

// ---- permute.cu
struct PermuteBuffers {
  int* counts;        // [E]
  int* offsets;       // [E+1]
  int* perm;          // [R]
  int* inv;           // [S*H*kc]
  int* rank;          // [S*H*kc] rank of the selection inside its token block
  int* blk_counts;    // [n_blocks][E]
  int* mt_group;      // [R/256 + E] tiles of 256 rows (one per CTA pair of the grouped GEMM): expert of each
  int* mt_row0;       //             and its first row
  int* n_mtiles;      // scalar
};
constexpr int kPermuteBlockTokens = 256;
// returns the number of kernels launched (1 for calls of at most 256 tokens, else 3)
int launch_permute(const int* idx, const PermuteBuffers& pb, int n_tokens, int sel_per_token, int E, int* status,
                   cudaStream_t st);

// ---- attention.cu
struct AttnArgs {
  const bf16* q;            // [S][n_q*dh] queries after RoPE
  bf16* out;                // [S][n_q*dh]
  const int* cu_q;          // [n_seqs+1]; nullptr in a decode step: sequence b's token is token b
  const int* context_lens;  // [n_seqs]
  const int* q_lens;        // [n_seqs] or nullptr (1 each)
  const int* block_table;   // [n_seqs][max_pages_per_seq]
  int n_seqs, max_pages_per_seq, num_pages;
  int n_tokens;             // tokens of the call (prefill)
  int n_q, n_kv, dh;        // dh: the real head_dim (64, 96 or 128); kernels are instantiated for 64 and 128 and read
                            // a 96-wide head zero-padded: q with a head stride of 128, K/V through the tensor maps
  int max_q_len;
  float scale_log2;         // log2(e) / sqrt(dh)
  int* status;
  // decode only
  float* part_o;            // [n_seqs][n_q][max_splits][dh] partial outputs of the segments of a (sequence, KV head) pair
  float* part_ml;           // [n_seqs][n_q][max_splits][2]
  int* split_done;          // [n_seqs][n_kv] segments finished so far (zero between calls)
  int max_splits;           // attn_decode_max_segments(max pages per sequence the layer was created for)
  int max_kv_pages;         // pages of a sequence the decode kernel looks at: min(block-table width, the layer's max_context / 64)
};
// tensor-core (tcgen05) prefill attention; tmQ maps the qkv buffer [S][(n_q+2n_kv)*dh] with 128-row boxes
void launch_attn_prefill_tc(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const AttnArgs& a,
                            cudaStream_t st);
void launch_attn_decode(const CUtensorMap& tmK, const CUtensorMap& tmV, const AttnArgs& a, int n_sms, cudaStream_t st);
int attn_decode_max_segments(int max_pages_per_seq);   // per (sequence, KV head): second-to-last extent of part_o / part_ml

// ---- gemm_tcgen05.cu
void launch_gemm(int epi, const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmArgs& args, int n_sms,
                 cudaStream_t st);
cudaError_t gemm_configure();   // opt in to the dynamic shared memory the kernels need
// The same for the other kernel families.  Kernel attributes belong to the device that is current when they are set, so
// every layer creation calls all of these (a process may create layers on several GPUs, from several host threads).
cudaError_t attn_decode_configure();
cudaError_t attn_prefill_configure();
cudaError_t router_tc_configure();
cudaError_t smallm_configure();
cudaError_t decode_proj_configure();

// ---- smallm.cu  (weight-streaming GEMMs for a handful of rows per group)
struct SmallMArgs {
  const bf16* W;            // [n_groups][N][K]  K contiguous
  const bf16* X;            // activation rows, K contiguous, row stride ldx
  int ldx;
  const int* row_index;     // optional gather: X row of logical row r is row_index[r]; nullptr = identity
  const int* group_offsets; // ragged: rows of group g are [off[g], off[g+1]); nullptr = uniform
  int n_groups;
  int rows_per_group;       // uniform
  int x_group_stride;       // uniform: first X row of group g = g * x_group_stride
  int N, K;
  int epi;                  // GemmEpilogue
  void* out; int ldo;
  float rms_eps;            // kEpiQKV: 1/rms of every activation row is computed from the staged rows themselves
  int q_cols, kv_cols, dh, n_kv;   // kEpiQKV: see GemmArgs (interleaved heads, RoPE, q -> out, k / v -> pages)
  int q_head_stride;
  const float2* rope_tab; const int* tok_pos; const int* tok_slot; bf16* k_pages; bf16* v_pages;
  const bf16* xsum; int x_count; size_t x_stride; float out_scale;
  int early_weights;        // kEpiBf16: the previous kernel writes X and nothing else this one reads, so the first weight
                            // tiles may be requested before waiting for it
  int* status;
};
// tmW: tensor map of W as [n_groups*N][K] with 64-column boxes of 64 rows (32 rows for the SwiGLU packing)
void launch_smallm(const CUtensorMap& tmW, const SmallMArgs& a, int n_sms, cudaStream_t st);

// ---- decode_proj.cu  (dense projections of a decode step on tcgen05, weights as the MMA's M operand)
struct DecodeProjArgs {
  int n_groups;
  int rows_per_group;       // tokens S (the same tokens for every group)
  int x_group_stride;       // activation row of (group g, token t) = g * x_group_stride + t
  int N, K;                 // weight rows per group (a multiple of 128), reduction length (a multiple of 64)
  int k_splits;             // set by the launcher: CTAs per cluster (1, 2, 4 or 8), each with its share of K
  int epi;                  // kEpiQKV or kEpiOProj
  int* status;
  void* out; int ldo;
  // kEpiQKV (see GemmArgs; 1/rms is computed from the staged activation rows)
  float rms_eps;
  int q_cols, kv_cols, dh, n_kv, q_head_stride;
  const float2* rope_tab; const int* tok_pos; const int* tok_slot; bf16* k_pages; bf16* v_pages;
  // kEpiQKV of a decode step (tok_pos == nullptr): token t is the one new token of sequence t; its position is
  // context_lens[t] and its cache slot comes from the block table, both looked up in the epilogue (no token-map kernel)
  const int* context_lens; const int* block_table; int max_pages_per_seq, num_pages, max_context;
  // kEpiOProj
  const bf16* xsum; int x_count; size_t x_stride; float out_scale;
  // kEpiOProj on one rank of a cluster-per-GPU group (push_span != 0, a multiple of the 128-row weight slab): the scaled
  // result goes as bf16 to the rank that owns its columns instead of `out` (see GemmArgs)
  bf16* push_base[8]; unsigned int* push_cnt[8]; int push_span; long long push_slot_off;
};
bool decode_proj_supported(int epi, int N, int K, int dh);
// tmW: the weights [n_groups * N][K] with 64-column boxes of 128 rows; tmX: the activations with 64 x 64 boxes
void launch_decode_proj(const CUtensorMap& tmW, const CUtensorMap& tmX, DecodeProjArgs a, int n_sms, cudaStream_t st);

// ---- shard.cu  (sync of a cluster-per-GPU group over peer memory)
// This rank's mappings of every rank's exchange buffer: receive slots ([2][H][S_cap][d/H] bf16), gather buffer
// ([2][S_cap][d] bf16), arrival counters of the slots (per exchange parity, source rank and block of kShardBlockRows
// rows, so that an owner can reduce a block of rows as soon as ITS partials have landed) and of the gather buffer ([H],
// one per owner, only ever growing).
struct ShardPeerTable {
  bf16* slots[8];
  bf16* gather[8];
  unsigned int* slot_cnt[8];      // slot_cnt[o]: on rank o, the counters [n_blocks] of THIS rank's pushes (parity 0; the
                                  // other parity's lie 8 * n_blocks further)
  unsigned int* gather_cnt[8];    // gather_cnt[p]: rank p's array of H counters (indexed by owner)
};
// src ([S][d] bf16 or fp32) * scale -> bf16 into this rank's slot on every owner; slot_off = element offset of that
// slot ((parity * H + rank) * S_cap * (d/H)); cnt_off = parity * 8 * n_blocks.  Adds rows * d/H to the counter of every
// block of rows on every owner.
void launch_shard_push(const void* src, int src_is_f32, float scale, int S, int d, int H, const ShardPeerTable& t,
                       long long slot_off, int cnt_off, cudaStream_t st);
// every block of 16 rows waits until the H counters of its row block (my_slot_cnt[h * n_blocks + block], this parity's)
// hold that block's rows * d/H, sums the H slots (my_slots = this parity's [H][S_cap][d/H]) and writes the bf16 result
// to gather[p] + gather_off + row * d + rank * d/H of every rank p; adds rows * d/H to gather_cnt[p][rank].
void launch_shard_reduce(const bf16* my_slots, const unsigned int* my_slot_cnt, int n_blocks, int S, size_t S_cap,
                         int d, int H, int rank, const ShardPeerTable& t, long long gather_off,
                         unsigned long long limit_ns, int* status, cudaStream_t st);
// waits until my_gather_cnt[0..H) reached `expect` and copies the [S][d] gathered tensor (my_gather = this parity's
// half) to dst_f32 and / or dst_bf16 (either may be null); zeroes this rank's own slot counters of the exchange
// (zero_cnt[0 .. zero_n)), which nobody reads any more and which the exchange after the next will count up again
void launch_shard_gather(const bf16* my_gather, const unsigned int* my_gather_cnt, unsigned int expect, int S, int d,
                         int H, float* dst_f32, bf16* dst_bf16, unsigned int* zero_cnt, int zero_n,
                         unsigned long long limit_ns, int* status, cudaStream_t st);

}  // namespace foe
