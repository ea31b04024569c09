// C ABI of the FoE block (see include/foe.h): argument checks, weight repacking, workspace, tensor maps and
// the launch sequences of prefill, decode and route.  No computation happens on the host.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>
#include <vector>

#include "../../include/foe.h"
#include "../../include/foe_shard.h"
#include "kernels.h"

using namespace foe;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// 2-D bf16 tensor [rows][cols] (cols contiguous), box [box_rows][64 cols], 128-byte swizzle.
bool make_map_2d(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  if (rows == 0) rows = 1;
  const cuuint64_t gdim[2] = {cols, rows};
  const cuuint64_t gstride[1] = {cols * 2};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

enum Stage { kStPrep = 0, kStQkv, kStAttn, kStOproj, kStRoute, kStPermute, kStGemm1, kStGemm2, kStCombine, kNumStages };
const char* kStageNames[kNumStages] = {"prep", "qkv_rope_kv_write", "attention", "o_proj_sync", "route",
                                       "permute", "expert_gemm1_swiglu", "expert_gemm2", "combine"};

}  // namespace

// Per-call scratch.  Layers of one stack run one after the other on a stream, so they can share one workspace
// (foe_layer_create_shared); it is freed with its last user.
struct foe_workspace {
  int refs;
  std::vector<void*> allocs;
  float *inv_rms, *inv_rms_f, *route_part, *r_full, *logits, *topk_w, *part_o, *part_ml;
  bf16 *qkv, *attn_o, *u, *hmid, *y;
  int *topk_idx, *cu_q, *tok_seq, *tok_pos, *tok_slot, *status, *split_done;
  size_t route_part_cap;                        // floats in route_part
  size_t split_done_count;                      // ints in split_done
  PermuteBuffers pb;
  CUtensorMap tm_attn_o, tm_hmid, tm_qkv;       // maps of workspace buffers (A operands, attention Q)
  CUtensorMap tm_attn_o64;                       // attention output with 64-row boxes (decode O-projection)
};

struct foe_layer {
  foe_config cfg;
  int H, g, c, dh, d, I, E, Ec, kc, n_q, n_kv, qkv_cols, S_max, R_max, n_sms;
  int dhp;               // head width the attention kernels work with: head_dim, or 128 for head_dim 96 (zero-padded)
  bool first, last;
  std::vector<void*> allocs;
  // repacked weights
  bf16 *wqkv_t, *wo_t, *wgu_t, *wd_t, *ffn_gain;
  float *router_w, *router_b;
  bf16* router_split;    // [3][E padded to 64][d]: bf16 terms of router weights x FFN-norm gain
  CUtensorMap tm_router;
  float2* rope_tab;
  foe_workspace* ws;
  int max_splits;
  // tensor maps of the weights
  CUtensorMap tm_wqkv, tm_wo, tm_wgu, tm_wd;       // weights; box = the rows of B one CTA of a pair stages per k-block
  CUtensorMap tms_wqkv, tms_wo, tms_wgu, tms_wd;   // same weights, boxes sized for the decode kernels
  CUtensorMap tmt_wqkv, tmt_wo;                    // 128-row boxes: slabs of the tensor-core decode projections
  bool dp_qkv, dp_oproj;                           // shapes those kernels take (else the weight-streaming kernels)
  // call state
  cudaStream_t last_stream;
  int last_tokens, launches;
  bool last_decode;
  int shard_stage;       // 0: no sharded call in flight; 1: foe_shard_attend done, foe_shard_ffn owed
  int profiling;                       // 0 off, else the number of recent calls whose stage events are kept
  std::vector<cudaEvent_t> ev;         // [profiling][kNumStages + 1]
  int prof_calls;                      // calls recorded since the times were last read
  bool ev_valid;
};

// One rank's end of the exchange of a cluster-per-GPU group.
struct foe_shard {
  foe_shard_config cfg;
  int span;                         // columns each rank owns
  size_t S_cap;
  uint8_t* buf[8];                  // every rank's exchange buffer as seen from here
  ShardPeerTable table;
  unsigned int epoch;               // exchanges started
  unsigned int gather_expect;       // running total the gather counters must reach for the current exchange
  int n_blk;                        // row blocks (of kShardBlockRows rows) that have slot counters
  int S;                            // tokens of the current exchange
  int stage;                        // 0 idle, 1 pushed, 2 reduced
  int* status;
  unsigned long long limit_ns;
  cudaStream_t last_stream;
};

namespace {

constexpr int kFewTokens = 256;                  // calls up to this size take the decode-step kernels where they fit
constexpr int kOverlapTokens = 2048;             // calls up to this size launch their kernels with programmatic dependent launch
// header of an exchange buffer: gather counters [8] at 0; slot counters [2 parities][8 sources][n_blk] from 128 on
int shard_blocks(const foe_shard_config* c) { return (c->max_tokens + kShardBlockRows - 1) / kShardBlockRows; }
size_t shard_header_bytes(const foe_shard_config* c) {
  return (128 + size_t(2) * 8 * shard_blocks(c) * sizeof(unsigned int) + 1023) / 1024 * 1024;
}

bool shard_config_ok(const foe_shard_config* c) {
  return c && c->n_ranks >= 1 && c->n_ranks <= 8 && c->rank >= 0 && c->rank < c->n_ranks && c->hidden > 0 &&
         c->hidden % (32 * c->n_ranks) == 0 && c->max_tokens > 0 && c->wait_limit_ms >= 0;
}
size_t shard_slots_bytes(const foe_shard_config* c) { return size_t(2) * c->max_tokens * c->hidden * sizeof(bf16); }

// floats of the split-K partial-score buffer of a workspace for calls of up to S tokens
size_t route_part_capacity(size_t S, size_t E) { return S * E > (size_t(1) << 21) ? S * E : (size_t(1) << 21); }

template <typename T>
bool dalloc(foe_layer* L, T** p, size_t count) {
  void* q = nullptr;
  if (count == 0) count = 1;
  if (cudaMalloc(&q, count * sizeof(T)) != cudaSuccess) { cudaGetLastError(); return false; }
  L->allocs.push_back(q);
  *p = static_cast<T*>(q);
  return true;
}

template <typename T>
bool walloc(foe_workspace* W, T** p, size_t count) {
  void* q = nullptr;
  if (count == 0) count = 1;
  if (cudaMalloc(&q, count * sizeof(T)) != cudaSuccess) { cudaGetLastError(); return false; }
  W->allocs.push_back(q);
  *p = static_cast<T*>(q);
  return true;
}

void ws_release(foe_workspace* W) {
  if (!W) return;
  if (--W->refs > 0) return;
  for (void* p : W->allocs) cudaFree(p);
  delete W;
}

foe_status validate(const foe_config* c) {
  if (c->hidden <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->n_clusters <= 0) return FOE_ERR_CONFIG;
  if (c->n_kv_heads % c->n_clusters || c->n_q_heads % c->n_kv_heads) return FOE_ERR_CONFIG;
  if (c->n_clusters > 8) return FOE_ERR_CONFIG;          // the sync epilogues add up to 8 residual streams
  if (c->head_dim != 64 && c->head_dim != 96 && c->head_dim != 128) return FOE_ERR_CONFIG;
  if (c->n_q_heads / c->n_kv_heads > 16) return FOE_ERR_CONFIG;
  if (c->experts_per_cluster < 1 || c->experts_per_cluster > 128) return FOE_ERR_CONFIG;
  if (c->top_k_per_cluster < 1 || c->top_k_per_cluster > c->experts_per_cluster || c->top_k_per_cluster > 32)
    return FOE_ERR_CONFIG;
  if (c->n_clusters * c->experts_per_cluster > 1024) return FOE_ERR_CONFIG;
  if (c->page_size != 64) return FOE_ERR_CONFIG;
  if (c->hidden % 128 || c->ffn_inter % 128 || c->ffn_inter <= 0) return FOE_ERR_CONFIG;
  if ((c->n_q_heads * c->head_dim) % 128) return FOE_ERR_CONFIG;
  if (c->max_tokens <= 0 || c->max_seqs <= 0 || c->max_context <= 0) return FOE_ERR_CONFIG;
  if (!(c->rope_theta > 0.f) || !(c->rms_eps >= 0.f)) return FOE_ERR_CONFIG;
  if (c->position < 0 || c->position > 3 || c->sync < 0 || c->sync > 1) return FOE_ERR_CONFIG;
  return FOE_OK;
}

void stage_mark(foe_layer* L, int i, cudaStream_t st) {
  if (L->profiling) cudaEventRecord(L->ev[size_t(L->prof_calls % L->profiling) * (kNumStages + 1) + i], st);
}

foe_status check_launch() { return cudaGetLastError() == cudaSuccess ? FOE_OK : FOE_ERR_CUDA; }

// routing + dispatch maps for n tokens whose synced residual is r (fp32 internal or bf16 from the caller)
void run_route_and_permute(foe_layer* L, const void* r, int r_is_bf16, int n, cudaStream_t st) {
  if (n <= kRouteSmallMaxTokens) {          // a decode step: two launches for norm, scores, top-k, gates and maps
    L->launches += launch_route_small(r, r_is_bf16, L->ffn_gain, L->router_w, L->router_b, L->ws->u, L->ws->route_part,
                                      L->ws->route_part_cap, L->ws->logits, L->ws->topk_idx, L->ws->topk_w, L->ws->pb, n, L->d, L->H, L->Ec,
                                      L->kc, L->cfg.rms_eps, L->ws->status, st);
    stage_mark(L, kStPermute, st);
    return;
  }
  L->launches += launch_route(r, r_is_bf16, L->ffn_gain, L->router_w, &L->tm_router, L->router_b, L->ws->u, L->ws->inv_rms_f, L->ws->route_part,
                              L->ws->route_part_cap, L->ws->logits, L->ws->topk_idx, L->ws->topk_w, n, L->d, L->H, L->Ec, L->kc, L->cfg.rms_eps, L->n_sms, L->ws->status, st);
  stage_mark(L, kStPermute, st);
  L->launches += launch_permute(L->ws->topk_idx, L->ws->pb, n, L->H * L->kc, L->E, L->ws->status, st);
}

// Attention half of the block: token map, QKV projection, attention core, output projection.  With `sh` the
// O-projection's result is this rank's partial of the synced residual and goes to the column owners' receive
// slots; otherwise it is r_full itself, in the workspace.
foe_status run_attend(foe_layer* L, const void* x, const foe_kv_cache* kv, cudaStream_t st, bool decode, foe_shard* sh) {
  const int S = decode ? kv->n_seqs : kv->n_tokens;
  // Launches of this call (this thread) overlap their predecessors' tails when the call is small; kernels that follow
  // a SHORT kernel do so at any size (the token map and statistics at the start of a call, the QKV projection after
  // them, the routing chain, expert GEMM 1 after the dispatch scatter): what costs at large sizes is a kernel's CTAs
  // sitting resident beside a long, power-bound predecessor.
  const bool overlap_call = decode || S <= kOverlapTokens;
  g_overlap_launches = true;
  L->last_stream = st;
  L->launches = 0;
  L->last_tokens = S;
  L->last_decode = decode;
  if (L->profiling <= 1) { L->ev_valid = false; L->prof_calls = 0; }
  if (S == 0) return FOE_OK;
  const int H = L->H, d = L->d, dh = L->dh;
  const bf16* xb = static_cast<const bf16*>(x);

  CUtensorMap tmK, tmV, tmX;
  const uint64_t page_rows = uint64_t(kv->num_pages) * L->n_kv * 64;
  if (!make_map_2d(&tmK, kv->k_pages, page_rows, dh, 64) || !make_map_2d(&tmV, kv->v_pages, page_rows, dh, 64))
    return FOE_ERR_CUDA;

  // ---- prep: token map and pre-attention RMS statistics
  stage_mark(L, kStPrep, st);
  // (a decode step whose QKV projection runs on the tensor-core kernel needs no token map: token b is sequence b,
  //  its position and cache slot are looked up where they are used)
  const bool inline_map = decode && L->dp_qkv;
  if (!inline_map) L->launches += launch_token_map(decode ? nullptr : kv->q_lens, kv->context_lens, kv->block_table, kv->n_seqs, kv->max_pages_per_seq,
                   kv->num_pages, 64, S, L->cfg.max_context, decode ? 1 : kv->max_q_len, L->ws->cu_q, L->ws->tok_seq, L->ws->tok_pos, L->ws->tok_slot, L->ws->status, st);
  const int x_rows = L->first ? S : H * S;
  // Kernel family of the two projections: a call of a few hundred tokens (any decode step, a short prompt chunk, a
  // small mixed batch) is a weight-streaming problem and takes the decode kernels, whatever entry point it came by.
  const bool few = decode || S <= kFewTokens;
  const bool qkv_dp = few && L->dp_qkv, qkv_gemm = !qkv_dp && !decode;
  const bool oproj_dp = few && L->dp_oproj, oproj_gemm = !oproj_dp && !decode;
  bool x_summed = false;   // r_full holds sum_h x[h] (fp32) for the output projection to add
  if (oproj_gemm && !L->first && H > 1 && !sh) {
    x_summed = launch_row_inv_rms_xsum(xb, L->ws->inv_rms, L->ws->r_full, S, d, H, L->cfg.rms_eps, st);
    if (x_summed) L->launches += 1;
  }
  if (qkv_gemm && !x_summed) {   // (the decode projections derive 1/rms from the rows they stage)
    launch_row_inv_rms(xb, L->ws->inv_rms, x_rows, d, L->cfg.rms_eps, st);
    L->launches += 1;
  }

  // ---- per-cluster QKV projection; its epilogue applies 1/rms (gain folded into the weights) and RoPE, writes q
  //      and puts K / V of the new tokens straight into their cache pages
  stage_mark(L, kStQkv, st);
  if (qkv_gemm) {
    if (!make_map_2d(&tmX, x, x_rows, d, kBM)) return FOE_ERR_CUDA;
    GemmArgs ga;
    memset(&ga, 0, sizeof(ga));
    ga.n_groups = H; ga.rows_per_group = S; ga.a_group_stride = L->first ? 0 : S;
    ga.N = (L->g + 2 * L->c) * dh; ga.K = d; ga.status = L->ws->status;
    ga.out = L->ws->qkv; ga.ldo = L->n_q * L->dhp; ga.q_head_stride = L->dhp;
    ga.row_scale = L->ws->inv_rms; ga.scale_group_stride = L->first ? 0 : S;
    ga.q_cols = L->g * dh; ga.kv_cols = L->c * dh; ga.dh = dh; ga.n_kv = L->n_kv;
    ga.rope_tab = L->rope_tab; ga.tok_pos = L->ws->tok_pos; ga.tok_slot = L->ws->tok_slot;
    ga.k_pages = static_cast<bf16*>(kv->k_pages); ga.v_pages = static_cast<bf16*>(kv->v_pages);
    launch_gemm(kEpiQKV, tmX, L->tm_wqkv, ga, L->n_sms, st);
  } else if (qkv_dp) {
    if (!make_map_2d(&tmX, x, x_rows, d, 64)) return FOE_ERR_CUDA;
    DecodeProjArgs pa;
    memset(&pa, 0, sizeof(pa));
    pa.n_groups = H; pa.rows_per_group = S; pa.x_group_stride = L->first ? 0 : S; pa.N = (L->g + 2 * L->c) * dh; pa.K = d;
    pa.epi = kEpiQKV; pa.status = L->ws->status;
    pa.out = L->ws->qkv; pa.ldo = L->n_q * L->dhp; pa.q_head_stride = L->dhp; pa.rms_eps = L->cfg.rms_eps;
    pa.q_cols = L->g * dh; pa.kv_cols = L->c * dh; pa.dh = dh; pa.n_kv = L->n_kv;
    pa.rope_tab = L->rope_tab; pa.tok_pos = L->ws->tok_pos; pa.tok_slot = L->ws->tok_slot;
    pa.k_pages = static_cast<bf16*>(kv->k_pages); pa.v_pages = static_cast<bf16*>(kv->v_pages);
    if (inline_map) {
      pa.tok_pos = nullptr; pa.tok_slot = nullptr;
      pa.context_lens = kv->context_lens; pa.block_table = kv->block_table; pa.max_pages_per_seq = kv->max_pages_per_seq;
      pa.num_pages = kv->num_pages; pa.max_context = L->cfg.max_context;
    }
    launch_decode_proj(L->tmt_wqkv, tmX, pa, L->n_sms, st);
  } else {
    SmallMArgs sa;
    memset(&sa, 0, sizeof(sa));
    sa.W = L->wqkv_t; sa.X = xb; sa.ldx = d; sa.n_groups = H; sa.rows_per_group = S; sa.x_group_stride = L->first ? 0 : S;
    sa.N = (L->g + 2 * L->c) * dh; sa.K = d; sa.epi = kEpiQKV;
    sa.out = L->ws->qkv; sa.ldo = L->n_q * L->dhp; sa.q_head_stride = L->dhp;
    sa.rms_eps = L->cfg.rms_eps;
    sa.q_cols = L->g * dh; sa.kv_cols = L->c * dh; sa.dh = dh; sa.n_kv = L->n_kv;
    sa.rope_tab = L->rope_tab; sa.tok_pos = L->ws->tok_pos; sa.tok_slot = L->ws->tok_slot;
    sa.k_pages = static_cast<bf16*>(kv->k_pages); sa.v_pages = static_cast<bf16*>(kv->v_pages);
    sa.status = L->ws->status;
    launch_smallm(L->tms_wqkv, sa, L->n_sms, st);
  }
  L->launches += 1;

  // ---- attention core over the paged cache
  g_overlap_launches = overlap_call;     // (attention follows the long QKV projection)
  stage_mark(L, kStAttn, st);
  AttnArgs aa;
  memset(&aa, 0, sizeof(aa));
  aa.q = L->ws->qkv; aa.out = L->ws->attn_o; aa.cu_q = inline_map ? nullptr : L->ws->cu_q; aa.context_lens = kv->context_lens;
  aa.q_lens = decode ? nullptr : kv->q_lens; aa.block_table = kv->block_table; aa.n_seqs = kv->n_seqs;
  aa.max_pages_per_seq = kv->max_pages_per_seq; aa.num_pages = kv->num_pages; aa.n_tokens = S; aa.n_q = L->n_q; aa.n_kv = L->n_kv;
  aa.dh = dh; aa.max_q_len = decode ? 1 : kv->max_q_len; aa.scale_log2 = float(1.4426950408889634 / sqrt(double(dh)));
  aa.status = L->ws->status; aa.part_o = L->ws->part_o; aa.part_ml = L->ws->part_ml; aa.max_splits = L->max_splits;
  aa.split_done = L->ws->split_done;
  aa.max_kv_pages = min(kv->max_pages_per_seq, (L->cfg.max_context + 63) / 64);   // part_o / part_ml were sized for this many
  if (decode) { launch_attn_decode(tmK, tmV, aa, L->n_sms, st); L->launches += 1; }
  else { launch_attn_prefill_tc(L->ws->tm_qkv, tmK, tmV, aa, st); L->launches += 1; }

  // ---- output projection; the cross-cluster sync is its K-reduction plus the sum of x[h] in the epilogue
  stage_mark(L, kStOproj, st);
  // one device: r_full = (sum_h (x[h] + Attn_h W_O[h])) / H, with the sum over h inside the GEMM's K loop.
  // one rank of a group: the partial (x[h] + Attn_h W_O[h]) / H; a first layer's shared x comes from rank 0 alone.
  float out_scale = (L->first || L->cfg.sync == FOE_SYNC_SUM) ? 1.0f : 1.0f / float(H);
  int x_count = L->first ? 1 : H;
  if (sh) {
    out_scale = (L->first || L->cfg.sync == FOE_SYNC_SUM) ? 1.0f : 1.0f / float(sh->cfg.n_ranks);
    x_count = (L->first && sh->cfg.rank != 0) ? 0 : 1;
  }
  const long long slot_off = sh ? (long long)((size_t(sh->epoch & 1) * sh->cfg.n_ranks + sh->cfg.rank) * sh->S_cap * sh->span) : 0;
  const int cnt_off = sh ? int(sh->epoch & 1) * 8 * sh->n_blk : 0;          // this exchange's half of the slot counters
  if (oproj_gemm) {
    GemmArgs ga;
    memset(&ga, 0, sizeof(ga));
    ga.n_groups = 1; ga.rows_per_group = S; ga.a_group_stride = 0; ga.N = d; ga.K = L->n_q * dh; ga.status = L->ws->status;
    ga.out = L->ws->r_full; ga.ldo = d; ga.xsum = xb; ga.x_count = x_count; ga.x_stride = size_t(S) * d;
    ga.out_scale = out_scale;
    if (x_summed) { ga.x_count = 0; ga.x_in_out = 1; }
    if (sh) {     // the epilogue stores each tile straight into the owners' slots
      for (int o = 0; o < sh->cfg.n_ranks; ++o) { ga.push_base[o] = sh->table.slots[o]; ga.push_cnt[o] = sh->table.slot_cnt[o] + cnt_off; }
      ga.push_span = sh->span;
      ga.push_slot_off = slot_off;
    }
    launch_gemm(kEpiOProj, L->ws->tm_attn_o, L->tm_wo, ga, L->n_sms, st);
  } else if (oproj_dp) {
    DecodeProjArgs pa;
    memset(&pa, 0, sizeof(pa));
    pa.n_groups = 1; pa.rows_per_group = S; pa.x_group_stride = 0; pa.N = d; pa.K = L->n_q * dh; pa.epi = kEpiOProj;
    pa.status = L->ws->status;
    pa.out = L->ws->r_full; pa.ldo = d; pa.xsum = xb; pa.x_count = x_count; pa.x_stride = size_t(S) * d; pa.out_scale = out_scale;
    const bool fused_push = sh && sh->span % 128 == 0;      // a 128-row weight slab then lies inside one owner's columns
    if (fused_push) {
      for (int o = 0; o < sh->cfg.n_ranks; ++o) { pa.push_base[o] = sh->table.slots[o]; pa.push_cnt[o] = sh->table.slot_cnt[o] + cnt_off; }
      pa.push_span = sh->span;
      pa.push_slot_off = slot_off;
    }
    launch_decode_proj(L->tmt_wo, L->ws->tm_attn_o64, pa, L->n_sms, st);
    if (sh && !fused_push) {
      launch_shard_push(L->ws->r_full, 1, 1.0f, S, d, sh->cfg.n_ranks, sh->table, slot_off, cnt_off, st);
      L->launches += 1;
    }
  } else {
    SmallMArgs sa;
    memset(&sa, 0, sizeof(sa));
    sa.W = L->wo_t; sa.X = L->ws->attn_o; sa.ldx = L->n_q * dh; sa.n_groups = 1; sa.rows_per_group = S; sa.N = d;
    sa.K = L->n_q * dh; sa.epi = kEpiOProj; sa.out = L->ws->r_full; sa.ldo = d; sa.xsum = xb; sa.x_count = x_count;
    sa.x_stride = size_t(S) * d; sa.out_scale = out_scale; sa.status = L->ws->status;
    launch_smallm(L->tms_wo, sa, L->n_sms, st);
    if (sh) {     // a decode step's partial is a few hundred KB: one more launch pushes it
      launch_shard_push(L->ws->r_full, 1, 1.0f, S, d, sh->cfg.n_ranks, sh->table, slot_off, cnt_off, st);
      L->launches += 1;
    }
  }
  L->launches += 1;
  return check_launch();
}

// FFN half of the block on the synced residual in the workspace: routing, dispatch maps, experts, combine.
foe_status run_ffn(foe_layer* L, void* out, cudaStream_t st) {
  const int S = L->last_tokens, H = L->H, d = L->d;
  const bool decode = L->last_decode;
  if (S == 0) return FOE_OK;
  g_overlap_launches = decode || S <= kOverlapTokens;

  // ---- router, top-k, gates, dispatch maps
  stage_mark(L, kStRoute, st);
  {
    // the routing and dispatch-map kernels are short at any call size: they always overlap their predecessors' tails
    const bool saved = g_overlap_launches;
    g_overlap_launches = true;
    run_route_and_permute(L, L->ws->r_full, 0, S, st);
    g_overlap_launches = saved;
  }
  const int R = S * H * L->kc;
  // experts: the weight-streaming kernels take 16 rows of an expert per pass over its weights; up to 8 rows per
  // expert on average (few experts need a second pass) they beat the tiled GEMMs, at 16 they no longer do
  const bool stream_experts = decode || (S <= kFewTokens && R <= 8 * L->E);

  if (!stream_experts) {
    stage_mark(L, kStGemm1, st);
    GemmArgs g1;
    memset(&g1, 0, sizeof(g1));
    g1.n_groups = L->E; g1.mt_group = L->ws->pb.mt_group; g1.mt_row0 = L->ws->pb.mt_row0; g1.group_end = L->ws->pb.offsets + 1;
    g1.n_mtiles = L->ws->pb.n_mtiles; g1.N = 2 * L->I; g1.K = d; g1.status = L->ws->status; g1.out = L->ws->hmid; g1.ldo = L->I;
    g1.a_gather = L->ws->u; g1.a_row_index = L->ws->pb.perm;      // rows of u gathered through the dispatch map
    {
      const bool saved = g_overlap_launches;
      g_overlap_launches = true;          // its predecessor (the dispatch scatter) is short: set up while it runs
      launch_gemm(kEpiSwiGLU, L->ws->tm_hmid, L->tm_wgu, g1, L->n_sms, st);   // the A map is unused with a gathered A
      g_overlap_launches = saved;
    }
    stage_mark(L, kStGemm2, st);
    GemmArgs g2 = g1;
    g2.a_gather = nullptr; g2.a_row_index = nullptr;
    g2.N = d; g2.K = L->I; g2.out = L->ws->y; g2.ldo = d;
    launch_gemm(kEpiBf16, L->ws->tm_hmid, L->tm_wd, g2, L->n_sms, st);
    L->launches += 2;
  } else {
    stage_mark(L, kStGemm1, st);
    SmallMArgs s1;
    memset(&s1, 0, sizeof(s1));
    s1.W = L->wgu_t; s1.X = L->ws->u; s1.ldx = d; s1.row_index = L->ws->pb.perm; s1.group_offsets = L->ws->pb.offsets;
    s1.n_groups = L->E; s1.N = 2 * L->I; s1.K = d; s1.epi = kEpiSwiGLU; s1.out = L->ws->hmid; s1.ldo = L->I;
    s1.status = L->ws->status;
    launch_smallm(L->tms_wgu, s1, L->n_sms, st);
    stage_mark(L, kStGemm2, st);
    SmallMArgs s2;
    memset(&s2, 0, sizeof(s2));
    s2.W = L->wd_t; s2.X = L->ws->hmid; s2.ldx = L->I; s2.group_offsets = L->ws->pb.offsets; s2.n_groups = L->E; s2.N = d;
    s2.K = L->I; s2.epi = kEpiBf16; s2.out = L->ws->y; s2.ldo = d;
    s2.status = L->ws->status;
    s2.early_weights = 1;
    launch_smallm(L->tms_wd, s2, L->n_sms, st);
    L->launches += 2;
  }

  // ---- weighted combine, residual, last-layer mean
  stage_mark(L, kStCombine, st);
  launch_combine(L->ws->r_full, L->ws->y, L->ws->topk_w, L->ws->pb.inv, static_cast<bf16*>(out), S, d, H, L->kc, L->last ? 1 : 0, st);
  L->launches += 1;
  if (L->profiling) { stage_mark(L, kNumStages, st); L->prof_calls += 1; L->ev_valid = true; }
  return check_launch();
}

foe_status run_block(foe_layer* L, const void* x, const foe_kv_cache* kv, void* out, cudaStream_t st, bool decode) {
  L->shard_stage = 0;
  const foe_status a = run_attend(L, x, kv, st, decode, nullptr);
  if (a != FOE_OK) return a;
  return run_ffn(L, out, st);
}

// argument checks shared by foe_prefill / foe_decode and foe_shard_attend (x and out are checked by the callers)
bool misaligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }

foe_status check_call(const foe_layer* L, const foe_kv_cache* kv, bool decode) {
  if (!kv->k_pages || !kv->v_pages || !kv->block_table || !kv->context_lens) return FOE_ERR_NULL;
  // pages are read through tensor maps and 16-byte accesses, the integer arrays element by element: a misaligned view
  // is refused here, before any launch, rather than found by the device
  if (misaligned(kv->k_pages, 16) || misaligned(kv->v_pages, 16) || misaligned(kv->block_table, 4) ||
      misaligned(kv->context_lens, 4) || (kv->q_lens && misaligned(kv->q_lens, 4)))
    return FOE_ERR_SHAPE;
  if (decode) {
    if (kv->n_seqs > L->cfg.max_seqs || kv->max_pages_per_seq <= 0 || kv->num_pages <= 0) return FOE_ERR_SHAPE;
    // the decode attention kernel numbers the pages of all (sequence, KV head) pairs with 32-bit integers
    const long long pages = (long long)kv->n_seqs * L->n_kv * min(kv->max_pages_per_seq, (L->cfg.max_context + 63) / 64);
    if (pages >= (1LL << 30)) return FOE_ERR_SHAPE;
    return FOE_OK;
  }
  if (!kv->q_lens) return FOE_ERR_NULL;
  if (kv->n_tokens > L->cfg.max_tokens || kv->n_seqs > L->cfg.max_seqs || kv->n_seqs == 0) return FOE_ERR_SHAPE;
  if (kv->max_q_len <= 0 || kv->max_q_len > kv->n_tokens || kv->max_pages_per_seq <= 0 || kv->num_pages <= 0)
    return FOE_ERR_SHAPE;
  return FOE_OK;
}

}  // namespace

extern "C" {

const char* foe_status_string(int s) {
  switch (s) {
    case FOE_OK: return "ok";
    case FOE_ERR_NULL: return "null pointer argument";
    case FOE_ERR_CONFIG: return "invalid layer configuration";
    case FOE_ERR_SHAPE: return "call exceeds the sizes the layer was created for";
    case FOE_ERR_UNSUPPORTED: return "unsupported";
    case FOE_ERR_OOM: return "device allocation failed";
    case FOE_ERR_CUDA: return "CUDA call failed";
    case FOE_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case FOE_ERR_BOUNDS: return "an index read on the device was out of range";
    default: return "unknown status";
  }
}

foe_status foe_layer_destroy(foe_layer* L) {
  if (!L) return FOE_OK;
  for (void* p : L->allocs) cudaFree(p);
  ws_release(L->ws);
  for (cudaEvent_t e : L->ev) cudaEventDestroy(e);
  delete L;
  return FOE_OK;
}

foe_status foe_layer_create(const foe_config* cfg, const foe_weights* w, foe_layer** out) {
  return foe_layer_create_shared(cfg, w, nullptr, out);
}

foe_status foe_layer_create_shared(const foe_config* cfg, const foe_weights* w, foe_layer* donor, foe_layer** out) {
  if (!cfg || !w || !out) return FOE_ERR_NULL;
  *out = nullptr;
  const foe_status v = validate(cfg);
  if (v != FOE_OK) return v;
  if (!w->attn_norm_g || !w->wq || !w->wk || !w->wv || !w->wo || !w->ffn_norm_g || !w->w_gate || !w->w_up ||
      !w->w_down || !w->router_w)
    return FOE_ERR_NULL;
  if (misaligned(w->attn_norm_g, 16) || misaligned(w->wq, 16) || misaligned(w->wk, 16) || misaligned(w->wv, 16) ||
      misaligned(w->wo, 16) || misaligned(w->ffn_norm_g, 16) || misaligned(w->w_gate, 16) || misaligned(w->w_up, 16) ||
      misaligned(w->w_down, 16) || misaligned(w->router_w, 16) || (w->router_b && misaligned(w->router_b, 4)))
    return FOE_ERR_SHAPE;
  int dev = 0, n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev == 0) { cudaGetLastError(); return FOE_ERR_CUDA; }
  if (cudaGetDevice(&dev) != cudaSuccess) return FOE_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return FOE_ERR_CUDA;
  if (prop.major != 10) return FOE_ERR_UNSUPPORTED;       // tcgen05/TMEM kernels: sm_100 only
  if (gemm_configure() != cudaSuccess || attn_decode_configure() != cudaSuccess || attn_prefill_configure() != cudaSuccess ||
      router_tc_configure() != cudaSuccess || smallm_configure() != cudaSuccess || decode_proj_configure() != cudaSuccess) {
    cudaGetLastError();
    return FOE_ERR_CUDA;
  }
  if (donor) {   // a shared workspace must have been sized for exactly these shapes
    const foe_config& a = donor->cfg;
    if (a.hidden != cfg->hidden || a.n_q_heads != cfg->n_q_heads || a.n_kv_heads != cfg->n_kv_heads ||
        a.n_clusters != cfg->n_clusters || a.head_dim != cfg->head_dim ||
        a.experts_per_cluster != cfg->experts_per_cluster || a.top_k_per_cluster != cfg->top_k_per_cluster ||
        a.ffn_inter != cfg->ffn_inter || a.max_tokens != cfg->max_tokens || a.max_seqs != cfg->max_seqs ||
        a.max_context != cfg->max_context)
      return FOE_ERR_SHAPE;
  }

  foe_layer* L = new (std::nothrow) foe_layer();
  if (!L) return FOE_ERR_OOM;
  L->cfg = *cfg;
  L->H = cfg->n_clusters; L->n_q = cfg->n_q_heads; L->n_kv = cfg->n_kv_heads; L->dh = cfg->head_dim; L->dhp = cfg->head_dim == 96 ? 128 : cfg->head_dim;
  L->g = L->n_q / L->H; L->c = L->n_kv / L->H; L->d = cfg->hidden; L->I = cfg->ffn_inter;
  L->Ec = cfg->experts_per_cluster; L->E = L->H * L->Ec; L->kc = cfg->top_k_per_cluster;
  L->qkv_cols = (L->n_q + 2 * L->n_kv) * L->dh;
  L->first = cfg->position == FOE_FIRST || cfg->position == FOE_SINGLE;
  L->last = cfg->position == FOE_LAST || cfg->position == FOE_SINGLE;
  L->S_max = cfg->max_tokens > cfg->max_seqs ? cfg->max_tokens : cfg->max_seqs;
  L->R_max = L->S_max * L->H * L->kc;
  L->n_sms = prop.multiProcessorCount;
  const int H = L->H, d = L->d, dh = L->dh, I = L->I, E = L->E, S = L->S_max, R = L->R_max;
  const int max_pages = (cfg->max_context + 63) / 64;
  L->max_splits = attn_decode_max_segments(max_pages);
  const int n_blocks = (S + kPermuteBlockTokens - 1) / kPermuteBlockTokens;
  const int qkvN = (L->g + 2 * L->c) * dh;

  bool ok = true;
  ok = ok && dalloc(L, &L->wqkv_t, size_t(H) * qkvN * d + 256 * size_t(d));
  ok = ok && dalloc(L, &L->wo_t, size_t(d) * L->n_q * dh + 256 * size_t(L->n_q) * dh);
  ok = ok && dalloc(L, &L->wgu_t, size_t(E) * 2 * I * d);
  ok = ok && dalloc(L, &L->wd_t, size_t(E) * d * I + 256 * size_t(I));
  ok = ok && dalloc(L, &L->ffn_gain, size_t(d));
  ok = ok && dalloc(L, &L->router_w, size_t(E) * d);
  ok = ok && dalloc(L, &L->router_b, size_t(E));
  ok = ok && dalloc(L, &L->router_split, size_t(3) * router_padded_experts(E) * d);
  ok = ok && dalloc(L, &L->rope_tab, size_t(cfg->max_context) * (dh / 2));
  if (!ok) { foe_layer_destroy(L); return FOE_ERR_OOM; }
  cudaStream_t st = 0;
  if (donor) {
    L->ws = donor->ws;
    L->ws->refs += 1;
  } else {
    foe_workspace* W = new (std::nothrow) foe_workspace();
    if (!W) { foe_layer_destroy(L); return FOE_ERR_OOM; }
    W->refs = 1;
    L->ws = W;
    ok = ok && walloc(W, &W->inv_rms, size_t(H) * S);
    ok = ok && walloc(W, &W->r_full, size_t(S) * d);
    ok = ok && walloc(W, &W->logits, size_t(S) * E);
    ok = ok && walloc(W, &W->inv_rms_f, size_t(S));
    W->route_part_cap = route_part_capacity(size_t(S), size_t(E));
    ok = ok && walloc(W, &W->route_part, W->route_part_cap);
    ok = ok && walloc(W, &W->topk_w, size_t(R));
    ok = ok && walloc(W, &W->topk_idx, size_t(R));
    ok = ok && walloc(W, &W->qkv, size_t(S + 128) * L->n_q * L->dhp);      // q after RoPE (k, v go to the pages)
    ok = ok && walloc(W, &W->attn_o, size_t(S + 128) * L->n_q * dh);
    ok = ok && walloc(W, &W->u, size_t(S) * d);
    ok = ok && walloc(W, &W->hmid, size_t(R + 128) * I);
    ok = ok && walloc(W, &W->y, size_t(R) * d);
    ok = ok && walloc(W, &W->cu_q, size_t(cfg->max_seqs) + 1);
    ok = ok && walloc(W, &W->tok_seq, size_t(S));
    ok = ok && walloc(W, &W->tok_pos, size_t(S));
    ok = ok && walloc(W, &W->tok_slot, size_t(S));
    ok = ok && walloc(W, &W->status, size_t(1));
    ok = ok && walloc(W, &W->part_o, size_t(cfg->max_seqs) * L->n_q * L->max_splits * L->dhp);
    ok = ok && walloc(W, &W->part_ml, size_t(cfg->max_seqs) * L->n_q * L->max_splits * 2);
    W->split_done_count = size_t(cfg->max_seqs) * L->n_kv;
    ok = ok && walloc(W, &W->split_done, W->split_done_count);
    ok = ok && walloc(W, &W->pb.counts, size_t(E));
    ok = ok && walloc(W, &W->pb.offsets, size_t(E) + 1);
    ok = ok && walloc(W, &W->pb.perm, size_t(R));
    ok = ok && walloc(W, &W->pb.inv, size_t(R));
    ok = ok && walloc(W, &W->pb.rank, size_t(R));
    ok = ok && walloc(W, &W->pb.blk_counts, size_t(n_blocks) * E);
    ok = ok && walloc(W, &W->pb.mt_group, size_t(R / 256 + E + 1));
    ok = ok && walloc(W, &W->pb.mt_row0, size_t(R / 256 + E + 1));
    ok = ok && walloc(W, &W->pb.n_mtiles, size_t(1));
    if (!ok) { foe_layer_destroy(L); return FOE_ERR_OOM; }
    cudaMemsetAsync(W->status, 0, sizeof(int), st);
    cudaMemsetAsync(W->split_done, 0, size_t(cfg->max_seqs) * L->n_kv * sizeof(int), st);
    cudaMemsetAsync(W->attn_o, 0, size_t(S + 128) * L->n_q * dh * sizeof(bf16), st);
    cudaMemsetAsync(W->qkv, 0, size_t(S + 128) * L->n_q * L->dhp * sizeof(bf16), st);   // padding columns stay zero
    cudaMemsetAsync(W->hmid, 0, size_t(R + 128) * I * sizeof(bf16), st);
    ok = make_map_2d(&W->tm_attn_o, W->attn_o, uint64_t(S), uint64_t(L->n_q) * dh, kBM) &&
         make_map_2d(&W->tm_hmid, W->hmid, uint64_t(R), I, kBM) &&
         make_map_2d(&W->tm_qkv, W->qkv, uint64_t(S), uint64_t(L->n_q) * L->dhp, 128) &&
         make_map_2d(&W->tm_attn_o64, W->attn_o, uint64_t(S), uint64_t(L->n_q) * dh, 64);
    if (!ok) { foe_layer_destroy(L); return FOE_ERR_CUDA; }
  }

  // K-major ("transposed") weights; the attention-norm gain is folded into W_q|k|v.
  const bf16* gain_a = static_cast<const bf16*>(w->attn_norm_g);
  const size_t qkv_batch = size_t(qkvN) * d;
  launch_transpose_batched(static_cast<const bf16*>(w->wq), size_t(d) * L->g * dh, L->g * dh, L->wqkv_t, qkv_batch, d, d,
                           L->g * dh, H, gain_a, dh, st);
  launch_transpose_batched(static_cast<const bf16*>(w->wk), size_t(d) * L->c * dh, L->c * dh,
                           L->wqkv_t + size_t(L->g) * dh * d, qkv_batch, d, d, L->c * dh, H, gain_a, dh, st);
  launch_transpose_batched(static_cast<const bf16*>(w->wv), size_t(d) * L->c * dh, L->c * dh,
                           L->wqkv_t + size_t(L->g + L->c) * dh * d, qkv_batch, d, d, L->c * dh, H, gain_a, dh, st);
  launch_transpose_batched(static_cast<const bf16*>(w->wo), 0, d, L->wo_t, 0, L->n_q * dh, L->n_q * dh, d, 1, nullptr, 0, st);
  launch_pack_gate_up(static_cast<const bf16*>(w->w_gate), static_cast<const bf16*>(w->w_up), L->wgu_t, E, d, I, st);
  for (int e0 = 0; e0 < E; e0 += 32768) {
    const int nb = E - e0 < 32768 ? E - e0 : 32768;
    launch_transpose_batched(static_cast<const bf16*>(w->w_down) + size_t(e0) * I * d, size_t(I) * d, d,
                             L->wd_t + size_t(e0) * d * I, size_t(d) * I, I, I, d, nb, nullptr, 0, st);
  }
  cudaMemcpyAsync(L->ffn_gain, w->ffn_norm_g, size_t(d) * sizeof(bf16), cudaMemcpyDeviceToDevice, st);
  cudaMemcpyAsync(L->router_w, w->router_w, size_t(E) * d * sizeof(float), cudaMemcpyDeviceToDevice, st);
  launch_split_router_weights(L->router_w, L->ffn_gain, L->router_split, E, d, st);
  if (w->router_b) cudaMemcpyAsync(L->router_b, w->router_b, size_t(E) * sizeof(float), cudaMemcpyDeviceToDevice, st);
  else cudaMemsetAsync(L->router_b, 0, size_t(E) * sizeof(float), st);
  // rotary table in double precision on the host: (cos, sin)(p * theta^(-2j/dh))
  {
    const int half = dh / 2;
    std::vector<float2> tab(size_t(cfg->max_context) * half);
    std::vector<double> inv_freq(half);
    for (int j = 0; j < half; ++j) inv_freq[j] = pow(double(cfg->rope_theta), -2.0 * j / double(dh));
    for (int p = 0; p < cfg->max_context; ++p)
      for (int j = 0; j < half; ++j) {
        const double ang = double(p) * inv_freq[j];
        tab[size_t(p) * half + j] = make_float2(float(cos(ang)), float(sin(ang)));
      }
    cudaMemcpy(L->rope_tab, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice);
  }
  if (cudaStreamSynchronize(st) != cudaSuccess || cudaGetLastError() != cudaSuccess) {
    foe_layer_destroy(L);
    return FOE_ERR_CUDA;
  }
  ok = make_map_2d(&L->tm_router, L->router_split, uint64_t(3) * router_padded_experts(E), d, kRouterChunk) &&
       make_map_2d(&L->tm_wqkv, L->wqkv_t, uint64_t(H) * qkvN, d, gemm_tile_rows_b(kEpiQKV, qkvN)) &&
       make_map_2d(&L->tm_wo, L->wo_t, uint64_t(d), uint64_t(L->n_q) * dh, gemm_tile_rows_b(kEpiOProj, d)) &&
       make_map_2d(&L->tm_wgu, L->wgu_t, uint64_t(E) * 2 * I, d, gemm_tile_rows_b(kEpiSwiGLU, 2 * I)) &&
       make_map_2d(&L->tm_wd, L->wd_t, uint64_t(E) * d, I, gemm_tile_rows_b(kEpiBf16, d)) &&
       make_map_2d(&L->tms_wqkv, L->wqkv_t, uint64_t(H) * qkvN, d, 64) &&
       make_map_2d(&L->tms_wo, L->wo_t, uint64_t(d), uint64_t(L->n_q) * dh, 64) &&
       make_map_2d(&L->tms_wgu, L->wgu_t, uint64_t(E) * 2 * I, d, 32) &&
       make_map_2d(&L->tms_wd, L->wd_t, uint64_t(E) * d, I, 64) &&
       make_map_2d(&L->tmt_wqkv, L->wqkv_t, uint64_t(H) * qkvN, d, 128) &&
       make_map_2d(&L->tmt_wo, L->wo_t, uint64_t(d), uint64_t(L->n_q) * dh, 128);
  L->dp_qkv = decode_proj_supported(kEpiQKV, qkvN, d, dh);
  L->dp_oproj = decode_proj_supported(kEpiOProj, d, L->n_q * dh, dh);
  if (!ok) { foe_layer_destroy(L); return FOE_ERR_CUDA; }
  *out = L;
  return FOE_OK;
}

foe_status foe_prefill(foe_layer* L, const void* x, const foe_kv_cache* kv, void* out, void* stream) {
  if (!L || !kv) return FOE_ERR_NULL;
  if (kv->n_tokens < 0 || kv->n_seqs < 0) return FOE_ERR_SHAPE;
  if (kv->n_tokens == 0) { L->launches = 0; L->last_tokens = 0; return FOE_OK; }
  if (!x || !out) return FOE_ERR_NULL;
  const foe_status c = check_call(L, kv, false);
  if (c != FOE_OK) return c;
  if (misaligned(x, 16) || misaligned(out, 16)) return FOE_ERR_SHAPE;
  if (x == out) return FOE_ERR_UNSUPPORTED;
  return run_block(L, x, kv, out, static_cast<cudaStream_t>(stream), false);
}

foe_status foe_decode(foe_layer* L, const void* x, const foe_kv_cache* kv, void* out, void* stream) {
  if (!L || !kv) return FOE_ERR_NULL;
  if (kv->n_seqs < 0) return FOE_ERR_SHAPE;
  if (kv->n_seqs == 0) { L->launches = 0; L->last_tokens = 0; return FOE_OK; }
  if (!x || !out) return FOE_ERR_NULL;
  const foe_status c = check_call(L, kv, true);
  if (c != FOE_OK) return c;
  if (misaligned(x, 16) || misaligned(out, 16)) return FOE_ERR_SHAPE;
  if (x == out) return FOE_ERR_UNSUPPORTED;
  return run_block(L, x, kv, out, static_cast<cudaStream_t>(stream), true);
}

foe_status foe_stack_forward(foe_layer* const* layers, int n_layers, const void* x, const foe_kv_cache* kvs, void* out,
                             void* work0, void* work1, int decode, void* stream) {
  if (!layers || !kvs || n_layers <= 0) return n_layers <= 0 && layers && kvs ? FOE_ERR_SHAPE : FOE_ERR_NULL;
  for (int l = 0; l < n_layers; ++l)
    if (!layers[l]) return FOE_ERR_NULL;
  if (n_layers > 1 && !work0) return FOE_ERR_NULL;
  if (n_layers > 2 && !work1) return FOE_ERR_NULL;
  if (work0 && (work0 == work1 || work0 == x || work0 == out)) return FOE_ERR_UNSUPPORTED;
  if (work1 && (work1 == x || work1 == out)) return FOE_ERR_UNSUPPORTED;
  // every layer's arguments are checked before the first one is launched
  for (int l = 0; l < n_layers; ++l) {
    const foe_kv_cache* kv = &kvs[l];
    if (kv->n_tokens < 0 || kv->n_seqs < 0) return FOE_ERR_SHAPE;
    const int S = decode ? kv->n_seqs : kv->n_tokens;
    const int S0 = decode ? kvs[0].n_seqs : kvs[0].n_tokens;
    if (S != S0) return FOE_ERR_SHAPE;
    if (S == 0) continue;
    const foe_status c = check_call(layers[l], kv, decode != 0);
    if (c != FOE_OK) return c;
    if (l > 0 && (layers[l]->first || layers[l]->d != layers[l - 1]->d ||
                  (layers[l - 1]->last ? 1 : layers[l - 1]->H) != layers[l]->H))
      return FOE_ERR_CONFIG;             // layer l must take what layer l-1 produces
  }
  const int S = decode ? kvs[0].n_seqs : kvs[0].n_tokens;
  if (S > 0 && (!x || !out)) return FOE_ERR_NULL;
  if (misaligned(x, 16) || misaligned(out, 16) || misaligned(work0, 16) || misaligned(work1, 16)) return FOE_ERR_SHAPE;
  if (S > 0 && x == out) return FOE_ERR_UNSUPPORTED;
  void* bufs[2] = {work0, work1};
  const void* in = x;
  for (int l = 0; l < n_layers; ++l) {
    void* dst = l == n_layers - 1 ? out : bufs[l & 1];
    if (S == 0) { layers[l]->launches = 0; layers[l]->last_tokens = 0; continue; }
    const foe_status r = run_block(layers[l], in, &kvs[l], dst, static_cast<cudaStream_t>(stream), decode != 0);
    if (r != FOE_OK) return r;
    in = dst;
  }
  return FOE_OK;
}

foe_status foe_context_advance(int* context_lens, int n_seqs, int by, void* stream) {
  if (!context_lens) return FOE_ERR_NULL;
  if (n_seqs < 0) return FOE_ERR_SHAPE;
  if (n_seqs == 0 || by == 0) return FOE_OK;
  launch_add_to_ints(context_lens, n_seqs, by, static_cast<cudaStream_t>(stream));
  return check_launch();
}

foe_status foe_route(foe_layer* L, const void* h, int n_tokens, int* topk_idx, float* topk_w, void* stream) {
  if (!L || !h || !topk_idx || !topk_w) return FOE_ERR_NULL;
  if (n_tokens < 0 || n_tokens > L->S_max) return FOE_ERR_SHAPE;
  if (misaligned(h, 16) || misaligned(topk_idx, 4) || misaligned(topk_w, 4)) return FOE_ERR_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  L->last_stream = st;
  L->launches = 0;
  L->last_tokens = n_tokens;
  L->ev_valid = false;
  if (n_tokens == 0) return FOE_OK;
  const int saved = L->profiling;
  L->profiling = 0;
  g_overlap_launches = n_tokens <= kOverlapTokens;
  run_route_and_permute(L, h, 1, n_tokens, st);
  L->profiling = saved;
  const size_t n = size_t(n_tokens) * L->H * L->kc;
  cudaMemcpyAsync(topk_idx, L->ws->topk_idx, n * sizeof(int), cudaMemcpyDeviceToDevice, st);
  cudaMemcpyAsync(topk_w, L->ws->topk_w, n * sizeof(float), cudaMemcpyDeviceToDevice, st);
  return check_launch();
}

foe_status foe_route_noalloc(int hidden, int n_clusters, int experts_per_cluster, int top_k_per_cluster, float rms_eps,
                             const void* ffn_norm_g, const float* router_w, const float* router_b, const void* h,
                             int n_tokens, int* topk_idx, float* topk_w, void* stream) {
  if (!ffn_norm_g || !router_w || !h || !topk_idx || !topk_w) return FOE_ERR_NULL;
  if (hidden <= 0 || hidden % 128 || n_clusters <= 0 || experts_per_cluster < 1 || experts_per_cluster > 128 ||
      top_k_per_cluster < 1 || top_k_per_cluster > experts_per_cluster || top_k_per_cluster > 32 ||
      n_clusters * experts_per_cluster > 1024 || !(rms_eps >= 0.f))
    return FOE_ERR_CONFIG;
  if (n_tokens < 0) return FOE_ERR_SHAPE;
  // the kernels read h and router_w 16 bytes at a time, the gain 8, the outputs 4: a misaligned view is refused here
  // instead of faulting on the device
  if (misaligned(h, 16) || misaligned(router_w, 16) || misaligned(ffn_norm_g, 8) || misaligned(topk_idx, 4) ||
      misaligned(topk_w, 4) || (router_b && misaligned(router_b, 4)))
    return FOE_ERR_SHAPE;
  const int rc = launch_route_noalloc(static_cast<const bf16*>(h), static_cast<const bf16*>(ffn_norm_g), router_w, router_b,
                                      topk_idx, topk_w, n_tokens, hidden, n_clusters, experts_per_cluster,
                                      top_k_per_cluster, rms_eps, static_cast<cudaStream_t>(stream));
  return rc == 0 ? FOE_OK : (rc == -3 ? FOE_ERR_SHAPE : FOE_ERR_CUDA);
}

size_t foe_route_partial_capacity(int max_tokens, int max_seqs, int n_experts) {
  if (max_tokens <= 0 || max_seqs <= 0 || n_experts <= 0) return 0;
  return route_part_capacity(size_t(max_tokens > max_seqs ? max_tokens : max_seqs), size_t(n_experts));
}

size_t foe_route_partial_floats(int hidden, int n_experts, int n_tokens, int n_sms, size_t capacity) {
  if (hidden <= 0 || n_experts <= 0 || n_tokens <= 0 || n_sms <= 0) return 0;
  int ks = 1;                                             // the tensor-core score kernel does not split
  if (n_tokens <= kRouteSmallMaxTokens) ks = clamp_k_splits(route_small_k_splits(hidden), n_tokens, n_experts, capacity);
  else if (n_tokens < kRouterTcMinTokens) ks = clamp_k_splits(route_k_splits(n_tokens, hidden, n_experts, n_sms), n_tokens, n_experts, capacity);
  return size_t(ks) * size_t(n_tokens) * size_t(n_experts);
}

foe_status foe_get_aux(foe_layer* L, foe_aux* a) {
  if (!L || !a) return FOE_ERR_NULL;
  a->n_tokens = L->last_tokens;
  a->r_full = L->ws->r_full; a->u = L->ws->u; a->logits = L->ws->logits; a->topk_idx = L->ws->topk_idx; a->topk_w = L->ws->topk_w;
  a->counts = L->ws->pb.counts; a->offsets = L->ws->pb.offsets; a->perm = L->ws->pb.perm; a->inv = L->ws->pb.inv;
  a->q = L->ws->qkv; a->attn_o = L->ws->attn_o;
  return FOE_OK;
}

foe_status foe_poll_status(foe_layer* L, int* device_status) {
  if (!L || !device_status) return FOE_ERR_NULL;
  if (cudaStreamSynchronize(L->last_stream) != cudaSuccess) { cudaGetLastError(); return FOE_ERR_CUDA; }
  int v = 0;
  if (cudaMemcpy(&v, L->ws->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return FOE_ERR_CUDA;
  *device_status = v;
  if (v != 0) {
    cudaMemset(L->ws->status, 0, sizeof(int));
    // the split counters of the decode attention re-arm themselves; after a reported failure make sure of it
    cudaMemset(L->ws->split_done, 0, L->ws->split_done_count * sizeof(int));
  }
  return FOE_OK;
}

int foe_last_launch_count(const foe_layer* L) { return L ? L->launches : 0; }

foe_status foe_set_profiling(foe_layer* L, int enabled) {
  if (!L) return FOE_ERR_NULL;
  const int ring = enabled < 0 ? 0 : (enabled > 256 ? 256 : enabled);
  const size_t want = size_t(ring) * (kNumStages + 1);
  while (L->ev.size() < want) {
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); return FOE_ERR_CUDA; }
    L->ev.push_back(e);
  }
  L->profiling = ring;
  L->prof_calls = 0;
  L->ev_valid = false;
  return FOE_OK;
}

int foe_num_stages(void) { return kNumStages; }

const char* foe_stage_name(int i) { return (i >= 0 && i < kNumStages) ? kStageNames[i] : ""; }

foe_status foe_get_stage_ms(foe_layer* L, float* ms, int n) {
  if (!L || !ms) return FOE_ERR_NULL;
  if (!L->ev_valid || n < kNumStages || L->profiling <= 0 || L->prof_calls <= 0) return FOE_ERR_UNSUPPORTED;
  const int ring = L->profiling;
  const int sets = L->prof_calls < ring ? L->prof_calls : ring;          // the most recent calls still in the ring
  const int last = (L->prof_calls - 1) % ring;
  if (cudaEventSynchronize(L->ev[size_t(last) * (kNumStages + 1) + kNumStages]) != cudaSuccess) { cudaGetLastError(); return FOE_ERR_CUDA; }
  for (int i = 0; i < kNumStages; ++i) ms[i] = 0.f;
  for (int c = 0; c < sets; ++c) {
    const size_t base = size_t((L->prof_calls - 1 - c) % ring) * (kNumStages + 1);
    for (int i = 0; i < kNumStages; ++i) {
      float t = 0.f;
      if (cudaEventElapsedTime(&t, L->ev[base + i], L->ev[base + i + 1]) != cudaSuccess) { cudaGetLastError(); return FOE_ERR_CUDA; }
      ms[i] += t;
    }
  }
  for (int i = 0; i < kNumStages; ++i) ms[i] /= float(sets);
  L->prof_calls = 0;
  L->ev_valid = false;
  return FOE_OK;
}

// ------------------------------------------------------------------ cluster-per-GPU group (include/foe_shard.h)

size_t foe_shard_buffer_bytes(const foe_shard_config* c) {
  if (!shard_config_ok(c)) return 0;
  return shard_header_bytes(c) + 2 * shard_slots_bytes(c);       // slots and gather buffer have the same size
}

foe_status foe_shard_buffer_alloc(const foe_shard_config* c, void** buffer) {
  if (!c || !buffer) return FOE_ERR_NULL;
  *buffer = nullptr;
  const size_t bytes = foe_shard_buffer_bytes(c);
  if (bytes == 0) return FOE_ERR_CONFIG;
  void* p = nullptr;
  if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); return FOE_ERR_OOM; }
  if (cudaMemset(p, 0, bytes) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
    cudaGetLastError();
    cudaFree(p);
    return FOE_ERR_CUDA;
  }
  *buffer = p;
  return FOE_OK;
}

foe_status foe_shard_buffer_free(void* buffer) {
  if (buffer && cudaFree(buffer) != cudaSuccess) { cudaGetLastError(); return FOE_ERR_CUDA; }
  return FOE_OK;
}

foe_status foe_shard_buffer_export(void* buffer, unsigned char handle[64]) {
  if (!buffer || !handle) return FOE_ERR_NULL;
  static_assert(sizeof(cudaIpcMemHandle_t) == 64, "IPC handle size");
  cudaIpcMemHandle_t h;
  if (cudaIpcGetMemHandle(&h, buffer) != cudaSuccess) { cudaGetLastError(); return FOE_ERR_CUDA; }
  memcpy(handle, &h, sizeof(h));
  return FOE_OK;
}

foe_status foe_shard_buffer_import(const unsigned char handle[64], void** buffer) {
  if (!handle || !buffer) return FOE_ERR_NULL;
  *buffer = nullptr;
  cudaIpcMemHandle_t h;
  memcpy(&h, handle, sizeof(h));
  void* p = nullptr;
  if (cudaIpcOpenMemHandle(&p, h, cudaIpcMemLazyEnablePeerAccess) != cudaSuccess) { cudaGetLastError(); return FOE_ERR_CUDA; }
  *buffer = p;
  return FOE_OK;
}

foe_status foe_shard_buffer_close(void* imported) {
  if (imported && cudaIpcCloseMemHandle(imported) != cudaSuccess) { cudaGetLastError(); return FOE_ERR_CUDA; }
  return FOE_OK;
}

foe_status foe_shard_create(const foe_shard_config* c, void* const* buffers, foe_shard** out) {
  if (!c || !buffers || !out) return FOE_ERR_NULL;
  *out = nullptr;
  if (!shard_config_ok(c)) return FOE_ERR_CONFIG;
  for (int r = 0; r < c->n_ranks; ++r)
    if (!buffers[r]) return FOE_ERR_NULL;
  foe_shard* sh = new (std::nothrow) foe_shard();
  if (!sh) return FOE_ERR_OOM;
  sh->cfg = *c;
  sh->span = c->hidden / c->n_ranks;
  sh->n_blk = shard_blocks(c);
  sh->S_cap = size_t(c->max_tokens);
  sh->limit_ns = (unsigned long long)(c->wait_limit_ms > 0 ? c->wait_limit_ms : 2000) * 1000000ull;
  for (int r = 0; r < c->n_ranks; ++r) {
    uint8_t* b = static_cast<uint8_t*>(buffers[r]);
    sh->buf[r] = b;
    sh->table.slots[r] = reinterpret_cast<bf16*>(b + shard_header_bytes(c));
    sh->table.gather[r] = reinterpret_cast<bf16*>(b + shard_header_bytes(c) + shard_slots_bytes(c));
    sh->table.slot_cnt[r] = reinterpret_cast<unsigned int*>(b + 128) + size_t(c->rank) * sh->n_blk;   // rank r's counters of MY pushes
    sh->table.gather_cnt[r] = reinterpret_cast<unsigned int*>(b);                // rank r's counters, one per owner
  }
  if (cudaMalloc(reinterpret_cast<void**>(&sh->status), sizeof(int)) != cudaSuccess) { cudaGetLastError(); delete sh; return FOE_ERR_OOM; }
  cudaMemset(sh->status, 0, sizeof(int));
  *out = sh;
  return FOE_OK;
}

foe_status foe_shard_destroy(foe_shard* sh) {
  if (!sh) return FOE_OK;
  cudaFree(sh->status);
  delete sh;
  return FOE_OK;
}

// starts exchange number epoch + 1 for S tokens: buffer half and the totals its counters will have to reach
static foe_status shard_begin(foe_shard* sh, int S, cudaStream_t st) {
  if (sh->stage != 0) return FOE_ERR_UNSUPPORTED;
  if (S < 0 || S > sh->cfg.max_tokens) return FOE_ERR_SHAPE;
  sh->epoch += 1;
  sh->S = S;
  sh->gather_expect += unsigned(S) * unsigned(sh->span);
  sh->stage = 1;
  sh->last_stream = st;
  return FOE_OK;
}

foe_status foe_shard_attend(foe_layer* L, foe_shard* sh, const void* x, const foe_kv_cache* kv, int decode, void* stream) {
  if (!L || !sh || !kv) return FOE_ERR_NULL;
  if (L->H != 1 || L->d != sh->cfg.hidden) return FOE_ERR_CONFIG;
  if (kv->n_tokens < 0 || kv->n_seqs < 0) return FOE_ERR_SHAPE;
  const int S = decode ? kv->n_seqs : kv->n_tokens;
  if (S > 0) {
    if (!x) return FOE_ERR_NULL;
    const foe_status c = check_call(L, kv, decode != 0);
    if (c != FOE_OK) return c;
    if (misaligned(x, 16)) return FOE_ERR_SHAPE;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const foe_status b = shard_begin(sh, S, st);
  if (b != FOE_OK) return b;
  L->shard_stage = 1;
  if (S == 0) { L->launches = 0; L->last_tokens = 0; return FOE_OK; }
  return run_attend(L, x, kv, st, decode != 0, sh);
}

foe_status foe_shard_push(foe_shard* sh, const void* src, int n_tokens, float scale, void* stream) {
  if (!sh) return FOE_ERR_NULL;
  if (n_tokens > 0 && !src) return FOE_ERR_NULL;
  if (misaligned(src, 16)) return FOE_ERR_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const foe_status b = shard_begin(sh, n_tokens, st);
  if (b != FOE_OK) return b;
  if (n_tokens == 0) return FOE_OK;
  const long long slot_off = (long long)((size_t(sh->epoch & 1) * sh->cfg.n_ranks + sh->cfg.rank) * sh->S_cap * sh->span);
  launch_shard_push(src, 0, scale, n_tokens, sh->cfg.hidden, sh->cfg.n_ranks, sh->table, slot_off,
                    int(sh->epoch & 1) * 8 * sh->n_blk, st);
  return check_launch();
}

foe_status foe_shard_reduce(foe_shard* sh, void* stream) {
  if (!sh) return FOE_ERR_NULL;
  if (sh->stage != 1) return FOE_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  sh->stage = 2;
  sh->last_stream = st;
  if (sh->S == 0) return FOE_OK;
  const int H = sh->cfg.n_ranks, me = sh->cfg.rank;
  const size_t half = size_t(sh->epoch & 1);
  const bf16* my_slots = sh->table.slots[me] + half * H * sh->S_cap * sh->span;
  const unsigned int* my_cnt = reinterpret_cast<const unsigned int*>(sh->buf[me] + 128) + half * 8 * sh->n_blk;
  launch_shard_reduce(my_slots, my_cnt, sh->n_blk, sh->S, sh->S_cap, sh->cfg.hidden, H, me, sh->table,
                      (long long)(half * sh->S_cap * sh->cfg.hidden), sh->limit_ns, sh->status, st);
  return check_launch();
}

static foe_status shard_finish(foe_shard* sh, float* dst_f32, bf16* dst_bf16, cudaStream_t st) {
  if (sh->stage != 2) return FOE_ERR_UNSUPPORTED;
  sh->stage = 0;
  sh->last_stream = st;
  if (sh->S == 0) return FOE_OK;
  const int me = sh->cfg.rank;
  const bf16* my_gather = sh->table.gather[me] + size_t(sh->epoch & 1) * sh->S_cap * sh->cfg.hidden;
  unsigned int* my_cnt = reinterpret_cast<unsigned int*>(sh->buf[me] + 128) + size_t(sh->epoch & 1) * 8 * sh->n_blk;
  launch_shard_gather(my_gather, sh->table.gather_cnt[me], sh->gather_expect, sh->S, sh->cfg.hidden, sh->cfg.n_ranks,
                      dst_f32, dst_bf16, my_cnt, 8 * sh->n_blk, sh->limit_ns, sh->status, st);
  return check_launch();
}

foe_status foe_shard_ffn(foe_layer* L, foe_shard* sh, void* out, void* stream) {
  if (!L || !sh) return FOE_ERR_NULL;
  if (L->shard_stage != 1 || L->last_tokens != sh->S) return FOE_ERR_UNSUPPORTED;
  if (sh->S > 0 && !out) return FOE_ERR_NULL;
  if (misaligned(out, 16)) return FOE_ERR_SHAPE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  g_overlap_launches = false;             // (the exchange kernels are launched the ordinary way)
  const foe_status f = shard_finish(sh, L->ws->r_full, nullptr, st);      // r_full of the whole group, as fp32
  if (f != FOE_OK) return f;
  L->shard_stage = 0;
  L->last_stream = st;
  if (sh->S == 0) return FOE_OK;
  L->launches += 1;
  return run_ffn(L, out, st);
}

foe_status foe_shard_gather(foe_shard* sh, void* dst, void* stream) {
  if (!sh) return FOE_ERR_NULL;
  if (sh->S > 0 && !dst) return FOE_ERR_NULL;
  if (misaligned(dst, 16)) return FOE_ERR_SHAPE;
  return shard_finish(sh, nullptr, static_cast<bf16*>(dst), static_cast<cudaStream_t>(stream));
}

foe_status foe_shard_poll_status(foe_shard* sh, int* device_status) {
  if (!sh || !device_status) return FOE_ERR_NULL;
  if (cudaStreamSynchronize(sh->last_stream) != cudaSuccess) { cudaGetLastError(); return FOE_ERR_CUDA; }
  int v = 0;
  if (cudaMemcpy(&v, sh->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return FOE_ERR_CUDA;
  *device_status = v;
  if (v != 0) cudaMemset(sh->status, 0, sizeof(int));
  return FOE_OK;
}

}  // extern "C"
