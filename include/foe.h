/*
 * foe.h -- C ABI of the B200 (sm_100a) forward pass of one Federation-of-Experts (FoE)
 * transformer block.
 *
 * The operation is the per-layer compute of the paper's Table 2 (right column) with the
 * layer-boundary rules and the group-limited routing rule of Section 3.1:
 *
 *     r[h,i]    = x[h,i] + Attn_h(x[h,:])[i]                      attention residual, per cluster h
 *     r_full[i] = (1/H) sum_h r[h,i]                              cross-cluster sync
 *     I_h[i], w_h[i] = TopK_{e in E_h}(Router(r_full[i]), k/H)    per-cluster routing
 *     x'[h,i]   = r_full[i] + sum_{e in I_h[i]} w_h[i,e] FFN_e(r_full[i])
 *
 * On one GPU the sync is a local reduction and dispatch/combine are local permutations.
 *
 * Conventions
 *  - Every pointer in foe_weights, foe_kv_cache and the x/out/h/topk arguments is a DEVICE
 *    pointer unless marked "host".  Structs themselves live in host memory.
 *  - bf16 tensors are row-major with the last index contiguous.  Tokens of a call are the
 *    sequences' new tokens concatenated in sequence order (S = sum of q_lens).
 *  - Cluster h owns query heads h*g..(h+1)*g-1 (g = n_q_heads / n_clusters), KV heads
 *    h*c..(h+1)*c-1 (c = n_kv_heads / n_clusters), rows h*g*head_dim.. of W_O and experts
 *    h*E_c..(h+1)*E_c-1.
 *  - All tensor memory belongs to the caller.  foe_layer_create copies and repacks the weights
 *    into library-owned device buffers, so the caller may release its copies afterwards.  The
 *    handle owns a workspace sized by max_tokens / max_seqs / max_context.
 *  - Calls are asynchronous on the given stream (a cudaStream_t passed as void*).  A handle is
 *    used from one stream at a time.  Same inputs give bit-identical outputs and maps.  After one
 *    ordinary call per entry point and call size class (it sets kernel attributes once) a call only
 *    launches kernels, so it can be captured into a CUDA graph.
 *  - Every function returns a foe_status; argument and shape checks happen on the host before
 *    anything is launched.  Conditions only the device can see (a bounded wait that ran out, an
 *    out-of-range page id) are recorded in a device status word read by foe_poll_status.
 *  - There is no CPU fallback: without a CUDA device every compute entry point fails.
 */
#ifndef FOE_H_
#define FOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FOE_OK = 0,
  FOE_ERR_NULL = -1,         /* a required pointer is NULL */
  FOE_ERR_CONFIG = -2,       /* foe_config violates a validity rule */
  FOE_ERR_SHAPE = -3,        /* call sizes exceed what the handle was created for */
  FOE_ERR_UNSUPPORTED = -4,
  FOE_ERR_OOM = -5,          /* device allocation failed */
  FOE_ERR_CUDA = -6,         /* a CUDA runtime/driver call failed */
  FOE_ERR_TIMEOUT = -7,      /* device status: a bounded wait inside a kernel ran out */
  FOE_ERR_BOUNDS = -8        /* device status: an index read from device memory was out of range */
} foe_status;

typedef enum { FOE_MIDDLE = 0, FOE_FIRST = 1, FOE_LAST = 2, FOE_SINGLE = 3 } foe_position;
typedef enum { FOE_SYNC_MEAN = 0, FOE_SYNC_SUM = 1 } foe_sync;

/* Layer description.  Validity: n_kv_heads % n_clusters == 0, n_q_heads % n_kv_heads == 0,
 * head_dim in {64, 96, 128}, 1 <= top_k_per_cluster <= experts_per_cluster <= 128, top_k_per_cluster <= 32,
 * page_size == 64, hidden % 128 == 0, (n_q_heads * head_dim) % 128 == 0, ffn_inter % 128 == 0,
 * n_clusters <= 8, n_clusters * experts_per_cluster <= 1024, n_q_heads / n_kv_heads <= 16, max_* > 0.
 * position: FOE_FIRST/FOE_SINGLE take x as [S, hidden] (one shared attention, its residual used
 * in place of r_full); FOE_LAST/FOE_SINGLE write out as [S, hidden] (mean over clusters of x').
 * Otherwise x and out are [n_clusters, S, hidden]. */
typedef struct {
  int hidden, n_q_heads, n_kv_heads, n_clusters, head_dim;
  int experts_per_cluster, top_k_per_cluster, ffn_inter;
  int page_size;
  int max_tokens;      /* largest S of a prefill call */
  int max_seqs;        /* largest n_seqs of any call (= largest S of a decode call) */
  int max_context;     /* largest context_len + q_len any sequence reaches */
  float rope_theta, rms_eps;
  int position;        /* foe_position */
  int sync;            /* foe_sync */
} foe_config;

/* Caller's weights (device pointers; bf16 unless stated). */
typedef struct {
  const void* attn_norm_g;   /* [hidden] gain of the RMSNorm before attention (shared by clusters) */
  const void* wq;            /* [H][hidden][g*head_dim] */
  const void* wk;            /* [H][hidden][c*head_dim] */
  const void* wv;            /* [H][hidden][c*head_dim] */
  const void* wo;            /* [n_q_heads*head_dim][hidden] */
  const void* ffn_norm_g;    /* [hidden] gain of the RMSNorm before router and experts */
  const void* w_gate;        /* [E][hidden][ffn_inter] */
  const void* w_up;          /* [E][hidden][ffn_inter] */
  const void* w_down;        /* [E][ffn_inter][hidden] */
  const float* router_w;     /* [E][hidden] fp32; rows h*E_c.. are cluster h's router */
  const float* router_b;     /* [E] fp32 additive score bias, or NULL */
} foe_weights;

/* Paged KV cache of one layer.  K is stored after RoPE.  The call writes K/V of the new tokens at
 * logical positions context_lens[s] .. context_lens[s]+q_len-1 through block_table (pages must be
 * assigned already) and attends over context_lens[s]+q_len entries.  It never changes context_lens. */
typedef struct {
  void* k_pages;              /* [num_pages][n_kv_heads][page_size][head_dim] bf16 */
  void* v_pages;
  const int* block_table;     /* [n_seqs][max_pages_per_seq] physical page ids */
  const int* context_lens;    /* [n_seqs] tokens cached before this call */
  const int* q_lens;          /* [n_seqs] new tokens in this call; NULL means 1 each (decode) */
  int n_seqs, max_pages_per_seq, num_pages;
  int n_tokens;               /* host copy of sum(q_lens) (ignored by foe_decode) */
  int max_q_len;              /* host upper bound of q_lens (ignored by foe_decode) */
} foe_kv_cache;

/* Device pointers to the intermediates of the last call on a handle (valid until the next call). */
typedef struct {
  int n_tokens;
  const float* r_full;      /* [S][hidden] fp32 synced residual */
  const void* u;            /* [S][hidden] bf16 FFN-normed r_full (expert input) */
  const float* logits;      /* [S][E] fp32 router scores */
  const int* topk_idx;      /* [S][H][k_c] global expert ids */
  const float* topk_w;      /* [S][H][k_c] gates */
  const int* counts;        /* [E] rows per expert */
  const int* offsets;       /* [E+1] exclusive scan of counts */
  const int* perm;          /* [S*H*k_c] slot -> token */
  const int* inv;           /* [S][H][k_c] -> slot */
  const void* q;            /* [S][n_q][head_dim, padded to 128 when it is 96] bf16 queries after RoPE (K and V of the
                               call are in the cache pages) */
  const void* attn_o;       /* [S][n_q*head_dim] bf16 attention output before W_O */
} foe_aux;

typedef struct foe_layer foe_layer;

/* Table 2 + Section 3.1: build a layer from its description and weights (host structs, device weight
 * pointers).  Allocates the repacked weights and the workspace; runs a few repack kernels on the
 * default stream and synchronises.  *out receives the handle. */
foe_status foe_layer_create(const foe_config* config, const foe_weights* weights, foe_layer** out);

/* Same as foe_layer_create, but the new layer borrows the workspace of `donor` instead of allocating its own
 * (a 16-layer stack needs one workspace, not sixteen).  The two layers must agree in every shape field and in
 * max_tokens / max_seqs / max_context (FOE_ERR_SHAPE otherwise); position, sync, rope_theta and rms_eps may differ.
 * Layers that share a workspace must not run concurrently; foe_get_aux of any of them shows the intermediates of
 * whichever ran last.  The workspace is released when its last user is destroyed.  donor == NULL allocates. */
foe_status foe_layer_create_shared(const foe_config* config, const foe_weights* weights, foe_layer* donor,
                                   foe_layer** out);

/* Frees everything the handle owns.  NULL is accepted. */
foe_status foe_layer_destroy(foe_layer* layer);

/* Alignment, all calls: device pointers to bf16 or fp32 tensors (weights, x, out, work buffers, K/V pages, h) must be
 * 16-byte aligned, int32 and per-expert fp32 arrays (block_table, context_lens, q_lens, router_b, topk_idx, topk_w)
 * 4-byte aligned.  A misaligned pointer is refused with FOE_ERR_SHAPE before anything is launched. */

/* Table 2 (all four rows) for S = kv->n_tokens new tokens of kv->n_seqs sequences: attention over the
 * paged cache plus the new tokens (causal), sync, routing, experts, combine.  x: [H][S][hidden] bf16
 * ([S][hidden] on a first layer); out likewise ([S][hidden] on a last layer); out must not alias x.
 * Calls of a few hundred tokens (short prompt chunks, small mixed batches) are run with the weight-streaming kernels
 * of the decode step where those fit; results do not depend on the entry point beyond rounding.
 * Errors: FOE_ERR_NULL, FOE_ERR_SHAPE (S > max_tokens, n_seqs > max_seqs, S == 0 is FOE_OK, no work). */
foe_status foe_prefill(foe_layer* layer, const void* x, const foe_kv_cache* kv, void* out, void* stream);

/* Same computation for one new token per sequence (S = kv->n_seqs, q_lens ignored), built for the
 * bandwidth-bound regime: split-KV paged attention and weight-streaming expert kernels.
 * x_step: [H][n_seqs][hidden] bf16 ([n_seqs][hidden] on a first layer). */
foe_status foe_decode(foe_layer* layer, const void* x_step, const foe_kv_cache* kv, void* out, void* stream);

/* A stack of layers (Section 3.1 "Layer boundaries": a first layer, middle layers, a last layer) in ONE host call:
 * layer l runs foe_prefill (decode == 0) or foe_decode (decode != 0) on the output of layer l-1 with its own cache
 * kvs[l] (host array of n_layers structs; they normally share block_table / context_lens / q_lens and differ in the
 * pages).  x is the first layer's input, out the last layer's output; work0 and work1 are two caller-owned device
 * buffers of n_clusters * S * hidden bf16 each for the activations between layers (work0 may be NULL for one layer,
 * work1 for up to two); none of x, out, work0, work1 may alias another.  Every layer's arguments are checked before
 * anything is launched; consecutive layers must fit (FOE_ERR_CONFIG: a first layer after another layer, a layer after
 * a last layer, different hidden sizes or cluster counts).  The layers may share one workspace.  Exactly the launches
 * of the single-layer calls, issued back to back: results are bit-identical to calling the layers one by one. */
foe_status foe_stack_forward(foe_layer* const* layers, int n_layers, const void* x, const foe_kv_cache* kvs, void* out,
                             void* work0, void* work1, int decode, void* stream);

/* context_lens[i] += by for i < n_seqs, on the stream (device array): after a decode step (by = 1) or a prompt chunk,
 * so that a generation loop keeps the lengths on the device and its steps can be replayed from a CUDA graph. */
foe_status foe_context_advance(int* context_lens, int n_seqs, int by, void* stream);

/* Section 3.1 "Routing": FFN RMSNorm, fp32 router scores, per-cluster top-k (larger score first, equal
 * scores -> lower expert id) and gates (softmax over the selected scores) for n_tokens rows of
 * h = r_full given as [n_tokens][hidden] bf16.  topk_idx: [n_tokens][H][k_c] int32 global expert ids;
 * topk_w: [n_tokens][H][k_c] fp32.  Also refreshes counts/offsets/perm/inv in the aux record. */
foe_status foe_route(foe_layer* layer, const void* h, int n_tokens, int* topk_idx, float* topk_w, void* stream);

/* The paper has no counterpart for this call; it exists for callers that cannot allocate device memory.
 * Examples: a server that gave all GPU memory to its own pool at start-up, so that cudaMalloc has nothing
 * left to hand out; a thread on a latency-critical path that must stay clear of the driver's allocator (its
 * lock, and the device-wide synchronisation that comes with freeing).  Such callers cannot create a handle
 * either, because foe_layer_create allocates.  foe_route_noalloc computes what foe_route computes -- FFN
 * RMSNorm of h, fp32 router scores, per-cluster top-k and gates -- from plain arguments and never calls
 * cudaMalloc, cudaFree or anything else that allocates.  Its scratch is a fixed array inside the library
 * image (about 6 MB, present on every GPU that loads the library until the process exits).
 *   ffn_norm_g [hidden] bf16, router_w [E][hidden] fp32, router_b [E] fp32 or NULL, h [n_tokens][hidden] bf16,
 *   topk_idx / topk_w [n_tokens][n_clusters][top_k_per_cluster] (int32 global expert ids / fp32 gates): all
 *   device pointers owned by the caller.  The dispatch maps and the expert input are not produced.
 * Limits: n_tokens <= 8192 and n_tokens * n_clusters * experts_per_cluster <= 524288; larger calls return
 * FOE_ERR_SHAPE and launch nothing.  Shape rules as for the layer description (FOE_ERR_CONFIG otherwise).
 * Alignment: h and router_w on 16 bytes, ffn_norm_g on 8, router_b / topk_idx / topk_w on 4 (FOE_ERR_SHAPE otherwise,
 * nothing launched): a sliced view that starts in the middle of a row group does not qualify.
 * The first call on each device looks up the device address of the scratch array (with that device current);
 * make that first call before any stream capture begins.  With lazy module loading that first call is also the
 * moment the driver places the library's code and this array on the device, so make it before your own pool takes
 * the memory that is left (it returns FOE_ERR_CUDA if the image cannot be loaded).  First calls from several host
 * threads at once are safe.  Every call on a device uses the same scratch, which
 * simply keeps the previous call's contents (nothing in it needs clearing: each call writes what it reads);
 * two calls that overlap on the GPU -- different streams, or different host threads -- race on it, so run
 * them one after the other. */
foe_status foe_route_noalloc(int hidden, int n_clusters, int experts_per_cluster, int top_k_per_cluster, float rms_eps,
                             const void* ffn_norm_g, const float* router_w, const float* router_b, const void* h,
                             int n_tokens, int* topk_idx, float* topk_w, void* stream);

/* Pointers to the last call's intermediates (host struct filled with device pointers). */
foe_status foe_get_aux(foe_layer* layer, foe_aux* out);

/* Synchronises the handle's last stream and reads the device status word into *device_status
 * (FOE_OK, FOE_ERR_TIMEOUT or FOE_ERR_BOUNDS); the word is reset to FOE_OK afterwards. */
foe_status foe_poll_status(foe_layer* layer, int* device_status);

/* Number of kernel launches the last prefill/decode/route call on this handle issued. */
int foe_last_launch_count(const foe_layer* layer);

/* Per-stage device timing of prefill/decode calls.  When enabled, every call records CUDA events on its
 * stream between the stages of the block; foe_get_stage_ms waits for the last call and writes the
 * foe_num_stages() elapsed times (milliseconds) into ms[0..n), n >= foe_num_stages().  foe_stage_name(i)
 * names stage i.  FOE_ERR_UNSUPPORTED if the last call was not recorded.
 * `enabled` is the number of most recent calls whose events are kept (0 = off, 1 = the last call, at most 256):
 * with enabled > 1 the calls can be issued back to back without reading anything in between, and foe_get_stage_ms
 * returns the mean over the calls recorded since it was last read (the most recent `enabled` of them), so that stage
 * times can be taken deep inside a long run of steps, at the clocks the GPU settles to. */
foe_status foe_set_profiling(foe_layer* layer, int enabled);
int foe_num_stages(void);
const char* foe_stage_name(int i);
foe_status foe_get_stage_ms(foe_layer* layer, float* ms, int n);

/* Host-only arithmetic, no device work (used by the tests; Section 3.1 "Routing" is the step they size).
 * The fp32 score kernels cut the hidden dimension into k_splits slices when a call has too few tokens to fill the
 * GPU; the slices' partial scores ([k_splits][n_tokens][n_experts] floats) go to a workspace buffer and are summed
 * in a fixed order.  foe_route_partial_capacity: floats of that buffer in a handle created with these sizes.
 * foe_route_partial_floats: floats a routing call of n_tokens tokens writes there on a device with n_sms SMs when
 * the buffer holds `capacity` floats (the number of slices is halved until they fit; 0 for n_tokens <= 0). */
size_t foe_route_partial_capacity(int max_tokens, int max_seqs, int n_experts);
size_t foe_route_partial_floats(int hidden, int n_experts, int n_tokens, int n_sms, size_t capacity);

/* Static description of a status code. */
const char* foe_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* FOE_H_ */
