/*
 * foe_shard.h -- C ABI for running one FoE block with ONE CLUSTER PER GPU (Section 3.2 of the paper: every
 * cluster keeps its attention heads, its experts and its KV cache on its own device, and the only traffic between
 * clusters is one all-reduce of the attention residual per layer -- Table 2, row "sync").
 *
 * Rank h of a group of H GPUs holds a layer handle created by foe_layer_create for cluster h alone:
 * n_clusters = 1, n_q_heads = g, n_kv_heads = c, experts_per_cluster = E_c, and the weight pointers of cluster h
 * (wq/wk/wv slice h, rows h*g*head_dim.. of wo, experts h*E_c.., router rows h*E_c..).  The block then runs as
 *
 *     foe_shard_attend   attention of cluster h; the O-projection pushes (x[h] + Attn_h)/H, tile by tile from
 *                        its epilogue, into the receive buffers of the ranks that own the columns
 *     foe_shard_reduce   this rank adds the H partials of the columns it owns and writes the result, r_full, into
 *                        every rank's gather buffer
 *     foe_shard_ffn      waits for r_full, then routing, experts and combine of cluster h: out = x'[h]
 *
 * queued back to back on one stream.  The exchange is a reduce-scatter followed by an all-gather, both as plain
 * stores into peer memory (bf16 payload, fp32 sums in rank order, so results do not depend on timing) with
 * arrival counters; no kernel of this library is given another GPU's memory through a tensor map.
 * foe_shard_push / foe_shard_reduce / foe_shard_gather run the same exchange on a tensor that already sits in
 * memory (the mean over clusters that ends the last layer, Section 3.1).
 * Precision: every partial and the reduced r_full cross the links as bf16, so the r_full a rank's routing and experts
 * see is the fp32 sum of bf16-rounded partials, rounded to bf16 once more.  The one-device block (foe_prefill /
 * foe_decode) keeps r_full in fp32 from the O-projection to the combine; the two ways of running a block therefore
 * agree within the output tolerance but not bit for bit.
 *
 * Exchange buffers.  Every rank allocates one buffer with foe_shard_buffer_alloc and makes it visible to the other
 * ranks: in one process driving several devices the pointers are used directly (with peer access enabled by the
 * caller); across processes foe_shard_buffer_export / foe_shard_buffer_import carry it through CUDA IPC.
 * foe_shard_create takes the table of all H buffers as this process sees them.
 *
 * Ordering rule.  A wait inside a kernel is bounded (wait_limit_ms; afterwards the device status becomes
 * FOE_ERR_TIMEOUT and the kernel returns), and it only ever waits for kernels that the other ranks queue EARLIER in
 * their own sequence.  With one rank per GPU every rank simply issues attend, reduce, ffn.  When several ranks are
 * driven on ONE device (a test, or a single-GPU emulation of the group) their kernels do not run concurrently, so
 * the caller must issue every rank's attend (or push) before any rank's reduce, and every reduce before any ffn
 * (or gather); then no wait ever has to spin.
 *
 * Conventions as in foe.h: device pointers unless marked host, calls asynchronous on the given stream, checks on
 * the host before anything is launched, no CPU fallback.
 */
#ifndef FOE_SHARD_H_
#define FOE_SHARD_H_

#include "foe.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Validity: 1 <= n_ranks <= 8, 0 <= rank < n_ranks, hidden % (32 * n_ranks) == 0, max_tokens > 0,
 * wait_limit_ms > 0 (0 selects the default of 2000). */
typedef struct {
  int rank, n_ranks;   /* this GPU's cluster h and the number of clusters H */
  int hidden;          /* d */
  int max_tokens;      /* largest S of any exchange */
  int wait_limit_ms;   /* bound of every device-side wait */
} foe_shard_config;

typedef struct foe_shard foe_shard;

/* Bytes of one rank's exchange buffer: a header of arrival counters (per owner for the gather buffer; per exchange
 * parity, source rank and block of 256 rows for the receive slots), receive slots [2][H][max_tokens][d/H] bf16 and the
 * gather buffer [2][max_tokens][d] bf16.  0 if the description is invalid. */
size_t foe_shard_buffer_bytes(const foe_shard_config* config);

/* Allocates (cudaMalloc on the current device) and zeroes one exchange buffer; synchronises.  The buffer belongs to the
 * caller until foe_shard_buffer_free. */
foe_status foe_shard_buffer_alloc(const foe_shard_config* config, void** buffer);
foe_status foe_shard_buffer_free(void* buffer);

/* CUDA IPC transport of a buffer to the other ranks' processes: export writes the 64-byte handle (host memory);
 * import maps a peer's buffer into this process (with peer access) and returns its address; close unmaps it. */
foe_status foe_shard_buffer_export(void* buffer, unsigned char handle[64]);
foe_status foe_shard_buffer_import(const unsigned char handle[64], void** buffer);
foe_status foe_shard_buffer_close(void* imported_buffer);

/* buffers: host array of n_ranks device pointers, entry r = rank r's exchange buffer as addressable from this
 * process (entry `rank` is this rank's own).  All ranks must use the same description apart from `rank`.  The
 * buffers must outlive the handle. */
foe_status foe_shard_create(const foe_shard_config* config, void* const* buffers, foe_shard** out);
foe_status foe_shard_destroy(foe_shard* shard);

/* Table 2, rows "attention" and "sync" (first half) on rank h.  layer: a handle with n_clusters == 1 and
 * hidden == config.hidden built from cluster h's weights; its position and sync fields keep their meaning
 * (FOE_FIRST/FOE_SINGLE: x is the shared [S][hidden] input and rank 0 alone contributes it to the sum).
 * x: [S][hidden] bf16 = x[h]; kv: cluster h's own cache ([num_pages][c][64][head_dim]).  decode != 0 selects the
 * one-token-per-sequence kernels (S = kv->n_seqs).  Errors as foe_prefill / foe_decode, FOE_ERR_SHAPE if S exceeds
 * config.max_tokens, FOE_ERR_UNSUPPORTED if the previous exchange on `shard` has not been finished. */
foe_status foe_shard_attend(foe_layer* layer, foe_shard* shard, const void* x, const foe_kv_cache* kv, int decode,
                            void* stream);

/* The same first half for a tensor in memory: src [n_tokens][hidden] bf16, multiplied by `scale` and rounded to bf16,
 * goes to the owners of its columns. */
foe_status foe_shard_push(foe_shard* shard, const void* src, int n_tokens, float scale, void* stream);

/* Second step of the exchange started by the last attend / push: sum over ranks of the columns this rank owns, result
 * written to every rank.  FOE_ERR_UNSUPPORTED if nothing was pushed. */
foe_status foe_shard_reduce(foe_shard* shard, void* stream);

/* Table 2, rows "routing", "experts", "combine" on rank h, after the exchange: waits for r_full, then
 * out = x'[h] = r_full + sum over cluster h's selected experts ([S][hidden] bf16; on a last layer the caller
 * averages x'[h] over the ranks with push(scale 1/H) / reduce / gather).  FOE_ERR_UNSUPPORTED unless the last calls
 * on (layer, shard) were foe_shard_attend and foe_shard_reduce. */
foe_status foe_shard_ffn(foe_layer* layer, foe_shard* shard, void* out, void* stream);

/* Third step for a pushed tensor: waits for the sum and writes it to dst ([n_tokens][hidden] bf16). */
foe_status foe_shard_gather(foe_shard* shard, void* dst, void* stream);

/* Synchronises the last stream used on `shard`, reads its device status word (FOE_OK or FOE_ERR_TIMEOUT) and resets
 * it.  After a timeout the exchange counters of the group no longer agree: destroy the handles and re-zero the buffers. */
foe_status foe_shard_poll_status(foe_shard* shard, int* device_status);

#ifdef __cplusplus
}
#endif
#endif /* FOE_SHARD_H_ */
