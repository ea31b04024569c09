// Argument block and epilogue kinds of the GEMM kernels (plain data, host and device).
#pragma once

#include <cuda_bf16.h>
#include <vector_types.h>
#include <stddef.h>

namespace foe {

constexpr int kBM = 128;   // GEMM tile rows per CTA (UMMA M of a CTA pair = 256)
constexpr int kBN = 256;   // widest GEMM tile (UMMA N); the launcher narrows it in steps of 64 so that N splits evenly

// Tile width for N columns per group: as few tiles as 256 allows, all of the same width (384 columns are two tiles
// of 192, not one of 256 and a half-empty one).
constexpr int gemm_tile_cols(int N) {
  const int tiles = (N + kBN - 1) / kBN;
  return tiles <= 0 ? kBN : ((((N + tiles - 1) / tiles) + 63) / 64) * 64;
}

enum GemmEpilogue : int {
  kEpiBf16 = 0,     // C -> bf16 [row][ldo]
  kEpiSwiGLU = 1,   // columns [0,128) gate, [128,256) up of one 128-wide block: silu(gate)*up -> bf16
  kEpiQKV = 2,      // row scale (1/rms), RoPE, q -> [S][n_q*dh], k and v -> cache pages
  kEpiOProj = 3     // r_full = scale * (C + sum_h x[h]) -> fp32 [row][ldo]; the sum either read as bf16 streams or found in r_full
};

// Rows of B one CTA of a pair stages per k-block = box rows of the B tensor map: half a tile.  The SwiGLU epilogue
// needs the full 256-wide tile (128 gate columns, 128 up columns).
constexpr int gemm_tile_rows_b(int epi, int N) { return (epi == kEpiSwiGLU ? kBN : gemm_tile_cols(N)) / 2; }

// rows per arrival counter of a cluster-per-GPU exchange (= the row tile of the O-projection GEMM that pushes)
constexpr int kShardBlockRows = 256;

struct GemmArgs {
  // uniform groups
  int n_groups;
  int rows_per_group;
  int a_group_stride;       // first A row of group g = g * a_group_stride
  // ragged groups (n_mtiles != nullptr)
  const int* mt_group;      // [n_mtiles] group of each m-tile
  const int* mt_row0;       // [n_mtiles] first A row of each m-tile
  const int* group_end;     // [n_groups] one past the last A row of the group
  const int* n_mtiles;      // device scalar
  int N;                    // columns per group (rows of B per group)
  int K;
  int bn;                   // tile width, set by the launcher (2 * gemm_tile_rows_b)
  int* status;              // device status word
  // gathered A operand (expert GEMM 1): A row r of a tile is a_gather[a_row_index[r]][:]; nullptr = A through tmA
  const __nv_bfloat16* a_gather;
  const int* a_row_index;
  // epilogue
  void* out;
  int ldo;                  // elements per output row
  // kEpiQKV: rows are tokens; the group's columns are its q heads, then its k heads, then its v heads, every head
  // stored with its two halves interleaved (packed column 2i = natural i, 2i+1 = natural i + dh/2) so that a
  // rotation pair sits in adjacent accumulator columns.  The epilogue applies 1/rms, rotates q and k (RoPE) in
  // fp32 and writes q to out[token][n_q*dh] and k / v straight into their cache pages.
  const float* row_scale;   // [n_groups * scale_group_stride]
  int scale_group_stride;
  int q_cols, kv_cols;      // g*dh and c*dh of one cluster
  int dh, n_kv;
  int q_head_stride;        // elements between the heads of a q row in out (head_dim, or 128 for head_dim 96: the
                            // attention kernels read q with zero padding up to their tile width)
  const float2* rope_tab;   // [max_context][dh/2] (cos, sin)
  const int* tok_pos;       // [tokens] position of the token in its sequence
  const int* tok_slot;      // [tokens] page * 64 + offset of the token in the cache, -1 = none
  __nv_bfloat16* k_pages;   // [num_pages][n_kv][64][dh]
  __nv_bfloat16* v_pages;
  // kEpiOProj
  const __nv_bfloat16* xsum; // one bf16 residual stream [rows][ldo] added to C when x_count == 1 (x_count is 0 or 1)
  int x_count;
  size_t x_stride;
  float out_scale;
  int x_in_out;              // `out` already holds the fp32 sum of the residual streams: out = scale * (C + out)
  // kEpiOProj on one rank of a cluster-per-GPU group (push_span != 0): the scaled tile is not written to `out` but
  // pushed as bf16 to the rank that owns its columns -- columns [o * push_span, (o + 1) * push_span) belong to rank
  // o -- at push_base[o] + push_slot_off + row * push_span + (column - o * push_span); push_cnt[o][row / 256] then grows
  // by the number of elements written (after a system-scope fence), which is what the owner's reduction of those rows
  // waits for.
  // The pointers are this rank's mappings of the owners' buffers (peer memory, or plain local memory).
  __nv_bfloat16* push_base[8];
  unsigned int* push_cnt[8];
  int push_span;
  long long push_slot_off;
};

}  // namespace foe
