// Host-side interface of the tensor-core all-boundary attention.
#pragma once
#include "attention_params.cuh"

namespace dpara {

struct TcPlan {
  bool eligible;        // false: shape outside what the tensor-core kernel handles (use the general kernel)
  int n_ji, n_pairs;    // (boundary, slot) rows per request; items (tile pairs, or single tiles) per (request, KV head), all head blocks
  int tiles_per_item;   // 2: an item is a pair of 128-row query tiles; 1: a single tile (small batches)
  int n_rows;           // query rows per request and head: n_ji, plus the spine rows when they are queries
  int n_hblk, hb_log2[4], h0[4], pair_start[5];  // head blocks (binary digits of the group size) and their tile pairs
  int nsplit;           // KV splits per (request, KV head, tile pair)
  int S8, cap0, cap;    // tail tiles: spine rows rounded up to 8; own blocks held by the first / by every later tail tile
  long long items;      // batch * Hkv * n_pairs
  size_t workspace_bytes;      // split-KV scratch this launch uses
  size_t workspace_max_bytes;  // ... and the most any context lengths within the same offsets can need
};

// host_ctx_lens may be null (request n fills rows host_ctx_offsets[n] .. host_ctx_offsets[n + 1])
TcPlan plan_attention_tc(const dpara_shape *s, const int64_t *host_ctx_offsets, const int64_t *host_ctx_lens);
dpara_status launch_attention_tc(const AttnParams &A, const TcPlan &plan, const int64_t *host_ctx_offsets,
                                 const int64_t *host_ctx_lens, void *workspace, cudaStream_t st);

}  // namespace dpara
