// Host-side interface of the tensor-core all-boundary attention.
#pragma once
#include "attention_params.cuh"

namespace dpara {

struct TcPlan {
  bool eligible;        // false: shape outside what the tensor-core kernel handles (use the general kernel)
  int n_ji, n_pairs;    // (boundary, slot) rows per request; tile pairs per (request, KV head), all head blocks
  int n_hblk, hb_log2[4], h0[4], pair_start[5];  // head blocks (binary digits of the group size) and their tile pairs
  int nsplit;           // KV splits per (request, KV head, tile pair)
  int S8, cap0, cap;    // tail tiles: spine rows rounded up to 8; own blocks held by the first / by every later tail tile
  long long items;      // batch * Hkv * n_pairs
  size_t workspace_bytes;
};

TcPlan plan_attention_tc(const dpara_shape *s, const int64_t *host_ctx_offsets);
dpara_status launch_attention_tc(const AttnParams &A, const TcPlan &plan, const int64_t *host_ctx_offsets, void *workspace,
                                 cudaStream_t st);

}  // namespace dpara
