// Host-side interface of the tensor-core all-boundary attention.
#pragma once
#include "attention_params.cuh"

namespace dpara {

struct TcPlan {
  bool eligible;        // false: shape outside what the tensor-core kernel handles (use the general kernel)
  int JI_T;             // (boundary, slot) rows per 128-row query tile = 128 / G
  int n_ji, n_tiles, n_pairs;
  int nsplit;           // KV splits per (request, KV head, tile pair)
  int S8, R_blk;        // tail tile: block keys start at row S8 and span R_blk rows
  long long items;      // batch * Hkv * n_pairs
  size_t workspace_bytes;
};

TcPlan plan_attention_tc(const dpara_shape *s, const int64_t *host_ctx_offsets);
dpara_status launch_attention_tc(const AttnParams &A, const TcPlan &plan, const int64_t *host_ctx_offsets, void *workspace,
                                 cudaStream_t st);

}  // namespace dpara
