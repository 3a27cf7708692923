// Host-side entry points shared between the translation units of the draft call.
#pragma once
#include "attention_params.cuh"

namespace dpara {

// attention-only scratch (split-KV partials); 0 when the chosen kernel needs none
size_t attention_workspace_bytes(const dpara_shape *shape, const int64_t *host_ctx_offsets);
// blk_req_rows / spine_req_rows: rows from one request's block (spine) keys to the next request's when they differ from
// J * Bq (S), e.g. when both live in one buffer of J * Bq + S rows per request; 0 = the default
dpara_status launch_attention(const dpara_shape *shape, const dpara_attn_io *io, void *workspace, int32_t *status_word,
                              cudaStream_t st, int blk_req_rows = 0, int spine_req_rows = 0);

// out[row] = bf16(x[row] / sqrt(mean(x^2) + eps) * gain) for M rows of H bf16 elements (gain may be null)
dpara_status launch_rmsnorm_bf16(const void *x, const void *gain, void *out, int M, int H, float eps, cudaStream_t st);

// a stack of blocks (each reads the previous one's bf16 output and its own context cache)
size_t backbone_workspace_bytes(const dpara_shape *shape, const int64_t *host_ctx_offsets, const dpara_backbone_io *bb);
dpara_status launch_backbone(const dpara_shape *shape, const dpara_attn_io *io, const dpara_backbone_io *bb, void *workspace,
                             int32_t *status_word, cudaStream_t st);

// full backbone block around the attention
size_t layer_workspace_bytes(const dpara_shape *shape, const dpara_layer_io *layer);
// byte offsets of xn, qkv, q, k, v, a, h1, hn, act inside the workspace of a full-layer call
void layer_workspace_offsets(const dpara_shape *shape, const dpara_layer_io *layer, size_t attn_bytes, size_t out[9]);
dpara_status launch_layer(const dpara_shape *shape, const dpara_attn_io *io, const dpara_layer_io *layer, void *workspace,
                          int32_t *status_word, cudaStream_t st);

}  // namespace dpara
