// Host-side entry points shared between the translation units of the draft call.
#pragma once
#include "attention_params.cuh"

namespace dpara {

// attention-only scratch (split-KV partials); 0 when the chosen kernel needs none
size_t attention_workspace_bytes(const dpara_shape *shape, const int64_t *host_ctx_offsets);
dpara_status launch_attention(const dpara_shape *shape, const dpara_attn_io *io, void *workspace, int32_t *status_word,
                              cudaStream_t st);

// out[row] = bf16(x[row] / sqrt(mean(x^2) + eps) * gain) for M rows of H bf16 elements (gain may be null)
dpara_status launch_rmsnorm_bf16(const void *x, const void *gain, void *out, int M, int H, float eps, cudaStream_t st);

// full backbone block around the attention
size_t layer_workspace_bytes(const dpara_shape *shape, const dpara_layer_io *layer);
// byte offsets of xn, qkv, q, k, v, a, h1, hn, act inside the workspace of a full-layer call
void layer_workspace_offsets(const dpara_shape *shape, const dpara_layer_io *layer, size_t attn_bytes, size_t out[9]);
dpara_status launch_layer(const dpara_shape *shape, const dpara_attn_io *io, const dpara_layer_io *layer, void *workspace,
                          int32_t *status_word, cudaStream_t st);

}  // namespace dpara
