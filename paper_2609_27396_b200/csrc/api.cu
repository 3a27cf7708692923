// C-ABI entry points of the draft call: argument validation, workspace sizing, kernel selection by shape.
#include "attention_params.cuh"
#include "layer.cuh"

#include <atomic>

using namespace dpara;

namespace dpara {

static std::atomic<long long> g_launches{0};
void count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

static dpara_status validate_shape(const dpara_shape *s) {
  if (!s) return DPARA_ERR_INVALID_ARG;
  if (s->batch <= 0 || s->n_boundaries <= 0 || s->block <= 0 || s->n_q_heads <= 0 || s->n_kv_heads <= 0) return DPARA_ERR_INVALID_ARG;
  if (s->n_spine < 0 || s->prefix_base < 0) return DPARA_ERR_INVALID_ARG;
  if (s->boundary_lo < 0 || s->boundary_hi > s->n_boundaries || s->boundary_lo > s->boundary_hi) return DPARA_ERR_INVALID_ARG;
  if (!(s->softmax_scale >= 0.f)) return DPARA_ERR_INVALID_ARG;
  if (s->spine_queries != 0 && s->spine_queries != 1) return DPARA_ERR_INVALID_ARG;
  if (s->spine_queries && (s->boundary_lo != 0 || s->boundary_hi != s->n_boundaries || s->n_spine == 0)) return DPARA_ERR_UNSUPPORTED;
  if (s->head_dim != 64 && s->head_dim != 128) return DPARA_ERR_UNSUPPORTED;
  if (s->n_q_heads % s->n_kv_heads != 0) return DPARA_ERR_UNSUPPORTED;
  if (s->n_q_heads / s->n_kv_heads > 16 || s->block > 64 || s->n_spine > 64) return DPARA_ERR_UNSUPPORTED;
  return DPARA_OK;
}

static dpara_status validate_offsets(const dpara_shape *s, const int64_t *h) {
  if (!h) return DPARA_ERR_INVALID_ARG;
  if (h[0] < 0) return DPARA_ERR_INVALID_ARG;
  for (int n = 0; n < s->batch; ++n)
    if (h[n + 1] < h[n]) return DPARA_ERR_INVALID_ARG;
  return DPARA_OK;
}

}  // namespace dpara

extern "C" size_t dpara_draft_workspace_bytes(const dpara_shape *shape, const int64_t *host_ctx_offsets,
                                              const dpara_layer_io *layer, int full_layer) {
  if (validate_shape(shape) != DPARA_OK || validate_offsets(shape, host_ctx_offsets) != DPARA_OK) return 0;
  size_t bytes = attention_workspace_bytes(shape, host_ctx_offsets);
  if (full_layer) {
    if (!layer) return 0;
    bytes += layer_workspace_bytes(shape, layer);
  }
  return bytes;
}

extern "C" dpara_status dpara_layer_workspace_layout(const dpara_shape *shape, const int64_t *host_ctx_offsets,
                                                     const dpara_layer_io *layer, size_t offsets[9]) {
  if (!layer || !offsets) return DPARA_ERR_INVALID_ARG;
  dpara_status s = validate_shape(shape);
  if (s != DPARA_OK) return s;
  s = validate_offsets(shape, host_ctx_offsets);
  if (s != DPARA_OK) return s;
  if (layer->hidden <= 0 || layer->intermediate <= 0) return DPARA_ERR_INVALID_ARG;
  layer_workspace_offsets(shape, layer, attention_workspace_bytes(shape, host_ctx_offsets), offsets);
  return DPARA_OK;
}

extern "C" dpara_status dpara_draft_all_boundaries(const dpara_shape *shape, const dpara_attn_io *io,
                                                   const dpara_layer_io *layer, void *workspace, size_t workspace_bytes,
                                                   int32_t *status_word, void *stream) {
  dpara_status s = validate_shape(shape);
  if (s != DPARA_OK) return s;
  if (!io) return DPARA_ERR_INVALID_ARG;
  s = validate_offsets(shape, io->host_ctx_offsets);
  if (s != DPARA_OK) return s;
  if (!io->ctx_offsets) return DPARA_ERR_INVALID_ARG;
  if ((io->ctx_lens == nullptr) != (io->host_ctx_lens == nullptr)) return DPARA_ERR_INVALID_ARG;
  if (io->host_ctx_lens)
    for (int n = 0; n < shape->batch; ++n)
      if (io->host_ctx_lens[n] < 0 || io->host_ctx_lens[n] > io->host_ctx_offsets[n + 1] - io->host_ctx_offsets[n]) return DPARA_ERR_INVALID_ARG;
  const bool has_ctx = io->host_ctx_offsets[shape->batch] > 0;
  if (has_ctx && (!io->k_ctx || !io->v_ctx)) return DPARA_ERR_INVALID_ARG;
  const bool spine_made_inside = layer && shape->spine_queries;  // a block with spine query rows produces the spine's keys/values
  if (shape->n_spine > 0 && !spine_made_inside && (!io->k_spine || !io->v_spine)) return DPARA_ERR_INVALID_ARG;
  if ((io->k_blk == nullptr) != (io->v_blk == nullptr)) return DPARA_ERR_INVALID_ARG;
  if (io->out_dtype != DPARA_BF16 && io->out_dtype != DPARA_F32) return DPARA_ERR_INVALID_ARG;
  if (!aligned16(io->k_ctx) || !aligned16(io->v_ctx) || !aligned16(io->k_spine) || !aligned16(io->v_spine) ||
      !aligned16(io->q) || !aligned16(io->k_blk) || !aligned16(io->v_blk) || !aligned16(io->out))
    return DPARA_ERR_INVALID_ARG;
  const size_t need = dpara_draft_workspace_bytes(shape, io->host_ctx_offsets, layer, layer != nullptr);
  if (need > 0 && (!workspace || workspace_bytes < need || !aligned16(workspace))) return DPARA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  if (layer) return launch_layer(shape, io, layer, workspace, status_word, st);

  if (!io->q || !io->out) return DPARA_ERR_INVALID_ARG;
  return launch_attention(shape, io, workspace, status_word, st);
}

extern "C" size_t dpara_backbone_workspace_bytes(const dpara_shape *shape, const int64_t *host_ctx_offsets, const dpara_backbone_io *bb) {
  if (validate_shape(shape) != DPARA_OK || validate_offsets(shape, host_ctx_offsets) != DPARA_OK) return 0;
  if (!bb || bb->n_layers <= 0 || !bb->host_layers || bb->host_layers[0].hidden <= 0 || bb->host_layers[0].intermediate <= 0) return 0;
  return backbone_workspace_bytes(shape, host_ctx_offsets, bb);
}

extern "C" dpara_status dpara_draft_backbone(const dpara_shape *shape, const dpara_attn_io *io, const dpara_backbone_io *bb,
                                             void *workspace, size_t workspace_bytes, int32_t *status_word, void *stream) {
  dpara_status s = validate_shape(shape);
  if (s != DPARA_OK) return s;
  if (!io || !bb || bb->n_layers <= 0 || !bb->host_layers || !bb->host_k_ctx || !bb->host_v_ctx) return DPARA_ERR_INVALID_ARG;
  s = validate_offsets(shape, io->host_ctx_offsets);
  if (s != DPARA_OK) return s;
  if (!io->ctx_offsets || (io->ctx_lens == nullptr) != (io->host_ctx_lens == nullptr)) return DPARA_ERR_INVALID_ARG;
  if (io->host_ctx_lens)
    for (int n = 0; n < shape->batch; ++n)
      if (io->host_ctx_lens[n] < 0 || io->host_ctx_lens[n] > io->host_ctx_offsets[n + 1] - io->host_ctx_offsets[n]) return DPARA_ERR_INVALID_ARG;
  if (shape->n_spine > 0 && !shape->spine_queries && (!io->k_spine || !io->v_spine)) return DPARA_ERR_INVALID_ARG;
  const bool has_ctx = io->host_ctx_offsets[shape->batch] > 0;
  for (int l = 0; l < bb->n_layers; ++l) {
    if (bb->host_layers[l].hidden != bb->host_layers[0].hidden || bb->host_layers[l].intermediate != bb->host_layers[0].intermediate)
      return DPARA_ERR_INVALID_ARG;
    if (has_ctx && (!bb->host_k_ctx[l] || !bb->host_v_ctx[l] || !aligned16(bb->host_k_ctx[l]) || !aligned16(bb->host_v_ctx[l])))
      return DPARA_ERR_INVALID_ARG;
  }
  if (!bb->host_layers[0].x || !bb->host_layers[bb->n_layers - 1].y_f32) return DPARA_ERR_INVALID_ARG;
  const size_t need = dpara_backbone_workspace_bytes(shape, io->host_ctx_offsets, bb);
  if (need == 0 || !workspace || workspace_bytes < need || !aligned16(workspace)) return DPARA_ERR_WORKSPACE;
  return launch_backbone(shape, io, bb, workspace, status_word, static_cast<cudaStream_t>(stream));
}

extern "C" const char *dpara_status_string(dpara_status s) {
  switch (s) {
    case DPARA_OK: return "ok";
    case DPARA_ERR_INVALID_ARG: return "invalid argument";
    case DPARA_ERR_UNSUPPORTED: return "unsupported shape";
    case DPARA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case DPARA_ERR_CUDA: return "CUDA call failed";
    case DPARA_ERR_TIMEOUT: return "device-side wait timed out";
    case DPARA_ERR_STATIC_LIMIT: return "request needs more scratch than the fixed-scratch entry point owns";
  }
  return "unknown status";
}

extern "C" int32_t dpara_version(void) { return 1000; }

extern "C" int64_t dpara_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

#include "gemm.cuh"

extern "C" dpara_status dpara_gemm_bf16(const dpara_gemm_io *io, int32_t *status_word, void *stream) {
  if (!io) return DPARA_ERR_INVALID_ARG;
  if (io->epilogue < 0 || io->epilogue > 3) return DPARA_ERR_INVALID_ARG;
  GemmArgs g;
  g.a = io->a; g.w = io->w; g.M = io->M; g.N = io->N; g.K = io->K; g.epi = io->epilogue;
  g.resid = io->resid; g.resid_bf16 = io->resid_dtype == DPARA_BF16; g.out = io->out; g.out_bf16 = io->out_bf16;
  return launch_gemm_tc(g, status_word, static_cast<cudaStream_t>(stream));
}

#include "head.cuh"

extern "C" size_t dpara_head_workspace_bytes(int32_t b, int32_t block, int32_t vocab) { return head_workspace_bytes(b, block, vocab); }

extern "C" dpara_status dpara_draft_head(const dpara_head_io *io, void *workspace, size_t workspace_bytes, int32_t *status_word,
                                         void *stream) {
  if (!io) return DPARA_ERR_INVALID_ARG;
  if (io->b <= 0 || io->block <= 0 || io->vocab <= 0) return DPARA_ERR_INVALID_ARG;
  const size_t need = head_workspace_bytes(io->b, io->block, io->vocab);
  if (!workspace || workspace_bytes < need || !aligned16(workspace)) return DPARA_ERR_WORKSPACE;
  HeadArgs h;
  h.sel_reps = io->sel_reps; h.w_lm = io->w_lm; h.ar_w = io->ar_w; h.ar_e = io->ar_e; h.bonus = io->bonus;
  h.next_tokens = io->next_tokens; h.b = io->b; h.block = io->block; h.hidden = io->hidden; h.vocab = io->vocab; h.rank = io->rank;
  h.uniforms = io->uniforms;
  return launch_head(h, workspace, status_word, static_cast<cudaStream_t>(stream));
}
