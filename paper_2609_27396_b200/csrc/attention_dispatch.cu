// Fills the attention kernel's parameters from the C-ABI structs and launches it.
#include <math.h>

#include "attention_tc.cuh"
#include "layer.cuh"

namespace dpara {

void fill_attn_params(AttnParams &P, const dpara_shape *s, const dpara_attn_io *io, int32_t *status_word) {
  P.q = static_cast<const uint16_t *>(io->q);
  P.k_ctx = static_cast<const uint16_t *>(io->k_ctx);
  P.v_ctx = static_cast<const uint16_t *>(io->v_ctx);
  P.ctx_offsets = io->ctx_offsets;
  P.ctx_lens = io->ctx_lens;
  P.k_spine = static_cast<const uint16_t *>(io->k_spine);
  P.v_spine = static_cast<const uint16_t *>(io->v_spine);
  P.k_blk = static_cast<const uint16_t *>(io->k_blk);
  P.v_blk = static_cast<const uint16_t *>(io->v_blk);
  P.out = io->out;
  P.out_lse = io->out_lse;
  P.out_f32 = io->out_dtype == DPARA_F32;
  P.b = s->batch; P.J = s->n_boundaries; P.Bq = s->block; P.Hq = s->n_q_heads; P.Hkv = s->n_kv_heads;
  P.D = s->head_dim; P.G = s->n_q_heads / s->n_kv_heads; P.S = s->n_spine; P.pb = s->prefix_base;
  P.lo = s->boundary_lo; P.hi = s->boundary_hi;
  P.Sq = s->spine_queries ? s->n_spine : 0;
  P.q_req_rows = s->n_boundaries * s->block + P.Sq;
  P.blk_req_rows = s->n_boundaries * s->block;
  P.spine_req_rows = s->n_spine;
  P.scale = s->softmax_scale > 0.f ? s->softmax_scale : 1.0f / sqrtf((float)s->head_dim);
  P.status_word = status_word;
}

size_t attention_workspace_bytes(const dpara_shape *shape, const int64_t *host_off) {
  TcPlan plan = plan_attention_tc(shape, host_off, nullptr);
  return plan.eligible ? align_up(plan.workspace_max_bytes, 256) : 0;
}

dpara_status launch_attention(const dpara_shape *shape, const dpara_attn_io *io, void *workspace, int32_t *status_word,
                              cudaStream_t st, int blk_req_rows, int spine_req_rows) {
  AttnParams P;
  fill_attn_params(P, shape, io, status_word);
  if (blk_req_rows) P.blk_req_rows = blk_req_rows;
  if (spine_req_rows) P.spine_req_rows = spine_req_rows;
  if (P.hi <= P.lo) return DPARA_OK;
  TcPlan plan = plan_attention_tc(shape, io->host_ctx_offsets, io->host_ctx_lens);
  if (!plan.eligible) return DPARA_ERR_UNSUPPORTED;  // group size > 16, block > 64, spine > 64, or more than 2^31 rows
  return launch_attention_tc(P, plan, io->host_ctx_offsets, io->host_ctx_lens, workspace, st);
}

}  // namespace dpara
