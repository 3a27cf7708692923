// Parameters of the attention kernel (plain struct, passed by value).
#pragma once
#include "common.cuh"

namespace dpara {

struct AttnParams {
  const uint16_t *q;                // [b][J][Bq][Hq][D]
  const uint16_t *k_ctx, *v_ctx;    // [sum L][Hkv][D]
  const int64_t *ctx_offsets;       // [b+1] device
  const int64_t *ctx_lens;          // [b] device or null (null: request n fills all of its rows)
  const uint16_t *k_spine, *v_spine;  // [b][S][Hkv][D]
  const uint16_t *k_blk, *v_blk;    // [b][J][Bq][Hkv][D] or null
  void *out;                        // [b][J][Bq][Hq][D] bf16 or fp32
  float *out_lse;                   // [b][J][Bq][Hq] or null
  int out_f32;
  int b, J, Bq, Hq, Hkv, D, G, S, pb, lo, hi;
  // Spine tokens as query rows (Sec. 3.2, Fig. 4: an anchor reads the cache, itself and the earlier anchors): Sq = S
  // extra rows per request behind the mask-slot rows, else 0.  q / out / out_lse then hold q_req_rows = J * Bq + Sq rows
  // per request.  blk_req_rows / spine_req_rows: rows from one request's block (spine) keys to the next request's
  // (J * Bq and S when the tensors are the caller's; J * Bq + S when both live in one per-request buffer).
  int Sq, q_req_rows, blk_req_rows, spine_req_rows;
  float scale;                      // softmax scale (natural-exp domain)
  int32_t *status_word;
};

}  // namespace dpara
