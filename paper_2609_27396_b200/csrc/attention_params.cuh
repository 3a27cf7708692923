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
  float scale;                      // softmax scale (natural-exp domain)
  int32_t *status_word;
};

}  // namespace dpara
