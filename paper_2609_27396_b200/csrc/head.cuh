// Host-side interface of the critical-path remainder: LM head on the selected branch + autoregressive head loop.
#pragma once
#include "common.cuh"

namespace dpara {

struct HeadArgs {
  const void *sel_reps;      // [b][block][hidden] bf16
  const void *w_lm;          // [vocab][hidden] bf16
  const void *ar_w;          // [vocab][rank] bf16
  const void *ar_e;          // [vocab][rank] bf16
  const int32_t *bonus;      // [b]
  int32_t *next_tokens;      // [b][block]
  int b, block, hidden, vocab, rank;
  const float *uniforms;     // [b][block] or null: null = greedy, else y_i is drawn from softmax(z_i) with uniforms[n][i-1]
};

size_t head_workspace_bytes(int b, int block, int vocab);
dpara_status launch_head(const HeadArgs &h, void *workspace, int32_t *status, cudaStream_t st);

}  // namespace dpara
