// Host-side interface of the tensor-core GEMM.
#pragma once
#include "common.cuh"

namespace dpara {

constexpr int kGemmMaxGroups = 8;

struct GemmArgs {
  const void *a;      // [M][K] bf16, row-major
  const void *w;      // [N][K] bf16 (epi 2: [2N][K], rows [0,N) gate and [N,2N) up)
  int M, N, K;        // N = output columns
  int epi;            // 0 bf16 store; 1 fp32 out = resid + acc (+ bf16 copy); 2 bf16 out = silu(gate) * up; 3 fp32 store
  const void *resid;  // epi 1: [M][N] bf16 or fp32
  int resid_bf16;
  void *out;          // [M][N] bf16 (epi 0, 2) or fp32 (epi 1, 3)
  void *out_bf16;     // epi 1: optional bf16 copy of out
  int perm_block = 0, perm_b = 0;  // epi 3 only, if set: output row (n * perm_block + i) is stored at row (i * perm_b + n)
  int split_k = 1;    // epi 3 and M > 128 only: the K range in split_k parts, out = [split_k][M][N] fp32 partial sums (the caller adds them)
  // Grouped launch (epi 3 and M > 128 only): n_groups products of this shape, product 0 = (a, w, out), product g > 0 =
  // (a_g[g], w_g[g], out_g[g]); the CTA pairs share out the work units of all of them
  int n_groups = 1;
  const void *a_g[kGemmMaxGroups] = {};
  const void *w_g[kGemmMaxGroups] = {};
  void *out_g[kGemmMaxGroups] = {};
};

dpara_status launch_gemm_tc(const GemmArgs &g, int32_t *status, cudaStream_t st);

}  // namespace dpara
