// Feature-cache append (Alg. 1, the cache update after the head loop: the verified features of t_0..t_r join the
// cache, the rejected suffix is dropped; App. D: the history is projected incrementally, never again).
//
// Per drafter layer: rmsnorm of the candidate feature rows -> one tensor-core GEMM against the layer's [keys | values]
// projection -> a row-wise kernel that applies the per-head key norm and the rotary embedding at the row's position
// and writes the r + 1 accepted rows of every request behind the filled part of that layer's cache.  The accepted
// length is read on the device (it is the output of the verify/select call queued before), so no host round trip
// sits between verification and the append.  All d + 1 candidate rows go through the GEMM: it is bound by reading the
// projection weights once (2 Hkv D x F bf16 per layer), not by the row count.
#include <math.h>

#include "gemm.cuh"
#include "layer.cuh"

namespace dpara {

struct AppendParams {
  const uint16_t *kv;       // [b * J][2 * Hkv * D] bf16: [keys | values] of every candidate row
  const uint16_t *knorm_w;  // [D] or null
  uint16_t *k_cache, *v_cache;
  const int64_t *row_start, *capacity, *ctx_len;
  const int32_t *accept_len;
  int32_t *status_word;
  int J, Hkv, D, use_rope;
  float eps, theta;
};

// One CTA per candidate row (request n, draft position i); rows above the accepted length leave at once.
__global__ void __launch_bounds__(128) append_rows_kernel(const AppendParams P) {
  extern __shared__ float s_cs[];  // cos[D/2], sin[D/2]
  const int n = blockIdx.x / P.J, i = blockIdx.x % P.J, tid = threadIdx.x;
  const int r = P.accept_len[n];
  const long long L = P.ctx_len[n];
  if (r < 0 || r >= P.J || L + r + 1 > P.capacity[n]) {  // does not fit (or no valid outcome): the request is left alone
    if (i == 0 && tid == 0 && P.status_word) atomicOr(reinterpret_cast<unsigned int *>(P.status_word), DPARA_STATUS_CACHE_FULL);
    return;
  }
  if (i > r) return;  // rejected suffix: dropped
  const int half = P.D / 2;
  if (P.use_rope) {
    const double pos = (double)(L + i);
    for (int d = tid; d < half; d += 128) {
      double sn, cs;
      sincos(pos * pow((double)P.theta, -2.0 * d / P.D), &sn, &cs);
      s_cs[d] = (float)cs;
      s_cs[half + d] = (float)sn;
    }
  }
  __syncthreads();
  const int warp = tid >> 5, lane = tid & 31;
  const size_t row = (size_t)(P.row_start[n] + L + i);
  const uint16_t *src = P.kv + (size_t)blockIdx.x * 2 * P.Hkv * P.D;
  const int E = P.D / 64;  // pairs (d, d + D/2) per lane
  for (int h = warp; h < P.Hkv; h += 4) {
    const uint16_t *ks = src + (size_t)h * P.D;
    uint16_t *kd = P.k_cache + (row * P.Hkv + h) * P.D;
    float x1[2], x2[2], ss = 0.f;
    for (int e = 0; e < E; ++e) {
      const int d = lane + 32 * e;
      x1[e] = bf16_bits_to_float(ks[d]);
      x2[e] = bf16_bits_to_float(ks[d + half]);
      ss += x1[e] * x1[e] + x2[e] * x2[e];
    }
    if (P.knorm_w) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      const float rs = rsqrtf(ss / (float)P.D + P.eps);
      for (int e = 0; e < E; ++e) {
        const int d = lane + 32 * e;
        x1[e] = __bfloat162float(__float2bfloat16_rn(x1[e] * rs * bf16_bits_to_float(P.knorm_w[d])));
        x2[e] = __bfloat162float(__float2bfloat16_rn(x2[e] * rs * bf16_bits_to_float(P.knorm_w[d + half])));
      }
    }
    for (int e = 0; e < E; ++e) {
      const int d = lane + 32 * e;
      float y1 = x1[e], y2 = x2[e];
      if (P.use_rope) {
        const float cs = s_cs[d], sn = s_cs[half + d];
        y1 = x1[e] * cs - x2[e] * sn;
        y2 = x2[e] * cs + x1[e] * sn;
      }
      kd[d] = __bfloat16_as_ushort(__float2bfloat16_rn(y1));
      kd[d + half] = __bfloat16_as_ushort(__float2bfloat16_rn(y2));
    }
  }
  const uint16_t *vs = src + (size_t)P.Hkv * P.D;
  uint16_t *vd = P.v_cache + row * P.Hkv * P.D;
  for (int c = tid * 8; c < P.Hkv * P.D; c += 128 * 8) *reinterpret_cast<uint4 *>(vd + c) = *reinterpret_cast<const uint4 *>(vs + c);
}

// After every layer has read the old lengths: L_n += r_n + 1 for the requests that fitted.
__global__ void append_commit_kernel(int64_t *ctx_len, const int64_t *capacity, const int32_t *accept_len, int b, int J) {
  for (int n = blockIdx.x * blockDim.x + threadIdx.x; n < b; n += gridDim.x * blockDim.x) {
    const int r = accept_len[n];
    const long long L = ctx_len[n];
    if (r >= 0 && r < J && L + r + 1 <= capacity[n]) ctx_len[n] = L + r + 1;
  }
}

size_t cache_append_workspace_bytes(const dpara_cache_io *io) {
  const size_t M = (size_t)io->batch * io->n_rows;
  return align_up(M * io->feat_dim * 2, 256) + align_up(M * 2 * io->n_kv_heads * io->head_dim * 2, 256);
}

dpara_status launch_cache_append(const dpara_cache_io *io, void *workspace, int32_t *status_word, cudaStream_t st) {
  const int M = io->batch * io->n_rows, F = io->feat_dim, N = 2 * io->n_kv_heads * io->head_dim;
  uint16_t *xn = static_cast<uint16_t *>(workspace);
  uint16_t *kv = reinterpret_cast<uint16_t *>(static_cast<uint8_t *>(workspace) + align_up((size_t)M * F * 2, 256));
  const void *prev_gain = nullptr;
  for (int l = 0; l < io->n_layers; ++l) {
    const void *gain = io->host_norm_w ? io->host_norm_w[l] : nullptr;
    if (l == 0 || gain != prev_gain) {  // layers that share the input norm share the normalised rows
      dpara_status s = launch_rmsnorm_bf16(io->features, gain, xn, M, F, io->rms_eps, st);
      if (s != DPARA_OK) return s;
      prev_gain = gain;
    }
    GemmArgs g{};
    g.a = xn; g.w = io->host_w_kv[l]; g.M = M; g.N = N; g.K = F; g.epi = 0; g.out = kv;
    dpara_status s = launch_gemm_tc(g, status_word, st);
    if (s != DPARA_OK) return s;
    AppendParams P;
    P.kv = kv;
    P.knorm_w = static_cast<const uint16_t *>(io->host_knorm_w ? io->host_knorm_w[l] : nullptr);
    P.k_cache = static_cast<uint16_t *>(io->host_k_ctx[l]);
    P.v_cache = static_cast<uint16_t *>(io->host_v_ctx[l]);
    P.row_start = io->row_start; P.capacity = io->capacity; P.ctx_len = io->ctx_len; P.accept_len = io->accept_len;
    P.status_word = status_word;
    P.J = io->n_rows; P.Hkv = io->n_kv_heads; P.D = io->head_dim; P.use_rope = io->use_rope;
    P.eps = io->rms_eps; P.theta = io->rope_theta;
    append_rows_kernel<<<M, 128, io->head_dim * sizeof(float), st>>>(P);
    DPARA_CHECK_LAUNCH();
    count_launches(1);
  }
  append_commit_kernel<<<(io->batch + 127) / 128, 128, 0, st>>>(io->ctx_len, io->capacity, io->accept_len, io->batch, io->n_rows);
  DPARA_CHECK_LAUNCH();
  count_launches(1);
  return DPARA_OK;
}

}  // namespace dpara

using namespace dpara;

static dpara_status validate_cache(const dpara_cache_io *io) {
  if (!io) return DPARA_ERR_INVALID_ARG;
  if (io->batch <= 0 || io->n_rows <= 0 || io->feat_dim <= 0 || io->n_kv_heads <= 0 || io->n_layers <= 0) return DPARA_ERR_INVALID_ARG;
  if (io->head_dim != 64 && io->head_dim != 128) return DPARA_ERR_UNSUPPORTED;
  if (io->feat_dim % 64 != 0) return DPARA_ERR_UNSUPPORTED;
  return DPARA_OK;
}

extern "C" size_t dpara_cache_append_workspace_bytes(const dpara_cache_io *io) {
  return validate_cache(io) == DPARA_OK ? cache_append_workspace_bytes(io) : 0;
}

extern "C" dpara_status dpara_cache_append(const dpara_cache_io *io, void *workspace, size_t workspace_bytes, int32_t *status_word,
                                           void *stream) {
  dpara_status s = validate_cache(io);
  if (s != DPARA_OK) return s;
  if (!io->features || !io->accept_len || !io->host_w_kv || !io->host_k_ctx || !io->host_v_ctx || !io->row_start || !io->capacity ||
      !io->ctx_len)
    return DPARA_ERR_INVALID_ARG;
  for (int l = 0; l < io->n_layers; ++l)
    if (!io->host_w_kv[l] || !io->host_k_ctx[l] || !io->host_v_ctx[l] || !aligned16(io->host_w_kv[l]) || !aligned16(io->host_k_ctx[l]) ||
        !aligned16(io->host_v_ctx[l]))
      return DPARA_ERR_INVALID_ARG;
  if (!aligned16(io->features)) return DPARA_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < cache_append_workspace_bytes(io) || !aligned16(workspace)) return DPARA_ERR_WORKSPACE;
  return launch_cache_append(io, workspace, status_word, static_cast<cudaStream_t>(stream));
}
