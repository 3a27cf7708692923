// Feature-cache append (Alg. 1, the cache update after the head loop: the verified features of t_0..t_r join the
// cache, the rejected suffix is dropped; App. D: the history is projected incrementally, never again).
//
// Per drafter layer: rmsnorm of the candidate feature rows -> one tensor-core GEMM against the layer's [keys | values]
// projection -> a row-wise kernel that applies the per-head key norm and the rotary embedding at the row's position
// and writes the r + 1 accepted rows of every request behind the filled part of that layer's cache.  One layer's product
// is skinny (a few hundred rows against a 2 Hkv D x F weight: 8 output tiles at the benchmark shape), so with more than
// 128 rows up to eight layers go into ONE grouped launch, their K ranges cut in parts where that evens out the rounds;
// the parts leave fp32 partial sums and ONE row-wise launch for the same layers adds them (rounding the sum to bf16, as
// a single product's bf16 store would).  The accepted
// length is read on the device (it is the output of the verify/select call queued before), so no host round trip
// sits between verification and the append.  All d + 1 candidate rows go through the GEMM: it is bound by reading the
// projection weights once (2 Hkv D x F bf16 per layer), not by the row count.
#include <math.h>

#include "gemm.cuh"
#include "layer.cuh"

namespace dpara {

struct AppendParams {
  const uint16_t *kv;       // [b * J][2 * Hkv * D] bf16: [keys | values] of every candidate row (n_parts == 0)
  const float *kv_parts;    // layer g of the launch: [n_parts][b * J][2 * Hkv * D] fp32 partial sums from kv_parts + g * n_parts * part_stride
  int n_parts;
  size_t part_stride;       // elements between two parts
  // per layer of the launch (blockIdx.y)
  const uint16_t *knorm_w[kGemmMaxGroups];  // [D] or null
  uint16_t *k_cache[kGemmMaxGroups], *v_cache[kGemmMaxGroups];
  const int64_t *row_start, *capacity, *ctx_len;
  const int32_t *accept_len;
  int32_t *status_word;
  int J, Hkv, D, use_rope;
  float eps, theta;
  double inv_freq[64];      // theta^(-2 d / D), d < D / 2, worked out on the host in double precision
};

// One CTA per (candidate row (request n, draft position i), layer of the launch); rows above the accepted length leave at once.
__global__ void __launch_bounds__(128) append_rows_kernel(const AppendParams P) {
  extern __shared__ float s_cs[];  // cos[D/2], sin[D/2]
  const int n = blockIdx.x / P.J, i = blockIdx.x % P.J, tid = threadIdx.x, g = blockIdx.y;
  pdl_wait();
  pdl_launch_dependents();
  const uint16_t *knorm_w = P.knorm_w[g];
  const float *kv_parts = P.kv_parts + (size_t)g * P.n_parts * P.part_stride;
  const int r = P.accept_len[n];
  const long long L = P.ctx_len[n];
  if (r < 0 || r >= P.J || L + r + 1 > P.capacity[n]) {  // does not fit (or no valid outcome): the request is left alone
    if (i == 0 && g == 0 && tid == 0 && P.status_word) atomicOr(reinterpret_cast<unsigned int *>(P.status_word), DPARA_STATUS_CACHE_FULL);
    return;
  }
  if (i > r) return;  // rejected suffix: dropped
  const int half = P.D / 2;
  if (P.use_rope) {
    const double pos = (double)(L + i);
    for (int d = tid; d < half; d += 128) {
      double sn, cs;
      sincos(pos * P.inv_freq[d], &sn, &cs);
      s_cs[d] = (float)cs;
      s_cs[half + d] = (float)sn;
    }
  }
  __syncthreads();
  const int warp = tid >> 5, lane = tid & 31;
  const size_t row = (size_t)(P.row_start[n] + L + i);
  const size_t src_off = (size_t)blockIdx.x * 2 * P.Hkv * P.D;
  // element `e` of this candidate row as the bf16 value the projection stores (split K: the rounded sum of the parts)
  auto kv_at = [&](size_t e) -> float {
    if (P.n_parts == 0) return bf16_bits_to_float(P.kv[src_off + e]);
    float acc = 0.f;
    for (int s = 0; s < P.n_parts; ++s) acc += __ldg(kv_parts + (size_t)s * P.part_stride + src_off + e);
    return __bfloat162float(__float2bfloat16_rn(acc));
  };
  const int E = P.D / 64;  // pairs (d, d + D/2) per lane
  for (int h = warp; h < P.Hkv; h += 4) {
    const size_t ks = (size_t)h * P.D;
    uint16_t *kd = P.k_cache[g] + (row * P.Hkv + h) * P.D;
    float x1[2], x2[2], ss = 0.f;
    for (int e = 0; e < E; ++e) {
      const int d = lane + 32 * e;
      x1[e] = kv_at(ks + d);
      x2[e] = kv_at(ks + d + half);
      ss += x1[e] * x1[e] + x2[e] * x2[e];
    }
    if (knorm_w) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
      const float rs = rsqrtf(ss / (float)P.D + P.eps);
      for (int e = 0; e < E; ++e) {
        const int d = lane + 32 * e;
        x1[e] = __bfloat162float(__float2bfloat16_rn(x1[e] * rs * bf16_bits_to_float(knorm_w[d])));
        x2[e] = __bfloat162float(__float2bfloat16_rn(x2[e] * rs * bf16_bits_to_float(knorm_w[d + half])));
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
  const size_t vs = (size_t)P.Hkv * P.D;
  uint16_t *vd = P.v_cache[g] + row * P.Hkv * P.D;
  if (P.n_parts == 0) {
    for (int c = tid * 8; c < P.Hkv * P.D; c += 128 * 8) *reinterpret_cast<uint4 *>(vd + c) = *reinterpret_cast<const uint4 *>(P.kv + src_off + vs + c);
  } else {
    for (int c = tid * 4; c < P.Hkv * P.D; c += 128 * 4) {
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int s = 0; s < P.n_parts; ++s) {
        const float4 x = __ldg(reinterpret_cast<const float4 *>(kv_parts + (size_t)s * P.part_stride + src_off + vs + c));
        acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
      }
      *reinterpret_cast<uint2 *>(vd + c) = make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
    }
  }
}

// After every layer has read the old lengths: L_n += r_n + 1 for the requests that fitted.
__global__ void append_commit_kernel(int64_t *ctx_len, const int64_t *capacity, const int32_t *accept_len, int b, int J) {
  pdl_wait();
  pdl_launch_dependents();
  for (int n = blockIdx.x * blockDim.x + threadIdx.x; n < b; n += gridDim.x * blockDim.x) {
    const int r = accept_len[n];
    const long long L = ctx_len[n];
    if (r >= 0 && r < J && L + r + 1 <= capacity[n]) ctx_len[n] = L + r + 1;
  }
}

// Layers per grouped launch and K parts per layer for `layers_left` remaining layers; parts = 0: one product per layer with
// a bf16 store (at most 128 rows: single CTAs, neither grouped nor split).  The parts are chosen to minimise
// rounds x (K slabs per part + ~8 slabs' worth of fixed cost per work unit) over the CTA pairs.
static void cache_group_plan(const dpara_cache_io *io, int layers_left, int *group, int *parts) {
  const int M = io->batch * io->n_rows, N = 2 * io->n_kv_heads * io->head_dim;
  *group = 1;
  *parts = 0;
  if (M <= 128) return;
  *group = layers_left < kGemmMaxGroups ? layers_left : kGemmMaxGroups;
  const int tiles = ((M + 255) / 256) * ((N + 255) / 256), pairs = kNumSM / 2, nkb = io->feat_dim / 64;
  int best = 1;
  long best_cost = -1;
  for (int s = 1; s <= 8; s *= 2) {
    if (s > 1 && nkb / s < 4) break;
    const long units = (long)*group * tiles * s;
    const long cost = ((units + pairs - 1) / pairs) * (nkb / s + 8);
    if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
  }
  *parts = best;
}

// normalised copies of the feature rows: one per run of layers that share the input norm
static int cache_norm_slots(const dpara_cache_io *io) {
  int slots = 1;
  for (int l = 1; l < io->n_layers; ++l)
    if (io->host_norm_w && io->host_norm_w[l] != io->host_norm_w[l - 1]) ++slots;
  return slots;
}

size_t cache_append_workspace_bytes(const dpara_cache_io *io) {
  const size_t M = (size_t)io->batch * io->n_rows, N = (size_t)2 * io->n_kv_heads * io->head_dim;
  int group, parts;
  cache_group_plan(io, io->n_layers, &group, &parts);
  if (!parts) return align_up(M * io->feat_dim * 2, 256) + align_up(M * N * 2, 256);
  // planes of partial sums: the first launch has the most layers, the last (smaller) one may cut K in more parts --
  // sized for the larger of the two
  size_t planes = (size_t)group * parts;
  const int rest = io->n_layers % kGemmMaxGroups;
  if (io->n_layers > kGemmMaxGroups && rest) {
    int g2, p2;
    cache_group_plan(io, rest, &g2, &p2);
    planes = planes > (size_t)g2 * p2 ? planes : (size_t)g2 * p2;
  }
  return (size_t)cache_norm_slots(io) * align_up(M * io->feat_dim * 2, 256) + align_up(planes * M * N * 4, 256);
}

dpara_status launch_cache_append(const dpara_cache_io *io, void *workspace, int32_t *status_word, cudaStream_t st) {
  const int M = io->batch * io->n_rows, F = io->feat_dim, N = 2 * io->n_kv_heads * io->head_dim;
  const size_t xn_bytes = align_up((size_t)M * F * 2, 256);
  int group0, parts0;
  cache_group_plan(io, io->n_layers, &group0, &parts0);
  const int slots = parts0 ? cache_norm_slots(io) : 1;
  uint8_t *ws = static_cast<uint8_t *>(workspace);
  uint16_t *kv = reinterpret_cast<uint16_t *>(ws + (size_t)slots * xn_bytes);
  AppendParams P;
  memset(&P, 0, sizeof(P));
  P.row_start = io->row_start; P.capacity = io->capacity; P.ctx_len = io->ctx_len; P.accept_len = io->accept_len;
  P.status_word = status_word;
  P.J = io->n_rows; P.Hkv = io->n_kv_heads; P.D = io->head_dim; P.use_rope = io->use_rope;
  P.eps = io->rms_eps; P.theta = io->rope_theta;
  for (int d = 0; d < io->head_dim / 2 && d < 64; ++d) P.inv_freq[d] = pow((double)io->rope_theta, -2.0 * d / io->head_dim);
  P.part_stride = (size_t)M * N;
  const void *prev_gain = nullptr;
  int slot = -1;
  for (int l0 = 0; l0 < io->n_layers;) {
    int group, parts;
    cache_group_plan(io, io->n_layers - l0, &group, &parts);
    GemmArgs g{};
    g.M = M; g.N = N; g.K = F; g.epi = parts ? 3 : 0; g.split_k = parts ? parts : 1; g.n_groups = group;
    for (int k = 0; k < group; ++k) {
      const int l = l0 + k;
      const void *gain = io->host_norm_w ? io->host_norm_w[l] : nullptr;
      if (l == 0 || gain != prev_gain) {  // layers that share the input norm share the normalised rows
        slot = parts ? slot + 1 : 0;
        dpara_status s = launch_rmsnorm_bf16(io->features, gain, ws + (size_t)slot * xn_bytes, M, F, io->rms_eps, st);
        if (s != DPARA_OK) return s;
        prev_gain = gain;
      }
      void *out = parts ? static_cast<void *>(reinterpret_cast<float *>(kv) + (size_t)k * parts * M * N) : static_cast<void *>(kv);
      if (k == 0) { g.a = ws + (size_t)slot * xn_bytes; g.w = io->host_w_kv[l]; g.out = out; }
      g.a_g[k] = ws + (size_t)slot * xn_bytes; g.w_g[k] = io->host_w_kv[l]; g.out_g[k] = out;
      P.knorm_w[k] = static_cast<const uint16_t *>(io->host_knorm_w ? io->host_knorm_w[l] : nullptr);
      P.k_cache[k] = static_cast<uint16_t *>(io->host_k_ctx[l]);
      P.v_cache[k] = static_cast<uint16_t *>(io->host_v_ctx[l]);
    }
    dpara_status s = launch_gemm_tc(g, status_word, st);
    if (s != DPARA_OK) return s;
    P.kv = kv;
    P.kv_parts = reinterpret_cast<const float *>(kv); P.n_parts = parts;
    launch_pdl(append_rows_kernel, dim3(M, group), dim3(128), io->head_dim * sizeof(float), st, P);
    DPARA_CHECK_LAUNCH();
    count_launches(1);
    l0 += group;
  }
  launch_pdl(append_commit_kernel, dim3((io->batch + 127) / 128), dim3(128), 0, st, io->ctx_len, io->capacity, io->accept_len, io->batch, io->n_rows);
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
