// One backbone block around the all-boundary attention (Sec. 3.1 lists a block's parts, no
// equations; the block equations are stated with dpara_draft_all_boundaries in the header):
//   rmsnorm -> QKV GEMM -> per-head RMS norm + rotary embedding -> all-boundary attention ->
//   O GEMM (+x) -> rmsnorm -> gate/up GEMM with fused SiLU*up -> down GEMM (+h1).
// The GEMMs and the attention are the tensor-core kernels; the three small kernels here are row-wise
// and HBM-bound (M rows of a few KB each).
#include <math.h>

#include "attention_tc.cuh"
#include "gemm.cuh"
#include "layer.cuh"

namespace dpara {

void fill_attn_params(AttnParams &P, const dpara_shape *s, const dpara_attn_io *io, int32_t *status_word);

// ------------------------------------------------------------------------------------------------ rmsnorm
// out[row] = bf16( x[row] / sqrt(mean(x^2) + eps) * gain ),  x bf16 or fp32, one 128-thread CTA per row.
template <bool kF32In>
__global__ void __launch_bounds__(128) rmsnorm_kernel(const void *__restrict__ x, const uint16_t *__restrict__ gain,
                                                      uint16_t *__restrict__ out, int H, float eps) {
  const int row = blockIdx.x, tid = threadIdx.x;
  pdl_wait();
  pdl_launch_dependents();
  float ss = 0.f;
  for (int c = tid * 8; c < H; c += 128 * 8) {
    float v[8];
    if (kF32In) {
      const float4 *p = reinterpret_cast<const float4 *>(static_cast<const float *>(x) + (size_t)row * H + c);
      float4 a = p[0], b = p[1];
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
      uint4 w = *reinterpret_cast<const uint4 *>(static_cast<const uint16_t *>(x) + (size_t)row * H + c);
      v[0] = bf16lo(w.x); v[1] = bf16hi(w.x); v[2] = bf16lo(w.y); v[3] = bf16hi(w.y);
      v[4] = bf16lo(w.z); v[5] = bf16hi(w.z); v[6] = bf16lo(w.w); v[7] = bf16hi(w.w);
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) ss = fmaf(v[e], v[e], ss);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  __shared__ float s_part[4];
  if ((tid & 31) == 0) s_part[tid >> 5] = ss;
  __syncthreads();
  const float tot = s_part[0] + s_part[1] + s_part[2] + s_part[3];
  const float rs = rsqrtf(tot / (float)H + eps);
  for (int c = tid * 8; c < H; c += 128 * 8) {
    float v[8], gw[8];
    if (kF32In) {
      const float4 *p = reinterpret_cast<const float4 *>(static_cast<const float *>(x) + (size_t)row * H + c);
      float4 a = p[0], b = p[1];
      v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    } else {
      uint4 w = *reinterpret_cast<const uint4 *>(static_cast<const uint16_t *>(x) + (size_t)row * H + c);
      v[0] = bf16lo(w.x); v[1] = bf16hi(w.x); v[2] = bf16lo(w.y); v[3] = bf16hi(w.y);
      v[4] = bf16lo(w.z); v[5] = bf16hi(w.z); v[6] = bf16lo(w.w); v[7] = bf16hi(w.w);
    }
    if (gain) {
      uint4 w = *reinterpret_cast<const uint4 *>(gain + c);
      gw[0] = bf16lo(w.x); gw[1] = bf16hi(w.x); gw[2] = bf16lo(w.y); gw[3] = bf16hi(w.y);
      gw[4] = bf16lo(w.z); gw[5] = bf16hi(w.z); gw[6] = bf16lo(w.w); gw[7] = bf16hi(w.w);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) gw[e] = 1.f;
    }
    uint4 o;
    o.x = pack_bf16(v[0] * rs * gw[0], v[1] * rs * gw[1]);
    o.y = pack_bf16(v[2] * rs * gw[2], v[3] * rs * gw[3]);
    o.z = pack_bf16(v[4] * rs * gw[4], v[5] * rs * gw[5]);
    o.w = pack_bf16(v[6] * rs * gw[6], v[7] * rs * gw[7]);
    *reinterpret_cast<uint4 *>(out + (size_t)row * H + c) = o;
  }
}

// ------------------------------------------------------------------------------------------------ q/k norm + rope, v copy
// One CTA per token row.  qkv row = [Hq*D | Hkv*D | Hkv*D].  q and k heads: optional RMS norm over D
// (rounded to bf16), then rotate-half rotary embedding at the row's position (rounded to bf16).
// Positions: slot i of boundary j of request n sits at L_n + j + 2 + i (spine row s at L_n + s, the
// unknown bonus of boundary j at L_n + j + 1).  Angles are formed in double precision.
// With spine query rows a request has J * Bq + S rows: the mask-slot rows, then the spine rows.
struct QkParams {
  const uint16_t *qkv;
  const uint16_t *qnorm_w, *knorm_w;
  uint16_t *q, *k, *v;
  const int64_t *ctx_offsets, *ctx_lens;
  int J, Bq, Hq, Hkv, D, Sq;
  int use_rope, use_norm;
  float eps, theta;
  double inv_freq[64];   // theta^(-2 d / D), d < D / 2, worked out on the host in double precision
};

__global__ void __launch_bounds__(128) qk_norm_rope_kernel(const QkParams P) {
  extern __shared__ float s_cs[];  // cos[D/2], sin[D/2]
  const int row = blockIdx.x, tid = threadIdx.x;
  const int half = P.D / 2;
  const int R = P.Bq * P.J + P.Sq;
  pdl_wait();
  pdl_launch_dependents();
  const int n = row / R, rr = row % R;
  if (P.use_rope) {
    const int rel = rr < P.Bq * P.J ? rr / P.Bq + 2 + rr % P.Bq : rr - P.Bq * P.J;  // mask slot (j, i): j + 2 + i; spine row s: s
    const double pos = (double)(P.ctx_lens ? P.ctx_lens[n] : P.ctx_offsets[n + 1] - P.ctx_offsets[n]) + rel;
    for (int d = tid; d < half; d += 128) {
      double sn, cs;
      sincos(pos * P.inv_freq[d], &sn, &cs);
      s_cs[d] = (float)cs;
      s_cs[half + d] = (float)sn;
    }
  }
  __syncthreads();
  const int warp = tid >> 5, lane = tid & 31;
  const size_t qkv_row = (size_t)row * (P.Hq + 2 * P.Hkv) * P.D;
  // A lane owns the element pairs (2 lane, 2 lane + 1) of both halves of a head (one 4-byte load each); a warp takes heads
  // warp, warp + 4, ... and fetches kChunk of them before it works on the first, so that a row costs a few global round
  // trips instead of one per head.
  constexpr int kChunk = 6;
  const bool active = 2 * lane < half;
  const int n_heads = P.Hq + P.Hkv;
  for (int hd0 = warp; hd0 < n_heads; hd0 += 4 * kChunk) {
    uint32_t lo[kChunk], hi[kChunk];
#pragma unroll
    for (int c = 0; c < kChunk; ++c) {
      const int hd = hd0 + 4 * c;
      lo[c] = hi[c] = 0u;
      if (hd < n_heads && active) {
        const uint16_t *src = P.qkv + qkv_row + (size_t)hd * P.D;
        lo[c] = *reinterpret_cast<const uint32_t *>(src + 2 * lane);
        hi[c] = *reinterpret_cast<const uint32_t *>(src + half + 2 * lane);
      }
    }
#pragma unroll
    for (int c = 0; c < kChunk; ++c) {
      const int hd = hd0 + 4 * c;
      if (hd >= n_heads) break;
      const bool is_q = hd < P.Hq;
      uint16_t *dst = is_q ? P.q + ((size_t)row * P.Hq + hd) * P.D : P.k + ((size_t)row * P.Hkv + (hd - P.Hq)) * P.D;
      const uint16_t *gain = is_q ? P.qnorm_w : P.knorm_w;
      float x1[2] = {bf16lo(lo[c]), bf16hi(lo[c])}, x2[2] = {bf16lo(hi[c]), bf16hi(hi[c])};
      if (P.use_norm) {
        float ss = x1[0] * x1[0] + x2[0] * x2[0] + x1[1] * x1[1] + x2[1] * x2[1];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        const float rs = rsqrtf(ss / (float)P.D + P.eps);
        if (active) {
          const uint32_t g1 = gain ? *reinterpret_cast<const uint32_t *>(gain + 2 * lane) : 0x3f803f80u;          // bf16 1.0 twice
          const uint32_t g2 = gain ? *reinterpret_cast<const uint32_t *>(gain + half + 2 * lane) : 0x3f803f80u;
          x1[0] = __bfloat162float(__float2bfloat16_rn(x1[0] * rs * bf16lo(g1)));
          x1[1] = __bfloat162float(__float2bfloat16_rn(x1[1] * rs * bf16hi(g1)));
          x2[0] = __bfloat162float(__float2bfloat16_rn(x2[0] * rs * bf16lo(g2)));
          x2[1] = __bfloat162float(__float2bfloat16_rn(x2[1] * rs * bf16hi(g2)));
        }
      }
      if (active) {
        float y1[2] = {x1[0], x1[1]}, y2[2] = {x2[0], x2[1]};
        if (P.use_rope) {
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const float cs = s_cs[2 * lane + e], sn = s_cs[half + 2 * lane + e];
            y1[e] = x1[e] * cs - x2[e] * sn;
            y2[e] = x2[e] * cs + x1[e] * sn;
          }
        }
        *reinterpret_cast<uint32_t *>(dst + 2 * lane) = pack_bf16(y1[0], y1[1]);
        *reinterpret_cast<uint32_t *>(dst + half + 2 * lane) = pack_bf16(y2[0], y2[1]);
      }
    }
  }
  // v: plain copy into its own contiguous tensor
  const uint16_t *vsrc = P.qkv + qkv_row + (size_t)(P.Hq + P.Hkv) * P.D;
  uint16_t *vdst = P.v + (size_t)row * P.Hkv * P.D;
  for (int c = tid * 8; c < P.Hkv * P.D; c += 128 * 8) *reinterpret_cast<uint4 *>(vdst + c) = *reinterpret_cast<const uint4 *>(vsrc + c);
}

// ------------------------------------------------------------------------------------------------ host
namespace {
struct LayerWs {
  size_t xn, qkv, q, k, v, a, h1, hn, act, attn, total;
};

LayerWs layer_ws_layout(const dpara_shape *s, const dpara_layer_io *l, size_t attn_bytes) {
  const size_t M = (size_t)s->batch * (s->n_boundaries * s->block + (s->spine_queries ? s->n_spine : 0));
  const size_t H = l->hidden, I = l->intermediate, QD = (size_t)s->n_q_heads * s->head_dim, KD = (size_t)s->n_kv_heads * s->head_dim;
  LayerWs w;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t r = o; o += align_up(bytes, 256); return r; };
  w.xn = take(M * H * 2);
  w.qkv = take(M * (QD + 2 * KD) * 2);
  w.q = take(M * QD * 2);
  w.k = take(M * KD * 2);
  w.v = take(M * KD * 2);
  w.a = take(M * QD * 2);
  w.h1 = take(M * H * 4);
  w.hn = take(M * H * 2);
  w.act = take(M * I * 2);
  w.attn = take(attn_bytes);
  w.total = o;
  return w;
}
}  // namespace

void layer_workspace_offsets(const dpara_shape *shape, const dpara_layer_io *layer, size_t attn_bytes, size_t out[9]) {
  const LayerWs w = layer_ws_layout(shape, layer, 0);
  const size_t o[9] = {w.xn, w.qkv, w.q, w.k, w.v, w.a, w.h1, w.hn, w.act};
  for (int i = 0; i < 9; ++i) out[i] = attn_bytes + o[i];
}

dpara_status launch_rmsnorm_bf16(const void *x, const void *gain, void *out, int M, int H, float eps, cudaStream_t st) {
  if (H % 8) return DPARA_ERR_UNSUPPORTED;
  launch_pdl(rmsnorm_kernel<false>, dim3(M), dim3(128), 0, st, x, static_cast<const uint16_t *>(gain), static_cast<uint16_t *>(out), H, eps);
  DPARA_CHECK_LAUNCH();
  count_launches(1);
  return DPARA_OK;
}

size_t layer_workspace_bytes(const dpara_shape *shape, const dpara_layer_io *layer) {
  if (layer->hidden <= 0 || layer->intermediate <= 0) return 0;
  return layer_ws_layout(shape, layer, 0).total;  // the attention's own scratch is added by the caller
}

dpara_status launch_layer(const dpara_shape *shape, const dpara_attn_io *io, const dpara_layer_io *L, void *workspace,
                          int32_t *status_word, cudaStream_t st) {
  if (!L->x || !L->w_qkv || !L->w_o || !L->w_gate_up || !L->w_down || !L->y_f32) return DPARA_ERR_INVALID_ARG;
  if (L->hidden <= 0 || L->intermediate <= 0) return DPARA_ERR_INVALID_ARG;
  if ((L->qnorm_w == nullptr) != (L->knorm_w == nullptr)) return DPARA_ERR_INVALID_ARG;
  if (shape->boundary_lo != 0 || shape->boundary_hi != shape->n_boundaries) return DPARA_ERR_UNSUPPORTED;
  const int Sq = shape->spine_queries ? shape->n_spine : 0;
  const int R = shape->n_boundaries * shape->block + Sq;  // rows per request: mask slots, then (if they are queries) the spine
  const int M = shape->batch * R;
  const int H = L->hidden, I = L->intermediate, D = shape->head_dim;
  const int QD = shape->n_q_heads * D, KD = shape->n_kv_heads * D;
  if (H % 64 || I % 64 || QD % 64 || H % 8) return DPARA_ERR_UNSUPPORTED;
  const size_t attn_ws = attention_workspace_bytes(shape, io->host_ctx_offsets);
  // layout: [attention scratch (as sized by attention_workspace_bytes)] [layer buffers]
  uint8_t *base = static_cast<uint8_t *>(workspace);
  const LayerWs w = layer_ws_layout(shape, L, 0);
  uint8_t *lw = base + attn_ws;
  uint16_t *xn = reinterpret_cast<uint16_t *>(lw + w.xn), *qkv = reinterpret_cast<uint16_t *>(lw + w.qkv);
  uint16_t *q = reinterpret_cast<uint16_t *>(lw + w.q), *k = reinterpret_cast<uint16_t *>(lw + w.k), *v = reinterpret_cast<uint16_t *>(lw + w.v);
  uint16_t *a = reinterpret_cast<uint16_t *>(lw + w.a), *hn = reinterpret_cast<uint16_t *>(lw + w.hn), *act = reinterpret_cast<uint16_t *>(lw + w.act);
  float *h1 = reinterpret_cast<float *>(lw + w.h1);

  launch_pdl(rmsnorm_kernel<false>, dim3(M), dim3(128), 0, st, L->x, static_cast<const uint16_t *>(L->rms1_w), xn, H, L->rms_eps);
  DPARA_CHECK_LAUNCH();
  count_launches(1);
  GemmArgs g{};
  g.a = xn; g.w = L->w_qkv; g.M = M; g.N = QD + 2 * KD; g.K = H; g.epi = 0; g.out = qkv;
  dpara_status s = launch_gemm_tc(g, status_word, st);
  if (s != DPARA_OK) return s;

  QkParams qp;
  qp.qkv = qkv; qp.qnorm_w = static_cast<const uint16_t *>(L->qnorm_w); qp.knorm_w = static_cast<const uint16_t *>(L->knorm_w);
  qp.q = q; qp.k = k; qp.v = v; qp.ctx_offsets = io->ctx_offsets; qp.ctx_lens = io->ctx_lens;
  qp.J = shape->n_boundaries; qp.Bq = shape->block; qp.Hq = shape->n_q_heads; qp.Hkv = shape->n_kv_heads; qp.D = D; qp.Sq = Sq;
  qp.use_rope = L->use_rope; qp.use_norm = L->qnorm_w != nullptr; qp.eps = L->rms_eps; qp.theta = L->rope_theta;
  for (int d = 0; d < D / 2 && d < 64; ++d) qp.inv_freq[d] = pow((double)L->rope_theta, -2.0 * d / D);
  launch_pdl(qk_norm_rope_kernel, dim3(M), dim3(128), D * sizeof(float), st, qp);
  DPARA_CHECK_LAUNCH();
  count_launches(1);

  dpara_attn_io aio = *io;
  aio.q = q; aio.k_blk = k; aio.v_blk = v; aio.out = a; aio.out_dtype = DPARA_BF16; aio.out_lse = nullptr;
  if (Sq) {
    // the spine's keys/values are the block's own: rows J * Bq .. of each request in the k / v buffers
    aio.k_spine = k + (size_t)shape->n_boundaries * shape->block * KD;
    aio.v_spine = v + (size_t)shape->n_boundaries * shape->block * KD;
  }
  s = launch_attention(shape, &aio, base, status_word, st, Sq ? R : 0, Sq ? R : 0);
  if (s != DPARA_OK) return s;

  g = GemmArgs{};
  g.a = a; g.w = L->w_o; g.M = M; g.N = H; g.K = QD; g.epi = 1; g.resid = L->x; g.resid_bf16 = 1; g.out = h1;
  s = launch_gemm_tc(g, status_word, st);
  if (s != DPARA_OK) return s;
  launch_pdl(rmsnorm_kernel<true>, dim3(M), dim3(128), 0, st, static_cast<const void *>(h1), static_cast<const uint16_t *>(L->rms2_w), hn, H, L->rms_eps);
  DPARA_CHECK_LAUNCH();
  count_launches(1);
  g = GemmArgs{};
  g.a = hn; g.w = L->w_gate_up; g.M = M; g.N = I; g.K = H; g.epi = 2; g.out = act;
  s = launch_gemm_tc(g, status_word, st);
  if (s != DPARA_OK) return s;
  g = GemmArgs{};
  g.a = act; g.w = L->w_down; g.M = M; g.N = H; g.K = I; g.epi = 1; g.resid = h1; g.resid_bf16 = 0; g.out = L->y_f32; g.out_bf16 = L->y_bf16;
  return launch_gemm_tc(g, status_word, st);
}

// ------------------------------------------------------------------------------------------------ stack of blocks
namespace {
struct BackboneWs { size_t x0, x1, yf, layer, total; };
BackboneWs backbone_ws_layout(const dpara_shape *s, const dpara_backbone_io *bb, size_t attn_bytes) {
  const size_t M = (size_t)s->batch * (s->n_boundaries * s->block + (s->spine_queries ? s->n_spine : 0));
  const size_t H = bb->host_layers[0].hidden;
  BackboneWs w;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t r = o; o += align_up(bytes, 256); return r; };
  w.layer = take(attn_bytes + layer_workspace_bytes(s, &bb->host_layers[0]));  // the attention scratch leads the block's scratch
  w.x0 = take(M * H * 2);
  w.x1 = take(M * H * 2);
  w.yf = take(M * H * 4);
  w.total = o;
  return w;
}
}  // namespace

size_t backbone_workspace_bytes(const dpara_shape *shape, const int64_t *host_ctx_offsets, const dpara_backbone_io *bb) {
  return backbone_ws_layout(shape, bb, attention_workspace_bytes(shape, host_ctx_offsets)).total;
}

dpara_status launch_backbone(const dpara_shape *shape, const dpara_attn_io *io, const dpara_backbone_io *bb, void *workspace,
                             int32_t *status_word, cudaStream_t st) {
  const BackboneWs w = backbone_ws_layout(shape, bb, attention_workspace_bytes(shape, io->host_ctx_offsets));
  uint8_t *base = static_cast<uint8_t *>(workspace);
  void *xbuf[2] = {base + w.x0, base + w.x1};
  const int last = bb->n_layers - 1;
  for (int l = 0; l <= last; ++l) {
    dpara_layer_io L = bb->host_layers[l];
    L.x = l == 0 ? bb->host_layers[0].x : xbuf[(l - 1) & 1];
    L.y_f32 = l == last ? bb->host_layers[last].y_f32 : reinterpret_cast<float *>(base + w.yf);
    L.y_bf16 = l == last ? bb->host_layers[last].y_bf16 : xbuf[l & 1];
    dpara_attn_io a = *io;
    a.k_ctx = bb->host_k_ctx[l];
    a.v_ctx = bb->host_v_ctx[l];
    dpara_status s = launch_layer(shape, &a, &L, base + w.layer, status_word, st);
    if (s != DPARA_OK) return s;
  }
  return DPARA_OK;
}

}  // namespace dpara
