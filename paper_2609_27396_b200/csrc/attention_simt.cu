// General-shape all-boundary attention on CUDA cores: one warp per query row (n, j, i, h).
// This is the path for shapes the tensor-core kernel is not built for (small tiles, odd group sizes);
// it walks the visible keys of the row's boundary in the order context, anchor prefix, own block
// (Fig. 4) with an online softmax.  Lanes split the head dimension, so every K/V row is one coalesced
// load per warp.
#include "attention_params.cuh"

namespace dpara {

template <int D>
struct RowAcc {
  static constexpr int E = D / 32;  // elements per lane
  float q[E], o[E];
  float m, l;
};

template <int D>
__device__ __forceinline__ void load_lane(const uint16_t *row, int lane, float (&x)[D / 32]) {
  if constexpr (D == 128) {
    uint2 w = __ldg(reinterpret_cast<const uint2 *>(row) + lane);
    x[0] = bf16lo(w.x); x[1] = bf16hi(w.x); x[2] = bf16lo(w.y); x[3] = bf16hi(w.y);
  } else {
    uint32_t w = __ldg(reinterpret_cast<const uint32_t *>(row) + lane);
    x[0] = bf16lo(w); x[1] = bf16hi(w);
  }
}

template <int D>
__device__ __forceinline__ void visit_key(RowAcc<D> &a, const uint16_t *krow, const uint16_t *vrow, int lane, float scale) {
  constexpr int E = D / 32;
  float k[E], v[E];
  load_lane<D>(krow, lane, k);
  load_lane<D>(vrow, lane, v);
  float s = 0.f;
#pragma unroll
  for (int e = 0; e < E; ++e) s = fmaf(a.q[e], k[e], s);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  s *= scale;
  float mn = fmaxf(a.m, s);
  float c = __expf(a.m - mn);  // 0 on the first key (a.m = -inf)
  float p = __expf(s - mn);
  a.l = a.l * c + p;
#pragma unroll
  for (int e = 0; e < E; ++e) a.o[e] = fmaf(p, v[e], a.o[e] * c);
  a.m = mn;
}

template <int D>
__global__ void __launch_bounds__(128) attn_simt_kernel(const AttnParams P) {
  constexpr int E = D / 32;
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * 4 + (threadIdx.x >> 5);
  const int nb = P.hi - P.lo;
  const long long total = (long long)P.b * nb * P.Bq * P.Hq;
  if (row >= total) return;
  int h = (int)(row % P.Hq);
  long long t = row / P.Hq;
  int i = (int)(t % P.Bq);
  t /= P.Bq;
  int j = P.lo + (int)(t % nb);
  int n = (int)(t / nb);
  const int g = h / P.G;
  const size_t kvs = (size_t)P.Hkv * D;  // elements between consecutive key rows

  RowAcc<D> a;
  const size_t qoff = ((((size_t)n * P.J + j) * P.Bq + i) * P.Hq + h) * D;
  load_lane<D>(P.q + qoff, lane, a.q);
#pragma unroll
  for (int e = 0; e < E; ++e) a.o[e] = 0.f;
  a.m = -INFINITY;
  a.l = 0.f;

  const long long c0 = P.ctx_offsets[n], c1 = P.ctx_offsets[n + 1];
  const uint16_t *kc = P.k_ctx + (size_t)c0 * kvs + (size_t)g * D;
  const uint16_t *vc = P.v_ctx + (size_t)c0 * kvs + (size_t)g * D;
  for (long long tkey = 0; tkey < c1 - c0; ++tkey) visit_key<D>(a, kc + tkey * kvs, vc + tkey * kvs, lane, P.scale);
  const int na = max(0, min(j + P.pb, P.S));
  const uint16_t *ks = P.k_spine + ((size_t)n * P.S) * kvs + (size_t)g * D;
  const uint16_t *vs = P.v_spine + ((size_t)n * P.S) * kvs + (size_t)g * D;
  for (int s = 0; s < na; ++s) visit_key<D>(a, ks + s * kvs, vs + s * kvs, lane, P.scale);
  if (P.k_blk) {
    const uint16_t *kb = P.k_blk + (((size_t)n * P.J + j) * P.Bq) * kvs + (size_t)g * D;
    const uint16_t *vb = P.v_blk + (((size_t)n * P.J + j) * P.Bq) * kvs + (size_t)g * D;
    for (int s = 0; s < P.Bq; ++s) visit_key<D>(a, kb + s * kvs, vb + s * kvs, lane, P.scale);
  }
  const float inv = a.l > 0.f ? 1.f / a.l : 0.f;
  if (P.out_f32) {
    float *o = static_cast<float *>(P.out) + qoff + lane * E;
#pragma unroll
    for (int e = 0; e < E; ++e) o[e] = a.o[e] * inv;
  } else {
    uint16_t *o = static_cast<uint16_t *>(P.out) + qoff + lane * E;
#pragma unroll
    for (int e = 0; e < E; e += 2) *reinterpret_cast<uint32_t *>(o + e) = pack_bf16(a.o[e] * inv, a.o[e + 1] * inv);
  }
  if (P.out_lse && lane == 0) P.out_lse[qoff / D] = a.l > 0.f ? a.m + logf(a.l) : -INFINITY;
}

dpara_status launch_attention_simt(const AttnParams &P, cudaStream_t st) {
  const long long total = (long long)P.b * (P.hi - P.lo) * P.Bq * P.Hq;
  if (total <= 0) return DPARA_OK;
  const long long blocks = (total + 3) / 4;
  if (blocks > 0x7fffffffLL) return DPARA_ERR_UNSUPPORTED;
  if (P.D == 128)
    attn_simt_kernel<128><<<(unsigned)blocks, 128, 0, st>>>(P);
  else
    attn_simt_kernel<64><<<(unsigned)blocks, 128, 0, st>>>(P);
  DPARA_CHECK_LAUNCH();
  count_launches(1);
  return DPARA_OK;
}

}  // namespace dpara
