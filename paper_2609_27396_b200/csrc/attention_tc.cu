// All-boundary attention on the 5th-generation tensor cores (Sec. 3.2, Fig. 4).
//
// Work item = (request n, KV head g, pair of 128-row query tiles, KV split).  The query rows of one
// (n, g) are ordered (boundary j, slot i, head-in-group), so one 128-row tile holds whole (j, i) rows
// of all G query heads that share the KV head, and every K/V byte streamed from HBM serves all
// boundaries and all heads of the group at once.
//
//   warp 8      TMA producer: Q tiles once, then K and V tiles of 128 keys through one ring of tile slots.
//               The context needs no mask at all (every row sees the whole cache); the spine prefix
//               and the boundaries' own blocks are packed into ONE extra "tail" tile per CTA.
//   warp 9      one thread issues tcgen05.mma:  S_t = Q_t K^T  (A, B from shared memory) and
//               O_t += P_t V  (A = P_t from tensor memory, B = V, MN-major), t = 0, 1 ping-pong so the
//               tensor pipe works on one tile while the other tile's softmax runs.
//   warps 0-3   softmax of tile 0, warps 4-7 softmax of tile 1: thread = row.  tcgen05.ld the S row,
//               mask (tail tile only: anchor prefix of the row's boundary + its own block), online
//               max/sum in registers with LAZY rescaling (O in TMEM is rescaled only when a row's max
//               grows by more than 2^8), P written back over S as bf16 with tcgen05.st.
// TMEM: S0 | S1 (128 fp32 columns each, P aliases the first 64) | O0 | O1 (D columns each).
// Every mbarrier wait is bounded; on expiry the CTA sets DPARA_STATUS_TIMEOUT and drains.
#include <math.h>

#include "attention_tc.cuh"
#include "sm100_ptx.cuh"

namespace dpara {
using namespace ptx;

namespace {
constexpr int kThreads = 320;
constexpr float kRescaleLog2 = 8.0f;
constexpr int kMaxOrdered = 128;
}  // namespace

struct TcParams {
  CUtensorMap map_q, map_kc, map_vc, map_ks, map_vs, map_kb, map_vb;
  AttnParams a;
  int JI_T, n_ji, n_tiles, n_pairs, nsplit, S8, R_blk, has_blk, has_tail;
  float *part_o;   // [item][2][128][D]
  float *part_ml;  // [item][2][128][2]
  float c_log2;    // softmax scale * log2(e)
  // requests in order of decreasing context length: the block scheduler hands out CTAs in grid order, so
  // launching the long requests first leaves the short ones to fill the tail of a ragged batch
  uint8_t req_order[kMaxOrdered];
  int use_order;
};

template <int D>
struct TcCfg {
  static constexpr int kSlabs = D / 64;
  static constexpr int kSlabBytes = 128 * 128;         // 128 rows x 64 bf16
  static constexpr int kTileBytes = kSlabs * kSlabBytes;  // Q, K or V tile
  // K and V tiles travel through ONE ring of tile-sized slots (K0 V0 K1 V1 ...), as deep as shared memory
  // allows next to the two Q tiles: the producer runs ~1.5 iterations ahead of the MMA issuer
  static constexpr int kSlots = (227 * 1024 - 2 * kTileBytes - 2048) / kTileBytes > 8 ? 8 : (227 * 1024 - 2 * kTileBytes - 2048) / kTileBytes;
  static constexpr int kSmemBytes = 2 * kTileBytes + kSlots * kTileBytes + 1024 + 512;
  static constexpr int kOBase = 256;                    // TMEM column of O0
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1) attn_tc_kernel(const __grid_constant__ TcParams P) {
  using Cfg = TcCfg<D>;
  const AttnParams &A = P.a;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *sQ = smem;                                   // 2 tiles
  uint8_t *sKV = smem + 2 * Cfg::kTileBytes;            // ring of K / V tile slots
  constexpr int kSlots = Cfg::kSlots;
  uint64_t *bars = reinterpret_cast<uint64_t *>(sKV + kSlots * Cfg::kTileBytes);
  uint64_t *kv_full = bars, *kv_empty = bars + kSlots, *q_full = bars + 2 * kSlots, *s_full = q_full + 1, *p_full = q_full + 3,
           *pv_done = q_full + 5;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(q_full + 7);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n = P.use_order ? (int)P.req_order[blockIdx.z] : (int)blockIdx.z, g = blockIdx.y;
  const int pair = blockIdx.x / P.nsplit, split = blockIdx.x % P.nsplit;
  const int ntq = min(2, P.n_tiles - pair * 2);
  const long long c0 = A.ctx_offsets[n];
  const int L = (int)(A.ctx_offsets[n + 1] - c0);
  const int nctx = (L + 127) >> 7;
  const int t0 = (int)((long long)split * nctx / P.nsplit), t1 = (int)((long long)(split + 1) * nctx / P.nsplit);
  const int n_ctx_it = t1 - t0;
  const bool do_tail = P.has_tail && split == P.nsplit - 1;
  const int n_iter = n_ctx_it + (do_tail ? 1 : 0);
  const int item = ((n * A.Hkv + g) * P.n_pairs + pair) * P.nsplit + split;
  const int jb0 = A.lo + (pair * 2 * P.JI_T) / A.Bq;    // first boundary whose block keys sit in the tail tile

  if (A.status_word && (*reinterpret_cast<volatile int32_t *>(A.status_word) & (int32_t)DPARA_STATUS_TIMEOUT)) return;

  if (n_iter == 0) {  // nothing visible to this work item
    for (int r = threadIdx.x; r < 256; r += kThreads) {
      if (P.nsplit > 1) {
        P.part_ml[((size_t)item * 256 + r) * 2] = -INFINITY;
        P.part_ml[((size_t)item * 256 + r) * 2 + 1] = 0.f;
      } else {
        const int t = r >> 7, rr = r & 127;
        const int ji = (pair * 2 + t) * P.JI_T + rr / A.G;
        if (t < ntq && rr < P.JI_T * A.G && ji < P.n_ji) {
          const int j = A.lo + ji / A.Bq, i = ji % A.Bq, h = g * A.G + rr % A.G;
          const size_t o = ((((size_t)n * A.J + j) * A.Bq + i) * A.Hq + h);
          for (int d = 0; d < D; ++d) {
            if (A.out_f32) static_cast<float *>(A.out)[o * D + d] = 0.f;
            else static_cast<uint16_t *>(A.out)[o * D + d] = 0;
          }
          if (A.out_lse) A.out_lse[o] = -INFINITY;
        }
      }
    }
    return;
  }

  if (threadIdx.x == 0) {
    for (int s = 0; s < kSlots; ++s) { mbar_init(kv_full + s, 1); mbar_init(kv_empty + s, 1); }
    mbar_init(q_full, 1);
    for (int t = 0; t < 2; ++t) { mbar_init(s_full + t, 1); mbar_init(p_full + t, 4); mbar_init(pv_done + t, 1); }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 9) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 8) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      prefetch_tensormap(&P.map_q);
      if (L > 0) { prefetch_tensormap(&P.map_kc); prefetch_tensormap(&P.map_vc); }
      const int qrow0 = (n * A.J + A.lo) * A.Bq + pair * 2 * P.JI_T;
      mbar_arrive_expect_tx(q_full, (uint32_t)(ntq * P.JI_T * A.G * 128 * Cfg::kSlabs));
      for (int t = 0; t < ntq; ++t)
        for (int sl = 0; sl < Cfg::kSlabs; ++sl)
          tma_load_3d(sQ + t * Cfg::kTileBytes + sl * Cfg::kSlabBytes, &P.map_q, q_full, sl * 64, g * A.G, qrow0 + t * P.JI_T);
    }
    // load q = 2 it is the K tile of iteration it, load 2 it + 1 its V tile; slot = q % kSlots
    for (int q = 0; q < 2 * n_iter; ++q) {
      const int it = q >> 1, is_v = q & 1;
      const int sl = q % kSlots;
      const uint32_t ph = (q / kSlots) & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(kv_empty + sl, ph ^ 1u, abort_flag))) break;
      uint8_t *dst = sKV + sl * Cfg::kTileBytes;
      if (it < n_ctx_it) {
        if (lane == 0) {
          const int row = (int)(c0 + (long long)(t0 + it) * 128);
          mbar_arrive_expect_tx(kv_full + sl, Cfg::kTileBytes);
          for (int sb = 0; sb < Cfg::kSlabs; ++sb)
            tma_load_3d(dst + sb * Cfg::kSlabBytes, is_v ? &P.map_vc : &P.map_kc, kv_full + sl, sb * 64, g, row);
        }
      } else {
        if (is_v) {
          // tail tile: rows the TMA boxes do not cover must still hold finite V (P = 0 there): clear the V tile
          for (int o = lane * 16; o < Cfg::kTileBytes; o += 32 * 16) *reinterpret_cast<uint4 *>(dst + o) = make_uint4(0, 0, 0, 0);
          fence_proxy_async();
          __syncwarp();
        }
        if (lane == 0) {
          uint32_t bytes = 0;
          if (A.S > 0) bytes += (uint32_t)A.S * 128 * Cfg::kSlabs;
          if (P.has_blk) bytes += (uint32_t)P.R_blk * 128 * Cfg::kSlabs;
          mbar_arrive_expect_tx(kv_full + sl, bytes);
          for (int sb = 0; sb < Cfg::kSlabs; ++sb) {
            if (A.S > 0) tma_load_3d(dst + sb * Cfg::kSlabBytes, is_v ? &P.map_vs : &P.map_ks, kv_full + sl, sb * 64, g, n * A.S);
            if (P.has_blk)
              tma_load_3d(dst + sb * Cfg::kSlabBytes + P.S8 * 128, is_v ? &P.map_vb : &P.map_kb, kv_full + sl, sb * 64, g,
                          (n * A.J + jb0) * A.Bq);
          }
        }
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = idesc_bf16_f32(128, 128, false, false);
      constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, false, true);
      const uint32_t q_addr = smem_u32(sQ), kv_addr = smem_u32(sKV);
      auto issue_qk = [&](int t, int it) {
        const uint32_t qa = q_addr + t * Cfg::kTileBytes, ka = kv_addr + ((2 * it) % kSlots) * Cfg::kTileBytes;
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk >> 2) * Cfg::kSlabBytes + (kk & 3) * 32;
          mma_ss(tmem + t * 128, smem_desc_sw128(qa + off, 16, 1024), smem_desc_sw128(ka + off, 16, 1024), idesc_qk, kk != 0);
        }
        mma_commit(s_full + t);
        if (t == ntq - 1) mma_commit(kv_empty + (2 * it) % kSlots);      // K tile consumed by every query tile
      };
      auto issue_pv = [&](int t, int it) {
        const uint32_t va = kv_addr + ((2 * it + 1) % kSlots) * Cfg::kTileBytes;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk)
          mma_ts(tmem + Cfg::kOBase + t * D, tmem + t * 128 + kk * 8, smem_desc_sw128(va + kk * 2048, Cfg::kSlabBytes, 1024),
                 idesc_pv, it > 0 || kk != 0);
        mma_commit(pv_done + t);
        if (t == ntq - 1) mma_commit(kv_empty + (2 * it + 1) % kSlots);  // V tile consumed
      };
      auto wait_load = [&](int q) { return mbar_wait(kv_full + q % kSlots, (q / kSlots) & 1, abort_flag); };
      bool ok = mbar_wait(q_full, 0, abort_flag) && wait_load(0);
      if (ok) {
        tc_fence_after();
        for (int t = 0; t < ntq; ++t) issue_qk(t, 0);
        for (int it = 0; it < n_iter && ok; ++it) {
          for (int t = 0; t < ntq && ok; ++t) {
            ok = mbar_wait(p_full + t, it & 1, abort_flag);
            if (ok && t == 0) ok = wait_load(2 * it + 1);
            if (!ok) break;
            tc_fence_after();
            issue_pv(t, it);
            if (it + 1 < n_iter) {
              if (t == 0) {
                ok = wait_load(2 * it + 2);
                if (!ok) break;
                tc_fence_after();
              }
              issue_qk(t, it + 1);
            }
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue: thread = row
    const int t = warp >> 2;
    if (t < ntq) {
      const int wq = warp & 3;
      const int r = wq * 32 + lane;
      const uint32_t lane_addr = tmem + ((uint32_t)(wq * 32) << 16);
      const int ji = (pair * 2 + t) * P.JI_T + r / A.G;
      const bool valid = (r < P.JI_T * A.G) && (ji < P.n_ji);
      const int j = A.lo + ji / A.Bq, i = ji % A.Bq, h = g * A.G + r % A.G;
      const int na = max(0, min(j + A.pb, A.S));
      const int b0 = P.has_blk ? P.S8 + (j - jb0) * A.Bq : 0, b1 = P.has_blk ? b0 + A.Bq : 0;
      const float c = P.c_log2;
      const float thr = kRescaleLog2 / c;
      float m_used = -INFINITY, l = 0.f;
      bool ok = true;

      for (int it = 0; it < n_iter; ++it) {
        ok = __all_sync(0xffffffffu, mbar_wait(s_full + t, it & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
#ifdef DPARA_EXP_SYNCONLY
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(p_full + t);
        continue;
#endif
        uint32_t su[128];
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) tmem_ld32(lane_addr + t * 128 + cc * 32, su + cc * 32);
        tmem_wait_ld();
        float s[128];
#pragma unroll
        for (int k = 0; k < 128; ++k) s[k] = __uint_as_float(su[k]);
        if (it >= n_ctx_it) {
#pragma unroll
          for (int k = 0; k < 128; ++k) s[k] = ((k < na) || (k >= b0 && k < b1)) ? s[k] : -INFINITY;
        } else if (it == n_ctx_it - 1 && t1 == nctx && (L & 127)) {
          const int nv = L & 127;
#pragma unroll
          for (int k = 0; k < 128; ++k) s[k] = k < nv ? s[k] : -INFINITY;
        }
#ifdef DPARA_EXP_NOMAX
        float mx = fmaxf(s[0], s[77]);
#else
        float mx = s[0];
#pragma unroll
        for (int k = 1; k < 128; ++k) mx = fmaxf(mx, s[k]);
#endif
        const bool need = mx > m_used + thr;  // also true when m_used = -inf and the tile has a visible key
        if (it == 0) {
          if (need) m_used = mx;
        } else if (__any_sync(0xffffffffu, need)) {
          ok = __all_sync(0xffffffffu, mbar_wait(pv_done + t, (it - 1) & 1, abort_flag));
          if (!ok) break;
          tc_fence_after();
          const float f = need ? ex2((m_used - mx) * c) : 1.0f;
#pragma unroll 1
          for (int cc = 0; cc < D / 32; ++cc) {
            uint32_t o[32];
            tmem_ld32(lane_addr + Cfg::kOBase + t * D + cc * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * f);
            tmem_st32(lane_addr + Cfg::kOBase + t * D + cc * 32, o);
          }
          tmem_wait_st();
          l *= f;
          if (need) m_used = mx;
        }
        const float mc = (m_used == -INFINITY ? 0.f : m_used) * c;
        uint32_t pk[64];
#pragma unroll
        for (int k = 0; k < 64; ++k) {
#ifdef DPARA_EXP_NOEX2
          const float p0 = fmaf(s[2 * k], c, -mc), p1 = fmaf(s[2 * k + 1], c, -mc);
#else
          const float p0 = ex2(fmaf(s[2 * k], c, -mc));
          const float p1 = ex2(fmaf(s[2 * k + 1], c, -mc));
#endif
          l += p0 + p1;
          pk[k] = pack_bf16(p0, p1);
        }
        tmem_st32(lane_addr + t * 128, pk);
        tmem_st32(lane_addr + t * 128 + 32, pk + 32);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(p_full + t);
      }

      // ---- epilogue
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(pv_done + t, (n_iter - 1) & 1, abort_flag));
      if (ok) {
        tc_fence_after();
        const size_t orow = (((size_t)n * A.J + j) * A.Bq + i) * A.Hq + h;
        const float inv = l > 0.f ? 1.0f / l : 0.f;
#pragma unroll 1
        for (int cc = 0; cc < D / 32; ++cc) {
          uint32_t o[32];
          tmem_ld32(lane_addr + Cfg::kOBase + t * D + cc * 32, o);
          tmem_wait_ld();
          if (P.nsplit > 1) {
            float4 *dst = reinterpret_cast<float4 *>(P.part_o + (((size_t)item * 2 + t) * 128 + r) * D + cc * 32);
#pragma unroll
            for (int v = 0; v < 8; ++v)
              dst[v] = make_float4(__uint_as_float(o[4 * v]), __uint_as_float(o[4 * v + 1]), __uint_as_float(o[4 * v + 2]),
                                   __uint_as_float(o[4 * v + 3]));
          } else if (valid) {
            if (A.out_f32) {
              float4 *dst = reinterpret_cast<float4 *>(static_cast<float *>(A.out) + orow * D + cc * 32);
#pragma unroll
              for (int v = 0; v < 8; ++v)
                dst[v] = make_float4(__uint_as_float(o[4 * v]) * inv, __uint_as_float(o[4 * v + 1]) * inv,
                                     __uint_as_float(o[4 * v + 2]) * inv, __uint_as_float(o[4 * v + 3]) * inv);
            } else {
              uint4 *dst = reinterpret_cast<uint4 *>(static_cast<uint16_t *>(A.out) + orow * D + cc * 32);
#pragma unroll
              for (int v = 0; v < 4; ++v) {
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
                  w[e] = pack_bf16(__uint_as_float(o[8 * v + 2 * e]) * inv, __uint_as_float(o[8 * v + 2 * e + 1]) * inv);
                dst[v] = make_uint4(w[0], w[1], w[2], w[3]);
              }
            }
          }
        }
        if (P.nsplit > 1) {
          P.part_ml[(((size_t)item * 2 + t) * 128 + r) * 2] = m_used;
          P.part_ml[(((size_t)item * 2 + t) * 128 + r) * 2 + 1] = l;
        } else if (valid && A.out_lse) {
          A.out_lse[orow] = l > 0.f ? (m_used * c + log2f(l)) * 0.6931471805599453f : -INFINITY;
        }
      }
    } else if (P.nsplit > 1) {
      // absent second tile of the last pair: its partial slots must read as empty
      const int r = (warp & 3) * 32 + lane;
      P.part_ml[(((size_t)item * 2 + 1) * 128 + r) * 2] = -INFINITY;
      P.part_ml[(((size_t)item * 2 + 1) * 128 + r) * 2 + 1] = 0.f;
    }
  }

  // ------------------------------------------------------------------ teardown
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // a wait gave up: give copies that may still be in flight a bounded time to land before the CTA's
    // shared memory is released, and report
    if (threadIdx.x == 0) {
      if (A.status_word) atomicOr(reinterpret_cast<unsigned int *>(A.status_word), DPARA_STATUS_TIMEOUT);
      for (int k = 0; k < 4096; ++k) __nanosleep(256);
    }
    __syncthreads();
  }
  if (warp == 9) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------------------------ split-KV combine
// One warp per (item pair, tile, row): merges the nsplit partial (m, l, O) triples of a query row.
template <int D>
__global__ void __launch_bounds__(128) attn_tc_combine_kernel(const TcParams P) {
  const AttnParams &A = P.a;
  const int lane = threadIdx.x & 31;
  const long long w = (long long)blockIdx.x * 4 + (threadIdx.x >> 5);
  const long long total = (long long)A.b * A.Hkv * P.n_pairs * 256;
  if (w >= total) return;
  const int r = (int)(w & 127), t = (int)((w >> 7) & 1);
  const long long base_item = (w >> 8);  // (n * Hkv + g) * n_pairs + pair
  const int pair = (int)(base_item % P.n_pairs);
  const int g = (int)((base_item / P.n_pairs) % A.Hkv), n = (int)(base_item / P.n_pairs / A.Hkv);
  const int ji = (pair * 2 + t) * P.JI_T + r / A.G;
  if (pair * 2 + t >= P.n_tiles || r >= P.JI_T * A.G || ji >= P.n_ji) return;
  const int j = A.lo + ji / A.Bq, i = ji % A.Bq, h = g * A.G + r % A.G;
  constexpr int E = D / 32;
  float mmax = -INFINITY;
  for (int s = 0; s < P.nsplit; ++s) mmax = fmaxf(mmax, P.part_ml[((((size_t)base_item * P.nsplit + s) * 2 + t) * 128 + r) * 2]);
  float l = 0.f, o[E];
#pragma unroll
  for (int e = 0; e < E; ++e) o[e] = 0.f;
  for (int s = 0; s < P.nsplit; ++s) {
    const size_t slot = (((size_t)base_item * P.nsplit + s) * 2 + t) * 128 + r;
    const float ms = P.part_ml[slot * 2], ls = P.part_ml[slot * 2 + 1];
    if (!(ls > 0.f)) continue;
    const float wgt = ptx::ex2((ms - mmax) * P.c_log2);
    l += wgt * ls;
    const float *po = P.part_o + slot * D + lane * E;
#pragma unroll
    for (int e = 0; e < E; ++e) o[e] = fmaf(wgt, po[e], o[e]);
  }
  const float inv = l > 0.f ? 1.0f / l : 0.f;
  const size_t orow = (((size_t)n * A.J + j) * A.Bq + i) * A.Hq + h;
  if (A.out_f32) {
    float *dst = static_cast<float *>(A.out) + orow * D + lane * E;
#pragma unroll
    for (int e = 0; e < E; ++e) dst[e] = o[e] * inv;
  } else {
    uint16_t *dst = static_cast<uint16_t *>(A.out) + orow * D + lane * E;
#pragma unroll
    for (int e = 0; e < E; e += 2) *reinterpret_cast<uint32_t *>(dst + e) = pack_bf16(o[e] * inv, o[e + 1] * inv);
  }
  if (A.out_lse && lane == 0) A.out_lse[orow] = l > 0.f ? (mmax * P.c_log2 + log2f(l)) * 0.6931471805599453f : -INFINITY;
}

// ------------------------------------------------------------------------------------------------ host
TcPlan plan_attention_tc(const dpara_shape *s, const int64_t *host_off) {
  TcPlan p{};
  const int G = s->n_q_heads / s->n_kv_heads;
  const int nb = s->boundary_hi - s->boundary_lo;
  if (nb <= 0) return p;
  p.JI_T = 128 / G;
  p.n_ji = nb * s->block;
  p.n_tiles = (p.n_ji + p.JI_T - 1) / p.JI_T;
  p.n_pairs = (p.n_tiles + 1) / 2;
  p.S8 = (s->n_spine + 7) & ~7;
  int nbmax = (2 * p.JI_T - 1) / s->block + 2;
  if (nbmax > nb) nbmax = nb;
  p.R_blk = nbmax * s->block;
  if (G > 16 || p.JI_T < 1 || p.JI_T > 256 || s->n_spine > 64 || p.R_blk > 256 || p.S8 + p.R_blk > 128) return p;
  long long max_l = 0, tot = host_off[s->batch] - host_off[0];
  for (int n = 0; n < s->batch; ++n) max_l = (host_off[n + 1] - host_off[n]) > max_l ? (host_off[n + 1] - host_off[n]) : max_l;
  if (tot + 128 >= (1ll << 31) || (long long)s->batch * s->n_boundaries * s->block >= (1ll << 31)) return p;
  const long long items = (long long)s->batch * s->n_kv_heads * p.n_pairs;
  const int max_tiles = (int)((max_l + 127) / 128);
  int nsplit = 1;
  if (items < 96 && max_tiles > 1) {
    nsplit = (int)((kNumSM + items - 1) / items);
    if (nsplit > max_tiles) nsplit = max_tiles;
    if (nsplit > 32) nsplit = 32;
    if (nsplit < 1) nsplit = 1;
  }
  p.nsplit = nsplit;
  p.items = items;
  p.workspace_bytes = nsplit > 1 ? (size_t)items * nsplit * 256 * ((size_t)s->head_dim + 2) * 4 : 0;
  p.eligible = true;
  return p;
}

template <int D>
static dpara_status launch_tc_d(const TcParams &P, const TcPlan &plan, cudaStream_t st) {
  using Cfg = TcCfg<D>;
  if (cudaFuncSetAttribute(attn_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes) != cudaSuccess) return DPARA_ERR_CUDA;
  dim3 grid(P.n_pairs * P.nsplit, P.a.Hkv, P.a.b);
  attn_tc_kernel<D><<<grid, kThreads, Cfg::kSmemBytes, st>>>(P);
  DPARA_CHECK_LAUNCH();
  count_launches(1);
  if (P.nsplit > 1) {
    const long long rows = plan.items * 256;
    attn_tc_combine_kernel<D><<<(unsigned)((rows + 3) / 4), 128, 0, st>>>(P);
    DPARA_CHECK_LAUNCH();
    count_launches(1);
  }
  return DPARA_OK;
}

dpara_status launch_attention_tc(const AttnParams &A, const TcPlan &plan, const int64_t *host_off, void *workspace, cudaStream_t st) {
  TcParams P;
  memset(&P, 0, sizeof(P));
  P.a = A;
  P.JI_T = plan.JI_T; P.n_ji = plan.n_ji; P.n_tiles = plan.n_tiles; P.n_pairs = plan.n_pairs; P.nsplit = plan.nsplit;
  P.S8 = plan.S8; P.R_blk = plan.R_blk; P.has_blk = A.k_blk != nullptr;
  P.has_tail = (A.S > 0) || P.has_blk;
  P.c_log2 = A.scale * 1.4426950408889634f;
  const int D = A.D;
  const uint64_t rs = (uint64_t)D * 2;
  const long long tot = host_off[A.b] - host_off[0];
  const uint64_t nq = (uint64_t)A.b * A.J * A.Bq;
  bool ok = make_tmap_bf16_3d(&P.map_q, A.q, D, A.Hq, nq, rs, rs * A.Hq, 64, A.G, plan.JI_T);
  if (tot > 0) {
    ok = ok && make_tmap_bf16_3d(&P.map_kc, A.k_ctx, D, A.Hkv, host_off[A.b], rs, rs * A.Hkv, 64, 1, 128);
    ok = ok && make_tmap_bf16_3d(&P.map_vc, A.v_ctx, D, A.Hkv, host_off[A.b], rs, rs * A.Hkv, 64, 1, 128);
  }
  if (A.S > 0) {
    ok = ok && make_tmap_bf16_3d(&P.map_ks, A.k_spine, D, A.Hkv, (uint64_t)A.b * A.S, rs, rs * A.Hkv, 64, 1, A.S);
    ok = ok && make_tmap_bf16_3d(&P.map_vs, A.v_spine, D, A.Hkv, (uint64_t)A.b * A.S, rs, rs * A.Hkv, 64, 1, A.S);
  }
  if (P.has_blk) {
    ok = ok && make_tmap_bf16_3d(&P.map_kb, A.k_blk, D, A.Hkv, nq, rs, rs * A.Hkv, 64, 1, plan.R_blk);
    ok = ok && make_tmap_bf16_3d(&P.map_vb, A.v_blk, D, A.Hkv, nq, rs, rs * A.Hkv, 64, 1, plan.R_blk);
  }
  if (!ok) return DPARA_ERR_CUDA;
  P.use_order = A.b <= kMaxOrdered && A.b > 1;
  if (P.use_order) {
    int idx[kMaxOrdered];
    for (int n = 0; n < A.b; ++n) idx[n] = n;
    for (int a = 1; a < A.b; ++a) {  // insertion sort by decreasing length (stable)
      const int v = idx[a];
      const long long lv = host_off[v + 1] - host_off[v];
      int c = a - 1;
      while (c >= 0 && host_off[idx[c] + 1] - host_off[idx[c]] < lv) { idx[c + 1] = idx[c]; --c; }
      idx[c + 1] = v;
    }
    for (int n = 0; n < A.b; ++n) P.req_order[n] = (uint8_t)idx[n];
  }
  if (plan.nsplit > 1) {
    P.part_o = static_cast<float *>(workspace);
    P.part_ml = P.part_o + (size_t)plan.items * plan.nsplit * 256 * D;
  }
  return D == 128 ? launch_tc_d<128>(P, plan, st) : launch_tc_d<64>(P, plan, st);
}

}  // namespace dpara
