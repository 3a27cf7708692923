// bf16 GEMM  out[M][N] = epilogue( a[M][K] * w[N][K]^T )  on the 5th-generation tensor cores.
//
// One CTA computes a 128 x 256 output tile: a TMA producer warp streams 64-wide K slabs of both
// operands (128-byte swizzle) through a 4-stage shared-memory ring, one elected thread issues
// tcgen05.mma (M = 128, N = 256, K = 16, fp32 accumulator in 256 TMEM columns), four warps read the
// accumulator back with tcgen05.ld and apply the epilogue:
//   0  bf16 store                                   (QKV projection)
//   1  fp32 out = resid + acc  (+ bf16 copy)        (O and down projections with the residual add)
//   2  bf16 out = silu(gate) * up                   (gate/up projection: the tile's 256 accumulator
//                                                    columns are 128 gate columns and the matching 128
//                                                    up columns, so the activation never leaves the SM)
//   3  fp32 store                                   (LM head: base logits)
// Every mbarrier wait is bounded; on expiry the CTA sets DPARA_STATUS_TIMEOUT and drains.
#include "gemm.cuh"
#include "sm100_ptx.cuh"

namespace dpara {
using namespace ptx;

namespace {
constexpr int kBM = 128, kBN = 256, kBK = 64, kStages = 4;
constexpr int kABytes = kBM * kBK * 2;         // 16 KB
constexpr int kBBytes = kBN * kBK * 2;         // 32 KB (two 128-row boxes)
constexpr int kStageBytes = kABytes + kBBytes;  // 48 KB
constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*align*/ + 256 /*barriers*/;
constexpr int kThreads = 192;                   // warps 0-3 epilogue, 4 TMA, 5 MMA
}  // namespace

struct GemmKernelParams {
  CUtensorMap map_a;
  CUtensorMap map_b;
  int M, N, K;
  int epi;
  int up_row_offset;
  void *out;
  const void *resid;
  int resid_bf16;
  void *out_bf16;
  int32_t *status;
  int perm_block, perm_b;
};

__device__ __forceinline__ float silu_f(float g) { return g / (1.0f + __expf(-g)); }

// Epilogue of one accumulator tile: thread = one accumulator row (`row` of the output), `taddr` = this warp's lanes
// of the accumulator buffer.
__device__ __forceinline__ void gemm_epilogue(const GemmKernelParams &P, uint32_t taddr, int row, int n_tile) {
      if (P.epi == 2) {
        const int col0 = n_tile * 128;
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t g[32], u[32];
          tmem_ld32(taddr + c * 32, g);
          tmem_ld32(taddr + 128 + c * 32, u);
          tmem_wait_ld();
          if (row < P.M) {
            uint16_t *o = static_cast<uint16_t *>(P.out) + (size_t)row * P.N + col0 + c * 32;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              if (col0 + c * 32 + v * 8 < P.N) {
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  float a0 = silu_f(__uint_as_float(g[v * 8 + 2 * e])) * __uint_as_float(u[v * 8 + 2 * e]);
                  float a1 = silu_f(__uint_as_float(g[v * 8 + 2 * e + 1])) * __uint_as_float(u[v * 8 + 2 * e + 1]);
                  w[e] = pack_bf16(a0, a1);
                }
                *reinterpret_cast<uint4 *>(o + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
              }
            }
          }
        }
      } else {
        const int col0 = n_tile * kBN;
#pragma unroll 1
        for (int c = 0; c < kBN / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(taddr + c * 32, r);
          tmem_wait_ld();
          if (row < P.M) {
            const int cb = col0 + c * 32;
            if (P.epi == 0) {
              uint16_t *o = static_cast<uint16_t *>(P.out) + (size_t)row * P.N + cb;
#pragma unroll
              for (int v = 0; v < 4; ++v) {
                if (cb + v * 8 < P.N) {
                  uint32_t w[4];
#pragma unroll
                  for (int e = 0; e < 4; ++e)
                    w[e] = pack_bf16(__uint_as_float(r[v * 8 + 2 * e]), __uint_as_float(r[v * 8 + 2 * e + 1]));
                  *reinterpret_cast<uint4 *>(o + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                }
              }
            } else {
              const int orow = P.perm_block ? (row % P.perm_block) * P.perm_b + row / P.perm_block : row;
              float *o = static_cast<float *>(P.out) + (size_t)orow * P.N + cb;
#pragma unroll
              for (int v = 0; v < 8; ++v) {
                if (cb + v * 4 < P.N) {
                  float x[4];
                  if (P.epi == 3) {
                    x[0] = x[1] = x[2] = x[3] = 0.f;
                  } else if (P.resid_bf16) {
                    uint2 rr = *reinterpret_cast<const uint2 *>(static_cast<const uint16_t *>(P.resid) + (size_t)row * P.N + cb + v * 4);
                    x[0] = bf16lo(rr.x); x[1] = bf16hi(rr.x); x[2] = bf16lo(rr.y); x[3] = bf16hi(rr.y);
                  } else {
                    float4 rr = *reinterpret_cast<const float4 *>(static_cast<const float *>(P.resid) + (size_t)row * P.N + cb + v * 4);
                    x[0] = rr.x; x[1] = rr.y; x[2] = rr.z; x[3] = rr.w;
                  }
#pragma unroll
                  for (int e = 0; e < 4; ++e) x[e] += __uint_as_float(r[v * 4 + e]);
                  *reinterpret_cast<float4 *>(o + v * 4) = make_float4(x[0], x[1], x[2], x[3]);
                  if (P.out_bf16) {
                    uint16_t *ob = static_cast<uint16_t *>(P.out_bf16) + (size_t)row * P.N + cb + v * 4;
                    *reinterpret_cast<uint2 *>(ob) = make_uint2(pack_bf16(x[0], x[1]), pack_bf16(x[2], x[3]));
                  }
                }
              }
            }
          }
        }
      }
}

__global__ void __launch_bounds__(kThreads, 1) gemm_tc_kernel(const __grid_constant__ GemmKernelParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + kStages * kStageBytes);
  uint64_t *empty = full + kStages;
  uint64_t *acc_full = empty + kStages;   // [2]: accumulator buffer ready for the epilogue
  uint64_t *acc_empty = acc_full + 2;     // [2]: accumulator buffer drained
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nkb = P.K / kBK;
  const int tile_cols = P.epi == 2 ? 128 : kBN;
  const int m_tiles = (P.M + kBM - 1) / kBM, n_tiles = (P.N + tile_cols - 1) / tile_cols;
  const int total_tiles = m_tiles * n_tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full + s, 1);
      mbar_init(empty + s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full + b, 1);
      mbar_init(acc_empty + b, 4);
    }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 5) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  // Persistent: CTA c computes tiles c, c + gridDim.x, ...; tile id = n_tile * m_tiles + m_tile, so the CTAs
  // running together cover all M rows of a few weight tiles (A stays in L2, each weight tile is read once).
  // Two accumulator buffers in TMEM let the epilogue of one tile overlap the main loop of the next.
  if (warp == 4) {
    if (lane == 0) {
      prefetch_tensormap(&P.map_a);
      prefetch_tensormap(&P.map_b);
      int stage = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        const int m_tile = tile % m_tiles, n_tile = tile / m_tiles;
        const int brow0 = P.epi == 2 ? n_tile * 128 : n_tile * kBN;
        const int brow1 = P.epi == 2 ? P.up_row_offset + n_tile * 128 : n_tile * kBN + 128;
        for (int kb = 0; kb < nkb; ++kb) {
          ok = mbar_wait(empty + stage, ph ^ 1u, abort_flag);
          if (!ok) break;
          uint8_t *sa = smem + stage * kStageBytes;
          mbar_arrive_expect_tx(full + stage, kStageBytes);
          tma_load_2d(sa, &P.map_a, full + stage, kb * kBK, m_tile * kBM);
          tma_load_2d(sa + kABytes, &P.map_b, full + stage, kb * kBK, brow0);
          tma_load_2d(sa + kABytes + 128 * kBK * 2, &P.map_b, full + stage, kb * kBK, brow1);
          if (++stage == kStages) { stage = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 5) {
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(kBM, kBN, false, false);
      // descriptors are built once; stage and K-step offsets are added in 16-byte units
      const uint64_t adesc0 = smem_desc_sw128(smem_u32(smem), 16, 1024);
      const uint64_t bdesc0 = smem_desc_sw128(smem_u32(smem) + kABytes, 16, 1024);
      int stage = 0, k = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++k) {
        const int buf = k & 1;
        ok = mbar_wait(acc_empty + buf, ((k >> 1) & 1) ^ 1u, abort_flag);  // epilogue of tile k - 2 has drained this buffer
        if (!ok) break;
        tc_fence_after();
        const uint32_t acc = tmem + buf * kBN;
        for (int kb = 0; kb < nkb; ++kb) {
          ok = mbar_wait(full + stage, ph, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint64_t so = (uint64_t)(stage * (kStageBytes >> 4));
          mma_ss(acc, adesc0 + so, bdesc0 + so, idesc, kb != 0);
#pragma unroll
          for (int kk = 1; kk < kBK / 16; ++kk) mma_ss_c<true>(acc, adesc0 + so + 2 * kk, bdesc0 + so + 2 * kk, idesc);
          mma_commit(empty + stage);
          if (++stage == kStages) { stage = 0; ph ^= 1u; }
        }
        if (ok) mma_commit(acc_full + buf);
      }
    }
  } else {
   int k = 0;
   bool live = true;
   for (int tile = blockIdx.x; tile < total_tiles && live; tile += gridDim.x, ++k) {
    const int m_tile = tile % m_tiles, n_tile = tile / m_tiles;
    const int buf = k & 1;
    // ---------------- epilogue: thread = one accumulator row
    const bool ok = __all_sync(0xffffffffu, mbar_wait(acc_full + buf, (k >> 1) & 1, abort_flag));  // warp-uniform: tcgen05.ld is warp-wide
    tc_fence_after();
    const int row = m_tile * kBM + warp * 32 + lane;
    const uint32_t taddr = tmem + buf * kBN + ((uint32_t)(warp * 32) << 16);
    live = ok;
    if (ok) {
      gemm_epilogue(P, taddr, row, n_tile);
    }
    // this warp has read its part of the accumulator: hand the buffer back to the MMA issuer
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(acc_empty + buf);
   }
  }
  // ---------------- teardown
  if (threadIdx.x == 0 && *abort_flag && P.status) atomicOr(reinterpret_cast<unsigned int *>(P.status), DPARA_STATUS_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  if (warp == 5) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------------------------ CTA pairs
// The same GEMM with a pair of CTAs (a cluster of two, tcgen05 cta_group::2) per 256 x 256 output tile.  Each CTA
// holds 128 rows of the activations, HALF of the weight tile (128 of its 256 rows) and the accumulator of its own
// 128 output rows; the even CTA's thread issues M = 256 products that read both halves.  Per pair and K slab
// 64 KB enter shared memory instead of the 96 KB two independent 128 x 256 tiles need: these shapes
// (M = 256..1024 rows against large weights) are bound by the L2 -> shared-memory fill rate, not by the tensor
// pipe.  Each CTA's producer fetches its own halves with ordinary tiled copies and counts the bytes on the LEADER's
// barrier; stage and accumulator hand-offs from the MMA thread reach both CTAs through one tcgen05.commit;
// the epilogue warps of both CTAs arrive on the leader's accumulator-empty barrier.
namespace {
constexpr int kStages2 = 6;
constexpr int kStageBytes2 = kABytes + 128 * kBK * 2;  // 32 KB: 128 activation rows + 128 weight rows
constexpr int kSmemBytes2 = kStages2 * kStageBytes2 + 1024 + 256;
}  // namespace

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1) gemm_tc2_kernel(const __grid_constant__ GemmKernelParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + kStages2 * kStageBytes2);   // used in the leader only
  uint64_t *empty = full + kStages2;                                              // local copy in each CTA
  uint64_t *acc_full = empty + kStages2;                                          // [2] local copy in each CTA
  uint64_t *acc_empty = acc_full + 2;                                             // [2] used in the leader only
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int nkb = P.K / kBK;
  const int tile_cols = P.epi == 2 ? 128 : kBN;
  const int m_pairs = (P.M + 2 * kBM - 1) / (2 * kBM), n_tiles = (P.N + tile_cols - 1) / tile_cols;
  const int total_tiles = m_pairs * n_tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages2; ++s) {
      mbar_init(full + s, 1);
      mbar_init(empty + s, 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full + b, 1);
      mbar_init(acc_empty + b, 8);   // four epilogue warps of each CTA
    }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 5) {
    tmem_alloc_pair(tmem_slot, 512);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // both CTAs' barriers exist before anything signals across the pair
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 4) {
    if (lane == 0) {
      prefetch_tensormap(&P.map_a);
      prefetch_tensormap(&P.map_b);
      int stage = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int tile = pair; tile < total_tiles && ok; tile += n_pairs) {
        const int m_pair = tile % m_pairs, n_tile = tile / m_pairs;
        // this CTA's half of the weight tile: rows [rank * 128, +128) of the tile (SwiGLU: gate rows / up rows)
        const int brow = P.epi == 2 ? (rank == 0 ? n_tile * 128 : P.up_row_offset + n_tile * 128) : n_tile * kBN + (int)rank * 128;
        const int arow = (m_pair * 2 + (int)rank) * kBM;
        for (int kb = 0; kb < nkb; ++kb) {
          ok = mbar_wait(empty + stage, ph ^ 1u, abort_flag, 2);
          if (!ok) break;
          uint8_t *sa = smem + stage * kStageBytes2;
          if (rank == 0) mbar_arrive_expect_tx(full + stage, 2u * kStageBytes2);
          tma_load_2d_pair(sa, &P.map_a, full + stage, kb * kBK, arow);
          tma_load_2d_pair(sa + kABytes, &P.map_b, full + stage, kb * kBK, brow);
          if (++stage == kStages2) { stage = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 5) {
    if (rank == 0 && lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(2 * kBM, kBN, false, false);
      const uint64_t adesc0 = smem_desc_sw128(smem_u32(smem), 16, 1024);
      const uint64_t bdesc0 = smem_desc_sw128(smem_u32(smem) + kABytes, 16, 1024);
      int stage = 0, k = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int tile = pair; tile < total_tiles && ok; tile += n_pairs, ++k) {
        const int buf = k & 1;
        ok = mbar_wait(acc_empty + buf, ((k >> 1) & 1) ^ 1u, abort_flag, 3);  // both CTAs' epilogues of tile k - 2 are done
        if (!ok) break;
        tc_fence_after();
        const uint32_t acc = tmem + buf * kBN;
        for (int kb = 0; kb < nkb; ++kb) {
          ok = mbar_wait(full + stage, ph, abort_flag, 4);
          if (!ok) break;
          tc_fence_after();
          const uint64_t so = (uint64_t)(stage * (kStageBytes2 >> 4));
          mma2_ss(acc, adesc0 + so, bdesc0 + so, idesc, kb != 0);
#pragma unroll
          for (int kk = 1; kk < kBK / 16; ++kk) mma2_ss_c<true>(acc, adesc0 + so + 2 * kk, bdesc0 + so + 2 * kk, idesc);
          mma2_commit_both(empty + stage);
          if (++stage == kStages2) { stage = 0; ph ^= 1u; }
        }
        if (ok) mma2_commit_both(acc_full + buf);
      }
    }
  } else {
    int k = 0;
    bool live = true;
    for (int tile = pair; tile < total_tiles && live; tile += n_pairs, ++k) {
      const int m_pair = tile % m_pairs, n_tile = tile / m_pairs;
      const int buf = k & 1;
      const bool ok = __all_sync(0xffffffffu, mbar_wait(acc_full + buf, (k >> 1) & 1, abort_flag, 5));
      tc_fence_after();
      const int row = (m_pair * 2 + (int)rank) * kBM + warp * 32 + lane;
      const uint32_t taddr = tmem + buf * kBN + ((uint32_t)(warp * 32) << 16);
      live = ok;
      if (ok) gemm_epilogue(P, taddr, row, n_tile);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(acc_empty + buf);
    }
  }
  // ---------------- teardown
  if (threadIdx.x == 0 && *abort_flag && P.status) atomicOr(reinterpret_cast<unsigned int *>(P.status), DPARA_STATUS_TIMEOUT);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // the peer may still signal this CTA's barriers or read its shared memory until here
  if (warp == 5) tmem_dealloc_pair(tmem, 512);
}

dpara_status launch_gemm_tc(const GemmArgs &g, int32_t *status, cudaStream_t st) {
  if (g.M <= 0 || g.N <= 0 || g.K <= 0) return DPARA_ERR_INVALID_ARG;
  if (g.K % kBK != 0 || g.N % 8 != 0) return DPARA_ERR_UNSUPPORTED;
  if (g.epi < 0 || g.epi > 3 || !g.a || !g.w || !g.out || (g.epi == 1 && !g.resid)) return DPARA_ERR_INVALID_ARG;
  if (!aligned16(g.a) || !aligned16(g.w) || !aligned16(g.out) || !aligned16(g.resid) || !aligned16(g.out_bf16)) return DPARA_ERR_INVALID_ARG;
  GemmKernelParams P;
  const int w_rows = g.epi == 2 ? 2 * g.N : g.N;
  if (!make_tmap_bf16_2d(&P.map_a, g.a, g.K, g.M, (uint64_t)g.K * 2, kBK, kBM)) return DPARA_ERR_CUDA;
  if (!make_tmap_bf16_2d(&P.map_b, g.w, g.K, w_rows, (uint64_t)g.K * 2, kBK, 128)) return DPARA_ERR_CUDA;
  P.M = g.M; P.N = g.N; P.K = g.K; P.epi = g.epi; P.up_row_offset = g.N;
  P.out = g.out; P.resid = g.resid; P.resid_bf16 = g.resid_bf16; P.out_bf16 = g.out_bf16; P.status = status;
  P.perm_block = g.epi == 3 ? g.perm_block : 0; P.perm_b = g.perm_b;
  if (cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return DPARA_ERR_CUDA;
  const int tile_cols = g.epi == 2 ? 128 : kBN;
  const int tiles = ((g.N + tile_cols - 1) / tile_cols) * ((g.M + kBM - 1) / kBM);
  int dev = 0, sms = kNumSM;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (g.M > kBM) {
    // more than one 128-row tile of activations: CTA pairs (one 256 x 256 tile per pair and round)
    if (cudaFuncSetAttribute(gemm_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes2) != cudaSuccess) return DPARA_ERR_CUDA;
    const int pair_tiles = ((g.N + tile_cols - 1) / tile_cols) * ((g.M + 2 * kBM - 1) / (2 * kBM));
    const int pairs = pair_tiles < sms / 2 ? pair_tiles : sms / 2;
    gemm_tc2_kernel<<<2 * pairs, kThreads, kSmemBytes2, st>>>(P);
    DPARA_CHECK_LAUNCH();
    count_launches(1);
    return DPARA_OK;
  }
  gemm_tc_kernel<<<tiles < sms ? tiles : sms, kThreads, kSmemBytes, st>>>(P);
  DPARA_CHECK_LAUNCH();
  count_launches(1);
  return DPARA_OK;
}

}  // namespace dpara
