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
constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*align*/ + 256 /*barriers*/ + 4 * 32 * 36 * 4 /*epilogue staging*/;
constexpr int kThreads = 192;                   // warps 0-3 epilogue, 4 TMA, 5 MMA
}  // namespace

struct GemmKernelParams {
  CUtensorMap map_a[kGemmMaxGroups];   // one entry per product of a grouped launch (a plain launch uses entry 0)
  CUtensorMap map_b[kGemmMaxGroups];
  void *out_g[kGemmMaxGroups];         // grouped launch: the products' outputs
  int n_groups;
  int M, N, K;
  int epi;
  int up_row_offset;
  void *out;
  const void *resid;
  int resid_bf16;
  void *out_bf16;
  int32_t *status;
  int perm_block, perm_b;
  int bn;        // output columns per tile of the CTA-pair kernel: 256, or 192 where that fills the rounds better (bf16 / fp32 stores)
  int split_k;   // > 1 (fp32 store only, CTA pairs): the K range in split_k parts, part s writes plane s of [split_k][M][N] partial sums
};

__device__ __forceinline__ float silu_f(float g) { return g / (1.0f + __expf(-g)); }

// Epilogue of one accumulator tile.  A thread reads one accumulator ROW from tensor memory (lane = row), 32 columns at
// a time; stored like that, one warp instruction would touch 32 rows x 16 bytes -- 32 cache lines for 512 bytes.  Each
// 32 x 32 block therefore goes through a per-warp shared-memory buffer (row pitch 36 floats: conflict-free both ways)
// and comes back with 8 lanes on one row: an instruction then covers 4 rows x 128 contiguous bytes, for the residual
// read as well as for the stores.  `row_base` = output row of lane 0, `stage` = this warp's 32 x 36 floats.
constexpr int kEpiPitch = 36;

__device__ __forceinline__ void gemm_epilogue(const GemmKernelParams &P, uint32_t taddr, int row_base, int n_tile, float *stage, int lane, int ks,
                                              int grp) {
  // fp32 output of this product; split K (fp32 store only): plane ks of the partial sums
  float *out_f32 = static_cast<float *>(P.n_groups > 1 ? P.out_g[grp] : P.out) + (size_t)ks * P.M * P.N;
  const int n_chunks = P.epi == 2 ? 4 : P.bn / 32;
  const int col0 = n_tile * (P.epi == 2 ? 128 : P.bn);
  const int sub_row = lane >> 3, piece = lane & 7;
#pragma unroll 1
  for (int c = 0; c < n_chunks; ++c) {
    uint32_t r[32];
    tmem_ld32(taddr + c * 32, r);
    if (P.epi == 2) {
      uint32_t u[32];
      tmem_ld32(taddr + 128 + c * 32, u);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(silu_f(__uint_as_float(r[e])) * __uint_as_float(u[e]));
    } else {
      tmem_wait_ld();
    }
    float4 *mine = reinterpret_cast<float4 *>(stage + lane * kEpiPitch);
#pragma unroll
    for (int v = 0; v < 8; ++v)
      mine[v] = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]), __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
    __syncwarp();
    const int col = col0 + c * 32 + piece * 4;
    if (col < P.N) {
      // the residual rows first, all in flight together
      float4 rr[8];
      if (P.epi == 1) {
        // (rows past M read row M - 1: an unconditional load the compiler can issue early; the value is not used)
        if (P.resid_bf16) {
          uint2 q[8];
#pragma unroll
          for (int i = 0; i < 8; ++i)
            q[i] = *reinterpret_cast<const uint2 *>(static_cast<const uint16_t *>(P.resid) + (size_t)min(row_base + i * 4 + sub_row, P.M - 1) * P.N + col);
#pragma unroll
          for (int i = 0; i < 8; ++i) rr[i] = make_float4(bf16lo(q[i].x), bf16hi(q[i].x), bf16lo(q[i].y), bf16hi(q[i].y));
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i)
            rr[i] = *reinterpret_cast<const float4 *>(static_cast<const float *>(P.resid) + (size_t)min(row_base + i * 4 + sub_row, P.M - 1) * P.N + col);
        }
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int rl = i * 4 + sub_row, row = row_base + rl;
        const float4 a = *reinterpret_cast<const float4 *>(stage + rl * kEpiPitch + piece * 4);
        if (row < P.M) {
          if (P.epi == 0 || P.epi == 2) {
            uint16_t *o = static_cast<uint16_t *>(P.out) + (size_t)row * P.N + col;
            *reinterpret_cast<uint2 *>(o) = make_uint2(pack_bf16(a.x, a.y), pack_bf16(a.z, a.w));
          } else {
            const int orow = P.perm_block ? (row % P.perm_block) * P.perm_b + row / P.perm_block : row;
            float4 x = a;
            if (P.epi == 1) { x.x += rr[i].x; x.y += rr[i].y; x.z += rr[i].z; x.w += rr[i].w; }
            *reinterpret_cast<float4 *>(out_f32 + (size_t)orow * P.N + col) = x;
            if (P.out_bf16)
              *reinterpret_cast<uint2 *>(static_cast<uint16_t *>(P.out_bf16) + (size_t)row * P.N + col) = make_uint2(pack_bf16(x.x, x.y), pack_bf16(x.z, x.w));
          }
        }
      }
    }
    __syncwarp();
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
  pdl_wait();  // nothing above touches global memory: the set-up overlaps the tail of the kernel before
  pdl_launch_dependents();

  // Persistent: CTA c computes tiles c, c + gridDim.x, ...; tile id = n_tile * m_tiles + m_tile, so the CTAs
  // running together cover all M rows of a few weight tiles (A stays in L2, each weight tile is read once).
  // Two accumulator buffers in TMEM let the epilogue of one tile overlap the main loop of the next.
  if (warp == 4) {
    if (lane == 0) {
      prefetch_tensormap(&P.map_a[0]);
      prefetch_tensormap(&P.map_b[0]);
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
          tma_load_2d(sa, &P.map_a[0], full + stage, kb * kBK, m_tile * kBM);
          tma_load_2d(sa + kABytes, &P.map_b[0], full + stage, kb * kBK, brow0);
          tma_load_2d(sa + kABytes + 128 * kBK * 2, &P.map_b[0], full + stage, kb * kBK, brow1);
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
    const int row_base = m_tile * kBM + warp * 32;
    const uint32_t taddr = tmem + buf * kBN + ((uint32_t)(warp * 32) << 16);
    live = ok;
    if (ok) {
      gemm_epilogue(P, taddr, row_base, n_tile, reinterpret_cast<float *>(smem + kStages * kStageBytes + 256) + warp * 32 * kEpiPitch, lane, 0, 0);
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
constexpr int kSmemBytes2 = kStages2 * kStageBytes2 + 1024 + 256 + 4 * 32 * 36 * 4;
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
  const int tile_cols = P.epi == 2 ? 128 : P.bn;
  const int m_pairs = (P.M + 2 * kBM - 1) / (2 * kBM), n_tiles = (P.N + tile_cols - 1) / tile_cols;
  const int group_units = m_pairs * n_tiles * P.split_k;   // work units of one product: (tile, K part), the parts of a tile adjacent
  const int total_tiles = group_units * P.n_groups;

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
  pdl_wait();  // nothing above touches global memory: the set-up overlaps the tail of the kernel before
  pdl_launch_dependents();

  if (warp == 4) {
    if (lane == 0) {
      for (int gi = 0; gi < P.n_groups; ++gi) {
        prefetch_tensormap(&P.map_a[gi]);
        prefetch_tensormap(&P.map_b[gi]);
      }
      int stage = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int unit0 = pair; unit0 < total_tiles && ok; unit0 += n_pairs) {
        const int grp = unit0 / group_units, unit = unit0 - grp * group_units;
        const int tile = unit / P.split_k, ks = unit - tile * P.split_k;
        const int m_pair = tile % m_pairs, n_tile = tile / m_pairs;
        const int kb0 = ks * nkb / P.split_k, kb1 = (ks + 1) * nkb / P.split_k;
        // this CTA's half of the weight tile: rows [rank * 128, +128) of the tile (SwiGLU: gate rows / up rows)
        const int half = P.epi == 2 ? 128 : P.bn / 2;   // weight rows each CTA of the pair holds
        const int brow = P.epi == 2 ? (rank == 0 ? n_tile * 128 : P.up_row_offset + n_tile * 128) : n_tile * P.bn + (int)rank * half;
        const uint32_t tx = 2u * ((uint32_t)kABytes + (uint32_t)half * kBK * 2u);
        const int arow = (m_pair * 2 + (int)rank) * kBM;
        for (int kb = kb0; kb < kb1; ++kb) {
          ok = mbar_wait(empty + stage, ph ^ 1u, abort_flag, 2);
          if (!ok) break;
          uint8_t *sa = smem + stage * kStageBytes2;
          if (rank == 0) mbar_arrive_expect_tx(full + stage, tx);
          tma_load_2d_pair(sa, &P.map_a[grp], full + stage, kb * kBK, arow);
          tma_load_2d_pair(sa + kABytes, &P.map_b[grp], full + stage, kb * kBK, brow);
          if (++stage == kStages2) { stage = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 5) {
    if (rank == 0 && lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(2 * kBM, P.epi == 2 ? kBN : P.bn, false, false);
      const uint64_t adesc0 = smem_desc_sw128(smem_u32(smem), 16, 1024);
      const uint64_t bdesc0 = smem_desc_sw128(smem_u32(smem) + kABytes, 16, 1024);
      int stage = 0, k = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int unit0 = pair; unit0 < total_tiles && ok; unit0 += n_pairs, ++k) {
        const int ks = (unit0 % group_units) % P.split_k;
        const int kb0 = ks * nkb / P.split_k, kb1 = (ks + 1) * nkb / P.split_k;
        const int buf = k & 1;
        ok = mbar_wait(acc_empty + buf, ((k >> 1) & 1) ^ 1u, abort_flag, 3);  // both CTAs' epilogues of tile k - 2 are done
        if (!ok) break;
        tc_fence_after();
        const uint32_t acc = tmem + buf * kBN;
        for (int kb = kb0; kb < kb1; ++kb) {
          ok = mbar_wait(full + stage, ph, abort_flag, 4);
          if (!ok) break;
          tc_fence_after();
          const uint64_t so = (uint64_t)(stage * (kStageBytes2 >> 4));
          mma2_ss(acc, adesc0 + so, bdesc0 + so, idesc, kb != kb0);
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
    for (int unit0 = pair; unit0 < total_tiles && live; unit0 += n_pairs, ++k) {
      const int grp = unit0 / group_units, unit = unit0 - grp * group_units;
      const int tile = unit / P.split_k, ks = unit - tile * P.split_k;
      const int m_pair = tile % m_pairs, n_tile = tile / m_pairs;
      const int buf = k & 1;
      const bool ok = __all_sync(0xffffffffu, mbar_wait(acc_full + buf, (k >> 1) & 1, abort_flag, 5));
      tc_fence_after();
      const int row_base = (m_pair * 2 + (int)rank) * kBM + warp * 32;
      const uint32_t taddr = tmem + buf * kBN + ((uint32_t)(warp * 32) << 16);
      live = ok;
      if (ok) gemm_epilogue(P, taddr, row_base, n_tile, reinterpret_cast<float *>(smem + kStages2 * kStageBytes2 + 256) + warp * 32 * kEpiPitch, lane, ks, grp);
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
  int dev = 0, sms = kNumSM;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int split = g.split_k > 1 ? g.split_k : 1, groups = g.n_groups > 1 ? g.n_groups : 1;
  // Tile width of the pair kernel: 192 columns when that evens out the rounds (QKV at 1024 x 6144: 96 tiles of 256 are two
  // rounds of the 74 pairs, the second a third full; 128 tiles of 192 are two rounds of 0.75 the length).  A 192-wide tile
  // pulls 28 KB per CTA and K slab for 0.75 of the flops of a 256-wide one: its rounds are weighted 1.14x.
  P.bn = kBN;
  if (g.M > kBM && g.epi != 2) {
    const long m_pairs = (g.M + 2 * kBM - 1) / (2 * kBM), pairs = sms / 2 > 0 ? sms / 2 : 1;
    const long u256 = m_pairs * ((g.N + 255) / 256) * split * groups, u192 = m_pairs * ((g.N + 191) / 192) * split * groups;
    const double c256 = (double)((u256 + pairs - 1) / pairs) * 256.0, c192 = (double)((u192 + pairs - 1) / pairs) * 192.0 * 1.14;
    if (c192 < 0.95 * c256) P.bn = 192;
  }
  P.n_groups = 1;
  if (g.n_groups > 1) {
    // several products of one shape in one launch (fp32 stores, CTA pairs): entry 0 of the lists is (a, w, out)
    if (g.epi != 3 || g.M <= kBM || g.n_groups > kGemmMaxGroups || g.perm_block) return DPARA_ERR_UNSUPPORTED;
    P.n_groups = g.n_groups;
  }
  for (int gi = 0; gi < P.n_groups; ++gi) {
    const void *a = gi ? g.a_g[gi] : g.a, *w = gi ? g.w_g[gi] : g.w;
    void *o = gi ? g.out_g[gi] : g.out;
    if (!a || !w || !o || !aligned16(a) || !aligned16(w) || !aligned16(o)) return DPARA_ERR_INVALID_ARG;
    if (!make_tmap_bf16_2d(&P.map_a[gi], a, g.K, g.M, (uint64_t)g.K * 2, kBK, kBM)) return DPARA_ERR_CUDA;
    if (!make_tmap_bf16_2d(&P.map_b[gi], w, g.K, w_rows, (uint64_t)g.K * 2, kBK, P.bn == kBN ? 128 : P.bn / 2)) return DPARA_ERR_CUDA;
    P.out_g[gi] = o;
  }
  P.M = g.M; P.N = g.N; P.K = g.K; P.epi = g.epi; P.up_row_offset = g.N;
  P.out = g.out; P.resid = g.resid; P.resid_bf16 = g.resid_bf16; P.out_bf16 = g.out_bf16; P.status = status;
  P.perm_block = g.epi == 3 ? g.perm_block : 0; P.perm_b = g.perm_b;
  P.split_k = 1;
  if (g.split_k > 1) {
    if (g.epi != 3 || g.M <= kBM || g.split_k > g.K / kBK) return DPARA_ERR_UNSUPPORTED;
    P.split_k = g.split_k;
  }
  if (cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return DPARA_ERR_CUDA;
  const int tile_cols = g.epi == 2 ? 128 : P.bn;
  const int tiles = ((g.N + tile_cols - 1) / tile_cols) * ((g.M + kBM - 1) / kBM);
  if (g.M > kBM) {
    // more than one 128-row tile of activations: CTA pairs (one 256 x 256 tile per pair and round)
    if (cudaFuncSetAttribute(gemm_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes2) != cudaSuccess) return DPARA_ERR_CUDA;
    const int pair_tiles = ((g.N + tile_cols - 1) / tile_cols) * ((g.M + 2 * kBM - 1) / (2 * kBM)) * P.split_k * P.n_groups;
    const int pairs = pair_tiles < sms / 2 ? pair_tiles : sms / 2;
    launch_pdl(gemm_tc2_kernel, dim3(2 * pairs), dim3(kThreads), kSmemBytes2, st, P);
    DPARA_CHECK_LAUNCH();
    count_launches(1);
    return DPARA_OK;
  }
  launch_pdl(gemm_tc_kernel, dim3(tiles < sms ? tiles : sms), dim3(kThreads), kSmemBytes, st, P);
  DPARA_CHECK_LAUNCH();
  count_launches(1);
  return DPARA_OK;
}

}  // namespace dpara
