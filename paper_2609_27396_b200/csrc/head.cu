// The critical-path remainder T_Head (Alg. 1 after the barrier; Sec. 3.2 "Loss" for the head's form):
//   base logits  l = h W_lm^T  of the SELECTED branch (b * d rows), one tensor-core GEMM with an fp32 store;
//   head loop    z_i = l_i + W E(y_{i-1}),  y_i = argmax z_i,  y_0 = bonus,  i = 1..d  (greedy).
//
// The loop is d dependent steps, each a skinny product: all vocab rows of W (vocab x rank, bf16) against the b
// embedding rows E(y_{i-1}) -- 0.6 GFLOP and one pass over W (78 MB at vocab 151 936, rank 256, which stays in
// L2) per step.  ONE persistent cooperative kernel runs all d steps:
//   warp 8      TMA producer: streams this CTA's 128-row tiles of W through a ring of shared-memory stages (the
//               tiles do not depend on the tokens, so the ring runs ahead across steps), and with each tile the
//               b x 128 block of base logits it will be added to (plain loads of those from the epilogue queued
//               behind the deep W stream and cost 1.6 us each; as part of the stage they cost nothing);
//   warp 9      one thread issues tcgen05.mma: D[128 vocab rows][nb] = W_tile[128][rank] * Ey[nb][rank]^T
//               (M = 128, N = nb = 16 or 32, both operands K-major in shared memory, 128-byte swizzle);
//   warps 0-7   build Ey in shared memory at the start of a step (gather of E rows, swizzled by hand), then for
//               every tile: tcgen05.ld the accumulator (thread = vocab row; warps w and w + 4 share the 32 rows
//               of a TMEM lane quarter and take the even / odd requests), add the base logit of each request
//               (from the stage), keep the running (value, index) maximum per request -- a thread meets its
//               rows in increasing order, so a strict compare keeps the lowest index; at the end of the step a
//               warp reduction, a CTA reduction and one 64-bit atomicMax per request and CTA.
// Between steps the CTAs meet at a grid barrier (a counter in global memory; the launch is cooperative, so all
// CTAs are resident; the wait is bounded by wall time and gives up with DPARA_STATUS_TIMEOUT).
// A maximum is carried as (order-preserving key of z) << 32 | ~index: the largest packed value is the largest
// logit, lowest index on ties; NaN ranks below every number.
#include "gemm.cuh"
#include "head.cuh"
#include "sm100_ptx.cuh"

namespace dpara {
using namespace ptx;

namespace {
constexpr int kThreads = 320;  // warps 0-7 epilogue, 8 TMA producer, 9 MMA issuer
constexpr int kEpiWarps = 8, kProducerWarp = 8, kMmaWarp = 9;
constexpr int kMaxBatch = 32;
constexpr int kAccCols = 32;  // TMEM columns per accumulator buffer (nb <= 32)
constexpr int kBestStride = 16;  // 64-bit words between two requests' maxima: one 128-byte line (one L2 atomic unit) each

__device__ __forceinline__ uint32_t head_key(float f) {
  if (f != f) return 0u;                    // NaN below everything
  if (f == 0.0f) f = 0.0f;                  // -0 == +0
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
}  // namespace

struct ArParams {
  CUtensorMap map_w;
  CUtensorMap map_l;          // base logits [block * b][vocab] fp32, box = 128 columns x nb rows
  const float *logits;        // [block][b][vocab]: the rows one step reads are contiguous
  const uint16_t *ar_e;       // [vocab][rank]
  const int32_t *bonus;       // [b]
  int32_t *next_tokens;       // [b][block]
  unsigned long long *best;   // [block][kMaxBatch][kBestStride], zeroed before the launch
  unsigned int *barrier;      // zeroed before the launch
  int32_t *status;
  int b, block, vocab, rank, n_tiles, nb, stages;
};

__global__ void __launch_bounds__(kThreads, 1) ar_head_kernel(const __grid_constant__ ArParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tile_bytes = 128 * P.rank * 2;
  const int lg_bytes = P.nb * 128 * 4;                   // base logits of one tile: [nb rows][128 vocab entries] fp32
  const int stage_bytes = tile_bytes + lg_bytes;
  const int slabs = P.rank / 64;
  uint8_t *sW = smem;                                    // ring of stages: W tile [slab][128 rows][128 B], then the logits block
  uint8_t *sE = smem + P.stages * stage_bytes;           // Ey: [slab][nb rows][128 B]
  uint64_t *bars = reinterpret_cast<uint64_t *>(sE + slabs * P.nb * 128);
  uint64_t *full = bars, *empty = bars + 4, *acc_full = bars + 8, *acc_empty = bars + 10, *e_ready = bars + 12, *epi_bar = bars + 13;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 14);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  int *s_tok = reinterpret_cast<int *>(tmem_slot + 2);   // [kMaxBatch] previous tokens of this step
  unsigned long long *s_red = reinterpret_cast<unsigned long long *>(s_tok + kMaxBatch);  // [4 warps][kMaxBatch]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < 4; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, 1 + kEpiWarps); }  // released by the MMA commit and the epilogue warps
    for (int a = 0; a < 2; ++a) { mbar_init(acc_full + a, 1); mbar_init(acc_empty + a, kEpiWarps); }
    mbar_init(e_ready, kEpiWarps);
    mbar_init(epi_bar, kEpiWarps);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == kMmaWarp) { tmem_alloc(tmem_slot, 64); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // this CTA's tiles: blockIdx.x, blockIdx.x + gridDim.x, ... (the same in every step)
  const int my_tiles = (P.n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

  if (warp == kProducerWarp) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      prefetch_tensormap(&P.map_w);
      int stage = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int step = 0; step < P.block && ok; ++step) {
        for (int k = 0; k < my_tiles; ++k) {
          ok = mbar_wait(empty + stage, ph ^ 1u, abort_flag, 2);
          if (!ok) break;
          const int row0 = ((int)blockIdx.x + k * (int)gridDim.x) * 128;
          mbar_arrive_expect_tx(full + stage, (uint32_t)stage_bytes);
          for (int sb = 0; sb < slabs; ++sb) tma_load_2d(sW + stage * stage_bytes + sb * 16384, &P.map_w, full + stage, sb * 64, row0);
          tma_load_2d(sW + stage * stage_bytes + tile_bytes, &P.map_l, full + stage, row0, step * P.b);
          if (++stage == P.stages) { stage = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = idesc_bf16_f32(128, P.nb, false, false);
      const uint64_t wdesc0 = smem_desc_sw128(smem_u32(sW), 16, 1024);
      const uint64_t edesc0 = smem_desc_sw128(smem_u32(sE), 16, 1024);
      int stage = 0, kt = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int step = 0; step < P.block && ok; ++step) {
        ok = mbar_wait(e_ready, step & 1, abort_flag, 3);   // Ey of this step is in shared memory
        for (int k = 0; k < my_tiles && ok; ++k, ++kt) {
          const int buf = kt & 1;
          ok = mbar_wait(acc_empty + buf, ((kt >> 1) & 1) ^ 1u, abort_flag, 4) && mbar_wait(full + stage, ph, abort_flag, 5);
          if (!ok) break;
          tc_fence_after();
          const uint64_t wd = wdesc0 + (uint64_t)((stage * stage_bytes) >> 4);
          for (int kk = 0; kk < P.rank / 16; ++kk) {
            const uint32_t woff = ((kk >> 2) * 16384 + (kk & 3) * 32) >> 4;
            const uint32_t eoff = ((kk >> 2) * (P.nb * 128) + (kk & 3) * 32) >> 4;
            mma_ss(tmem + buf * kAccCols, wd + woff, edesc0 + eoff, idesc, kk > 0);
          }
          mma_commit(empty + stage);
          mma_commit(acc_full + buf);
          if (++stage == P.stages) { stage = 0; ph ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ Ey build + epilogue: thread = vocab row of the tile
    const int quarter = warp & 3, nh = warp >> 2;  // TMEM lane quarter; this warp takes requests n = 2 j + nh
    const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16);
    int kt = 0, stage = 0;
    bool ok = true;
    uint32_t ph_epi = 0, ph_full = 0;
    // barrier of the epilogue warps (bounded like every other wait; orders their shared-memory writes)
    auto epi_sync = [&]() {
      __syncwarp();
      if (lane == 0) mbar_arrive(epi_bar);
      const bool r = __all_sync(0xffffffffu, mbar_wait(epi_bar, ph_epi, abort_flag, 8));
      ph_epi ^= 1u;
      return r;
    };
    for (int step = 0; step < P.block && ok; ++step) {
      // previous tokens: the bonus for the first step, else the winners of the previous step
      if (threadIdx.x < kMaxBatch) {
        int tok = 0;
        if ((int)threadIdx.x < P.b) {
          if (step == 0) {
            tok = P.bonus[threadIdx.x];
            if (tok < 0 || tok >= P.vocab) {
              if (P.status) atomicOr(reinterpret_cast<unsigned int *>(P.status), DPARA_STATUS_BAD_TOKEN);
              tok = 0;
            }
          } else {
            const unsigned long long w = __ldcg(P.best + ((size_t)(step - 1) * kMaxBatch + threadIdx.x) * kBestStride);
            tok = (int)(0xffffffffu - (uint32_t)(w & 0xffffffffull));
            if (w == 0ull) tok = 0;  // (all-NaN row)
            if (blockIdx.x == 0) P.next_tokens[(size_t)threadIdx.x * P.block + (step - 1)] = tok;
          }
        }
        s_tok[threadIdx.x] = tok;
      }
      ok = epi_sync();
      if (!ok) break;
      // Ey[n][k] = E[tok_n][k] in the K-major 128-byte-swizzle layout the MMA reads: slab = k / 64, row n at
      // 128 B pitch, 16-byte chunk c of the row stored at chunk position c ^ (n & 7); rows n >= b are zero
      const int chunks_per_row = P.rank / 8;
      for (int q = threadIdx.x; q < P.nb * chunks_per_row; q += kEpiWarps * 32) {
        const int n = q / chunks_per_row, c = q % chunks_per_row;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (n < P.b) v = *reinterpret_cast<const uint4 *>(P.ar_e + (size_t)s_tok[n] * P.rank + c * 8);
        const int sb = c >> 3, cc = c & 7;
        *reinterpret_cast<uint4 *>(sE + sb * (P.nb * 128) + n * 128 + ((cc ^ (n & 7)) << 4)) = v;
      }
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(e_ready);

      float bz[kMaxBatch / 2];
      int bv[kMaxBatch / 2];
#pragma unroll
      for (int j = 0; j < kMaxBatch / 2; ++j) { bz[j] = -INFINITY; bv[j] = -1; }
      for (int k = 0; k < my_tiles; ++k, ++kt) {
        const int buf = kt & 1;
        ok = __all_sync(0xffffffffu, mbar_wait(acc_full + buf, (kt >> 1) & 1, abort_flag, 6));
        if (!ok) break;
        tc_fence_after();
        uint32_t acc[32];
        tmem_ld32(taddr + buf * kAccCols, acc);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty + buf);
        const int v = ((int)blockIdx.x + k * (int)gridDim.x) * 128 + quarter * 32 + lane;
        // (acc_full implies the stage's loads have landed: the MMA issuer waited for them; this wait is the
        //  epilogue threads' own acquire of the TMA-written logits and returns at once)
        ok = __all_sync(0xffffffffu, mbar_wait(full + stage, ph_full, abort_flag, 9));
        if (!ok) break;
        const bool live = v < P.vocab;
        const float *sl = reinterpret_cast<const float *>(sW + stage * stage_bytes + tile_bytes) + quarter * 32 + lane;
#pragma unroll
        for (int j = 0; j < kMaxBatch / 2; ++j) {
          const int n = 2 * j + nh;
          if (n < P.b) {
            const float z = __uint_as_float(nh ? acc[2 * j + 1] : acc[2 * j]) + sl[n * 128];
            // larger, or the first number this thread sees (NaN never wins; -inf can, at the lowest index)
            if (live && (z > bz[j] || (bv[j] < 0 && z == z))) { bz[j] = z; bv[j] = v; }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty + stage);
        if (++stage == P.stages) { stage = 0; ph_full ^= 1u; }
      }
      if (!ok) break;
      // step maximum: warp reduction, CTA reduction through shared memory, then ONE atomic per request and CTA,
      // each request on its own 128-byte line (atomics on one line are serialised by a single L2 unit)
#pragma unroll
      for (int j = 0; j < kMaxBatch / 2; ++j) {
        const int n = 2 * j + nh;
        if (n < P.b) {
          unsigned long long x = bv[j] < 0 ? 0ull : (((unsigned long long)head_key(bz[j]) << 32) | (unsigned long long)(0xffffffffu - (uint32_t)bv[j]));
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long y = __shfl_xor_sync(0xffffffffu, x, o);
            x = y > x ? y : x;
          }
          if (lane == 0) s_red[quarter * kMaxBatch + n] = x;
        }
      }
      ok = epi_sync();
      if (!ok) break;
      if ((int)threadIdx.x < P.b) {
        unsigned long long x = s_red[threadIdx.x];
#pragma unroll
        for (int w = 1; w < 4; ++w) x = s_red[w * kMaxBatch + threadIdx.x] > x ? s_red[w * kMaxBatch + threadIdx.x] : x;
        atomicMax(P.best + ((size_t)step * kMaxBatch + threadIdx.x) * kBestStride, x);
      }
      // ---- grid barrier: every CTA's maxima of this step are in before anyone reads them
      __threadfence();
      ok = epi_sync();
      if (!ok) break;
      if (threadIdx.x == 0) {
        atomicAdd(P.barrier, 1u);
        const unsigned int target = (unsigned int)(step + 1) * gridDim.x;
        const uint64_t t0 = global_timer_ns();
        while (*reinterpret_cast<volatile unsigned int *>(P.barrier) < target) {
          if (*abort_flag || global_timer_ns() - t0 > kWaitLimitNs) { *abort_flag = 7; break; }
        }
        __threadfence();
      }
      ok = epi_sync() && !*abort_flag;
    }
    // the last step's winners
    if (ok && blockIdx.x == 0 && (int)threadIdx.x < P.b) {
      const unsigned long long w = __ldcg(P.best + ((size_t)(P.block - 1) * kMaxBatch + threadIdx.x) * kBestStride);
      P.next_tokens[(size_t)threadIdx.x * P.block + (P.block - 1)] = w == 0ull ? 0 : (int)(0xffffffffu - (uint32_t)(w & 0xffffffffull));
    }
  }
  // ------------------------------------------------------------------ teardown
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) {
      if (P.status) atomicOr(reinterpret_cast<unsigned int *>(P.status), DPARA_STATUS_TIMEOUT);
      for (int k = 0; k < 4096; ++k) __nanosleep(256);  // copies that may still be in flight get a bounded time to land
    }
    __syncthreads();
  }
  if (warp == kMmaWarp) tmem_dealloc(tmem, 64);
}

size_t head_workspace_bytes(int b, int block, int vocab) {
  if (b <= 0 || block <= 0 || vocab <= 0) return 0;
  const size_t logits = (((size_t)b * block * vocab * sizeof(float)) + 255) & ~size_t(255);
  return logits + (size_t)block * kMaxBatch * kBestStride * sizeof(unsigned long long) + 256;
}

dpara_status launch_head(const HeadArgs &h, void *workspace, int32_t *status, cudaStream_t st) {
  if (h.b <= 0 || h.block <= 0 || h.hidden <= 0 || h.vocab <= 0 || h.rank <= 0) return DPARA_ERR_INVALID_ARG;
  if (h.b > kMaxBatch || h.rank % 64 != 0 || h.rank > 256 || h.hidden % 64 != 0 || h.vocab % 8 != 0 || h.block > 64) return DPARA_ERR_UNSUPPORTED;
  if (!h.sel_reps || !h.w_lm || !h.ar_w || !h.ar_e || !h.bonus || !h.next_tokens || !workspace) return DPARA_ERR_INVALID_ARG;
  if (!aligned16(h.sel_reps) || !aligned16(h.w_lm) || !aligned16(h.ar_w) || !aligned16(h.ar_e) || !aligned16(workspace)) return DPARA_ERR_INVALID_ARG;
  uint8_t *ws = static_cast<uint8_t *>(workspace);
  float *logits = reinterpret_cast<float *>(ws);
  const size_t logits_bytes = (((size_t)h.b * h.block * h.vocab * sizeof(float)) + 255) & ~size_t(255);
  unsigned long long *best = reinterpret_cast<unsigned long long *>(ws + logits_bytes);
  unsigned int *barrier = reinterpret_cast<unsigned int *>(best + (size_t)h.block * kMaxBatch * kBestStride);
  if (cudaMemsetAsync(best, 0, (size_t)h.block * kMaxBatch * kBestStride * sizeof(unsigned long long) + 256, st) != cudaSuccess) return DPARA_ERR_CUDA;

  // base logits of the selected branches, fp32, stored step-major [block][b][vocab] (GEMM row n * block + i goes
  // to row i * b + n): the b rows a step reads then lie in one contiguous range instead of b ranges
  // block * vocab * 4 bytes apart
  GemmArgs g;
  g.a = h.sel_reps; g.w = h.w_lm; g.M = h.b * h.block; g.N = h.vocab; g.K = h.hidden; g.epi = 3;
  g.resid = nullptr; g.resid_bf16 = 0; g.out = logits; g.out_bf16 = nullptr; g.perm_block = h.block; g.perm_b = h.b;
  dpara_status rc = launch_gemm_tc(g, status, st);
  if (rc != DPARA_OK) return rc;

  ArParams P;
  memset(&P, 0, sizeof(P));
  if (!make_tmap_bf16_2d(&P.map_w, h.ar_w, h.rank, h.vocab, (uint64_t)h.rank * 2, 64, 128)) return DPARA_ERR_CUDA;
  if (!make_tmap_f32_2d(&P.map_l, logits, h.vocab, (uint64_t)h.block * h.b, (uint64_t)h.vocab * 4, 128, h.b <= 16 ? 16 : 32)) return DPARA_ERR_CUDA;
  P.logits = logits; P.ar_e = static_cast<const uint16_t *>(h.ar_e); P.bonus = h.bonus; P.next_tokens = h.next_tokens;
  P.best = best; P.barrier = barrier; P.status = status;
  P.b = h.b; P.block = h.block; P.vocab = h.vocab; P.rank = h.rank;
  P.n_tiles = (h.vocab + 127) / 128;
  P.nb = h.b <= 16 ? 16 : 32;
  const int stage_bytes = 128 * h.rank * 2 + P.nb * 128 * 4;
  const int fixed = (h.rank / 64) * P.nb * 128 + 1024 + 2048;   // Ey, alignment slack, barriers and reduction scratch
  P.stages = (227 * 1024 - fixed) / stage_bytes > 4 ? 4 : (227 * 1024 - fixed) / stage_bytes;
  const int smem = P.stages * stage_bytes + fixed;
  if (cudaFuncSetAttribute(ar_head_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return DPARA_ERR_CUDA;
  int dev = 0, sms = kNumSM;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  // cooperative launch: the grid barrier needs every CTA resident (one CTA per SM fits by construction)
  const int grid = P.n_tiles < sms ? P.n_tiles : sms;
  void *args[] = {&P};
  if (cudaLaunchCooperativeKernel(reinterpret_cast<void *>(ar_head_kernel), dim3(grid), dim3(kThreads), args, smem, st) != cudaSuccess) {
    cudaGetLastError();
    return DPARA_ERR_CUDA;
  }
  count_launches(1);
  return DPARA_OK;
}

}  // namespace dpara
