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
  float *z_out;               // sampling: [b][vocab] fp32, the logits z of step `step0`
  int step0;                  // sampling: the one step this launch computes
};

// kSample = false: the whole greedy loop in one cooperative launch.  kSample = true: ONE step (P.step0) of the sampling
// loop -- the same producer / MMA / epilogue pipeline, but the epilogue writes z = l + W E(y_prev) to P.z_out instead of
// tracking maxima, the previous tokens come from P.next_tokens (written by the draw of the step before), and there is no
// grid barrier (the draw is a launch of its own).
template <bool kSample>
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
  pdl_wait();  // nothing above touches global memory
  pdl_launch_dependents();
  // this CTA's tiles: blockIdx.x, blockIdx.x + gridDim.x, ... (the same in every step)
  const int my_tiles = (P.n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
  const int step_begin = kSample ? P.step0 : 0, step_end = kSample ? P.step0 + 1 : P.block;

  if (warp == kProducerWarp) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      prefetch_tensormap(&P.map_w);
      int stage = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int step = step_begin; step < step_end && ok; ++step) {
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
      for (int step = step_begin; step < step_end && ok; ++step) {
        ok = mbar_wait(e_ready, (step - step_begin) & 1, abort_flag, 3);   // Ey of this step is in shared memory
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
    for (int step = step_begin; step < step_end && ok; ++step) {
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
          } else if (kSample) {
            tok = __ldcg(P.next_tokens + (size_t)threadIdx.x * P.block + (step - 1));
            if (tok < 0 || tok >= P.vocab) tok = 0;
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
            if (kSample) {
              if (live) P.z_out[(size_t)n * P.vocab + v] = z;       // a warp writes 32 consecutive entries of one row
            } else if (live && (z > bz[j] || (bv[j] < 0 && z == z))) {
              // larger, or the first number this thread sees (NaN never wins; -inf can, at the lowest index)
              bz[j] = z; bv[j] = v;
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty + stage);
        if (++stage == P.stages) { stage = 0; ph_full ^= 1u; }
      }
      if (!ok || kSample) break;
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
    if (!kSample && ok && blockIdx.x == 0 && (int)threadIdx.x < P.b) {
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

// ------------------------------------------------------------------------------------------------ sampling head loop
// y_i ~ softmax(z_i) with a supplied uniform (App. C: temperature 1, top-p 1).  Two launches per step: the head kernel
// above in its one-step form writes z = l_i + W E(y_{i-1}) (fp32, [b][vocab]), then the draw, spread over
// (vocabulary chunk, request) CTAs: each CTA leaves its chunk's maximum m_c and weight sum s_c = sum exp(z - m_c) and
// takes a ticket; the CTA that takes a request's last ticket (no CTA ever waits) rescales the chunk sums to the row
// maximum, finds the chunk the threshold u * total falls into, rescans that one chunk in vocabulary order for the
// crossing element, writes the token and puts the ticket back to zero.
// Exponentials are fp32 (relative error ~1e-7, far below the fp32 logits' own), every sum is fp64.
namespace {
constexpr int kPickThreads = 256;
constexpr int kPickMaxChunks = 256;          // one chunk per thread in the finishing CTA

struct PickPart { float m; float pad; double s; };

__host__ __device__ inline int pick_chunk_elems(int vocab) {
  int chunk = 2048;
  while ((vocab + chunk - 1) / chunk > kPickMaxChunks) chunk *= 2;
  return chunk;
}

__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// inclusive block scan of one double per thread (kPickThreads threads); returns the inclusive value, total in *total
__device__ __forceinline__ double block_scan(double x, double *s_warp, double *total) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  double inc = x;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();                       // s_warp free again
  if (lane == 31) s_warp[w] = inc;
  __syncthreads();
  double before = 0.0, tot = 0.0;
#pragma unroll
  for (int k = 0; k < kPickThreads / 32; ++k) { if (k < w) before += s_warp[k]; tot += s_warp[k]; }
  *total = tot;
  return before + inc;
}

__global__ void __launch_bounds__(kPickThreads) head_sample_kernel(const float *__restrict__ z, const float *__restrict__ uniforms,
                                                                   int32_t *__restrict__ next_tokens, PickPart *__restrict__ part,
                                                                   unsigned int *__restrict__ tick, int vocab, int block,
                                                                   int step, int chunk) {
  const int n = blockIdx.y, c = blockIdx.x, n_chunks = gridDim.x, tid = threadIdx.x;
  const float *row = z + (size_t)n * vocab;
  pdl_wait();
  pdl_launch_dependents();
  __shared__ float s_max[kPickThreads / 32];
  __shared__ double s_warp[kPickThreads / 32];
  __shared__ int s_flag;
  __shared__ int s_tok;
  __shared__ double s_base;

  // ---- phase 1: this chunk's maximum and weight sum (vocab % 8 == 0 and chunk % 1024 == 0: float4 loads never straddle)
  const int c0 = c * chunk, c1 = min(vocab, c0 + chunk);
  float mx = -INFINITY;
  for (int v = c0 + tid * 4; v < c1; v += kPickThreads * 4) {
    const float4 x = __ldcg(reinterpret_cast<const float4 *>(row + v));
    mx = fmaxf(mx, fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w)));          // fmaxf drops NaN operands
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((tid & 31) == 0) s_max[tid >> 5] = mx;
  __syncthreads();
  mx = s_max[0];
#pragma unroll
  for (int w = 1; w < kPickThreads / 32; ++w) mx = fmaxf(mx, s_max[w]);
  double loc = 0.0;
  if (mx > -INFINITY && mx < INFINITY) {
    for (int v = c0 + tid * 4; v < c1; v += kPickThreads * 4) {
      const float4 x = __ldcg(reinterpret_cast<const float4 *>(row + v));
      if (x.x == x.x) loc += (double)expf(x.x - mx);
      if (x.y == x.y) loc += (double)expf(x.y - mx);
      if (x.z == x.z) loc += (double)expf(x.z - mx);
      if (x.w == x.w) loc += (double)expf(x.w - mx);
    }
  }
  loc = warp_sum(loc);
  if ((tid & 31) == 0) s_warp[tid >> 5] = loc;
  __syncthreads();
  if (tid == 0) {
    double s = 0.0;
    for (int w = 0; w < kPickThreads / 32; ++w) s += s_warp[w];
    PickPart pp; pp.m = mx; pp.pad = 0.f; pp.s = s;
    part[(size_t)n * kPickMaxChunks + c] = pp;
    __threadfence();
    s_flag = atomicAdd(tick + n, 1u) == (unsigned)(n_chunks - 1);
  }
  __syncthreads();
  if (!s_flag) return;
  __threadfence();

  // ---- phase 2 (the CTA that took the request's last ticket): thread t holds chunk t
  float m_c = -INFINITY;
  double s_c = 0.0;
  if (tid < n_chunks) {
    const uint4 raw = __ldcg(reinterpret_cast<const uint4 *>(part + (size_t)n * kPickMaxChunks + tid));
    m_c = __uint_as_float(raw.x);
    s_c = __hiloint2double((int)raw.w, (int)raw.z);
  }
  float M = m_c;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  __syncthreads();
  if ((tid & 31) == 0) s_max[tid >> 5] = M;
  if (tid == 0) { s_tok = -1; s_flag = -1; }
  __syncthreads();
  M = s_max[0];
#pragma unroll
  for (int w = 1; w < kPickThreads / 32; ++w) M = fmaxf(M, s_max[w]);
  int tok = 0;
  if (M > -INFINITY && M < INFINITY) {
    const double scale = (m_c > -INFINITY) ? exp((double)m_c - (double)M) : 0.0;
    const double S = s_c * scale;
    double total;
    const double inc = block_scan(S, s_warp, &total);
    const double T = (double)uniforms[(size_t)n * block + step] * total;
    // the chunk the threshold falls into; when rounding puts the threshold at or past the total, the last chunk with weight
    if (S > 0.0 && inc - S <= T && T < inc) { s_flag = tid; s_base = inc - S; }
    __syncthreads();
    if (s_flag < 0) {
      if (S > 0.0) atomicMax(&s_flag, tid);
      __syncthreads();
      if (tid == s_flag) s_base = inc - S;
      __syncthreads();
    }
    const int cs = s_flag;                               // >= 0: total > 0 because the row maximum is finite
    __syncthreads();
    if (tid == cs) { s_max[0] = m_c; s_warp[0] = scale; }
    __syncthreads();
    const float mcs = s_max[0];
    const double scs = s_warp[0];
    double running = s_base;
    const int r0 = cs * chunk, r1 = min(vocab, r0 + chunk);
    int last_w = -1;                                     // the last element with weight seen by this thread
    for (int v0 = r0; v0 < r1; v0 += kPickThreads * 4) {
      const int v = v0 + tid * 4;
      double w[4] = {0.0, 0.0, 0.0, 0.0};
      if (v < r1) {
        const float4 x = __ldcg(reinterpret_cast<const float4 *>(row + v));
        if (x.x == x.x) w[0] = (double)expf(x.x - mcs) * scs;
        if (x.y == x.y) w[1] = (double)expf(x.y - mcs) * scs;
        if (x.z == x.z) w[2] = (double)expf(x.z - mcs) * scs;
        if (x.w == x.w) w[3] = (double)expf(x.w - mcs) * scs;
#pragma unroll
        for (int k = 0; k < 4; ++k) if (w[k] > 0.0) last_w = v + k;
      }
      const double l4 = (w[0] + w[1]) + (w[2] + w[3]);
      double sub_total;
      const double inc4 = block_scan(l4, s_warp, &sub_total);
      double acc = running + inc4 - l4;
      if (l4 > 0.0 && acc <= T && T < acc + l4) {
        int pick = -1;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          if (pick < 0 && w[k] > 0.0) { acc += w[k]; if (acc > T) pick = v + k; }
        }
        if (pick < 0) pick = last_w;                     // rounding inside the four: their last with weight
        s_tok = pick;
      }
      __syncthreads();
      if (s_tok >= 0) break;
      running += sub_total;
    }
    if (s_tok < 0) {
      // summation order put the threshold past this chunk's end: its last element with weight
      atomicMax(&s_tok, last_w);
      __syncthreads();
    }
    tok = s_tok < 0 ? 0 : s_tok;
  }
  if (tid == 0) {
    next_tokens[(size_t)n * block + step] = tok;
    tick[n] = 0u;                                        // the next step finds the ticket at zero
  }
}
}  // namespace

size_t head_workspace_bytes(int b, int block, int vocab) {
  if (b <= 0 || block <= 0 || vocab <= 0) return 0;
  const size_t logits = (((size_t)b * block * vocab * sizeof(float)) + 255) & ~size_t(255);
  const size_t zstep = (((size_t)b * vocab * sizeof(float)) + 255) & ~size_t(255);   // sampling: one step's logits
  return logits + (size_t)block * kMaxBatch * kBestStride * sizeof(unsigned long long) + 256 + zstep +
         (size_t)kMaxBatch * kPickMaxChunks * sizeof(PickPart);
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
  float *zstep = reinterpret_cast<float *>(reinterpret_cast<uint8_t *>(barrier) + 256);
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
  if (cudaFuncSetAttribute(ar_head_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess ||
      cudaFuncSetAttribute(ar_head_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return DPARA_ERR_CUDA;
  int dev = 0, sms = kNumSM;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int grid = P.n_tiles < sms ? P.n_tiles : sms;
  if (h.uniforms) {
    // ---- sampling: per step the logits z (one-step head kernel), then the draw.  The tickets live in the zeroed 256 bytes
    // after the greedy path's barrier word (kMaxBatch words from byte 128).
    unsigned int *tick = barrier + 32;
    PickPart *part = reinterpret_cast<PickPart *>(reinterpret_cast<uint8_t *>(zstep) + ((((size_t)h.b * h.vocab * sizeof(float)) + 255) & ~size_t(255)));
    const int chunk = pick_chunk_elems(h.vocab), n_chunks = (h.vocab + chunk - 1) / chunk;
    P.z_out = zstep;
    for (int i = 0; i < h.block; ++i) {
      P.step0 = i;
      launch_pdl(ar_head_kernel<true>, dim3(grid), dim3(kThreads), (size_t)smem, st, P);
      DPARA_CHECK_LAUNCH();
      launch_pdl(head_sample_kernel, dim3(n_chunks, h.b), dim3(kPickThreads), 0, st, static_cast<const float *>(zstep), h.uniforms, h.next_tokens, part, tick, h.vocab, h.block, i, chunk);
      DPARA_CHECK_LAUNCH();
      count_launches(2);
    }
    return DPARA_OK;
  }
  // cooperative launch: the grid barrier needs every CTA resident (one CTA per SM fits by construction)
  void *args[] = {&P};
  if (cudaLaunchCooperativeKernel(reinterpret_cast<void *>(ar_head_kernel<false>), dim3(grid), dim3(kThreads), args, smem, st) != cudaSuccess) {
    cudaGetLastError();
    return DPARA_ERR_CUDA;
  }
  count_launches(1);
  return DPARA_OK;
}

}  // namespace dpara
