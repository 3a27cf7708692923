// Verification outcome + branch selection (Alg. 1 lines 2-3; Sec. 2.1; App. C).
//
// Both modes are ONE launch: the vocabulary work is spread over the whole GPU (CTAs over
// (request row, vocabulary chunk), 16-byte streaming loads), partial results meet in a small
// workspace, and the last CTA to finish a request does that request's position scan, writes
// (accept_len, bonus, out_tokens) and gathers the selected branch's representation.
// No CTA ever waits for another: "last" is decided by an atomic ticket.
#include "common.cuh"

namespace dpara {

constexpr int kVsThreads = 256;
constexpr int kMaxGreedyLoads = 16;  // 16-byte loads in flight per thread (1, 2, 4, 8 or 16: chosen per shape so that the grid fills the GPU)
constexpr int kSampChunk = 4096;    // floats per CTA and per row
constexpr int kMaxJ = 64;

// Monotone map float -> uint32 (a < b  <=>  key(a) < key(b)), -0 folded onto +0, NaN -> 0 (below -inf).
__device__ __forceinline__ uint32_t order_key(float f) {
  f = __fadd_rn(f, 0.0f);
  uint32_t u = __float_as_uint(f);
  uint32_t k = u ^ (((uint32_t)((int32_t)u >> 31)) | 0x80000000u);
  return (f != f) ? 0u : k;
}

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    unsigned long long t = __shfl_xor_sync(0xffffffffu, v, o);
    v = t > v ? t : v;
  }
  return v;
}

__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Copy of the selected branch: reps[n][r] -> selected[n], `bytes` per request.
__device__ __forceinline__ void gather_branch(const uint8_t *__restrict__ reps, uint8_t *__restrict__ selected, int n,
                                              size_t req_bytes, int r, size_t bytes, int tid, int nthreads) {
  const uint8_t *src = reps + (size_t)n * req_bytes + (size_t)r * bytes;
  uint8_t *dst = selected + (size_t)n * bytes;
  if ((bytes & 15) == 0 && ((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15) == 0) {
    const uint4 *s = reinterpret_cast<const uint4 *>(src);
    uint4 *d = reinterpret_cast<uint4 *>(dst);
    const size_t nv = bytes >> 4;
    // 8 independent 16-byte loads in flight per thread: the copy is one CTA's job, so latency matters
    size_t i = tid;
    for (; i + 7 * (size_t)nthreads < nv; i += 8 * (size_t)nthreads) {
      uint4 v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = __ldcs(s + i + k * (size_t)nthreads);
#pragma unroll
      for (int k = 0; k < 8; ++k) d[i + k * (size_t)nthreads] = v[k];
    }
    for (; i < nv; i += nthreads) d[i] = __ldcs(s + i);
  } else {
    for (size_t i = tid; i < bytes; i += nthreads) dst[i] = src[i];
  }
}

struct VerifyParams {
  const float *target;
  const float *draft_probs;
  const int32_t *tokens;
  const float *uniforms;
  const uint8_t *reps;
  int32_t *accept_len, *bonus, *gather_idx, *out_tokens;
  uint8_t *selected;
  int32_t *status_word;
  // The workspace is all zero when a call starts and all zero again when it ends: the CTA that finishes last
  // puts back what the call dirtied (no clearing launch in front of the kernel).
  unsigned long long *ws64;  // greedy: keys[b*J]; sampling: chunk sums [b][nchunks][2]
  unsigned int *counters;    // greedy: [b*J] row counters, then one "rows finished" counter; sampling: [b]
  unsigned long long *masks; // greedy: [b] completed-row masks
  int b, J, V, nchunks, vec_ok;
  int early;         // early start: no wait for the preceding kernel until `reps` is read / the workspace is handed back
  size_t rep_bytes;  // Bq * hidden * 2
  size_t req_bytes;  // from one request's representations to the next request's (J * rep_bytes when packed)
};

// Outputs of request n, written by the first J threads of the finishing CTA.
__device__ __forceinline__ void write_result(const VerifyParams &P, int n, int r, int tok, bool bad, int tid) {
  if (tid == 0) {
    P.accept_len[n] = r;
    P.bonus[n] = tok;
    P.gather_idx[n] = r;
    if (bad && P.status_word) atomicOr(reinterpret_cast<unsigned int *>(P.status_word), DPARA_STATUS_BAD_TOKEN);
  }
  if (P.out_tokens && tid < P.J)
    P.out_tokens[(size_t)n * P.J + tid] = tid < r ? P.tokens[(size_t)n * (P.J - 1) + tid] : (tid == r ? tok : -1);
}

// ------------------------------------------------------------------------------------------ greedy
template <int kGreedyLoads>
__global__ void __launch_bounds__(kVsThreads, kGreedyLoads >= 16 ? 3 : (kGreedyLoads >= 8 ? 4 : 6)) verify_greedy_kernel(const VerifyParams P) {
  constexpr int kGreedyChunk = kGreedyLoads * 1024;  // floats per CTA
  const int tid = threadIdx.x;
  if (!P.early) {
    pdl_wait();
    pdl_launch_dependents();
  }
  // rows are handed out position-major (every request's row 0 first, then every row 1, ...): the early rows,
  // which decide the accepted length, finish early for ALL requests
  const int n = blockIdx.y % P.b;
  const int row = n * P.J + blockIdx.y / P.b;
  const float *__restrict__ p = P.target + (size_t)row * P.V;
  const int base = blockIdx.x * kGreedyChunk;
  const int end = min(P.V, base + kGreedyChunk);

  // Fast path: plain float compares (3 instructions per element).  A strict '>' from -inf keeps the
  // lowest index among equal values, never selects a NaN, and treats -0 and +0 as equal.  What it cannot
  // rank are -inf and NaN themselves; a chunk in which nothing beat -inf is redone with the exact
  // integer keys below (rare, CTA-uniform).
  __shared__ unsigned long long s_k[kVsThreads / 32];
  __shared__ int s_flag;
  float bv = -INFINITY;
  uint32_t bi = 0xffffffffu;
  if (P.vec_ok) {
    float4 v[kGreedyLoads];
#pragma unroll
    for (int it = 0; it < kGreedyLoads; ++it) {
      int idx = base + (it * kVsThreads + tid) * 4;
      v[it] = idx < end ? __ldcs(reinterpret_cast<const float4 *>(p + idx)) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    }
#pragma unroll
    for (int it = 0; it < kGreedyLoads; ++it) {
      const uint32_t idx = base + (it * kVsThreads + tid) * 4;
      if (v[it].x > bv) { bv = v[it].x; bi = idx; }
      if (v[it].y > bv) { bv = v[it].y; bi = idx + 1; }
      if (v[it].z > bv) { bv = v[it].z; bi = idx + 2; }
      if (v[it].w > bv) { bv = v[it].w; bi = idx + 3; }
    }
  } else {
    for (int idx = base + tid; idx < end; idx += kVsThreads) {
      const float x = __ldcs(p + idx);
      if (x > bv) { bv = x; bi = idx; }
    }
  }
  unsigned long long key = bi == 0xffffffffu ? 0ull : (((unsigned long long)order_key(bv) << 32) | (unsigned long long)(0xffffffffu - bi));
  key = warp_max_u64(key);
  if ((tid & 31) == 0) s_k[tid >> 5] = key;
  __syncthreads();
  {
    unsigned long long m = s_k[0];
#pragma unroll
    for (int w = 1; w < kVsThreads / 32; ++w) m = s_k[w] > m ? s_k[w] : m;
    __syncthreads();
    if (m == 0ull) {  // only -inf / NaN in this chunk: exact ranking with integer keys
      uint32_t bk = 0;
      bi = 0xffffffffu;
      for (int idx = base + tid; idx < end; idx += kVsThreads) {
        uint32_t k = order_key(p[idx]);
        if (k > bk) { bk = k; bi = idx; }
      }
      key = warp_max_u64(((unsigned long long)bk << 32) | (unsigned long long)(0xffffffffu - bi));
      if ((tid & 31) == 0) s_k[tid >> 5] = key;
      __syncthreads();
    }
  }
  // Completion protocol (no CTA waits for another):
  //   row counter   -- the CTA that brings a row's counter to nchunks has completed that row;
  //   request mask  -- it then ORs the row's bit into the request's mask.  The accepted length is decided
  //                    as soon as rows 0..k are complete and either draft k+1 disagrees with row k's maximum or
  //                    k is the last row.  Exactly one CTA sees the mask go from "undecided" to "decided"
  //                    (the atomic OR serialises them); it writes the results and gathers the branch -- usually
  //                    while most of the request's later rows are still streaming, so the gather is hidden.
  __shared__ unsigned long long s_old, s_new;
  if (tid == 0) {
    unsigned long long m = s_k[0];
#pragma unroll
    for (int w = 1; w < kVsThreads / 32; ++w) m = s_k[w] > m ? s_k[w] : m;
    if (m) atomicMax(P.ws64 + row, m);
    __threadfence();
    s_flag = 0;
    if (atomicAdd(P.counters + row, 1u) == (unsigned int)P.nchunks - 1u) {
      __threadfence();
      const unsigned long long bit = 1ull << (row - n * P.J);
      const unsigned long long old = atomicOr(P.masks + n, bit);
      s_old = old;
      s_new = old | bit;
      s_flag = 1;
    }
  }
  __syncthreads();
  if (!s_flag) return;

  // ---- this CTA completed a row: is the request's outcome decided now, and was it not before?
  __threadfence();
  __shared__ int s_a[kMaxJ], s_t[kMaxJ];
  __shared__ int s_r, s_bad, s_act, s_last;
  const unsigned long long mask_new = s_new, mask_old = s_old;
  if (tid < P.J) {
    const bool done = (mask_new >> tid) & 1ull;
    unsigned long long k = done ? __ldcg(P.ws64 + (size_t)n * P.J + tid) : 0ull;
    s_a[tid] = k == 0ull ? 0 : (int)(0xffffffffu - (uint32_t)(k & 0xffffffffull));  // all-NaN row -> 0
    s_t[tid] = tid < P.J - 1 ? P.tokens[(size_t)n * (P.J - 1) + tid] : -1;           // all tokens in one round trip
  }
  __syncthreads();
  if (tid == 0) {
    // scan with the new mask; remember how far the OLD mask would have allowed the same scan to go
    int r = -1;
    bool bad = false, decided_before = false;
    for (int k = 0; k < P.J; ++k) {
      if (!((mask_new >> k) & 1ull)) break;  // row k not complete yet: undecided
      bool stop = (k == P.J - 1);
      if (!stop) {
        const int t = s_t[k];
        if (t < 0 || t >= P.V) { bad = true; stop = true; }
        else if (t != s_a[k]) stop = true;
      }
      if (stop) {
        r = k;
        // decided before iff rows 0..k were all complete in the old mask as well
        const unsigned long long need = (k == 63) ? ~0ull : ((1ull << (k + 1)) - 1ull);
        decided_before = (mask_old & need) == need;
        break;
      }
    }
    s_act = (r >= 0) && !decided_before;
    s_r = r;
    s_bad = bad;
  }
  __syncthreads();
  if (s_act) {
    if (P.early) pdl_wait();   // the selected branch comes from the kernel before
    const int r = s_r;
    if (tid == 0) {
      P.accept_len[n] = r;
      P.bonus[n] = s_a[r];
      P.gather_idx[n] = r;
      if (s_bad && P.status_word) atomicOr(reinterpret_cast<unsigned int *>(P.status_word), DPARA_STATUS_BAD_TOKEN);
    }
    if (P.out_tokens && tid < P.J) P.out_tokens[(size_t)n * P.J + tid] = tid < r ? s_t[tid] : (tid == r ? s_a[r] : -1);
    if (P.reps) gather_branch(P.reps, P.selected, n, P.req_bytes, r, P.rep_bytes, tid, kVsThreads);
  }
  // ---- leave the workspace as it was found.  Every row-completing CTA checks in here as its LAST access to
  // the workspace; a CTA that did not complete a row touched it last before its row counter moved, i.e. before
  // that row's completer got here.  So the CTA that checks in last is alone with the workspace and zeroes it.
  __syncthreads();
  if (tid == 0) {
    __threadfence();
    s_last = atomicAdd(P.counters + (size_t)P.b * P.J, 1u) == (unsigned int)(P.b * P.J) - 1u;
  }
  __syncthreads();
  if (!s_last) return;
  if (P.early) pdl_wait();     // (the call does not complete before the work in front of it has)
  for (int i = tid; i < P.b * P.J; i += kVsThreads) { P.ws64[i] = 0ull; P.counters[i] = 0u; }
  for (int i = tid; i < P.b; i += kVsThreads) P.masks[i] = 0ull;
  if (tid == 0) P.counters[(size_t)P.b * P.J] = 0u;
}

// ------------------------------------------------------------------------------------------ sampling
__device__ __forceinline__ unsigned long long fx_weight(float d) {
  d = d > 0.0f ? d : 0.0f;  // negatives and NaN carry no weight
  return __float2ull_rz(d * 4294967296.0f);
}

// primary weight (residual, or p itself when no draft was rejected) and fallback weight (p)
__device__ __forceinline__ void weights_of(float p, float q, bool residual, unsigned long long &w0, unsigned long long &w1) {
  w1 = fx_weight(p);
  w0 = residual ? fx_weight(__fsub_rn(p, q)) : w1;
}

__global__ void __launch_bounds__(kVsThreads) verify_sampling_kernel(const VerifyParams P) {
  const int tid = threadIdx.x;
  if (!P.early) {
    pdl_wait();
    pdl_launch_dependents();
  }
  const int n = blockIdx.y;
  const int c = blockIdx.x;
  const int g = P.J - 1;
  __shared__ int s_r, s_bad, s_flag;
  __shared__ unsigned long long s_w[2][kVsThreads / 32];

  // accepted length: every CTA of the request repeats this 2*gamma-scalar scan (L2 hits)
  if (tid < 32) {
    unsigned int rej = 0, badm = 0;
    for (int i0 = 0; i0 < g; i0 += 32) {
      int i = i0 + tid;
      bool reject = false, bad = false;
      if (i < g) {
        int t = P.tokens[(size_t)n * g + i];
        if (t < 0 || t >= P.V) {
          reject = bad = true;
        } else {
          float qv = P.draft_probs[((size_t)n * g + i) * P.V + t];
          float pv = P.target[((size_t)n * P.J + i) * P.V + t];
          float u = P.uniforms[(size_t)n * P.J + i];
          reject = !(__fmul_rn(u, qv) < pv);
        }
      }
      rej = __ballot_sync(0xffffffffu, reject);
      badm = __ballot_sync(0xffffffffu, bad);
      if (rej) {
        if (tid == 0) {
          int f = __ffs(rej) - 1;
          s_r = i0 + f;
          s_bad = (badm >> f) & 1u;
        }
        break;
      }
    }
    if (!rej && tid == 0) { s_r = g; s_bad = 0; }
  }
  __syncthreads();
  const int r = s_r;
  const bool residual = r < g;
  const float *__restrict__ prow = P.target + ((size_t)n * P.J + r) * P.V;
  const float *__restrict__ qrow = residual ? P.draft_probs + ((size_t)n * g + r) * P.V : prow;

  // chunk sums of both weightings
  const int base = c * kSampChunk;
  const int end = min(P.V, base + kSampChunk);
  unsigned long long a0 = 0, a1 = 0;
  if (P.vec_ok) {
#pragma unroll
    for (int it = 0; it < kSampChunk / (kVsThreads * 4); ++it) {
      int idx = base + (it * kVsThreads + tid) * 4;
      if (idx < end) {
        float4 pv = __ldg(reinterpret_cast<const float4 *>(prow + idx));
        float4 qv = residual ? __ldg(reinterpret_cast<const float4 *>(qrow + idx)) : pv;
        unsigned long long w0, w1;
        weights_of(pv.x, qv.x, residual, w0, w1); a0 += w0; a1 += w1;
        weights_of(pv.y, qv.y, residual, w0, w1); a0 += w0; a1 += w1;
        weights_of(pv.z, qv.z, residual, w0, w1); a0 += w0; a1 += w1;
        weights_of(pv.w, qv.w, residual, w0, w1); a0 += w0; a1 += w1;
      }
    }
  } else {
    for (int idx = base + tid; idx < end; idx += kVsThreads) {
      unsigned long long w0, w1;
      weights_of(prow[idx], qrow[idx], residual, w0, w1);
      a0 += w0; a1 += w1;
    }
  }
  a0 = warp_sum_u64(a0);
  a1 = warp_sum_u64(a1);
  if ((tid & 31) == 0) { s_w[0][tid >> 5] = a0; s_w[1][tid >> 5] = a1; }
  __syncthreads();
  if (tid == 0) {
    unsigned long long t0 = 0, t1 = 0;
#pragma unroll
    for (int w = 0; w < kVsThreads / 32; ++w) { t0 += s_w[0][w]; t1 += s_w[1][w]; }
    unsigned long long *cs = P.ws64 + ((size_t)n * P.nchunks + c) * 2;
    __stcg(cs, t0);
    __stcg(cs + 1, t1);
    __threadfence();
    unsigned int t = atomicAdd(P.counters + n, 1u);
    s_flag = (t == (unsigned int)P.nchunks - 1u);
  }
  __syncthreads();
  if (!s_flag) return;

  // ---- last CTA of request n: total weight, threshold, locate the crossing
  if (P.early) pdl_wait();     // before the branch is read and before the request's part of the call completes
  __threadfence();
  __shared__ unsigned long long s_T, s_basepref;
  __shared__ int s_chunk, s_which, s_tok;
  if (P.nchunks <= kVsThreads) {
    // thread k holds chunk k's two sums: totals by a block reduction, the crossing chunk by a block scan (one L2 round trip
    // for all the sums; a single thread walking the chunks paid one round trip per chunk, ~0.7 us each)
    unsigned long long c0 = 0, c1 = 0;
    if (tid < P.nchunks) {
      c0 = __ldcg(P.ws64 + ((size_t)n * P.nchunks + tid) * 2);
      c1 = __ldcg(P.ws64 + ((size_t)n * P.nchunks + tid) * 2 + 1);
    }
    unsigned long long r0 = warp_sum_u64(c0), r1 = warp_sum_u64(c1);
    if ((tid & 31) == 0) { s_w[0][tid >> 5] = r0; s_w[1][tid >> 5] = r1; }
    if (tid == 0) { s_tok = 0; s_chunk = 0; }
    __syncthreads();
    unsigned long long W0 = 0, W1 = 0;
#pragma unroll
    for (int w = 0; w < kVsThreads / 32; ++w) { W0 += s_w[0][w]; W1 += s_w[1][w]; }
    const int which = W0 ? 0 : (W1 ? 1 : 2);
    __syncthreads();   // s_w is reused by the scan
    if (tid == 0) s_which = which;
    if (which < 2) {
      const unsigned long long Wt = which ? W1 : W0;
      // a uniform is m * 2^-24 with m < 2^24; anything at or above 1 is taken as the largest uniform, so the
      // threshold stays below the total weight and the draw inside the vocabulary
      unsigned int m = __float2uint_rn(fminf(P.uniforms[(size_t)n * P.J + g], 1.0f) * 16777216.0f);
      m = m > 16777215u ? 16777215u : m;
      const unsigned long long lo = (unsigned long long)m * Wt;  // low 64 bits
      const unsigned long long hi = __umul64hi((unsigned long long)m, Wt);
      const unsigned long long T = (hi << 40) | (lo >> 24);  // (m * W) >> 24, m < 2^24 so it fits
      const unsigned long long sel = which ? c1 : c0;
      unsigned long long inc = sel;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long t = __shfl_up_sync(0xffffffffu, inc, o);
        if ((tid & 31) >= o) inc += t;
      }
      if ((tid & 31) == 31) s_w[0][tid >> 5] = inc;
      __syncthreads();
      unsigned long long before = 0;
      for (int w = 0; w < (tid >> 5); ++w) before += s_w[0][w];
      inc += before;
      // the first chunk whose inclusive sum exceeds the threshold (T < total: there is exactly one such first chunk)
      if (tid < P.nchunks && inc > T && inc - sel <= T) { s_chunk = tid; s_T = T; s_basepref = inc - sel; }
    }
  } else if (tid == 0) {
    unsigned long long W0 = 0, W1 = 0;
    for (int k = 0; k < P.nchunks; ++k) {
      W0 += __ldcg(P.ws64 + ((size_t)n * P.nchunks + k) * 2);
      W1 += __ldcg(P.ws64 + ((size_t)n * P.nchunks + k) * 2 + 1);
    }
    int which = W0 ? 0 : (W1 ? 1 : 2);
    s_which = which;
    s_tok = 0;
    s_chunk = 0;
    if (which < 2) {
      unsigned long long Wt = which ? W1 : W0;
      // a uniform is m * 2^-24 with m < 2^24; anything at or above 1 is taken as the largest uniform, so the
      // threshold stays below the total weight and the draw inside the vocabulary
      unsigned int m = __float2uint_rn(fminf(P.uniforms[(size_t)n * P.J + g], 1.0f) * 16777216.0f);
      m = m > 16777215u ? 16777215u : m;
      unsigned long long lo = (unsigned long long)m * Wt;  // low 64 bits
      unsigned long long hi = __umul64hi((unsigned long long)m, Wt);
      unsigned long long T = (hi << 40) | (lo >> 24);  // (m * W) >> 24, m < 2^24 so it fits
      unsigned long long pref = 0;
      int k = 0;
      for (; k < P.nchunks - 1; ++k) {
        unsigned long long s = __ldcg(P.ws64 + ((size_t)n * P.nchunks + k) * 2 + which);
        if (pref + s > T) break;
        pref += s;
      }
      s_chunk = k;
      s_T = T;
      s_basepref = pref;
    }
  }
  __syncthreads();
  const int which = s_which;
  if (which < 2) {
    // thread t owns elements [cb + 16 t, cb + 16 t + 16) of the crossing chunk
    const int cb = s_chunk * kSampChunk;
    const int per = kSampChunk / kVsThreads;
    unsigned long long w[kSampChunk / kVsThreads];
    unsigned long long loc = 0;
#pragma unroll
    for (int e = 0; e < per; ++e) {
      int idx = cb + tid * per + e;
      unsigned long long w0 = 0, w1 = 0;
      if (idx < P.V) weights_of(prow[idx], qrow[idx], residual, w0, w1);
      w[e] = which ? w1 : w0;
      loc += w[e];
    }
    // block exclusive scan of loc
    unsigned long long inc = loc;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      unsigned long long t = __shfl_up_sync(0xffffffffu, inc, o);
      if ((tid & 31) >= o) inc += t;
    }
    if ((tid & 31) == 31) s_w[0][tid >> 5] = inc;
    __syncthreads();
    unsigned long long woff = 0;
    for (int k = 0; k < (tid >> 5); ++k) woff += s_w[0][k];
    unsigned long long excl = s_basepref + woff + inc - loc;
    const unsigned long long T = s_T;
    if (excl <= T && excl + loc > T) {  // exactly one thread
      unsigned long long acc = excl;
      int tok = cb + tid * per;
#pragma unroll
      for (int e = 0; e < per; ++e) {
        acc += w[e];
        if (acc > T) { tok = cb + tid * per + e; break; }
      }
      s_tok = tok;
    }
    __syncthreads();
  } else {
    // no weight anywhere in p_r: lowest-index maximum of the row
    uint32_t bk = 0, bi = 0xffffffffu;
    for (int idx = tid; idx < P.V; idx += kVsThreads) {
      uint32_t k = order_key(prow[idx]);
      if (k > bk) { bk = k; bi = idx; }
    }
    unsigned long long key = warp_max_u64(((unsigned long long)bk << 32) | (unsigned long long)(0xffffffffu - bi));
    if ((tid & 31) == 0) s_w[0][tid >> 5] = key;
    __syncthreads();
    if (tid == 0) {
      unsigned long long m = 0;
      for (int k = 0; k < kVsThreads / 32; ++k) m = s_w[0][k] > m ? s_w[0][k] : m;
      s_tok = m == 0ull ? 0 : (int)(0xffffffffu - (uint32_t)(m & 0xffffffffull));
    }
    __syncthreads();
  }
  write_result(P, n, r, s_tok, s_bad != 0, tid);
  // this CTA is the request's last: nobody reads the chunk sums or the ticket again -- leave them zeroed
  __syncthreads();
  for (int i = tid; i < 2 * P.nchunks; i += kVsThreads) P.ws64[(size_t)n * P.nchunks * 2 + i] = 0ull;
  if (tid == 0) P.counters[n] = 0u;
  if (P.reps) gather_branch(P.reps, P.selected, n, P.req_bytes, r, P.rep_bytes, tid, kVsThreads);
}

// Greedy: 16-byte loads in flight per thread.  As many as possible (fewer, larger CTAs amortise the reduction
// and the completion atomics: measured 37 / 38 / 43 / 64 us at 16 / 8 / 4 / 2 loads for 16 requests x 16 rows),
// but few enough that rows x chunks gives every SM a CTA (a single request's 8 rows: 8 loads, 152 CTAs).
static int greedy_loads_of(const dpara_verify_io *io) {
  const long long rows = (long long)io->batch * io->n_boundaries;
  for (int l = kMaxGreedyLoads; l > 1; l >>= 1)
    if (rows * ((io->vocab + l * 1024 - 1) / (l * 1024)) >= kNumSM) return l;
  return 1;
}

static int chunks_of(const dpara_verify_io *io) {
  int ch = io->mode == 0 ? greedy_loads_of(io) * 1024 : kSampChunk;
  return (io->vocab + ch - 1) / ch;
}

// workspace: [64-bit area][counters]
static size_t ws64_count(const dpara_verify_io *io) {
  return io->mode == 0 ? (size_t)io->batch * io->n_boundaries : (size_t)io->batch * chunks_of(io) * 2;
}

static dpara_status validate_dims(const dpara_verify_io *io) {
  if (!io) return DPARA_ERR_INVALID_ARG;
  if (io->batch <= 0 || io->n_boundaries <= 0 || io->vocab <= 0) return DPARA_ERR_INVALID_ARG;
  if (io->mode != 0 && io->mode != 1) return DPARA_ERR_INVALID_ARG;
  if (io->n_boundaries > kMaxJ) return DPARA_ERR_UNSUPPORTED;
  if (io->batch > 65535) return DPARA_ERR_UNSUPPORTED;
  if ((long long)io->batch * io->n_boundaries > 65535 && io->mode == 0) return DPARA_ERR_UNSUPPORTED;
  return DPARA_OK;
}

static dpara_status validate_verify(const dpara_verify_io *io) {
  dpara_status s = validate_dims(io);
  if (s != DPARA_OK) return s;
  if (!io->target || !io->accept_len || !io->bonus || !io->gather_idx) return DPARA_ERR_INVALID_ARG;
  if (io->flags & ~DPARA_VERIFY_EARLY_START) return DPARA_ERR_INVALID_ARG;
  if (io->n_boundaries > 1 && !io->draft_tokens) return DPARA_ERR_INVALID_ARG;
  if (io->mode == 1 && (!io->uniforms || (io->n_boundaries > 1 && !io->draft_probs))) return DPARA_ERR_INVALID_ARG;
  if (io->reps) {
    if (!io->selected || io->block <= 0 || io->hidden <= 0) return DPARA_ERR_INVALID_ARG;
    if (io->rep_req_rows < 0 || (io->rep_req_rows > 0 && io->rep_req_rows < io->n_boundaries * io->block)) return DPARA_ERR_INVALID_ARG;
  }
  return DPARA_OK;
}

}  // namespace dpara

using namespace dpara;

extern "C" size_t dpara_verify_workspace_bytes(const dpara_verify_io *io) {
  if (validate_dims(io) != DPARA_OK) return 0;
  const size_t ncnt = io->mode == 0 ? (size_t)io->batch * io->n_boundaries + 1 : (size_t)io->batch;
  return align_up(ws64_count(io) * 8, 256) + align_up((size_t)io->batch * 8, 256) + align_up(ncnt * 4, 256);
}

namespace dpara {
// Shared by the public entry point; `ws` must hold dpara_verify_workspace_bytes(io) bytes.
dpara_status launch_verify(const dpara_verify_io *io, void *ws, int32_t *status_word, cudaStream_t st) {
  VerifyParams P;
  P.target = io->target;
  P.draft_probs = io->draft_probs;
  P.tokens = io->draft_tokens;
  P.uniforms = io->uniforms;
  P.reps = static_cast<const uint8_t *>(io->reps);
  P.accept_len = io->accept_len;
  P.bonus = io->bonus;
  P.gather_idx = io->gather_idx;
  P.out_tokens = io->out_tokens;
  P.selected = static_cast<uint8_t *>(io->selected);
  P.status_word = status_word;
  P.b = io->batch;
  P.J = io->n_boundaries;
  P.V = io->vocab;
  P.nchunks = chunks_of(io);
  P.rep_bytes = (size_t)io->block * io->hidden * 2;
  P.early = (io->flags & DPARA_VERIFY_EARLY_START) ? 1 : 0;
  P.req_bytes = io->rep_req_rows > 0 ? (size_t)io->rep_req_rows * io->hidden * 2 : (size_t)io->n_boundaries * P.rep_bytes;
  size_t n64 = ws64_count(io);
  const size_t mask_off = align_up(n64 * 8, 256);
  const size_t cnt_off = mask_off + align_up((size_t)io->batch * 8, 256);
  P.ws64 = static_cast<unsigned long long *>(ws);
  P.masks = reinterpret_cast<unsigned long long *>(static_cast<uint8_t *>(ws) + mask_off);
  P.counters = reinterpret_cast<unsigned int *>(static_cast<uint8_t *>(ws) + cnt_off);
  bool vec = (io->vocab % 4 == 0) && aligned16(io->target) && (io->mode == 0 || io->n_boundaries == 1 || aligned16(io->draft_probs));
  P.vec_ok = vec ? 1 : 0;
  // keys, masks and counters are zero on entry (the previous call put them back); nothing is cleared here
  if (io->mode == 0) {
    dim3 grid(P.nchunks, io->batch * io->n_boundaries);
    // The 16-load form is chosen when the grid is several waves deep (b = 16: 2560 CTAs): launched early behind a long
    // kernel it measured 5 us SLOWER than a plain launch, so only the small-grid forms ask for the early launch
    // (b = 1: 152 CTAs, 3 us faster).
    switch (greedy_loads_of(io)) {
      case 16:
        if (P.early) launch_pdl(verify_greedy_kernel<16>, dim3(grid), dim3(kVsThreads), 0, st, P);
        else verify_greedy_kernel<16><<<grid, kVsThreads, 0, st>>>(P);
        break;
      case 8: launch_pdl(verify_greedy_kernel<8>, dim3(grid), dim3(kVsThreads), 0, st, P); break;
      case 4: launch_pdl(verify_greedy_kernel<4>, dim3(grid), dim3(kVsThreads), 0, st, P); break;
      case 2: launch_pdl(verify_greedy_kernel<2>, dim3(grid), dim3(kVsThreads), 0, st, P); break;
      default: launch_pdl(verify_greedy_kernel<1>, dim3(grid), dim3(kVsThreads), 0, st, P); break;
    }
  } else {
    dim3 grid(P.nchunks, io->batch);
    launch_pdl(verify_sampling_kernel, dim3(grid), dim3(kVsThreads), 0, st, P);
  }
  DPARA_CHECK_LAUNCH();
  count_launches(1);
  return DPARA_OK;
}
}  // namespace dpara

extern "C" dpara_status dpara_verify_select(const dpara_verify_io *io, void *workspace, size_t workspace_bytes,
                                            int32_t *status_word, void *stream) {
  dpara_status s = validate_verify(io);
  if (s != DPARA_OK) return s;
  size_t need = dpara_verify_workspace_bytes(io);
  if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 7u)) return DPARA_ERR_WORKSPACE;
  return launch_verify(io, workspace, status_word, static_cast<cudaStream_t>(stream));
}

// ------------------------------------------------------------------------------------------ fixed-scratch variant
// For callers that cannot allocate (all device memory already handed to their own pool, or an
// allocation would stall the decode loop): the scratch lives in the library's device image.
// `g_verify_scratch` below is only a host-side stand-in for the array when named in host code; the
// device address a kernel can use comes from cudaGetSymbolAddress, looked up once per device with
// that device current.
#include <mutex>

static __device__ __align__(256) unsigned char g_verify_scratch[DPARA_VERIFY_STATIC_SCRATCH_BYTES];

namespace dpara {
constexpr int kMaxDevices = 64;
static void *g_scratch_addr[kMaxDevices] = {nullptr};
static std::mutex g_scratch_mutex;

// Device address of the fixed scratch on the CURRENT device (set-up on first use per device).
static dpara_status static_scratch_ptr(void **out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return DPARA_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return DPARA_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_addr[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_verify_scratch) != cudaSuccess || !p) return DPARA_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return DPARA_OK;
}
}  // namespace dpara

extern "C" dpara_status dpara_verify_select_static(const dpara_verify_io *io, int32_t *status_word, void *stream) {
  dpara_status s = validate_verify(io);
  if (s != DPARA_OK) return s;
  if (dpara_verify_workspace_bytes(io) > (size_t)DPARA_VERIFY_STATIC_SCRATCH_BYTES) return DPARA_ERR_STATIC_LIMIT;
  void *scratch = nullptr;
  s = static_scratch_ptr(&scratch);
  if (s != DPARA_OK) return s;
  // the array is zero when the library is loaded, and every call puts back the zeros it consumed (the
  // CTA that finishes last clears the keys, masks and counters), so nothing has to be cleared up front
  return launch_verify(io, scratch, status_word, static_cast<cudaStream_t>(stream));
}
