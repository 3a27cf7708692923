// All-boundary attention on the 5th-generation tensor cores (Sec. 3.2, Fig. 4).
//
// Work item = (request n, KV head g, pair of 128-row query tiles, KV split).  Every K/V byte streamed from
// HBM serves all boundaries and all query heads of the group that share the KV head.  The G heads of a
// group are cut into "head blocks" of 8, 4, 2 or 1 heads (the binary digits of G: G = 5 -> 4 + 1); a
// query tile holds hb heads x (128 / hb) consecutive (boundary j, slot i) rows of one head block, ordered
// (j, i, head), which is one 3-D TMA box of the q tensor -- so every tile is full whatever G is (a tile of
// 128 / G whole (j, i) rows of all G heads leaves rows idle and a part-filled last tile when G is not a
// power of two).
//
//   warp 8      TMA producer: Q tiles once, then K and V tiles of 128 keys through one ring of tile slots
//               (order K0 K1 V0 K2 V1 ...).  The context needs no mask at all (every row sees the whole
//               cache); the spine prefix and the own blocks of the boundaries a tile pair touches are
//               packed into extra "tail" tiles (the first holds the spine and as many blocks as fit next to
//               it; usually it is the only one).
//   warps 9, 10 one thread per query tile issues tcgen05.mma:  S = Q_t K^T  (A, B from shared memory) and
//               O_t += P_t V  (A = P_t from tensor memory, B = V, MN-major).
//   warps 0-3   softmax of tile 0, warps 4-7 softmax of tile 1: thread = row.  tcgen05.ld the S row into
//               registers and hand the S buffer back at once; mask (tail tile only: anchor prefix of the
//               row's boundary + its own block), online max/sum in registers with LAZY rescaling (O in
//               TMEM is rescaled only when a row's max grows by more than 2^8), P_t written as bf16 with
//               tcgen05.st to its own columns.
// TMEM: O0 | O1 (128 columns reserved each) | S (128 fp32 columns, ONE buffer that the two tiles take in
// turns) | P0 | P1 (64 columns each).  S lives only from its QK to the softmax warps' load, and P_t does not
// alias it, so QK(t, i+1) never waits for softmax(t, i): a tile's softmax finds its next scores ready, and
// the tensor pipe and the softmax warps are coupled only through buffer hand-offs, not through a
// score -> probability -> score chain.
// Every mbarrier wait is bounded; on expiry the CTA sets DPARA_STATUS_TIMEOUT and drains.
#include <math.h>

#include <algorithm>
#include <mutex>
#include <queue>
#include <utility>
#include <vector>

#include "attention_tc.cuh"
#include "sm100_ptx.cuh"

namespace dpara {
using namespace ptx;

namespace {
constexpr int kThreads = 384;  // warps 0-7 softmax, 8 TMA producer, 9 and 10 MMA issuers, 11 idle (completes the third warpgroup)
constexpr float kRescaleLog2 = 8.0f;
constexpr int kMaxOrdered = 128;
constexpr int kMaxSched = 3072;  // items a host-built schedule can hold (kernel parameter space)
constexpr int kMaxHeadBlocks = 4;  // G <= 16: at most four binary digits unless G == 16 (one block)
constexpr int kMaxSeg = 224;       // segments of the cut schedule (groups + teams)
constexpr int kMaxPairs = 256;     // 64 boundaries x 64 slots in tiles of 8 (j, i) rows = 512 tiles
}  // namespace


struct TcParams {
  CUtensorMap map_q[kMaxHeadBlocks], map_kc, map_vc, map_ks, map_vs, map_kb0, map_vb0, map_kb, map_vb;
  AttnParams a;
  // head blocks: block k covers heads [h0[k], h0[k] + (1 << hb_log2[k])) of every group; its tiles hold
  // 128 >> hb_log2[k] (j, i) rows; its tile pairs are pair_start[k] .. pair_start[k + 1] - 1
  int n_hblk, hb_log2[kMaxHeadBlocks], h0[kMaxHeadBlocks], pair_start[kMaxHeadBlocks + 1];
  // per tile pair, worked out on the host so that taking up an item costs a few loads, not a dozen divisions
  // (the two tiles of an item may come from DIFFERENT head blocks: the odd last tiles of two blocks share one K/V stream)
  struct PairInfo {
    int16_t ji0[2];   // first (j, i) row of each tile
    int16_t jb0_rel;  // first boundary whose block keys sit in the tail tiles, relative to boundary_lo
    uint8_t blk[2], hs[2], h0[2];  // per tile: head block, log2(heads per row group), first head
    uint8_t ntq, n_tail;
  } pair[kMaxPairs];
  int nsplit_log2;

  // tail tiles: the first holds the spine (S8 = S rounded up to 8 rows) and cap0 blocks, the others cap blocks
  int n_ji, n_pairs, nsplit, S8, cap0, cap, has_blk, has_tail, n_items;
  int n_rows;  // query rows per request and head: n_ji mask-slot rows, then the spine rows when they are queries
  float *part_o;   // split-KV partials [item slot][2][D / 4][128 rows] float4 (unnormalised rows; a warp's lanes are
                   // consecutive rows, so its stores and the merge's loads are contiguous 512-byte runs)
  float2 *part_ml; // [item slot][2][128] (row max in raw-score units, row sum)
  float c_log2;    // softmax scale * log2(e)
  // requests in order of decreasing context length: the block scheduler hands out CTAs in grid order, so
  // launching the long requests first leaves the short ones to fill the tail of a ragged batch
  uint8_t req_order[kMaxOrdered];
  int use_order;
  // context offsets and lengths of small batches travel in the parameters (saves every CTA two dependent global
  // loads, ~1 us, before it can start)
  int use_ctx_p;
  int ctx_len_p[kMaxOrdered];
  long long ctx_off_p[kMaxOrdered];
  // Work schedule of the persistent CTAs (no KV split, more items than CTAs): CTA c runs items
  // sched[cta_first[c]] .. sched[cta_first[c + 1] - 1].  The host balances the CTAs' loads (longest processing
  // time first, each item to the least loaded CTA); a ragged batch has few items per CTA (about five at the
  // benchmark shape), so handing them out round-robin leaves the most loaded CTA ~20 % above the mean.
  int use_sched;
  // Cut schedule.  The X tile pairs of one (request, KV head) read the same K/V stream; run by X CTAs side by side (a
  // TEAM: CTAs team * X .. team * X + X - 1, member x takes pair x) they stay in step and every K/V tile comes from HBM
  // once and from L2 for the other members.  The host cuts the groups' key-tile ranges into CONTIGUOUS SEGMENTS of
  // near-equal cost, one run of segments per team (team_first), so that all teams finish together whatever the number of
  // groups (32 groups do not fill 37 teams otherwise, and a ragged batch does not balance).  A cut group's pieces leave
  // unnormalised rows in scratch; when a CTA has finished its run it takes a ticket for each of its cut items, and
  // whoever draws an item's last ticket merges the pieces and writes the output (no waiting).
  int use_seg, seg_X, seg_teams;
  struct Seg {
    uint16_t group, t0, t1, slot0;  // (request, KV head) group; context tiles [t0, t1); scratch slot base of the group's piece 0
    uint8_t piece, npieces, pad[2];
  } seg[kMaxSeg];
  uint16_t team_first[kNumSM + 1];
  unsigned int *seg_count;  // [items] tickets, zeroed before the launch
  uint16_t cta_first[kNumSM + 1];
  uint16_t sched[kMaxSched];
};

template <int D>
struct TcCfg {
  static constexpr int kSlabs = D / 64;
  static constexpr int kSlabBytes = 128 * 128;         // 128 rows x 64 bf16
  static constexpr int kTileBytes = kSlabs * kSlabBytes;  // Q, K or V tile
  // K and V tiles travel through ONE ring of tile-sized slots (K0 K1 V0 K2 V1 ...), as deep as shared memory
  // allows next to the two Q tiles: the producer runs ~1.5 iterations ahead of the MMA issuer
  static constexpr int kSlots = (227 * 1024 - 2 * kTileBytes - 2048) / kTileBytes > 8 ? 8 : (227 * 1024 - 2 * kTileBytes - 2048) / kTileBytes;
  static constexpr int kSmemBytes = 2 * kTileBytes + kSlots * kTileBytes + 1024 + 512;
  static constexpr int kColO = 0, kColS = 256, kColP = 384;  // TMEM columns: O_t at kColO + 128 t, S, P_t at kColP + 64 t
};

// One unit of work of a persistent CTA.
struct Item {
  int n, g, pair, split, ntq, L, t0, t1, nctx, n_ctx_it, n_tail, n_iter, jb0, slot;
  int npieces, slot0, item;    // KV pieces of the item (1: whole), scratch slot of piece 0, item id
  uint32_t geo0, geo1;  // per tile, packed (selected with a ternary, never indexed: the struct stays in registers):
                        // first (j, i) row | log2(heads per row group) << 16 | first head << 20 | head block << 28
  long long c0;
};

__device__ __forceinline__ uint32_t tile_geo(const Item &I, int t) { return t ? I.geo1 : I.geo0; }
__device__ __forceinline__ int geo_ji0(uint32_t g) { return (int)(g & 0xffffu); }
__device__ __forceinline__ int geo_hs(uint32_t g) { return (int)((g >> 16) & 0xfu); }
__device__ __forceinline__ int geo_h0(uint32_t g) { return (int)((g >> 20) & 0xffu); }
__device__ __forceinline__ int geo_blk(uint32_t g) { return (int)(g >> 28); }

// The low k bits set (k <= 0: none, k >= 32: all).
__device__ __forceinline__ uint32_t bits_below(int k) { return k <= 0 ? 0u : (k >= 32 ? 0xffffffffu : ((1u << k) - 1u)); }

// 4 x 4 transpose of 16-byte pieces among the four lanes of a quad: on return x[v] of lane c is what lane v of the
// quad held in x[c].
__device__ __forceinline__ void quad_transpose(uint4 (&x)[4], int lane) {
  auto swap_step = [&](int mask, uint4 &lo0, uint4 &lo1, uint4 &hi0, uint4 &hi1) {
    // lanes with the mask bit clear send (hi0, hi1) and receive into them; the others send (lo0, lo1) and receive into them
    const bool up = lane & mask;
    uint4 a = up ? lo0 : hi0, b = up ? lo1 : hi1;
    a.x = __shfl_xor_sync(0xffffffffu, a.x, mask); a.y = __shfl_xor_sync(0xffffffffu, a.y, mask);
    a.z = __shfl_xor_sync(0xffffffffu, a.z, mask); a.w = __shfl_xor_sync(0xffffffffu, a.w, mask);
    b.x = __shfl_xor_sync(0xffffffffu, b.x, mask); b.y = __shfl_xor_sync(0xffffffffu, b.y, mask);
    b.z = __shfl_xor_sync(0xffffffffu, b.z, mask); b.w = __shfl_xor_sync(0xffffffffu, b.w, mask);
    if (up) { lo0 = a; lo1 = b; } else { hi0 = a; hi1 = b; }
  };
  swap_step(2, x[0], x[1], x[2], x[3]);  // exchange the off-diagonal 2 x 2 blocks
  swap_step(1, x[0], x[2], x[1], x[3]);  // transpose inside the 2 x 2 blocks
}

// Tail tiles a tile pair needs: its boundaries' own blocks, cap0 of them next to the spine in the first tile.
__host__ __device__ __forceinline__ int tail_tiles(int has_tail, int has_blk, int nbk, int cap0, int cap) {
  if (!has_tail) return 0;
  if (!has_blk || nbk <= cap0) return 1;
  return 1 + (nbk - cap0 + cap - 1) / cap;
}

__device__ __forceinline__ Item decode_item(const TcParams &P, int id) {
  const AttnParams &A = P.a;
  Item I;
  const unsigned X = (unsigned)(P.n_pairs << P.nsplit_log2);
  const unsigned yz = (unsigned)id / X, x = (unsigned)id - yz * X;
  const unsigned z = yz / (unsigned)A.Hkv;
  I.g = (int)(yz - z * (unsigned)A.Hkv);
  I.n = P.use_order ? (int)P.req_order[z] : (int)z;
  I.pair = (int)(x >> P.nsplit_log2);
  I.split = (int)(x & ((1u << P.nsplit_log2) - 1u));
  const TcParams::PairInfo pi = P.pair[I.pair];
  I.geo0 = (uint32_t)(uint16_t)pi.ji0[0] | ((uint32_t)pi.hs[0] << 16) | ((uint32_t)pi.h0[0] << 20) | ((uint32_t)pi.blk[0] << 28);
  I.geo1 = (uint32_t)(uint16_t)pi.ji0[1] | ((uint32_t)pi.hs[1] << 16) | ((uint32_t)pi.h0[1] << 20) | ((uint32_t)pi.blk[1] << 28);
  I.ntq = pi.ntq;
  if (P.use_ctx_p) {
    I.c0 = P.ctx_off_p[I.n];
    I.L = P.ctx_len_p[I.n];
  } else {
    I.c0 = A.ctx_offsets[I.n];
    I.L = (int)(A.ctx_lens ? A.ctx_lens[I.n] : A.ctx_offsets[I.n + 1] - I.c0);
  }
  I.nctx = (I.L + 127) >> 7;
  I.t0 = (int)(((unsigned)I.split * (unsigned)I.nctx) >> P.nsplit_log2);  // nctx < 2^24, split < 8
  I.t1 = (int)(((unsigned)(I.split + 1) * (unsigned)I.nctx) >> P.nsplit_log2);
  I.n_ctx_it = I.t1 - I.t0;
  I.jb0 = A.lo + pi.jb0_rel;  // first boundary whose block keys sit in the tail tiles
  I.n_tail = I.split == (1 << P.nsplit_log2) - 1 ? pi.n_tail : 0;
  I.n_iter = I.n_ctx_it + I.n_tail;
  I.slot = (((I.n * A.Hkv + I.g) * P.n_pairs + I.pair) << P.nsplit_log2) + I.split;
  I.npieces = 1 << P.nsplit_log2;
  I.slot0 = I.slot - I.split;
  I.item = id;
  return I;
}

// Entry qi of this CTA's work list: a whole item (or one of its cluster splits), or a segment of a cut group.
__device__ __forceinline__ Item fetch_item(const TcParams &P, int qi) {
  if (!P.use_seg) return decode_item(P, P.use_sched ? (int)P.sched[qi] : qi);
  const TcParams::Seg e = P.seg[qi];
  const int x = (int)blockIdx.x % P.seg_X;  // this CTA's tile pair within its team
  Item I = decode_item(P, (int)e.group * P.seg_X + x);
  I.t0 = e.t0;
  I.t1 = e.t1;
  I.n_ctx_it = e.t1 - e.t0;
  if (e.piece + 1 != e.npieces) I.n_tail = 0;  // the tail tiles go with the last piece
  I.n_iter = I.n_ctx_it + I.n_tail;
  I.split = e.piece;
  I.npieces = e.npieces;
  I.slot0 = (int)e.slot0 * P.seg_X + x * e.npieces;
  I.slot = I.slot0 + e.piece;
  return I;
}

// Merge of the KV pieces of an item: rows [row_begin, row_begin + n_rows) of the item's 256 (two tiles of 128; n_rows
// divides 256).  Every piece has left its unnormalised rows and (max, sum) in its scratch slot (slot0 + piece); the caller
// has made them visible.  A thread owns one row (its weights are worked out once) and walks over that row's 16-column
// parts.  kNp = compile-time bound on the pieces (2, 4 or 8): every loop over pieces is fully unrolled and predicated, so
// the loads of a part (of two parts when kNp = 2) are all in flight together.
template <int D, int kNp>
__device__ __forceinline__ void merge_pieces_n(const TcParams &P, const Item &I, int np, int row_begin, int n_rows, int tid) {
  const AttnParams &A = P.a;
  const float c = P.c_log2;
  const size_t slot0 = (size_t)I.slot0;
  constexpr int kParts = D / 16;
  constexpr int kUnroll = kNp == 2 ? 2 : 1;  // parts whose loads are in flight together
  const int R = row_begin + tid % n_rows;
  const int t = R >> 7, r = R & 127;
  const uint32_t geo = tile_geo(I, t);
  const int ji = geo_ji0(geo) + (r >> geo_hs(geo));
  if (t >= I.ntq || ji >= P.n_rows) return;
  const int h = I.g * A.G + geo_h0(geo) + (r & ((1 << geo_hs(geo)) - 1));
  const size_t orow = ((size_t)I.n * A.q_req_rows + A.lo * A.Bq + ji) * A.Hq + h;
  // weights of the pieces for this row: exp2((m_piece - m) c) / sum; a piece without visible keys wrote no rows (its slot
  // may hold anything) and gets weight 0
  float2 ml[kNp];
#pragma unroll
  for (int sp = 0; sp < kNp; ++sp)
    ml[sp] = sp < np ? __ldcg(P.part_ml + ((slot0 + sp) * 2 + t) * 128 + r) : make_float2(-INFINITY, 0.f);
  float mmax = -INFINITY, lsum = 0.f, wgt[kNp];
#pragma unroll
  for (int sp = 0; sp < kNp; ++sp) if (ml[sp].y > 0.f) mmax = fmaxf(mmax, ml[sp].x);
#pragma unroll
  for (int sp = 0; sp < kNp; ++sp) {
    wgt[sp] = ml[sp].y > 0.f ? ex2((ml[sp].x - mmax) * c) : 0.f;
    lsum = fmaf(wgt[sp], ml[sp].y, lsum);
  }
  const float inv = lsum > 0.f ? 1.0f / lsum : 0.f;
#pragma unroll
  for (int sp = 0; sp < kNp; ++sp) wgt[sp] *= inv;
  const int step = 256 / n_rows;
  const float4 *po = reinterpret_cast<const float4 *>(P.part_o) + ((slot0 * 2 + t) * (D / 4)) * 128 + r;
  constexpr size_t kPieceStride = (size_t)2 * (D / 4) * 128;  // float4 from one piece's tile to the next piece's
  for (int part0 = tid / n_rows; part0 < kParts; part0 += step * kUnroll) {
    float4 x[kUnroll][kNp < 4 ? kNp : 4][4];
    float acc[kUnroll][16];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u)
#pragma unroll
      for (int e = 0; e < 16; ++e) acc[u][e] = 0.f;
#pragma unroll
    for (int sp0 = 0; sp0 < kNp; sp0 += 4) {
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int part = part0 + u * step;
#pragma unroll
        for (int q = 0; q < (kNp < 4 ? kNp : 4); ++q)
#pragma unroll
          for (int v = 0; v < 4; ++v)
            x[u][q][v] = (sp0 + q < np && part < kParts) ? __ldcg(po + (size_t)(sp0 + q) * kPieceStride + (size_t)(part * 4 + v) * 128)
                                                        : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u)
#pragma unroll
        for (int q = 0; q < (kNp < 4 ? kNp : 4); ++q) {
          const float w = wgt[sp0 + q];   // 0 for a piece that does not exist or saw no key: its (undefined) rows are not read above or weigh nothing
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            if (w > 0.f) {
              acc[u][4 * v] = fmaf(w, x[u][q][v].x, acc[u][4 * v]);
              acc[u][4 * v + 1] = fmaf(w, x[u][q][v].y, acc[u][4 * v + 1]);
              acc[u][4 * v + 2] = fmaf(w, x[u][q][v].z, acc[u][4 * v + 2]);
              acc[u][4 * v + 3] = fmaf(w, x[u][q][v].w, acc[u][4 * v + 3]);
            }
          }
        }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int part = part0 + u * step;
      if (part >= kParts) break;
      if (A.out_f32) {
        float4 *dst = reinterpret_cast<float4 *>(static_cast<float *>(A.out) + orow * D + part * 16);
#pragma unroll
        for (int v = 0; v < 4; ++v) dst[v] = make_float4(acc[u][4 * v], acc[u][4 * v + 1], acc[u][4 * v + 2], acc[u][4 * v + 3]);
      } else {
        uint4 *dst = reinterpret_cast<uint4 *>(static_cast<uint16_t *>(A.out) + orow * D + part * 16);
#pragma unroll
        for (int v = 0; v < 2; ++v)
          dst[v] = make_uint4(pack_bf16(acc[u][8 * v], acc[u][8 * v + 1]), pack_bf16(acc[u][8 * v + 2], acc[u][8 * v + 3]),
                              pack_bf16(acc[u][8 * v + 4], acc[u][8 * v + 5]), pack_bf16(acc[u][8 * v + 6], acc[u][8 * v + 7]));
      }
    }
  }
  if (A.out_lse && tid / n_rows == 0) A.out_lse[orow] = lsum > 0.f ? (mmax * c + log2f(lsum)) * 0.6931471805599453f : -INFINITY;
}

template <int D>
__device__ __forceinline__ void merge_pieces(const TcParams &P, const Item &I, int np, int row_begin, int n_rows, int tid) {
  if (np <= 2) merge_pieces_n<D, 2>(P, I, np, row_begin, n_rows, tid);
  else if (np <= 4) merge_pieces_n<D, 4>(P, I, np, row_begin, n_rows, tid);
  else merge_pieces_n<D, 8>(P, I, np, row_begin, n_rows, tid);
}

// Persistent kernel: CTA c works through items c, c + gridDim.x, ... of the (longest request first) item
// list; barrier phases and the K/V slot ring run on across items, so the producer already streams the next
// item's Q/K/V while the softmax warps write the previous item's output.
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
  uint64_t *kv_full = bars, *kv_empty = bars + kSlots, *q_full = bars + 2 * kSlots, *q_empty = q_full + 1, *s_full = q_full + 2,
           *p_full = q_full + 4, *pv_done = q_full + 6, *sf_a = q_full + 8, *sf_b = q_full + 9;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(q_full + 10);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  volatile int *merge_flag = reinterpret_cast<volatile int *>(tmem_slot + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // this CTA's items: its slice of the host-built schedule, else items blockIdx.x, blockIdx.x + gridDim.x, ...
  const int team = P.use_seg ? (int)blockIdx.x / P.seg_X : 0;  // (CTAs behind the last whole team have no work)
  const int q_begin = P.use_seg ? (team < P.seg_teams ? (int)P.team_first[team] : 0) : (P.use_sched ? (int)P.cta_first[blockIdx.x] : (int)blockIdx.x);
  const int q_end = P.use_seg ? (team < P.seg_teams ? (int)P.team_first[team + 1] : 0) : (P.use_sched ? (int)P.cta_first[blockIdx.x + 1] : P.n_items);
  const int q_step = (P.use_seg || P.use_sched) ? 1 : (int)gridDim.x;
  pdl_wait();  // nothing above touches global memory
  pdl_launch_dependents();
  // (a CTA of a cluster must not leave early: its peers meet it at the cluster barriers below)
  if (P.nsplit == 1 && A.status_word && (*reinterpret_cast<volatile int32_t *>(A.status_word) & (int32_t)DPARA_STATUS_TIMEOUT)) return;

  if (threadIdx.x == 0) {
    // K/V slots and the Q buffer are released by BOTH MMA issuers
    for (int s = 0; s < kSlots; ++s) { mbar_init(kv_full + s, 1); mbar_init(kv_empty + s, 2); }
    mbar_init(q_full, 1);
    mbar_init(q_empty, 2);
    for (int t = 0; t < 2; ++t) { mbar_init(s_full + t, 1); mbar_init(p_full + t, 4); mbar_init(pv_done + t, 1); }
    // S hand-off: sf_a is waited for by tile 0's issuer only, sf_b by tile 1's only (one waiter per barrier, so
    // every phase is consumed in order); the softmax warps arrive on the one the NEXT user of S waits for
    mbar_init(sf_a, 4);
    mbar_init(sf_b, 4);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 9) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  // register budget: the softmax warpgroups need the registers (a 128-wide score row per thread), the
  // producer / MMA warpgroup almost none
  if (warp >= 8) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 96;");
  if (warp == 8) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      prefetch_tensormap(&P.map_q[0]);
    }
    int ld = 0, k = 0;  // running K/V load counter, processed-item counter
    bool ok = true;
    for (int qi = q_begin; qi < q_end && ok; qi += q_step) {
      const Item I = fetch_item(P, qi);
      if (I.n_iter == 0) continue;
      // the Q buffer is free once the previous item's last QK has completed
      ok = __all_sync(0xffffffffu, mbar_wait(q_empty, (k & 1) ^ 1u, abort_flag));
      if (!ok) break;
      if (lane == 0) {
        const int qrow0 = I.n * A.q_req_rows + A.lo * A.Bq;
        mbar_arrive_expect_tx(q_full, (uint32_t)(I.ntq * Cfg::kTileBytes));
        for (int t = 0; t < I.ntq; ++t) {
          const uint32_t geo = tile_geo(I, t);
          for (int sb = 0; sb < Cfg::kSlabs; ++sb)
            tma_load_3d(sQ + t * Cfg::kTileBytes + sb * Cfg::kSlabBytes, &P.map_q[geo_blk(geo)], q_full, sb * 64, I.g * A.G + geo_h0(geo),
                        qrow0 + geo_ji0(geo));
        }
      }
      // load order K0 K1 V0 K2 V1 ... K(n-1) V(n-2) V(n-1): the order the MMA issuer consumes them in
      // (the scores of iteration it + 1 are issued before the PV product of iteration it); slot = (ld + q) % kSlots
      for (int q = 0; q < 2 * I.n_iter; ++q) {
        const bool is_v = q > 0 && (((q & 1) == 0) || ((q + 1) >> 1) >= I.n_iter);
        const int it = q == 0 ? 0 : (is_v ? ((q & 1) ? I.n_iter - 1 : (q >> 1) - 1) : (q + 1) >> 1);
        const int sl = (ld + q) % kSlots;
        const uint32_t ph = ((ld + q) / kSlots) & 1;
        ok = __all_sync(0xffffffffu, mbar_wait(kv_empty + sl, ph ^ 1u, abort_flag));
        if (!ok) break;
        uint8_t *dst = sKV + sl * Cfg::kTileBytes;
        if (it < I.n_ctx_it) {
          if (lane == 0) {
            const int row = (int)(I.c0 + (long long)(I.t0 + it) * 128);
            mbar_arrive_expect_tx(kv_full + sl, Cfg::kTileBytes);
            for (int sb = 0; sb < Cfg::kSlabs; ++sb)
              tma_load_3d(dst + sb * Cfg::kSlabBytes, is_v ? &P.map_vc : &P.map_kc, kv_full + sl, sb * 64, I.g, row);
          }
        } else {
          if (is_v) {
            // tail tile: rows the TMA boxes do not cover must still hold finite V (P = 0 there): clear the V tile
            for (int o = lane * 16; o < Cfg::kTileBytes; o += 32 * 16) *reinterpret_cast<uint4 *>(dst + o) = make_uint4(0, 0, 0, 0);
            fence_proxy_async();
            __syncwarp();
          }
          if (lane == 0) {
            const int tk = it - I.n_ctx_it;  // tail tile 0: spine rows, then cap0 blocks; tail tile k >= 1: cap blocks
            if (tk == 0) {
              uint32_t bytes = 0;
              if (A.S > 0) bytes += (uint32_t)A.S * 128 * Cfg::kSlabs;
              if (P.has_blk) bytes += (uint32_t)(P.cap0 * A.Bq) * 128 * Cfg::kSlabs;
              mbar_arrive_expect_tx(kv_full + sl, bytes);
              for (int sb = 0; sb < Cfg::kSlabs; ++sb) {
                if (A.S > 0) tma_load_3d(dst + sb * Cfg::kSlabBytes, is_v ? &P.map_vs : &P.map_ks, kv_full + sl, sb * 64, I.g, I.n * A.spine_req_rows);
                if (P.has_blk)
                  tma_load_3d(dst + sb * Cfg::kSlabBytes + P.S8 * 128, is_v ? &P.map_vb0 : &P.map_kb0, kv_full + sl, sb * 64, I.g,
                              I.n * A.blk_req_rows + I.jb0 * A.Bq);
              }
            } else {
              mbar_arrive_expect_tx(kv_full + sl, (uint32_t)(P.cap * A.Bq) * 128 * Cfg::kSlabs);
              for (int sb = 0; sb < Cfg::kSlabs; ++sb)
                tma_load_3d(dst + sb * Cfg::kSlabBytes, is_v ? &P.map_vb : &P.map_kb, kv_full + sl, sb * 64, I.g,
                            I.n * A.blk_req_rows + (I.jb0 + P.cap0 + (tk - 1) * P.cap) * A.Bq);
            }
          }
        }
      }
      ld += 2 * I.n_iter;
      ++k;
    }
  } else if (warp == 9 || warp == 10) {
    // ------------------------------------------------------------------ MMA issuers: warp 9 for tile 0, warp 10 for tile 1
    // One issuing thread per query tile.  A tcgen05.mma block issued into a drained pipe pays a start-up latency
    // and the issuing thread spends the block's whole execution time issuing it (the queue is shallow); with
    // one thread per tile, one tile's waits and commits overlap the other tile's products and the tensor pipe
    // stays fed.  The two threads meet only through barriers (the S hand-off below, the K/V ring).
    if (lane == 0) {
      const int ti = warp - 9;
      constexpr uint32_t idesc_qk = idesc_bf16_f32(128, 128, false, false);
      constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, false, true);
      constexpr uint32_t kTile16 = Cfg::kTileBytes >> 4;
      const uint64_t qdesc = smem_desc_sw128(smem_u32(sQ) + ti * Cfg::kTileBytes, 16, 1024);
      const uint64_t kdesc0 = smem_desc_sw128(smem_u32(sKV), 16, 1024);                 // K tile: K-major operand
      const uint64_t vdesc0 = smem_desc_sw128(smem_u32(sKV), Cfg::kSlabBytes, 1024);    // V tile: MN-major operand
      const uint32_t s_t = tmem + Cfg::kColS, o_t = tmem + Cfg::kColO + ti * 128, p_t = tmem + Cfg::kColP + ti * 64;
      uint64_t *sf = ti == 0 ? sf_a : sf_b;
      int ring_slot = 0, k = 0;
      uint32_t ring_phase = 0, ph_p = 0, ph_sf = 0;
      bool ok = true, first_qk = (ti == 0);
      auto next_load = [&](int &slot_out) {  // wait for the next tile of the K/V ring (both issuers take every tile, in order)
        slot_out = ring_slot;
        const bool r = mbar_wait(kv_full + ring_slot, ring_phase, abort_flag, 2);
        if (++ring_slot == kSlots) { ring_slot = 0; ring_phase ^= 1u; }
        return r;
      };
      // The S buffer comes back from whichever tile's softmax warps loaded it last (also across items).
      auto wait_s_free = [&]() {
        if (first_qk) { first_qk = false; return true; }
        const bool r = mbar_wait(sf, ph_sf, abort_flag, 3);
        ph_sf ^= 1u;
        return r;
      };
      auto issue_qk = [&](int kslot, bool last_it) {
        const uint64_t ka = kdesc0 + (uint64_t)(kslot * kTile16);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = ((kk >> 2) * Cfg::kSlabBytes + (kk & 3) * 32) >> 4;
          if (kk == 0) mma_ss_c<false>(s_t, qdesc + off, ka + off, idesc_qk);
          else mma_ss_c<true>(s_t, qdesc + off, ka + off, idesc_qk);
        }
        mma_commit(s_full + ti);
        mma_commit(kv_empty + kslot);        // this tile is done with the K tile
        if (last_it) mma_commit(q_empty);    // ... and with its Q tile
      };
      auto issue_pv = [&](int vslot, bool acc) {
        const uint64_t va = vdesc0 + (uint64_t)(vslot * kTile16);
        mma_ts(o_t, p_t, va, idesc_pv, acc);
#pragma unroll
        for (int kk = 1; kk < 8; ++kk) mma_ts_c<true>(o_t, p_t + kk * 8, va + (uint64_t)(kk * (2048 >> 4)), idesc_pv);
        mma_commit(pv_done + ti);
        mma_commit(kv_empty + vslot);
      };
      for (int qi = q_begin; qi < q_end && ok; qi += q_step) {
      const Item I = fetch_item(P, qi);
        if (I.n_iter == 0) continue;
        const int n_iter = I.n_iter;
        int kslot = 0, vslot = 0;
        ok = mbar_wait(q_full, k & 1, abort_flag, 4);
        ++k;
        if (!ok) break;
        if (ti >= I.ntq) {
          // no second tile in this item: keep the ring and Q-buffer protocols in step (a slot is released only
          // after its load has landed, so this thread cannot run ahead of the other issuer by a ring cycle)
          for (int q = 0; q < 2 * n_iter && ok; ++q) {
            ok = next_load(kslot);
            if (ok) mbar_arrive(kv_empty + kslot);
          }
          if (ok) mbar_arrive(q_empty);
          continue;
        }
        // per iteration: QK(it + 1), then PV(it) -- the scores of the next iteration are issued as soon as
        // the S buffer and the K tile are there, the PV product when this tile's softmax has written P
        ok = next_load(kslot) && wait_s_free();
        if (!ok) break;
        tc_fence_after();
        issue_qk(kslot, n_iter == 1);
        for (int it = 0; it < n_iter && ok; ++it) {
          if (it + 1 < n_iter) {
            ok = next_load(kslot) && wait_s_free();
            if (!ok) break;
            tc_fence_after();
            issue_qk(kslot, it + 2 == n_iter);
          }
          ok = next_load(vslot) && mbar_wait(p_full + ti, ph_p, abort_flag, 5);
          ph_p ^= 1u;
          if (!ok) break;
          tc_fence_after();
          issue_pv(vslot, it > 0);
        }
      }
    }
  }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue: thread = row
    asm volatile("setmaxnreg.inc.sync.aligned.u32 200;");
    const int t = warp >> 2;
    const int wq = warp & 3;
    const int r = wq * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(wq * 32) << 16);
    const float c = P.c_log2;
    const float thr = kRescaleLog2 / c;
    int cnt = 0;  // iterations this tile's barriers have been through
    uint32_t ph_pv = 0;  // pv_done[t] completes once per (item, iteration); every phase is waited for exactly once, in order
    bool ok = true;
    for (int qi = q_begin; qi < q_end && ok; qi += q_step) {
      // ---- what the iteration loop needs, in as few registers as possible (the score row takes 128 of them); the item
      // is decoded again after the loop for the output addresses
      int n_iter, n_ctx_it, ragged_nv, jrel, na_row;
      bool two_tiles, skip;
      {
        const Item I = fetch_item(P, qi);
        skip = I.n_iter == 0 || t >= I.ntq;  // nothing visible to this work item, or no second tile in the last pair
        n_iter = skip ? 0 : I.n_iter;
        n_ctx_it = I.n_ctx_it;
        two_tiles = I.ntq == 2;
        ragged_nv = (I.t1 == I.nctx) ? (I.L & 127) : 0;  // valid keys of a part-filled last context tile (0: it is full or not ours)
        // a mask-slot row: its boundary, counted from the first one whose block sits in the tail tiles, and its anchor
        // prefix; a spine row (an anchor as a query): no own block (-1), and anchors 0 .. itself
        const int ji = geo_ji0(tile_geo(I, t)) + (r >> geo_hs(tile_geo(I, t)));
        const bool is_spine = ji >= P.n_ji;
        jrel = is_spine ? -1 : A.lo + ji / A.Bq - I.jb0;
        na_row = is_spine ? ji - P.n_ji + 1 : max(0, min(A.lo + ji / A.Bq + A.pb, A.S));
      }
      float m_used = -INFINITY, l = 0.f;

      for (int it = 0; it < n_iter; ++it) {
        // tail tile tk: the anchor prefix sits in tile 0; this row's own block in tile kt at key rows [boff, boff + Bq)
        // (worked out before the score row occupies the registers)
        // The visible keys of the tile as a 128-bit mask (four words), so that masking a score is one bit test.
        uint32_t vis[4] = {0u, 0u, 0u, 0u};
        if (it >= n_ctx_it) {
          const int tk = it - n_ctx_it;
          const int kt = (!P.has_blk || jrel < 0) ? -1 : (jrel < P.cap0 ? 0 : 1 + (jrel - P.cap0) / P.cap);
          const int boff = jrel < P.cap0 ? P.S8 + jrel * A.Bq : ((jrel - P.cap0) % P.cap) * A.Bq;
          const int na_t = tk == 0 ? na_row : 0;
          const int b0 = tk == kt ? boff : 0, b1 = tk == kt ? boff + A.Bq : 0;
#pragma unroll
          for (int w = 0; w < 4; ++w) vis[w] = bits_below(na_t - 32 * w) | (bits_below(b1 - 32 * w) & ~bits_below(b0 - 32 * w));
        }
        ok = __all_sync(0xffffffffu, mbar_wait(s_full + t, (cnt + it) & 1, abort_flag, 6));
        if (!ok) break;
        tc_fence_after();
        uint32_t su[128];
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) tmem_ld32(lane_addr + Cfg::kColS + cc * 32, su + cc * 32);
        tmem_wait_ld();
        // the scores are in registers: hand the S buffer to the next QK product
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive((t == 0 && two_tiles) ? sf_b : sf_a);  // next user: tile 1 of this iteration, else tile 0
        bool pv_waited = (it == 0);  // PV(t, it-1) must be complete before O_t is rescaled or P_t overwritten
        float s[128];
#pragma unroll
        for (int kx = 0; kx < 128; ++kx) s[kx] = __uint_as_float(su[kx]);
        if (it >= n_ctx_it) {
#pragma unroll
          for (int kx = 0; kx < 128; ++kx) s[kx] = ((vis[kx >> 5] >> (kx & 31)) & 1u) ? s[kx] : -INFINITY;
        } else if (it == n_ctx_it - 1 && ragged_nv) {
          const int nv = ragged_nv;
#pragma unroll
          for (int kx = 0; kx < 128; ++kx) s[kx] = kx < nv ? s[kx] : -INFINITY;
        }
        float mxa = fmaxf(s[0], s[1]), mxb = fmaxf(s[2], s[3]), mxc = fmaxf(s[4], s[5]), mxd = fmaxf(s[6], s[7]);
#pragma unroll
        for (int kx = 8; kx < 128; kx += 8) {  // four independent chains
          mxa = max3(mxa, s[kx], s[kx + 1]);
          mxb = max3(mxb, s[kx + 2], s[kx + 3]);
          mxc = max3(mxc, s[kx + 4], s[kx + 5]);
          mxd = max3(mxd, s[kx + 6], s[kx + 7]);
        }
        const float mx = fmaxf(fmaxf(mxa, mxb), fmaxf(mxc, mxd));
        const bool need = mx > m_used + thr;  // also true when m_used = -inf and the tile has a visible key
        if (it == 0) {
          if (need) m_used = mx;
        } else if (__any_sync(0xffffffffu, need)) {
          ok = __all_sync(0xffffffffu, mbar_wait(pv_done + t, ph_pv, abort_flag, 7));
          ph_pv ^= 1u;
          pv_waited = true;
          if (!ok) break;
          tc_fence_after();
          const float f = need ? ex2((m_used - mx) * c) : 1.0f;
#pragma unroll 1
          for (int cc = 0; cc < D / 32; ++cc) {
            uint32_t o[32];
            tmem_ld32(lane_addr + Cfg::kColO + t * 128 + cc * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int kx = 0; kx < 32; ++kx) o[kx] = __float_as_uint(__uint_as_float(o[kx]) * f);
            tmem_st32(lane_addr + Cfg::kColO + t * 128 + cc * 32, o);
          }
          tmem_wait_st();
          l *= f;
          if (need) m_used = mx;
        }
        const float mc = (m_used == -INFINITY ? 0.f : m_used) * c;
        uint32_t pk[64];
        {
          // packed fp32x2 scale/shift and row sum (half the FMA/ADD issue slots of the scalar form)
          const uint64_t c2 = pack2(c, c), nmc2 = pack2(-mc, -mc);
          uint64_t l2 = pack2(0.f, 0.f);
#pragma unroll
          for (int kx = 0; kx < 64; ++kx) {
            float x0, x1;
            unpack2(fma2(pack2(s[2 * kx], s[2 * kx + 1]), c2, nmc2), x0, x1);
            const float p0 = ex2(x0), p1 = ex2(x1);
            l2 = add2(l2, pack2(p0, p1));
            pk[kx] = pack_bf16(p0, p1);
          }
          float la, lb;
          unpack2(l2, la, lb);
          l += la + lb;
        }
        if (!pv_waited) {
          ok = __all_sync(0xffffffffu, mbar_wait(pv_done + t, ph_pv, abort_flag, 8));
          ph_pv ^= 1u;
          if (!ok) break;
          tc_fence_after();
        }
        tmem_st32(lane_addr + Cfg::kColP + t * 64, pk);
        tmem_st32(lane_addr + Cfg::kColP + t * 64 + 32, pk + 32);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(p_full + t);
      }

      // ---- output of this item (the MMA issuer cannot touch O_t again before this tile's next p_full arrive)
      if (!ok) break;
      const Item I = fetch_item(P, qi);
      const uint32_t geo = tile_geo(I, t);
      const int ji = geo_ji0(geo) + (r >> geo_hs(geo));
      const bool valid = (t < I.ntq) && (ji < P.n_rows);
      const int h = I.g * A.G + geo_h0(geo) + (r & ((1 << geo_hs(geo)) - 1));
      const size_t orow = ((size_t)I.n * A.q_req_rows + A.lo * A.Bq + ji) * A.Hq + h;
      // split-KV: this CTA's partial rows go to an L2-resident scratch slot and are merged later
      const size_t pslot = ((size_t)I.slot * 2 + t) * 128 + r;
      const bool partial = I.npieces > 1;  // one KV piece of several: unnormalised rows to scratch
      if (skip) {
        if (partial) {
          __stcg(P.part_ml + pslot, make_float2(-INFINITY, 0.f));
        } else if (valid) {
          for (int d = 0; d < D; ++d) {
            if (A.out_f32) static_cast<float *>(A.out)[orow * D + d] = 0.f;
            else static_cast<uint16_t *>(A.out)[orow * D + d] = 0;
          }
          if (A.out_lse) A.out_lse[orow] = -INFINITY;
        }
        continue;
      }
      ok = __all_sync(0xffffffffu, mbar_wait(pv_done + t, ph_pv, abort_flag, 9));
      ph_pv ^= 1u;
      if (!ok) break;
      tc_fence_after();
      const float inv = l > 0.f ? 1.0f / l : 0.f;
      // output rows of the four lanes of this thread's quad (all ones: no such row)
      size_t qrow[4];
#pragma unroll
      for (int v = 0; v < 4; ++v)
        qrow[v] = (size_t)__shfl_sync(0xffffffffu, valid ? (unsigned long long)orow : ~0ull, (lane & ~3) + v);
#pragma unroll 1
      for (int cc = 0; cc < D / 32; ++cc) {
        uint32_t o[32];
        tmem_ld32(lane_addr + Cfg::kColO + t * 128 + cc * 32, o);
        tmem_wait_ld();
        if (partial) {
          float4 *dst = reinterpret_cast<float4 *>(P.part_o) + (((size_t)I.slot * 2 + t) * (D / 4) + cc * 8) * 128 + r;
#pragma unroll
          for (int v = 0; v < 8; ++v)
            __stcg(dst + v * 128, make_float4(__uint_as_float(o[4 * v]), __uint_as_float(o[4 * v + 1]), __uint_as_float(o[4 * v + 2]),
                                        __uint_as_float(o[4 * v + 3])));
        } else if (valid) {
          if (A.out_f32) {
            float4 *dst = reinterpret_cast<float4 *>(static_cast<float *>(A.out) + orow * D + cc * 32);
#pragma unroll
            for (int v = 0; v < 8; ++v)
              dst[v] = make_float4(__uint_as_float(o[4 * v]) * inv, __uint_as_float(o[4 * v + 1]) * inv,
                                   __uint_as_float(o[4 * v + 2]) * inv, __uint_as_float(o[4 * v + 3]) * inv);
          }
        }
        if (!partial && !A.out_f32) {
          // bf16 output: the thread's 32 columns are four 16-byte pieces of its row.  Written as they are, one store
          // instruction of a warp touches 32 rows (32 partial sectors).  The four lanes of a quad swap pieces (a 4 x 4
          // transpose by two butterfly steps) so that store v of a quad is 64 contiguous bytes of row 4q + v.
          uint4 x[4];
#pragma unroll
          for (int v = 0; v < 4; ++v)
            x[v] = make_uint4(pack_bf16(__uint_as_float(o[8 * v]) * inv, __uint_as_float(o[8 * v + 1]) * inv),
                              pack_bf16(__uint_as_float(o[8 * v + 2]) * inv, __uint_as_float(o[8 * v + 3]) * inv),
                              pack_bf16(__uint_as_float(o[8 * v + 4]) * inv, __uint_as_float(o[8 * v + 5]) * inv),
                              pack_bf16(__uint_as_float(o[8 * v + 6]) * inv, __uint_as_float(o[8 * v + 7]) * inv));
          quad_transpose(x, lane);
#pragma unroll
          for (int v = 0; v < 4; ++v)
            if (qrow[v] != ~size_t(0))
              *reinterpret_cast<uint4 *>(static_cast<uint16_t *>(A.out) + qrow[v] * D + cc * 32 + (lane & 3) * 8) = x[v];
        }
      }
      tc_fence_before();  // the O_t reads above are ordered before this warp's next p_full arrive
      if (partial) {
        __stcg(P.part_ml + pslot, make_float2(m_used, l));
      } else if (valid && A.out_lse) {
        A.out_lse[orow] = l > 0.f ? (m_used * c + log2f(l)) * 0.6931471805599453f : -INFINITY;
      }
      cnt += n_iter;
    }
  }

  // ------------------------------------------------------------------ split-KV merge across the cluster
  // The nsplit CTAs that share (request, KV head, tile pair) form one thread-block cluster.  Each has written
  // its unnormalised rows and (max, sum) to its scratch slot (which stays in L2); after a cluster barrier CTA
  // `rank` merges 256 / nsplit of the rows from all peers' slots and writes the final output.  No second launch.
  if (P.nsplit > 1) {
    __threadfence();
    __syncwarp();
    cluster_sync_all();
    if (warp < 8 && !*abort_flag) {
      const Item I = decode_item(P, blockIdx.x);
      const uint32_t rank = cluster_ctarank();
      const int rows_per = I.ntq * 128 / P.nsplit;  // the item's rows (one tile or two), shared out over the cluster
      merge_pieces<D>(P, I, P.nsplit, (int)rank * rows_per, rows_per, threadIdx.x);
    }
  }

  // ------------------------------------------------------------------ cut schedule: tickets and merges
  if (P.use_seg && q_end > q_begin) {
    // The pieces written early in the kernel have long left L2 (the K/V stream passed through it since): ask for every
    // cut item's scratch rows now, so that a merge finds them in L2 instead of paying an HBM round trip per dependent load.
    for (int qi = q_begin; qi < q_end; ++qi) {
      const Item I = fetch_item(P, qi);
      if (I.npieces <= 1) continue;
      const char *base = reinterpret_cast<const char *>(P.part_o) + (size_t)I.slot0 * 2 * 128 * D * 4;
      const int lines = I.npieces * 2 * 128 * D * 4 / 128;
      for (int k = threadIdx.x; k < lines; k += kThreads) prefetch_l2(base + (size_t)k * 128);
      if (threadIdx.x < I.npieces * 2 * 8) prefetch_l2(reinterpret_cast<const char *>(P.part_ml + (size_t)I.slot0 * 2 * 128) + threadIdx.x * 128);
    }
    __threadfence();
    __syncthreads();  // every partial row of this CTA is written
    for (int qi = q_begin; qi < q_end; ++qi) {
      const Item I = fetch_item(P, qi);
      if (I.npieces <= 1) continue;
      if (threadIdx.x == 0) *merge_flag = !*abort_flag && atomicAdd(P.seg_count + I.item, 1u) == (unsigned)I.npieces - 1u;
      __syncthreads();
      if (*merge_flag && warp < 8) {
        __threadfence();
        merge_pieces<D>(P, I, I.npieces, 0, 256, threadIdx.x);
      }
      __syncthreads();
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

// ------------------------------------------------------------------------------------------------ host
// Clusters of `size` CTAs of this kernel that the device runs at the same time (one CTA per SM, a cluster inside one
// GPC: fewer than SMs / size).  Asked once per (head dim, size); without a device, a careful guess.
static int max_active_clusters(int D, int size) {
  static std::mutex mu;
  static int cached[2][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}};
  const int di = D == 128 ? 1 : 0, si = size == 8 ? 3 : (size == 4 ? 2 : (size == 2 ? 1 : 0));
  std::lock_guard<std::mutex> lock(mu);
  if (cached[di][si] > 0) return cached[di][si];
  int n = 0;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  cfg.gridDim = dim3(size * kNumSM);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = D == 128 ? TcCfg<128>::kSmemBytes : TcCfg<64>::kSmemBytes;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = size; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  cudaError_t e = D == 128 ? cudaFuncSetAttribute(attn_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cfg.dynamicSmemBytes)
                           : cudaFuncSetAttribute(attn_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cfg.dynamicSmemBytes);
  if (e == cudaSuccess)
    e = D == 128 ? cudaOccupancyMaxActiveClusters(&n, attn_tc_kernel<128>, &cfg) : cudaOccupancyMaxActiveClusters(&n, attn_tc_kernel<64>, &cfg);
  if (e != cudaSuccess || n <= 0) {
    cudaGetLastError();
    return (kNumSM * 3 / 4) / size;   // not cached: a later call with a device asks again
  }
  cached[di][si] = n;
  return n;
}

TcPlan plan_attention_tc(const dpara_shape *s, const int64_t *host_off, const int64_t *host_lens) {
  auto len_of = [&](int n) { return host_lens ? host_lens[n] : host_off[n + 1] - host_off[n]; };
  TcPlan p{};
  const int G = s->n_q_heads / s->n_kv_heads;
  const int nb = s->boundary_hi - s->boundary_lo;
  if (nb <= 0) return p;
  if (G > 16 || s->n_spine > 64 || s->block > 64) return p;
  p.n_ji = nb * s->block;
  p.n_rows = p.n_ji + (s->spine_queries ? s->n_spine : 0);
  // head blocks = binary digits of G, widest first; block k's tiles hold 128 / hb (j, i) rows
  auto lay_out_items = [&](int tiles_per_item) {
    p.tiles_per_item = tiles_per_item;
    p.n_hblk = 0;
    p.n_pairs = 0;
    int n_odd = 0;
    for (int bit = 4, h0 = 0; bit >= 0; --bit) {
      if (!(G & (1 << bit))) continue;
      const int ji_t = 128 >> bit, tiles = (p.n_rows + ji_t - 1) / ji_t;
      p.hb_log2[p.n_hblk] = bit;
      p.h0[p.n_hblk] = h0;
      p.pair_start[p.n_hblk] = p.n_pairs;
      p.n_pairs += tiles / tiles_per_item;
      n_odd += tiles_per_item == 2 ? (tiles & 1) : 0;
      h0 += 1 << bit;
      ++p.n_hblk;
    }
    p.pair_start[p.n_hblk] = p.n_pairs;
    p.n_pairs += (n_odd + 1) / 2;   // the blocks' odd last tiles, two by two
  };
  lay_out_items(2);
  p.S8 = (s->n_spine + 7) & ~7;
  p.cap = 128 / s->block;
  p.cap0 = (128 - p.S8) / s->block;  // >= 1: S8 <= 64 and block <= 64
  long long max_l = 0, tot = host_off[s->batch] - host_off[0];
  for (int n = 0; n < s->batch; ++n) max_l = len_of(n) > max_l ? len_of(n) : max_l;
  if (tot + 128 >= (1ll << 31) || (long long)s->batch * s->n_boundaries * s->block >= (1ll << 31)) return p;
  const int max_tiles = (int)((max_l + 127) / 128);
  // A small batch is latency-bound: when one-tile items with their splits still fit the GPU in a single wave, an item is
  // ONE query tile instead of two -- twice the CTAs, each with half the Q load, half the partial rows and half the merge
  int split_cap = 8;  // largest cluster size whose clusters all run at once
  long long items1 = 0;
  {
    const int pairs2 = p.n_pairs;
    lay_out_items(1);
    items1 = (long long)s->batch * s->n_kv_heads * p.n_pairs;
    int split1 = 0;
    for (int c = 8; c >= 2 && !split1; c >>= 1)
      if (c <= max_tiles && items1 <= max_active_clusters(s->head_dim, c)) split1 = c;
    if (p.n_pairs == pairs2 || items1 >= 96 || split1 < 4) lay_out_items(2); else split_cap = split1;
  }
  const long long items = (long long)s->batch * s->n_kv_heads * p.n_pairs;
  // split the KV range over a cluster of 2, 4 or 8 CTAs when the batch alone cannot fill the GPU
  int nsplit = 1;
  if (items < 96 && max_tiles > 1) {
    const long long want = (kNumSM + items - 1) / items;
    for (int c = 8; c >= 2; c >>= 1)
      if (c <= want && c <= max_tiles && c <= split_cap) { nsplit = c; break; }
  }
  p.nsplit = nsplit;
  p.items = items;
  p.workspace_bytes = nsplit > 1 ? (size_t)items * nsplit * 256 * ((size_t)s->head_dim + 2) * 4 : 0;
  // (sized for the one-tile layout, the larger of the two: which layout is taken depends on how many clusters the device
  //  runs at once, and the size must not)
  p.workspace_max_bytes = items < 96 ? (size_t)std::max(items, items1) * 8 * 256 * ((size_t)s->head_dim + 2) * 4 : 0;
  // the cut schedule (items >= 96): at most two pieces per team and member plus seven per group of a degenerate cut,
  // bounded here by 2 * SMs piece slots; plus one ticket per item
  if (items >= 96 && p.n_pairs <= 16)
    p.workspace_max_bytes = (size_t)(2 * kNumSM) * 256 * ((size_t)s->head_dim + 2) * 4 + align_up((size_t)items * 4, 256);
  p.eligible = true;
  return p;
}

template <int D>
static dpara_status launch_tc_d(const TcParams &P, const TcPlan &plan, cudaStream_t st) {
  using Cfg = TcCfg<D>;
  if (cudaFuncSetAttribute(attn_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes) != cudaSuccess) return DPARA_ERR_CUDA;
  int dev = 0, sms = kNumSM;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = Cfg::kSmemBytes;
  cfg.stream = st;
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (P.nsplit > 1) {
    // one CTA per (item, split); the splits of an item are consecutive CTAs = one cluster
    cfg.gridDim = dim3(P.n_items);
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = P.nsplit;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  } else {
    cfg.gridDim = dim3(P.use_seg || P.n_items >= sms ? sms : P.n_items);  // persistent: at most one CTA per SM
  }
  if (cudaLaunchKernelEx(&cfg, attn_tc_kernel<D>, P) != cudaSuccess) {
    cudaGetLastError();
    return DPARA_ERR_CUDA;
  }
  count_launches(1);
  return DPARA_OK;
}

// The last host-built work schedule and the tile counts it was built for (guarded by the mutex; a pure function of
// the key, kept only to save host time on repeated shapes).
static std::mutex g_sched_mu;
static std::vector<int> g_sched_key;
static std::vector<uint16_t> g_sched_items;
static uint16_t g_sched_first[kNumSM + 1];

dpara_status launch_attention_tc(const AttnParams &A, const TcPlan &plan, const int64_t *host_off, const int64_t *host_lens,
                                 void *workspace, cudaStream_t st) {
  auto len_of = [&](int n) { return host_lens ? host_lens[n] : host_off[n + 1] - host_off[n]; };
  TcParams P;
  memset(&P, 0, sizeof(P));
  P.a = A;
  P.n_ji = plan.n_ji; P.n_rows = plan.n_rows; P.n_pairs = plan.n_pairs; P.nsplit = plan.nsplit;
  P.n_hblk = plan.n_hblk;
  for (int k = 0; k < plan.n_hblk; ++k) { P.hb_log2[k] = plan.hb_log2[k]; P.h0[k] = plan.h0[k]; }
  for (int k = 0; k <= plan.n_hblk; ++k) P.pair_start[k] = plan.pair_start[k];
  P.S8 = plan.S8; P.cap0 = plan.cap0; P.cap = plan.cap; P.has_blk = A.k_blk != nullptr;
  P.nsplit_log2 = plan.nsplit == 8 ? 3 : (plan.nsplit == 4 ? 2 : (plan.nsplit == 2 ? 1 : 0));
  P.has_tail = (A.S > 0) || P.has_blk;
  P.n_items = (int)(plan.items * plan.nsplit);
  {
    // the items of a (request, KV head): per head block its tiles two by two (or one by one); the odd last tiles of the
    // blocks, which all cover the highest (j, i) rows, are paired with one another
    struct Tile { int blk, idx; };
    std::vector<std::vector<Tile>> items;
    std::vector<Tile> odd;
    const int tpi = plan.tiles_per_item;
    for (int blk = 0; blk < plan.n_hblk; ++blk) {
      const int ji_t = 128 >> plan.hb_log2[blk], tiles = (plan.n_rows + ji_t - 1) / ji_t;
      for (int i = 0; i + tpi <= tiles; i += tpi) items.push_back(tpi == 2 ? std::vector<Tile>{{blk, i}, {blk, i + 1}} : std::vector<Tile>{{blk, i}});
      if (tpi == 2 && (tiles & 1)) odd.push_back({blk, tiles - 1});
    }
    for (size_t i = 0; i < odd.size(); i += 2) items.push_back(i + 1 < odd.size() ? std::vector<Tile>{odd[i], odd[i + 1]} : std::vector<Tile>{odd[i]});
    if ((int)items.size() != plan.n_pairs) return DPARA_ERR_INVALID_ARG;   // (plan and table disagree: cannot happen)
    for (int x = 0; x < plan.n_pairs; ++x) {
      TcParams::PairInfo &pi = P.pair[x];
      memset(&pi, 0, sizeof(pi));
      pi.ntq = (uint8_t)items[x].size();
      // boundaries whose own blocks the item's mask-slot rows need (none if it holds spine rows only)
      int jb_first = 1 << 30, jb_last = -1;
      for (int t = 0; t < pi.ntq; ++t) {
        const int blk = items[x][t].blk, ji_t = 128 >> plan.hb_log2[blk], ji0 = items[x][t].idx * ji_t;
        pi.ji0[t] = (int16_t)ji0;
        pi.blk[t] = (uint8_t)blk; pi.hs[t] = (uint8_t)plan.hb_log2[blk]; pi.h0[t] = (uint8_t)plan.h0[blk];
        const int ji_last = std::min(ji0 + ji_t, plan.n_ji) - 1;
        if (ji_last >= ji0) { jb_first = std::min(jb_first, ji0 / A.Bq); jb_last = std::max(jb_last, ji_last / A.Bq); }
      }
      pi.jb0_rel = (int16_t)(jb_last >= 0 ? jb_first : 0);
      pi.n_tail = (uint8_t)tail_tiles(P.has_tail, P.has_blk, jb_last >= 0 ? jb_last - jb_first + 1 : 0, plan.cap0, plan.cap);
    }
  }

  P.c_log2 = A.scale * 1.4426950408889634f;
  const int D = A.D;
  const uint64_t rs = (uint64_t)D * 2;
  const long long tot = host_off[A.b] - host_off[0];
  const uint64_t nq = (uint64_t)A.b * A.q_req_rows;
  const uint64_t n_blk_rows = (uint64_t)(A.b - 1) * A.blk_req_rows + (uint64_t)A.J * A.Bq;
  const uint64_t n_spine_rows = (uint64_t)(A.b - 1) * A.spine_req_rows + (uint64_t)A.S;
  bool ok = true;
  for (int k = 0; k < plan.n_hblk; ++k)
    ok = ok && make_tmap_bf16_3d(&P.map_q[k], A.q, D, A.Hq, nq, rs, rs * A.Hq, 64, 1u << plan.hb_log2[k], 128u >> plan.hb_log2[k]);
  if (tot > 0) {
    ok = ok && make_tmap_bf16_3d(&P.map_kc, A.k_ctx, D, A.Hkv, host_off[A.b], rs, rs * A.Hkv, 64, 1, 128);
    ok = ok && make_tmap_bf16_3d(&P.map_vc, A.v_ctx, D, A.Hkv, host_off[A.b], rs, rs * A.Hkv, 64, 1, 128);
  }
  if (A.S > 0) {
    ok = ok && make_tmap_bf16_3d(&P.map_ks, A.k_spine, D, A.Hkv, n_spine_rows, rs, rs * A.Hkv, 64, 1, A.S);
    ok = ok && make_tmap_bf16_3d(&P.map_vs, A.v_spine, D, A.Hkv, n_spine_rows, rs, rs * A.Hkv, 64, 1, A.S);
  }
  if (P.has_blk) {
    ok = ok && make_tmap_bf16_3d(&P.map_kb0, A.k_blk, D, A.Hkv, n_blk_rows, rs, rs * A.Hkv, 64, 1, plan.cap0 * A.Bq);
    ok = ok && make_tmap_bf16_3d(&P.map_vb0, A.v_blk, D, A.Hkv, n_blk_rows, rs, rs * A.Hkv, 64, 1, plan.cap0 * A.Bq);
    ok = ok && make_tmap_bf16_3d(&P.map_kb, A.k_blk, D, A.Hkv, n_blk_rows, rs, rs * A.Hkv, 64, 1, plan.cap * A.Bq);
    ok = ok && make_tmap_bf16_3d(&P.map_vb, A.v_blk, D, A.Hkv, n_blk_rows, rs, rs * A.Hkv, 64, 1, plan.cap * A.Bq);
  }
  if (!ok) return DPARA_ERR_CUDA;
  P.use_ctx_p = A.b <= kMaxOrdered;
  if (P.use_ctx_p)
    for (int n = 0; n < A.b; ++n) { P.ctx_off_p[n] = host_off[n]; P.ctx_len_p[n] = (int)len_of(n); }
  P.use_order = A.b <= kMaxOrdered && A.b > 1;
  if (P.use_order) {
    int idx[kMaxOrdered];
    for (int n = 0; n < A.b; ++n) idx[n] = n;
    for (int a = 1; a < A.b; ++a) {  // insertion sort by decreasing length (stable)
      const int v = idx[a];
      const long long lv = len_of(v);
      int c = a - 1;
      while (c >= 0 && len_of(idx[c]) < lv) { idx[c + 1] = idx[c]; --c; }
      idx[c + 1] = v;
    }
    for (int n = 0; n < A.b; ++n) P.req_order[n] = (uint8_t)idx[n];
  }
  int sms = kNumSM, dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  std::vector<int> sched_key;
  bool sched_hit = false;
  if (plan.nsplit == 1 && P.n_items > sms && P.n_items <= kMaxSched && sms <= kNumSM) {
    // the schedule is a function of the tile counts alone: the last one built is kept and reused while they stay the same
    sched_key.reserve(8 + 2 * plan.n_pairs + A.b);
    sched_key.push_back(sms); sched_key.push_back(A.b); sched_key.push_back(A.Hkv); sched_key.push_back(plan.n_pairs);
    for (int x = 0; x < plan.n_pairs; ++x) { sched_key.push_back(P.pair[x].ntq); sched_key.push_back(P.pair[x].n_tail); }
    for (int z = 0; z < A.b; ++z) sched_key.push_back((int)((len_of(P.use_order ? (int)P.req_order[z] : z) + 127) >> 7));
    std::lock_guard<std::mutex> lock(g_sched_mu);
    if (g_sched_key == sched_key) {
      memcpy(P.cta_first, g_sched_first, sizeof(P.cta_first));
      memcpy(P.sched, g_sched_items.data(), g_sched_items.size() * sizeof(uint16_t));
      P.use_sched = 1;
      sched_hit = true;
    }
  }
  if (!sched_hit && plan.nsplit == 1 && P.n_items > sms && P.n_items <= kMaxSched && sms <= kNumSM) {
    // cost model in SM clocks, from traces of this kernel: an iteration (128 keys) of a two-tile item, of a
    // one-tile item, and the fixed part of an item (Q load, first scores, epilogue)
    const int X = plan.n_pairs, per_req = X * A.Hkv;
    std::vector<std::pair<int, int>> cost(P.n_items);  // (cost, id)
    for (int id = 0; id < P.n_items; ++id) {
      const int z = id / per_req, x = id % X;
      const int n = P.use_order ? (int)P.req_order[z] : z;
      const long long L = len_of(n);
      const int ntq = P.pair[x].ntq;
      const int n_iter = (int)((L + 127) >> 7) + P.pair[x].n_tail;
      cost[id] = {n_iter * (ntq == 2 ? 3300 : 2700) + 11000, id};
    }
    std::stable_sort(cost.begin(), cost.end(), [](const std::pair<int, int> &a, const std::pair<int, int> &b) { return a.first > b.first; });
    typedef std::pair<long long, int> Load;  // (load, CTA): least loaded first, ties to the lower CTA
    std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
    for (int c = 0; c < sms; ++c) heap.push({0, c});
    std::vector<std::vector<uint16_t>> lists(sms);
    for (const auto &ci : cost) {
      Load l = heap.top();
      heap.pop();
      lists[l.second].push_back((uint16_t)ci.second);
      heap.push({l.first + ci.first, l.second});
    }
    // ---- local search on top of the greedy packing: with about four items per CTA in a handful of cost classes the
    // greedy result leaves the fullest CTA ~10 % above the mean; moving an item of the fullest CTA elsewhere, or swapping
    // it for a cheaper item of another CTA, whichever lowers the larger of the two loads most, closes that to < 1 %
    {
      std::vector<int> cost_of(P.n_items, 0);
      for (const auto &ci : cost) cost_of[ci.second] = ci.first;
      std::vector<long long> load(sms, 0);
      for (int c = 0; c < sms; ++c) for (uint16_t id : lists[c]) load[c] += cost_of[id];
      const int n_cand = std::min(16, sms);  // partners: the least loaded CTAs (as good as trying all of them, a tenth of the work)
      std::vector<int> by_load(sms);
      for (int iter = 0; iter < 8 * sms; ++iter) {
        int hi = 0;
        for (int c = 1; c < sms; ++c) if (load[c] > load[hi]) hi = c;
        for (int c = 0; c < sms; ++c) by_load[c] = c;
        std::partial_sort(by_load.begin(), by_load.begin() + n_cand, by_load.end(),
                          [&](int x, int y) { return load[x] != load[y] ? load[x] < load[y] : x < y; });
        long long best = load[hi] - 500;  // worth at least 500 clocks
        int ba = -1, bc = -1, bb = -1;
        for (size_t ai = 0; ai < lists[hi].size(); ++ai) {
          const int ca = cost_of[lists[hi][ai]];
          for (int k = 0; k < n_cand; ++k) {
            const int c = by_load[k];
            if (c == hi) continue;
            if (load[c] + ca < best && load[hi] - ca < best) {           // move
              const long long nm = std::max(load[hi] - ca, load[c] + ca);
              if (nm < best) { best = nm; ba = (int)ai; bc = c; bb = -1; }
            }
            if (load[c] >= best) continue;
            for (size_t bi = 0; bi < lists[c].size(); ++bi) {           // swap
              const int d = ca - cost_of[lists[c][bi]];
              if (d <= 0) continue;
              const long long nm = std::max(load[hi] - d, load[c] + d);
              if (nm < best) { best = nm; ba = (int)ai; bc = c; bb = (int)bi; }
            }
          }
        }
        if (ba < 0) break;
        const uint16_t a = lists[hi][ba];
        if (bb < 0) {
          lists[hi].erase(lists[hi].begin() + ba);
          lists[bc].push_back(a);
          load[hi] -= cost_of[a]; load[bc] += cost_of[a];
        } else {
          const uint16_t b2 = lists[bc][bb];
          lists[hi][ba] = b2; lists[bc][bb] = a;
          const int d = cost_of[a] - cost_of[b2];
          load[hi] -= d; load[bc] += d;
        }
      }
      // longest first within a CTA (the short items fill the end, where CTAs finish at slightly different times)
      for (int c = 0; c < sms; ++c)
        std::stable_sort(lists[c].begin(), lists[c].end(), [&](uint16_t x, uint16_t y) { return cost_of[x] > cost_of[y]; });
    }
    int q = 0;
    for (int c = 0; c < sms; ++c) {
      P.cta_first[c] = (uint16_t)q;
      for (uint16_t id : lists[c]) P.sched[q++] = id;
    }
    for (int c = sms; c <= kNumSM; ++c) P.cta_first[c] = (uint16_t)q;
    P.use_sched = 1;
    std::lock_guard<std::mutex> lock(g_sched_mu);
    g_sched_key = sched_key;
    memcpy(g_sched_first, P.cta_first, sizeof(P.cta_first));
    g_sched_items.assign(P.sched, P.sched + q);
  }
  if (plan.nsplit > 1) {
    P.part_o = static_cast<float *>(workspace);
    P.part_ml = reinterpret_cast<float2 *>(P.part_o + (size_t)plan.items * plan.nsplit * 256 * D);
  }
  const int X = plan.n_pairs, n_groups = A.b * A.Hkv, teams = X > 0 ? sms / X : 0;
  // Used for few, long items (up to 2.5 per SM): with more, handing whole items to the least loaded CTA balances as well
  // and averages out the pairs' different tail-tile counts, which a team pays in full (measured at 640 items of ~22 key
  // tiles: 207 us against 255 us).
  if (plan.nsplit == 1 && P.n_items >= 96 && 2 * P.n_items <= 5 * sms && X <= 16 && teams >= 2 && n_groups + teams <= kMaxSeg &&
      sms <= kNumSM && workspace) {
    // ---- cut schedule: the groups' key tiles laid end to end (each group counted with its tail tiles and a fixed
    // cost of ~3 tiles), cut at the multiples of total / teams; a cut snaps to the nearest allowed place -- a group
    // boundary, or inside a group at least kMinPiece context tiles from either end
    const int kFixedTiles = 3, kMinPiece = 4;
    int max_tail = 0;
    for (int x = 0; x < X; ++x) max_tail = std::max(max_tail, (int)P.pair[x].n_tail);
    std::vector<int> nctx(n_groups);
    std::vector<long long> pre(n_groups + 1, 0);
    int longest = 0;
    for (int gr = 0; gr < n_groups; ++gr) {
      const int z = gr / A.Hkv, n = P.use_order ? (int)P.req_order[z] : z;
      nctx[gr] = (int)((len_of(n) + 127) >> 7);
      pre[gr + 1] = pre[gr] + nctx[gr] + max_tail + kFixedTiles;
      longest = std::max(longest, nctx[gr]);
    }
    if (longest >= 4 * kMinPiece && longest < 65536) {
      struct Piece { int group, t0, t1, team; };
      std::vector<Piece> pieces;
      // cut k (k = 1 .. teams - 1) as a position (group, tile): tile 0 = the group's start
      int cg = 0, ct = 0, team = 0, cuts_in_group = 0;  // current start position, team under construction
      auto emit_until = [&](int g1, int t1) {             // pieces of `team` from (cg, ct) up to (g1, t1), t1 == 0: the group's start
        while (cg < g1 || (cg == g1 && ct < t1)) {
          const int end = cg < g1 ? nctx[cg] : t1;
          if (end > ct || nctx[cg] == 0) pieces.push_back({cg, ct, end, team});
          if (cg < g1) { ++cg; ct = 0; cuts_in_group = 0; } else { ct = t1; }
        }
      };
      for (int k = 1; k < teams; ++k) {
        const long long target = pre[n_groups] * k / teams;
        int g = cg;
        while (g < n_groups && pre[g + 1] <= target) ++g;
        if (g >= n_groups) break;
        const long long off = target - pre[g];           // units into group g
        // candidates: the start of g, the start of g + 1, a place inside g
        long long best = off;                            // distance to the start of g
        int bg = g, bt = 0;
        if (pre[g + 1] - target < best) { best = pre[g + 1] - target; bg = g + 1; bt = 0; }
        if (nctx[g] >= 2 * kMinPiece && cuts_in_group + (g == cg ? 0 : -cuts_in_group) < 7) {
          long long t = std::min<long long>(std::max<long long>(off, kMinPiece), nctx[g] - kMinPiece);
          if (g == cg) t = std::max<long long>(t, (long long)ct + kMinPiece);
          if (t <= nctx[g] - kMinPiece && std::llabs(t - off) + 1 < best) { best = std::llabs(t - off); bg = g; bt = (int)t; }
        }
        if (bg < cg || (bg == cg && bt <= ct)) continue;  // nothing between the previous cut and this one: the team stays empty
        emit_until(bg, bt);
        if (bt > 0) ++cuts_in_group;
        ++team;
      }
      team = std::min(team, teams - 1);
      emit_until(n_groups, 0);
      if ((int)pieces.size() <= kMaxSeg) {
        std::vector<int> np(n_groups, 0), slot0(n_groups, 0), seen(n_groups, 0);
        for (const Piece &pc : pieces) ++np[pc.group];
        int slots = 0;  // per team member
        for (int gr = 0; gr < n_groups; ++gr) { slot0[gr] = slots; slots += np[gr] > 1 ? np[gr] : 0; }
        const size_t part_bytes = (size_t)slots * X * 256 * ((size_t)D + 2) * 4;
        if (slots < 65536 && part_bytes + align_up((size_t)P.n_items * 4, 256) <= plan.workspace_max_bytes) {
          int q = 0, c = 0;
          for (const Piece &pc : pieces) {
            while (c <= pc.team) P.team_first[c++] = (uint16_t)q;
            TcParams::Seg &e = P.seg[q++];
            e.group = (uint16_t)pc.group; e.t0 = (uint16_t)pc.t0; e.t1 = (uint16_t)pc.t1; e.slot0 = (uint16_t)slot0[pc.group];
            e.piece = (uint8_t)seen[pc.group]++; e.npieces = (uint8_t)np[pc.group];
          }
          while (c <= kNumSM) P.team_first[c++] = (uint16_t)q;
          P.use_seg = 1; P.seg_X = X; P.seg_teams = teams;
          P.use_sched = 0;
          P.part_o = static_cast<float *>(workspace);
          P.part_ml = reinterpret_cast<float2 *>(P.part_o + (size_t)slots * X * 256 * D);
          P.seg_count = reinterpret_cast<unsigned int *>(static_cast<uint8_t *>(workspace) + align_up(part_bytes, 256));
          if (cudaMemsetAsync(P.seg_count, 0, (size_t)P.n_items * 4, st) != cudaSuccess) return DPARA_ERR_CUDA;
        }
      }
    }
  }
  return D == 128 ? launch_tc_d<128>(P, plan, st) : launch_tc_d<64>(P, plan, st);
}

}  // namespace dpara

