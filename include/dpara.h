/* dpara.h -- C ABI of the B200 (sm_100a) all-boundary draft step.
 *
 * The method (paper Alg. 1): while the target model verifies the draft block t_{0:d}, the drafter
 * backbone precomputes, in one pass, draft representations for EVERY acceptance boundary r = 0..d
 * (Alg. 1 line 1, Sec. 3.2, Fig. 4); when verification returns the accepted length r and the bonus
 * token b (Alg. 1 line 2, Sec. 2.1), branch r is selected (Alg. 1 line 3) and handed to the
 * autoregressive head.  This library implements those two calls:
 *
 *   dpara_draft_all_boundaries  -- Alg. 1 line 1 for one backbone block: the tree-masked attention
 *                                  of Fig. 4 for all boundaries at once (optionally wrapped in the
 *                                  block's projections, norms and MLP).
 *   dpara_verify_select         -- Alg. 1 lines 2-3 after the target forward: accepted length, bonus
 *                                  token (greedy, or the rejection rule of App. C) and the gather of
 *                                  the selected branch's representation.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its name starts with host_.  The caller owns every
 *     buffer; the library allocates nothing.  The only state it keeps between calls is a process-wide
 *     launch counter (dpara_kernel_launches), the last attention work schedule with the key-tile counts
 *     it was built for (a pure function of those counts, kept in host memory to save host time when they
 *     repeat) and, for the fixed-scratch entry point, that entry's scratch array and its cached device
 *     address.
 *   - Calls enqueue kernels on `stream` (a cudaStream_t passed as void*) and return without
 *     synchronising.  Outputs are valid once the stream has reached the end of the call's work.
 *   - The return code reports host-detectable errors.  Argument errors (INVALID_ARG, UNSUPPORTED,
 *     WORKSPACE, STATIC_LIMIT) are found before anything is launched.  DPARA_ERR_CUDA can also come from
 *     the middle of a multi-kernel call (a launch or tensor-map encode that fails after earlier kernels
 *     of the same call were queued); outputs are then undefined.
 *     Conditions only the device can see (a draft token outside the vocabulary, a bounded wait that
 *     expired) OR a bit into *status_word (may be NULL) and the kernels still finish with defined
 *     outputs.
 *   - bf16 tensors are row-major with the last index contiguous and must be 16-byte aligned.
 *   - J = n_boundaries = d + 1.  Boundary j reads spine rows [0, min(j + prefix_base, n_spine)).
 */
#ifndef DPARA_H_
#define DPARA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DPARA_OK = 0,
  DPARA_ERR_INVALID_ARG = -1, /* null pointer, non-positive size, misaligned buffer, bad range */
  DPARA_ERR_UNSUPPORTED = -2, /* shape outside what the kernels are built for (see each call) */
  DPARA_ERR_WORKSPACE = -3,   /* workspace missing or smaller than *_workspace_bytes() */
  DPARA_ERR_CUDA = -4,        /* a CUDA runtime/driver call failed (launch, tensor-map encode) */
  DPARA_ERR_TIMEOUT = -5,     /* never returned by a call (calls do not synchronise); the code and its string exist
                                 for callers that turn DPARA_STATUS_TIMEOUT in *status_word into a status */
  DPARA_ERR_STATIC_LIMIT = -6 /* request needs more scratch than a fixed-scratch entry point owns */
} dpara_status;

/* bits OR-ed into *status_word by kernels */
#define DPARA_STATUS_BAD_TOKEN 1u /* a draft token outside [0, vocab): rejected at that position */
#define DPARA_STATUS_TIMEOUT 2u   /* a bounded device-side wait gave up; outputs of that tile are undefined */
#define DPARA_STATUS_CACHE_FULL 4u /* dpara_cache_append: a request's new rows did not fit its cache; it was left as it was */

typedef enum { DPARA_BF16 = 0, DPARA_F32 = 1 } dpara_dtype;

/* Shapes of one draft call (Sec. 3.2: d+1 boundaries, each a block of mask slots). */
typedef struct {
  int32_t batch;        /* b requests */
  int32_t n_boundaries; /* J = d + 1 */
  int32_t block;        /* Bq mask slots (query rows) per boundary */
  int32_t n_q_heads;    /* Hq */
  int32_t n_kv_heads;   /* Hkv; Hq % Hkv == 0; query head h reads KV head h / (Hq/Hkv) */
  int32_t head_dim;     /* D: 64 or 128 */
  int32_t prefix_base;  /* anchors visible to boundary j = j + prefix_base; paper (k = r + 1): 1 */
  int32_t n_spine;      /* S spine rows stored per request (normally J) */
  int32_t boundary_lo;  /* boundaries computed: [boundary_lo, boundary_hi); all = [0, J);        */
  int32_t boundary_hi;  /* a conventional single-anchor-set draft step = [j, j + 1)               */
  float softmax_scale;  /* 0 selects 1/sqrt(D) */
  int32_t spine_queries; /* 0: only the mask slots are query rows (the spine's keys/values are inputs).  1: the S spine
                            tokens are query rows as well (Sec. 3.2, Fig. 4: an anchor reads the cache, itself and the
                            earlier anchors) -- q, out and out_lse then hold J*Bq + S rows per request, the mask-slot rows
                            in (boundary, slot) order followed by the spine rows; needs boundary_lo = 0, boundary_hi = J */
} dpara_shape;

/* Tensors of the attention (Fig. 4).  Context keys/values are the drafter-side projection of the
 * cached target features C (Alg. 1 Require); spine keys/values belong to the feature-less draft block
 * t_{0:d}; block keys/values belong to the mask slots themselves (branches attend bidirectionally
 * within their own block).  In full-layer mode q, k_blk, v_blk and out may be NULL: they are
 * produced inside the call. */
typedef struct {
  const void *q;                   /* [b][J][Bq][Hq][D] bf16 */
  const void *k_ctx, *v_ctx;       /* [sum_n L_n][Hkv][D] bf16; request n owns rows ctx_offsets[n]..ctx_offsets[n+1) */
  const int64_t *ctx_offsets;      /* [b+1] device copy */
  const int64_t *host_ctx_offsets; /* [b+1] HOST copy of the same values (needed to size the grid) */
  const void *k_spine, *v_spine;   /* [b][S][Hkv][D] bf16 */
  const void *k_blk, *v_blk;       /* [b][J][Bq][Hkv][D] bf16; both NULL: slots read no block keys */
  void *out;                       /* [b][J][Bq][Hq][D], dtype out_dtype; rows of boundaries outside [lo,hi) untouched */
  int32_t out_dtype;               /* dpara_dtype */
  float *out_lse;                  /* optional [b][J][Bq][Hq]: natural-log sum-exp of the scaled scores (NULL ok) */
  /* Caches kept with slack for in-place appends (dpara_cache_append): both NULL = packed (request n's context is all
   * of rows ctx_offsets[n]..ctx_offsets[n+1)); both given = only the first ctx_lens[n] of those rows are context.
   * The unused rows must hold finite numbers (clear the cache once when it is allocated): the last, part-filled key
   * tile of a request carries them through the tensor core with weight exactly 0, and 0 x NaN is NaN. */
  const int64_t *ctx_lens;         /* [b] device */
  const int64_t *host_ctx_lens;    /* [b] HOST copy of the same values */
} dpara_attn_io;

/* Full-layer mode (one pre-norm backbone block; Sec. 3.1 lists the block's trainable parts without giving
 * equations -- the equations are this library's reading, stated with the call). */
typedef struct {
  const void *x;                                   /* [b][J][Bq][hidden] bf16 hidden states of the mask slots; with
                                                      shape->spine_queries: [b][J*Bq + S][hidden], each request's spine rows
                                                      behind its mask-slot rows (y_f32 / y_bf16 likewise) */
  const void *w_qkv;                               /* [(Hq + 2 Hkv) D][hidden] bf16, rows = [q | k | v] */
  const void *w_o;                                 /* [hidden][Hq D] bf16 */
  const void *w_gate_up;                           /* [2 inter][hidden] bf16, rows [0,inter) gate, [inter,2 inter) up */
  const void *w_down;                              /* [hidden][inter] bf16 */
  const void *rms1_w, *rms2_w;                     /* [hidden] bf16 gains; NULL = ones */
  const void *qnorm_w, *knorm_w;                   /* [D] bf16 gains of the per-head q/k RMS norm; both NULL = no QK-norm */
  float rms_eps;
  float rope_theta;
  int32_t use_rope;                                /* slot i of boundary j of request n sits at position L_n + j + 2 + i */
  int32_t hidden, intermediate;
  float *y_f32;                                    /* [b][J][Bq][hidden] fp32 output (required) */
  void *y_bf16;                                    /* optional bf16 copy of y (NULL ok) */
} dpara_layer_io;

/* Bytes of scratch dpara_draft_all_boundaries needs for these shapes (0 is possible).
 * host_ctx_offsets: [b+1] host array.  full_layer != 0: include the block's intermediates
 * (hidden/intermediate are taken from `layer`, which may be NULL when full_layer == 0).  The figure is an upper bound
 * over all context lengths that fit the offsets, so one workspace serves a cache that grows in place. */
size_t dpara_draft_workspace_bytes(const dpara_shape *shape, const int64_t *host_ctx_offsets,
                                   const dpara_layer_io *layer, int full_layer);

/* Alg. 1 line 1 / Sec. 3.2 / Fig. 4.  For every request n, boundary j in [lo,hi), slot i, head h:
 *   out = softmax(scale * q K^T) V over the keys  context[0..L_n)  ++  spine[0..min(j+prefix_base,S))
 *   ++  block j (all Bq slots; omitted when k_blk == NULL),  fp32 accumulation, bf16 inputs.
 * A row with no visible key gives out = 0 and lse = -inf.
 * layer == NULL: attention only, on io->q / io->k_blk / io->v_blk.
 * layer != NULL: xn = bf16(rmsnorm(x) g1); [q|k|v] = bf16(xn Wqkv^T); per-head RMS norm and rotary
 *   embedding (rotate-half) on q, k, each rounded to bf16; the slots' own k, v are the block
 *   keys/values; a = bf16(attention); h1 = x + a Wo^T (fp32); hn = bf16(rmsnorm(h1) g2);
 *   act = bf16(silu(hn Wg^T) * (hn Wu^T)); y = h1 + act Wd^T (fp32).
 * workspace: device scratch of at least dpara_draft_workspace_bytes(); contents need not be
 *   initialised and are garbage afterwards; two calls in flight must not share it.
 * Errors: INVALID_ARG (null/misaligned/ranges, ctx_offsets not non-decreasing), UNSUPPORTED
 *   (head_dim not 64/128, Hq % Hkv != 0, Hq/Hkv > 16, block > 64, n_spine > 64), WORKSPACE, CUDA. */
dpara_status dpara_draft_all_boundaries(const dpara_shape *shape, const dpara_attn_io *io,
                                        const dpara_layer_io *layer, void *workspace,
                                        size_t workspace_bytes, int32_t *status_word, void *stream);

/* A stack of backbone blocks in one call (Alg. 1 line 1 runs the whole M-DFlash backbone on the spine; Sec. 3.2 / Fig. 4
 * give the mask every block uses).  Block l reads block l-1's bf16 output (the residual stream between blocks is bf16)
 * and its own context cache.  Meant for shape->spine_queries = 1, where every block produces the spine's keys/values
 * itself (with spine_queries = 0 all blocks would read the same supplied spine keys/values); x and the outputs then hold
 * J*Bq + S rows per request, the mask-slot rows followed by the spine rows.
 *   host_layers   HOST array [n_layers] of dpara_layer_io: weights and flags of each block (all with the same hidden and
 *                 intermediate sizes); x is taken from entry 0 only, y_f32 (required) and y_bf16 from the last entry only
 *   host_k_ctx, host_v_ctx   HOST arrays [n_layers] of DEVICE pointers: each block's context keys/values, all laid out
 *                 by io->ctx_offsets (and io->ctx_lens); io->k_ctx / io->v_ctx are ignored
 * Workspace: dpara_backbone_workspace_bytes().  Errors: as dpara_draft_all_boundaries. */
typedef struct {
  int32_t n_layers;
  const dpara_layer_io *host_layers;
  const void *const *host_k_ctx;
  const void *const *host_v_ctx;
} dpara_backbone_io;
size_t dpara_backbone_workspace_bytes(const dpara_shape *shape, const int64_t *host_ctx_offsets, const dpara_backbone_io *bb);
dpara_status dpara_draft_backbone(const dpara_shape *shape, const dpara_attn_io *io, const dpara_backbone_io *bb, void *workspace,
                                  size_t workspace_bytes, int32_t *status_word, void *stream);

/* Where a full-layer call leaves the block's intermediates (the quantities named in the equations above;
 * the paper, Sec. 3.1, lists the block's parts without equations).  offsets[0..8] receive the byte offsets,
 * inside the call's workspace, of  xn [M][hidden] bf16,  qkv [M][(Hq+2Hkv)D] bf16,  q [M][Hq D] bf16,
 * k [M][Hkv D] bf16,  v [M][Hkv D] bf16,  a [M][Hq D] bf16,  h1 [M][hidden] fp32,  hn [M][hidden] bf16,
 * act [M][inter] bf16, with M = b * J * Bq rows in (request, boundary, slot) order (b * (J * Bq + S) rows, each request's
 * spine rows behind its mask-slot rows, when shape->spine_queries is set).  They hold the last call's
 * values until the workspace is reused.  Host-only; nothing is launched.  For stage-by-stage checks.
 * Errors: INVALID_ARG, UNSUPPORTED (as dpara_draft_all_boundaries). */
dpara_status dpara_layer_workspace_layout(const dpara_shape *shape, const int64_t *host_ctx_offsets,
                                          const dpara_layer_io *layer, size_t offsets[9]);

/* Verification-side tensors (Sec. 2.1; App. C for mode 1).  Row i of `target` is the target's
 * prediction for the token after t_0..t_i, so draft t_{i+1} is judged by row i and the bonus comes
 * from row r. */
typedef struct {
  int32_t batch;               /* b */
  int32_t n_boundaries;        /* J = d + 1 target rows per request */
  int32_t vocab;               /* V */
  int32_t block;               /* Bq rows per representation */
  int32_t hidden;              /* elements per representation row */
  int32_t mode;                /* 0 greedy on logits, 1 rejection sampling on probabilities */
  const float *target;         /* [b][J][V] fp32: logits (mode 0) or probabilities (mode 1) */
  const float *draft_probs;    /* [b][J-1][V] fp32, mode 1 only: row i is the drafter distribution t_{i+1} was drawn from */
  const int32_t *draft_tokens; /* [b][J-1] = t_1..t_d */
  const float *uniforms;       /* [b][J] fp32, mode 1 only; each = m * 2^-24, m integer in [0, 2^24):
                                  u[i] tests draft t_{i+1}; u[J-1] draws the bonus */
  const void *reps;            /* [b][J][Bq][hidden] bf16 (e.g. `out`/`y_bf16` of the draft call); NULL: no gather */
  int32_t *accept_len;         /* [b] r */
  int32_t *bonus;              /* [b] b */
  int32_t *gather_idx;         /* [b] index of the selected branch (= r) */
  int32_t *out_tokens;         /* optional [b][J]: t_1..t_r, bonus, then -1 */
  void *selected;              /* [b][Bq][hidden] bf16 = reps[n][r] (required when reps != NULL) */
  int32_t rep_req_rows;        /* rows of `hidden` elements from one request's representations to the next request's;
                                  0 = J * Bq (packed).  J * Bq + S for the output of a call with spine query rows */
  int32_t flags;               /* 0, or DPARA_VERIFY_EARLY_START */
} dpara_verify_io;

/* dpara_verify_io.flags.  EARLY_START: the call may begin before the work enqueued immediately before it on the stream
 * has finished -- it reads target / draft_probs / draft_tokens / uniforms and uses its workspace and its small outputs
 * straight away, and waits for that work only before it reads `reps` (and before it completes).  The caller promises that
 * the immediately preceding work writes none of those inputs and touches neither this call's workspace nor its outputs:
 * the case of Alg. 1 when verification has resolved while the drafter's precompute (the producer of `reps`) is still
 * running on the same stream.  Only work that releases its dependents early is affected (this library's own kernels do);
 * behind anything else the flag changes nothing. */
#define DPARA_VERIFY_EARLY_START 1

/* Bytes of scratch dpara_verify_select needs; only the sizes and mode of `io` are read. 0 on bad sizes. */
size_t dpara_verify_workspace_bytes(const dpara_verify_io *io);

/* Alg. 1 lines 2-3.  mode 0: a_i = lowest index of the maximum of row i (-0 == +0, NaN below every
 * number); r = number of leading drafts with t_i == a_{i-1}; bonus = a_r.
 * mode 1: draft t_i accepted iff fl32(u[i-1] * q_{i-1}(t_i)) < p_{i-1}(t_i), scan stops at the first
 * rejection; bonus drawn by inverse CDF in vocabulary order from integer weights
 * trunc(max(fl32(p_r - q_r), 0) * 2^32) (r < d) or trunc(p_d * 2^32) (r = d) with threshold
 * (m * W) >> 24; empty residual falls back to p_r, then to the lowest-index maximum of p_r.
 * A draft token outside [0, V) is rejected and sets DPARA_STATUS_BAD_TOKEN.
 * selected[n] = reps[n][r] copied bit for bit.
 * workspace: at least dpara_verify_workspace_bytes() bytes, 8-byte aligned, ZERO-FILLED before its first use
 *   (one cudaMemset when it is allocated).  Every call leaves it zero-filled again -- the CTA that finishes
 *   last puts back what the call used, so no clearing launch precedes the kernel -- and it can be handed to
 *   the next call as it is, in either mode, as long as that call's size request is not larger.  Two calls in
 *   flight must not share it.
 * Errors: INVALID_ARG, UNSUPPORTED (J > 64), WORKSPACE, CUDA. */
dpara_status dpara_verify_select(const dpara_verify_io *io, void *workspace, size_t workspace_bytes,
                                 int32_t *status_word, void *stream);

/* dpara_verify_select for callers that cannot hand over scratch memory.  (The paper has no
 * counterpart; this is a packaging variant of the call above.)
 *
 * Who needs it: a serving process that has given all free device memory to its own KV-cache pool at
 * start-up, or a decode loop in which an allocation would stall the device between two rounds, has
 * no way to obtain the workspace the normal call asks for.  This variant computes exactly what
 * dpara_verify_select computes -- same kernels, same outputs, bit for bit -- but keeps its scratch
 * in a fixed array of DPARA_VERIFY_STATIC_SCRATCH_BYTES that lives inside the library's device
 * image.  Every GPU that loads the library carries that array until the process exits.
 *
 *  - The call performs no cudaMalloc/cudaFree and calls no allocating routine.  Inputs and outputs
 *    are still the caller's buffers, as in dpara_verify_io.
 *  - The first call on each device looks up the array's device address (with that device current)
 *    and remembers it.  Make that first call during start-up, before any stream capture begins on
 *    that device.
 *  - Requests whose scratch need (dpara_verify_workspace_bytes) exceeds the fixed size are refused
 *    with DPARA_ERR_STATIC_LIMIT and nothing is launched.  For scale: greedy mode with 16 requests
 *    x 16 boundaries needs 3.3 KB, sampling mode with 8 requests over a 151 936-token vocabulary
 *    5.3 KB; the need grows with batch * n_boundaries (greedy) or batch * ceil(vocab / 4096) (sampling).
 *  - All calls on a device share the one array and it keeps whatever the previous call left; the
 *    array is zero when the library is loaded and each call, before it ends, clears again the parts
 *    that the next call needs at zero.  Two calls that overlap on the same GPU
 *    (different streams, or different host threads without ordering) race on it and give undefined
 *    results: order them on one stream or with events.
 * Errors: as dpara_verify_select, plus DPARA_ERR_STATIC_LIMIT; DPARA_ERR_CUDA if the address lookup
 * fails. */
#define DPARA_VERIFY_STATIC_SCRATCH_BYTES (256u * 1024u)
dpara_status dpara_verify_select_static(const dpara_verify_io *io, int32_t *status_word, void *stream);

/* The critical-path remainder T_Head (Alg. 1, the lines after the barrier: starting from the bonus token, each of
 * the d head steps adds a correction computed from the previous step's token to the selected branch's base logits
 * and picks the next token; Sec. 3.2 "Loss" gives the formula: the head has its own low-rank token embedding E and
 * a projection W of it to the vocabulary, and reads only the preceding token).  The base
 * logits l_i are the language-model head applied to the selected branch's final hidden states (App. D runs the
 * language-model head on shipped hidden states right before the head loop).  uniforms == NULL: greedy decoding (Table 1),
 * y_i is the lowest index holding the maximum of z_i; NaN ranks below every number.  uniforms != NULL: sampling (App. C:
 * temperature 1, top-p 1), y_i is drawn from softmax(z_i) by the inverse CDF in vocabulary order with the supplied
 * uniform u = uniforms[n][i-1] = m * 2^-24: the lowest v with sum_{v' <= v} w_v' > u * sum w, w_v = exp(z_v - max z)
 * (exponentials and sums in double precision; NaN logits weigh nothing).
 *   sel_reps     device [b][block][hidden] bf16: the selected branches (the `selected` output of dpara_verify_select)
 *   w_lm         device [vocab][hidden] bf16 (weights stored [out][in])
 *   ar_w, ar_e   device [vocab][rank] bf16: W (one row per vocabulary entry) and E (one row per token)
 *   bonus        device [b] int32: y_0 of each request; a value outside [0, vocab) sets DPARA_STATUS_BAD_TOKEN in
 *                *status_word and is treated as token 0
 *   next_tokens  device [b][block] int32 out: y_1 .. y_d
 * bf16 products with fp32 accumulation; z_i = (fp32 base logit) + (fp32 correction), compared in fp32.
 * Workspace: dpara_head_workspace_bytes(b, block, vocab) bytes of device memory, 16-byte aligned, owned by the
 * caller and private to the call while it runs (it holds the fp32 base logits [b * block][vocab] and, for sampling, one
 * step's logits z [b][vocab]).  The greedy loop is ONE persistent kernel; the sampling loop is two launches per step
 * (the skinny product with the base logits added, then one CTA per request that draws the token).
 * All work is queued on `stream`; nothing is allocated.  Errors: INVALID_ARG (null or misaligned pointer,
 * non-positive size), UNSUPPORTED (b > 32, block > 64, rank not a multiple of 64 or > 256, hidden % 64 != 0,
 * vocab % 8 != 0), CUDA.  A device-side wait that runs out sets DPARA_STATUS_TIMEOUT in *status_word. */
typedef struct {
  const void *sel_reps;
  const void *w_lm;
  const void *ar_w;
  const void *ar_e;
  const int32_t *bonus;
  int32_t *next_tokens;
  int32_t b, block, hidden, vocab, rank;
  const float *uniforms;      /* device [b][block] fp32 or NULL (greedy) */
} dpara_head_io;
size_t dpara_head_workspace_bytes(int32_t b, int32_t block, int32_t vocab);
dpara_status dpara_draft_head(const dpara_head_io *io, void *workspace, size_t workspace_bytes, int32_t *status_word, void *stream);

/* Feature-cache update (Alg. 1, the line after the head loop: the verified features of t_0..t_r are appended to the
 * cache and the rejected drafts t_{r+1..d} dropped; Sec. 3.3 states it in words; App. D, single-GPU paragraph: history
 * features are projected incrementally).  The drafter layers read the cache as keys and values; this call projects the
 * new rows for every layer and appends them in place.  Reading of the projection (the paper gives no equations), per
 * layer l and feature row c at position p:  cn = bf16(rmsnorm(c) g_l);  [k | v] = bf16(cn Wkv_l^T);
 * k = bf16(rmsnorm_over_D(k) gk_l) when knorm is given;  k = bf16(rope(k, p)) (rotate-half) when use_rope.
 * Cache layout: request n owns rows [row_start[n], row_start[n] + capacity[n]) of every layer's k/v tensor
 * ([rows][Hkv][D] bf16); the first ctx_len[n] are filled.  The call writes the r_n + 1 rows of t_0..t_{r_n}
 * (r_n = accept_len[n], read on the device: queue this call behind dpara_verify_select) at rows
 * row_start[n] + ctx_len[n] + i, positions ctx_len[n] + i, then adds r_n + 1 to ctx_len[n].  A request whose rows do not
 * fit (or whose accept_len is outside [0, n_rows)) is left untouched and DPARA_STATUS_CACHE_FULL is OR-ed into
 * *status_word.  The draft call reads such a cache through dpara_attn_io.ctx_lens.
 *   features      device [b][n_rows][feat_dim] bf16: target features of t_0..t_d from the verification forward
 *   host_*        HOST arrays of n_layers DEVICE pointers: w_kv [2 Hkv D][feat_dim] bf16 (rows = keys, then values),
 *                 norm_w [feat_dim] and knorm_w [D] bf16 gains (array or entries may be NULL), k_ctx / v_ctx caches
 *   row_start, capacity   device [b] int64;   ctx_len   device [b] int64, in/out
 * Workspace: dpara_cache_append_workspace_bytes(), 16-byte aligned, private to the call while it runs.
 * Errors: INVALID_ARG, UNSUPPORTED (head_dim not 64/128, feat_dim % 64 != 0), WORKSPACE, CUDA. */
typedef struct {
  int32_t batch, n_rows, feat_dim, n_kv_heads, head_dim, n_layers;
  const void *features;
  const int32_t *accept_len;
  const void *const *host_w_kv;
  const void *const *host_norm_w;
  const void *const *host_knorm_w;
  void *const *host_k_ctx;
  void *const *host_v_ctx;
  const int64_t *row_start;
  const int64_t *capacity;
  int64_t *ctx_len;
  float rms_eps, rope_theta;
  int32_t use_rope;
} dpara_cache_io;
size_t dpara_cache_append_workspace_bytes(const dpara_cache_io *io);
dpara_status dpara_cache_append(const dpara_cache_io *io, void *workspace, size_t workspace_bytes, int32_t *status_word, void *stream);

const char *dpara_status_string(dpara_status s);

/* Library/ABI version: major * 1000 + minor. */
int32_t dpara_version(void);

/* The projection GEMM of the backbone block on its own (Sec. 3.1, trainable parts of the backbone block;
 * bf16 operands, fp32 accumulation on the tensor cores):
 *   out[M][N] = epilogue( a[M][K] * w[N][K]^T ),  a and w bf16 row-major (weights stored [out][in]).
 * epilogue 0: out bf16.   epilogue 1: out fp32 = resid + product (resid [M][N], bf16 when
 * resid_dtype == DPARA_BF16 else fp32), optional bf16 copy in out_bf16.   epilogue 2: w holds 2N rows,
 * [0,N) gate and [N,2N) up; out bf16 = silu(a Wg^T) * (a Wu^T).   epilogue 3: out fp32 = product.
 * No workspace.  Errors: INVALID_ARG (null/misaligned), UNSUPPORTED (K % 64 != 0 or N % 8 != 0), CUDA. */
typedef struct {
  const void *a;
  const void *w;
  int32_t M, N, K;
  int32_t epilogue;
  const void *resid;
  int32_t resid_dtype;
  void *out;
  void *out_bf16;
} dpara_gemm_io;
dpara_status dpara_gemm_bf16(const dpara_gemm_io *io, int32_t *status_word, void *stream);

/* Failure-detection self-test (the paper has no counterpart): launches one CTA that waits, with the
 * same bounded wait all kernels here use, on a barrier nothing arrives at.  After `limit_us`
 * microseconds (1 .. 1 000 000) the wait gives up, DPARA_STATUS_TIMEOUT is OR-ed into *status_word
 * (device, required), the time actually waited is stored in *waited_ns (device, optional) and the kernel
 * ends normally; the CUDA context stays usable.  Errors: INVALID_ARG, CUDA. */
dpara_status dpara_selftest_bounded_wait(int32_t *status_word, uint32_t limit_us, uint64_t *waited_ns, void *stream);

/* Number of kernels this library has launched in this process so far (all calls, all streams).
 * Bookkeeping for benchmarks; the paper has no counterpart. */
int64_t dpara_kernel_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* DPARA_H_ */
