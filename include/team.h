/*
 * team.h -- C ABI of the TEAM MoE-layer library for NVIDIA B200 (sm_100a).
 *
 * One call of team_moe_forward() is the MoE feed-forward layer of one
 * denoising step of a block-diffusion MoE language model, with the expert
 * activation rule of TEAM (arXiv 2602.08404):
 *
 *   - Sec. 4.1 (delayed caching, DCD): tokens decoded two or more steps ago
 *     are not recomputed; only masked tokens and tokens accepted in the
 *     previous step enter the layer.
 *   - Sec. 4.2, Eq. 4: a masked token is "hot" if its last confidence exceeds
 *     tau_hot or it lies within L_hot positions of a decoded token, else "cold".
 *   - Sec. 4.3, Algorithm 1 (limited activation, LAC): newly accepted and hot
 *     tokens are routed over all experts; the union of their top-k sets is the
 *     necessary set E_A; cold tokens are routed inside E_A only.
 *   - Sec. 4.2 (speculative exploration, SEH): the caller lays the branches of
 *     a sequence out as extra rows with a branch id; rows of one group share
 *     E_A and one pass over the expert weights.
 *   - The layer itself: fp32 router, softmax, top-k, renormalised routing
 *     weights, expert dispatch, SwiGLU experts, weighted combine (Sec. 1 and
 *     Algorithm 1 "Router"; the paper leaves the arithmetic to the base model).
 *
 * Conventions
 *   - Every pointer inside team_weights, team_step_state, team_routing and the
 *     x / y arguments is DEVICE memory owned by the caller.  The library
 *     borrows weight pointers from team_set_weights() until they are replaced
 *     or the context is destroyed, and never frees caller memory.
 *   - team_config, team_weights, team_step_state and team_routing structs
 *     themselves live in HOST memory and are read during the call only.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*,
 *     NULL = default stream).  The return value reports argument and launch
 *     errors only; conditions detected on the device (an index out of range,
 *     a bounded wait that gave up, a layout contract broken) set a status word
 *     read back with team_read_status(); kernels always terminate.
 *   - No global state; a context may be used from one thread at a time.  Calls
 *     on one context must be stream-ordered with respect to each other because
 *     they share the context's workspace.
 *   - There is no CPU fallback: without a usable CUDA device every compute
 *     entry point returns TEAM_ERR_CUDA.
 *
 * Row layout.  A call presents T = n_rows rows.  Rows that share (group,
 * branch) must be contiguous and form one decoding block (at most
 * TEAM_MAX_BLOCK rows); `pos` is the position inside that block.  `group` is
 * the scope of E_A (normally the sequence), 0 <= group < max_groups.  A run
 * longer than TEAM_MAX_BLOCK, or a group / branch index out of range, is
 * reported as TEAM_ERR_STATE in the device status; rows of one (group,
 * branch) that are NOT contiguous are not detected: each run then counts as a
 * block of its own for the distance test of Eq. 4.
 *
 * Slot ids.  Row t's j-th routed choice is slot t*top_k + j.  Shared expert s
 * (expert id n_experts + s) applied to row t is slot T*top_k + s*T + t and has
 * combine weight 1.
 */
#ifndef TEAM_H_
#define TEAM_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct team_ctx team_ctx;

enum {
  TEAM_OK = 0,
  TEAM_ERR_ARG = -1,     /* NULL pointer, n_rows out of range, missing weights         */
  TEAM_ERR_SHAPE = -2,   /* configuration the kernels do not support                   */
  TEAM_ERR_CUDA = -3,    /* CUDA runtime / driver error (see team_last_cuda_error)     */
  TEAM_ERR_TIMEOUT = -4, /* device status: a bounded wait expired                      */
  TEAM_ERR_STATE = -5,   /* device status: row layout contract broken / index range    */
  TEAM_ERR_CAPACITY = -6 /* more rows than a fixed-size scratch area holds               */
};

enum { TEAM_TOK_MASKED = 0, TEAM_TOK_NEW = 1, TEAM_TOK_CACHED = 2 };   /* team_step_state.tok_state */
enum { TEAM_CLS_SKIP = 0, TEAM_CLS_FIRST = 1, TEAM_CLS_COLD = 2 };     /* team_routing.tok_class    */
enum { TEAM_F_DCD = 1, TEAM_F_LAC = 2 };                               /* team_config.flags; 0 = vanilla top-k */
enum { TEAM_DTYPE_F32 = 0, TEAM_DTYPE_BF16 = 1 };

#define TEAM_MAX_EXPERTS 256   /* routed experts                       */
#define TEAM_MAX_TOPK 16
#define TEAM_MAX_SHARED 4
#define TEAM_MAX_ROWS 2048     /* rows per call                        */
#define TEAM_MAX_GROUPS 1024
#define TEAM_MAX_BLOCK 64      /* rows of one (group, branch)          */
#define TEAM_STATIC_ROUTE_MAX_ROWS 256   /* rows per team_route_static call */

typedef struct {
  int32_t hidden;      /* H; multiple of 128 for bf16, of 4 for fp32                     */
  int32_t n_experts;   /* E routed experts, top_k <= E <= TEAM_MAX_EXPERTS               */
  int32_t top_k;       /* k <= min(E, TEAM_MAX_TOPK)                                    */
  int32_t inter;       /* I; multiple of 64 for bf16, of 16 for fp32                     */
  int32_t n_shared;    /* always-on experts appended after the routed ones              */
  int32_t max_rows;    /* largest n_rows of any call on this context; it also picks the
                          expert kernel (bf16).  Hidden size 1024 or 2048 and fewer than 96
                          rows: the weight-streaming kernel on the row-major / slab layout
                          (<= 8 rows all resident, else work items of 8 token-slots).
                          Otherwise: the tensor-memory (tcgen05) grouped GEMMs on the
                          tile-major layout of team_pack_w_tiles()                      */
  int32_t max_groups;  /* group ids are in [0, max_groups), <= TEAM_MAX_GROUPS; branch ids in [0, 256) */
  int32_t dtype;       /* TEAM_DTYPE_F32: x and expert weights fp32 (plain FMA kernels);
                          TEAM_DTYPE_BF16: x and expert weights bf16, fp32 accumulation
                          on tensor cores.  Router weights and y are fp32 in both.      */
  int32_t flags;       /* TEAM_F_* bits                                                 */
  float tau_hot;       /* Eq. 4 confidence threshold (paper default 0.7)                */
  int32_t L_hot;       /* Eq. 4 distance bound (paper default 3)                        */
  int32_t hot_dist_inclusive; /* 1: |k-j| <= L_hot (Sec. 5.1 wording), 0: < (Eq. 4 as printed) */
  int32_t prefix_decoded;     /* 1: position -1 (previous block) counts as decoded      */
  int32_t norm_topk;          /* 1: routing weights renormalised over the k chosen      */
  int32_t refresh_every;      /* Sec. 4.1 / Table 3 (Refresh-4, Refresh-8): N > 0 recomputes every token on the
                                 steps with step_index % N == 0 (cached tokens are treated as newly accepted
                                 there); 0 = never, the paper's refresh-free choice                        */
  int32_t ep_rank;            /* expert parallelism: this context computes the experts                    */
  int32_t ep_world;           /* [ep_rank * E / ep_world, (ep_rank + 1) * E / ep_world) only; 0 or 1 = all.  With
                                 ep_world > 1: n_experts must be a multiple of ep_world, n_shared must be 0, the
                                 expert-weight tensors given to team_set_weights hold the context's OWN experts
                                 only (E / ep_world of them, in order), router weights and routing are complete
                                 and identical on every rank, and y receives this rank's PARTIAL sums for the
                                 computed rows: the layer output is the sum over the ranks (an all-reduce of
                                 the computed rows of y, which is the caller's to run)                     */
} team_config;

typedef struct {
  const void *w_router; /* fp32 [E, H] row-major                                          */
  /* Expert weights come in two layouts; a context needs the one its expert kernel reads (see max_rows in
     team_config) and accepts both.  Set the pointers of a layout you do not provide to NULL. */
  const void *w_gate;   /* [E + n_shared, I, H] row-major, dtype per config               */
  const void *w_up;     /* [E + n_shared, I, H]                                           */
  const void *w_down;   /* [E + n_shared, I/16, H, 16]: Eq. 1's W_down [H, I] of every expert
                           stored in slabs of 16 columns, as team_pack_w_down() writes it */
  const void *w_gu_tiles;   /* bf16 only: gate and up projections as 16 KB tensor-core tiles, */
  const void *w_down_tiles; /* and the down projection likewise, as team_pack_w_tiles() writes them */
} team_weights;

/* State carried from the previous denoising step (Algorithm 1 inputs D, M; Eq. 4). */
typedef struct {
  int32_t n_rows;           /* T, 1 <= T <= max_rows                                      */
  const uint8_t *tok_state; /* [T] TEAM_TOK_*                                             */
  const float *conf;        /* [T] confidence c_k of the previous step's prediction       */
  const int32_t *pos;       /* [T] position in the block                                  */
  const int32_t *group;     /* [T] scope of E_A                                           */
  const int32_t *branch;    /* [T] speculative branch id (scope of "decoded" in Eq. 4)    */
  int32_t step_index;       /* denoising step inside the block, 0-based (read only when refresh_every > 0) */
} team_step_state;

/* Optional outputs; any pointer may be NULL.  team_route fills probs, topk_idx,
 * topk_w, margin with the plain (unrestricted) top-k of every computed row;
 * team_select_experts / team_moe_forward fill everything with TEAM's choice. */
typedef struct {
  float *probs;           /* [T, E] softmax over all experts (computed rows; others 0)     */
  int32_t *topk_idx;      /* [T, k] descending score, ties to the lower id; -1 if skipped  */
  float *topk_w;          /* [T, k] routing weights                                        */
  float *margin;          /* [T] logit gap between the last expert taken and the best one
                             left out of the candidate set (+inf if none, or skipped)     */
  uint8_t *tok_class;     /* [T] TEAM_CLS_*                                                */
  uint64_t *group_mask;   /* [max_groups, ceil(E/64)] necessary set E_A per group          */
  int32_t *expert_count;  /* [E + n_shared] slots per expert                               */
  int32_t *expert_offset; /* [E + n_shared + 1] exclusive prefix sum of expert_count       */
  int32_t *perm;          /* [T*(k+n_shared)] slot ids grouped by expert (ascending expert,
                             ascending slot id inside); unused tail -1                    */
  int32_t *active;        /* [E + n_shared] ascending ids of experts with count > 0        */
  int32_t *n_active;      /* [1] size of the activated set (the layer's APF, Table 1)      */
  int32_t *n_rows_active; /* [1] rows computed this step                                   */
} team_routing;

/* Create / destroy a context.  team_create allocates the context's device
 * workspace (a few MB at max_rows = 1024) on the current device.
 * Errors: TEAM_ERR_ARG, TEAM_ERR_SHAPE, TEAM_ERR_CUDA. */
int team_create(const team_config *cfg, team_ctx **out);
int team_destroy(team_ctx *ctx);

/* Borrow the layer's weights (device pointers, 16-byte aligned; bf16 expert
 * weights 128-byte aligned).  w_router is required, and at least one complete
 * layout of the expert weights; a call whose expert kernel needs a layout that
 * was not given returns TEAM_ERR_ARG.  May be called again to switch layers; the switch
 * takes effect for calls issued afterwards (pointers are passed by value at
 * launch). */
int team_set_weights(team_ctx *ctx, const team_weights *w);

/* Convert down-projection weights from row-major [n_experts_total, H, I] (src)
 * to the slab layout [n_experts_total, I/16, H, 16] (dst) that team_weights.w_down
 * expects: element (e, h, c) moves to (((e * I/16 + c/16) * H + h) * 16 + c%16).
 * The expert kernels give each group of 16 intermediate columns to one CTA
 * (Eq. 1's down projection, summed over groups); in this layout the 16 columns
 * of all H rows are one contiguous block.  Done once per layer when weights are
 * loaded; needs no context.  src and dst are device pointers, 16-byte aligned,
 * of the same size, not overlapping; both stay owned by the caller.  inter must
 * be a multiple of 16.  Asynchronous on `stream`.
 * Errors: TEAM_ERR_ARG, TEAM_ERR_SHAPE, TEAM_ERR_CUDA. */
int team_pack_w_down(const void *src, void *dst, int n_experts_total, int hidden,
                     int inter, int dtype, void *stream);

/* Tile-major copy of a layer's expert weights for the tensor-memory kernels (bf16): Eq. 1's three projections
 * cut into [128 rows x 64 k] tiles of 16 KB, each contiguous and already in the 128-byte-swizzled K-major layout
 * the tensor core reads, so that a pipeline stage is one bulk copy.
 *   gu_tiles   [n_experts_total][I/64][H/64][128][64]: tile row blk*32 + m*16 + i holds row (u*64 + blk*16 + i) of
 *              W_gate (m = 0) or W_up (m = 1), k-block kb; 16-byte piece p of tile row r is stored at p ^ (r & 7).
 *   down_tiles [n_experts_total][H/128][I/64][128][64]: tile row r holds row ht*128 + r of W_down [H, I], columns
 *              kb*64 ...; same piece swizzle.
 * Sources are row-major device tensors ([.., I, H], [.., I, H], [.., H, I]), 16-byte aligned; destinations are
 * device buffers of the same total size (gu_tiles: both matrices), 128-byte aligned, not overlapping the
 * sources; all stay owned by the caller, who may free the row-major copies afterwards.  hidden must be a
 * multiple of 128, inter of 64.  Asynchronous on `stream`; needs no context.
 * Errors: TEAM_ERR_ARG, TEAM_ERR_SHAPE, TEAM_ERR_CUDA. */
int team_pack_w_tiles(const void *w_gate, const void *w_up, const void *w_down, void *gu_tiles, void *down_tiles,
                      int n_experts_total, int hidden, int inter, void *stream);

/* Change flags / tau_hot / L_hot / hot_dist_inclusive / prefix_decoded /
 * norm_topk / refresh_every of an existing context (shapes and dtype must be unchanged). */
int team_set_policy(team_ctx *ctx, const team_config *cfg);

/* Router (Algorithm 1 "Router", Sec. 4.1 row selection): logits = x W_r^T in
 * fp32 for every computed row, softmax over all experts, plain top-k with
 * renormalised weights and the decision margin.  x: [T, H] row-major, dtype per
 * config.  Logits stay in the context for team_select_experts. */
int team_route(team_ctx *ctx, const void *x, const team_step_state *st, team_routing *out, void *stream);

/* The router step without any allocation.  (The paper has no counterpart; this is a deployment
 * variant of team_route.)
 *
 * Who needs it: code that runs where device allocation is off limits -- a serving loop whose device
 * memory is planned up front and frozen, a plug-in called from inside another framework's stream
 * callback or capture region, a latency-critical path that must not hit the allocator's implicit
 * device synchronisation, or a process whose memory pool is owned by someone else.  Such callers
 * cannot create a team_ctx, because team_create allocates the workspace that holds the logits.
 *
 * What it does: the same two router kernels as team_route (fp32 logits, softmax, plain top-k with
 * renormalised weights, decision margin; cached rows skipped when TEAM_F_DCD is set), with the logits
 * kept in a fixed scratch array that is part of the library image: TEAM_STATIC_ROUTE_MAX_ROWS x
 * TEAM_MAX_EXPERTS floats = 256 KiB on every GPU that loads the library, held until the process
 * exits.  No context is involved: shapes, dtype and policy come from `cfg` (hidden, n_experts, top_k,
 * dtype, flags, norm_topk are read; the rest is ignored), x [T, H] and w_router [E, H] fp32 are
 * caller-owned device memory, `st->tok_state` must be set, and `out` receives probs / topk_idx /
 * topk_w / margin exactly as team_route writes them (NULL members are skipped).
 *
 * Limits and caveats:
 *   - st->n_rows > TEAM_STATIC_ROUTE_MAX_ROWS returns TEAM_ERR_CAPACITY and launches nothing.
 *   - The call never calls cudaMalloc / cudaFree or any allocating routine.  The first call on a
 *     device looks up the scratch array's device address and opts the kernels in to their shared
 *     memory; make that first call outside any stream capture.
 *   - All calls on a device share the one scratch array, which keeps the previous call's contents
 *     (nothing in it needs clearing: every row that is read is rewritten first).  Two calls whose
 *     kernels overlap on the GPU (different streams) race on it; keep them stream-ordered.
 * Errors: TEAM_ERR_ARG, TEAM_ERR_SHAPE, TEAM_ERR_CAPACITY, TEAM_ERR_CUDA. */
int team_route_static(const team_config *cfg, const void *x, const void *w_router, const team_step_state *st,
                      team_routing *out, void *stream);

/* TEAM selection (Eq. 4, Algorithm 1 steps 1-3) and dispatch tables, from the
 * logits left by the preceding team_route on the same context, stream and rows. */
int team_select_experts(team_ctx *ctx, const team_step_state *st, team_routing *out, void *stream);

/* The whole layer step: route, select, dispatch, SwiGLU experts, weighted
 * combine.  y: fp32 [T, H]; rows with class TEAM_CLS_SKIP are left untouched
 * (they keep the previous step's output), all other rows are overwritten.
 * `out` may be NULL; tables nobody asked for may not be built at all (with at
 * most 8 rows the expert kernel works from the rows' choices alone). */
int team_moe_forward(team_ctx *ctx, const void *x, const team_step_state *st, team_routing *out,
                     float *y, void *stream);

/* The same layer step for callers whose buffers live in HOST memory (pageable
 * or pinned): x_host [T, H] in the config's dtype, the five arrays of st_host
 * as host pointers, y_host fp32 [T, H].  The call packs the inputs into a pinned
 * staging block owned by the context, moves them to the device with one copy,
 * runs team_moe_forward on `stream`, copies y back and synchronises the stream
 * before it returns, so y_host is valid on return.  Rows with class
 * TEAM_CLS_SKIP receive what the previous call on this context left in the
 * context's device-side y (zero before the first call): use one context per
 * layer to get "the previous step's output" there.  `out`, if given, holds
 * DEVICE pointers as in team_moe_forward.  The first call on a context allocates
 * the staging block (device and pinned host, (6 H + 17) bytes per row of
 * max_rows for bf16); team_destroy frees it.  Not reentrant per context.
 * On a stream that can be captured (not the legacy default stream, not already
 * capturing) and with `out` NULL, the sequence copy in / kernels / copy out is
 * recorded once per context and row count as a graph and replayed afterwards;
 * team_set_weights, team_set_policy and team_debug_force_simt discard it.
 * Errors: as team_moe_forward. */
int team_moe_forward_host(team_ctx *ctx, const void *x_host, const team_step_state *st_host,
                          team_routing *out, float *y_host, void *stream);

/* Stack glue for a MoE-only multi-layer model: x[t,:] <- x[t,:] + y[t,:] for
 * every row computed by the preceding team_moe_forward (fp32 add, stored in
 * x's dtype, round to nearest even). */
int team_residual_add(team_ctx *ctx, void *x, const float *y, int32_t n_rows, void *stream);

/* Synchronise `stream` and return the device status word (TEAM_OK or the first
 * TEAM_ERR_TIMEOUT / TEAM_ERR_STATE recorded since the last read; reading
 * clears it).  detail_out (optional, host) receives a kernel-specific code. */
int team_read_status(team_ctx *ctx, void *stream, int32_t *detail_out);

/* Number of kernels the last compute call on this context launched. */
int team_last_launch_count(const team_ctx *ctx);

/* Average device time (ms) of the expert kernel over the launches made since
 * the counters were last reset, measured with CUDA events on the launching
 * stream when timing is enabled.  Synchronises the stream. */
int team_expert_timing(team_ctx *ctx, int32_t enable, void *stream, float *avg_ms_out, int32_t *launches_out);

/* Name of the expert kernel this context's team_moe_forward launches (static string), e.g. for labelling a
 * measurement.  NULL context: "". */
const char *team_expert_kernel_name(const team_ctx *ctx);

/* Diagnostic: run the expert FFNs of a bf16 context through the plain-FMA
 * kernels instead of the tensor-core kernel (allocates scratch on first use).
 * Meant for triage of a parity failure, not for production. */
int team_debug_force_simt(team_ctx *ctx, int on);

/* Decode-loop glue of a block (Eq. 2-3; Sec. 4.2 "Speculative Exploration for Hot Tokens"; Sec. 5.4 "Aligned Token
 * Candidates in SEH"): from the outputs of one forward pass over the block's branches -- predicted token and
 * confidence per branch and position -- accept the confident positions (c > tau), verify the speculative branches
 * in a chain, pick the next two candidates, and lay out the rows of the next forward pass for team_moe_forward.
 *
 * Branches (n_branches = 4; Sec. 5.1): 0 = base, 1 = base + 1st-confidence candidate accepted, 2 = base + 2nd,
 * 3 = base + both.  A candidate is confirmed in a branch when that branch predicts the speculated token at its
 * position with c > tau.  The base branch is always trusted; branch 1 after it if the 1st candidate is confirmed in
 * the base branch, then branch 3 if the 2nd is confirmed in branch 1; else branch 2 if the 2nd is confirmed in the
 * base branch, then branch 3 if the 1st is confirmed in branch 2.  Every masked position with c > tau in a trusted
 * branch is accepted with the prediction of the first trusted branch that accepts it; confirmed candidates are
 * accepted with their speculated tokens.  Accepted tokens are TEAM_TOK_NEW at the next step, the previous NEW ones
 * TEAM_TOK_CACHED (Sec. 4.1).  The next candidates are the two masked positions with the highest confidences in the
 * last trusted ("adopted") branch, ties to the lower position.  n_branches = 1 is plain threshold decoding (Eq. 3).
 *
 * All pointers are device memory owned by the caller.  team_seh_state persists over the steps of a block:
 *   token [S, L] int32 (-1 while masked), state [S, L] uint8 TEAM_TOK_*, spec_pos / spec_tok [S, 2] int32 (the
 *   candidates the given forward pass was run with; rewritten with the next ones), counters [S, 2] int32 (forward
 *   passes, accepted tokens; optional).
 * pred int32 / conf fp32 [S, n_branches, L]: the forward pass's outputs; both NULL begins a block (everything masked,
 *   no candidates, counters zeroed).
 * team_seh_rows: the next forward pass's step state, [S * n_branches * L] each, rows ordered [sequence][branch]
 *   [position], group = sequence; conf is the adopted branch's for masked positions and 1 for decoded ones.
 * adopted_out [S] int32 (optional): the adopted branch.  block <= TEAM_MAX_BLOCK, S * n_branches * block <=
 * TEAM_MAX_ROWS.  Asynchronous on `stream`; needs no context.
 * Errors: TEAM_ERR_ARG, TEAM_ERR_SHAPE, TEAM_ERR_CUDA. */
typedef struct { int32_t n_seqs, block, n_branches; float tau; } team_seh_config;
typedef struct { int32_t *token; uint8_t *state; int32_t *spec_pos; int32_t *spec_tok; int32_t *counters; } team_seh_state;
typedef struct { uint8_t *tok_state; float *conf; int32_t *pos; int32_t *group; int32_t *branch; } team_seh_rows;
int team_seh_step(const team_seh_config *cfg, const team_seh_state *state, const int32_t *pred, const float *conf,
                  const team_seh_rows *rows, int32_t *adopted_out, void *stream);

/* The attention half of delayed caching (Sec. 4.1; block diffusion, Sec. 2): one attention layer of one denoising
 * step over the block being decoded.  Attention is bidirectional inside the block and runs over the cached keys /
 * values of earlier blocks (the prefix).  Rows of cached tokens are not computed (flags & TEAM_F_DCD): they have no
 * query, their output rows are left untouched, and the other rows see their keys / values from the in-block cache;
 * after the pass the keys / values of the decoded rows computed in the base branch (branch 0) -- the tokens newly
 * accepted in the previous step -- are inserted into that cache at their positions (delayed insertion).  A token
 * that only a speculative branch treats as accepted is not inserted: the cache is shared by a sequence's branches.
 *
 * Rows are ordered [sequence][branch][position] and every (sequence, branch) presents its whole block:
 * st->n_rows = n_seqs * n_branches * block, pos = 0 .. block-1 inside each run, group = sequence (a row that breaks
 * this sets TEAM_ERR_STATE in `status`; conf is not read).  All pointers are device memory owned by the caller, 16-byte
 * aligned; bf16 unless stated:
 *   q [T, n_heads, head_dim]; k_new, v_new [T, n_kv_heads, head_dim] (this pass's projections of the rows);
 *   k_prefix, v_prefix [n_seqs, max_prefix, n_kv_heads, head_dim] with prefix_len [n_seqs] int32 valid entries;
 *   k_block, v_block [n_seqs, block, n_kv_heads, head_dim]: the in-block cache, read and then updated;
 *   out fp32 [T, n_heads, head_dim]: softmax(q k^T / sqrt(head_dim)) v over prefix + block, computed rows only;
 *   status int32 [2] (optional): first device-detected problem (code, detail), to be zeroed by the caller.
 * Query head h uses key / value head h / (n_heads / n_kv_heads).  head_dim is 64 or 128, block <= TEAM_MAX_BLOCK.
 * Asynchronous on `stream`; needs no context.  Errors: TEAM_ERR_ARG, TEAM_ERR_SHAPE, TEAM_ERR_CUDA. */
typedef struct { int32_t n_heads, n_kv_heads, head_dim, block, n_seqs, n_branches, max_prefix, flags; } team_attn_config;
int team_block_attention(const team_attn_config *cfg, const team_step_state *st, const void *q, const void *k_new,
                         const void *v_new, const void *k_prefix, const void *v_prefix, const int32_t *prefix_len,
                         void *k_block, void *v_block, float *out, int32_t *status, void *stream);

/* Diagnostic knobs of a context (not for production use).
 *   TEAM_KNOB_NO_FUSE (value 0/1): with at most 8 rows and no dispatch table asked for, team_moe_forward runs the
 *     whole step as one kernel; 1 keeps the three-kernel sequence (router, selection, experts) instead.
 *   TEAM_KNOB_WAIT_LIMIT_US (1 .. 10,000,000): how long a device-side wait (the one-kernel step's grid barrier) may
 *     last before the kernel gives up, records TEAM_ERR_TIMEOUT in the status word and returns; default about 1 s.
 *   TEAM_KNOB_EXTRA_ARRIVALS (0/1): 1 makes that barrier wait for one arrival that never comes, so that the
 *     give-up path can be exercised (with a short limit) without any kernel hanging; y is then left unspecified
 *     for the computed rows of that call.
 *   TEAM_KNOB_EXPERT_KERNEL (0/1/2): 0 lets max_rows choose the expert kernel of a bf16 context, 1 asks for the
 *     weight-streaming kernel, 2 for the tensor-memory kernels (ignored where the shape does not allow the kernel);
 *     the weight layout that kernel reads must have been given.
 *   TEAM_KNOB_ORDERED_COMBINE (0/1): the weighted combine normally adds the experts' contributions into y with fp32
 *     reductions, whose order (hence the last bits of y) varies from run to run.  1 makes the one-kernel step keep
 *     one partial output per CTA and sum them in CTA order behind a second grid barrier: two runs are then identical
 *     bit for bit, which tells a race from a rounding difference.  Allocates n_SMs x max_rows x H floats on first
 *     use; only for contexts of at most 8 rows on hidden size 1024 or 2048 (else TEAM_ERR_SHAPE); a few us slower.
 * Errors: TEAM_ERR_ARG, TEAM_ERR_SHAPE, TEAM_ERR_CUDA. */
enum { TEAM_KNOB_NO_FUSE = 1, TEAM_KNOB_EXTRA_ARRIVALS = 2, TEAM_KNOB_WAIT_LIMIT_US = 3, TEAM_KNOB_EXPERT_KERNEL = 4,
       TEAM_KNOB_ORDERED_COMBINE = 5 };
int team_debug_knob(team_ctx *ctx, int knob, long long value);

const char *team_strerror(int code);
const char *team_last_cuda_error(const team_ctx *ctx);
int team_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TEAM_H_ */
