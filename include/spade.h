/* spade.h -- C ABI of the B200 (sm_100a) SPADE hot path: input-adaptive 3-D block-sparse
 * self-attention for video diffusion transformers.
 *
 * One attention layer is four device stages, called in this order on one CUDA stream:
 *
 *   spade_plan       scheme generation: SICS / Aggregation Score of every blocking candidate per
 *                    head (Eq. 3-5, Algorithm 1), argmax candidate per head (Sec. 3.2), budget ->
 *                    per-head keep count, heads grouped by chosen scheme (Sec. 3.3, optimisation 2)
 *   spade_summarize  Summarizer: mean of Q and of K over each 3-D block of the chosen scheme
 *                    (Sec. 3.1 "Summarizer Expression", Sec. 3.3: summaries Q', K')
 *   spade_select     Estimator + index search: block scores <Q'_i, K'_j>/sqrt(d), softmax over KV
 *                    blocks, Top-K or Top-P (cumulative mass) per (head, query block), emitted as
 *                    ascending index lists (Sec. 3.1, Fig. 4c; Sec. 3.3 "ranked BSR")
 *   spade_attn       flash block-sparse attention over the listed blocks only (Eq. 2; Sec. 3.3,
 *                    optimisation 3), output in the original token order
 *
 * Conventions
 *   - Q, K, V, O: DEVICE pointers, bf16, contiguous [B, heads, N, d], d = 128, 16-byte aligned.
 *     N = T*H*W + n_text; token n = (t*H + h)*W + w (Sec. 2.1); the n_text text tokens are the
 *     LAST rows of N.  Every query block always attends all text blocks and every text query
 *     block attends all blocks; text is outside scoring and outside the Aggregation Score.
 *   - A blocking candidate (bt, bh, bw) (order T, H, W, Fig. 3) must have bt*bh*bw in {64, 128}.
 *     Grids need not divide: edge blocks are partial, absent positions take part in nothing.
 *   - `ws` is a caller-allocated DEVICE workspace of spade_workspace_bytes() bytes, 256-byte
 *     aligned, passed to every stage; it carries all tables between stages.  The library
 *     allocates device memory only inside spade_plan_create (small per-candidate tables, freed
 *     by spade_plan_destroy).  A plan and a workspace serve one layer at a time: calls on the same
 *     plan must not overlap in time (host threads) and a workspace must not be used by two layers
 *     that may run concurrently (streams); use one plan and one workspace per concurrent layer.
 *     The attention and estimator kernels take their tensor-memory columns with tcgen05.alloc, the one
 *     device-side wait of this library that has no time limit (the instruction has none): two layers
 *     launched on two streams are correct but take turns on an SM's tensor memory rather than overlap.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Stage calls are
 *     asynchronous and never synchronise the host.  Every call makes the plan's device current
 *     while it runs and restores the caller's current device before it returns.
 *   - B * heads may be at most 4096.
 *   - Every function returns SPADE_OK (0) or a negative spade_error_t; arguments are validated
 *     before anything is launched; nothing aborts.  spade_last_error() gives the message.
 *   - There is no CPU path: without a CUDA device every stage returns SPADE_ERR_CUDA.
 *   - Debug build (compile the sources with -DSPADE_DEBUG; the Python binding loads it when the environment
 *     has SPADE_DEBUG=1): every index a kernel takes from an index list, a histogram or a table is checked
 *     before use.  A failed check never traps or faults: it is counted in the status words with the site and
 *     the offending value, the access is skipped, and spade_status returns SPADE_ERR_DEBUG_CHECK.  The
 *     workspace then also carries a 256-byte guard word behind every region (spade_workspace_bytes grows
 *     accordingly), written by spade_plan and verified by spade_status.
 */
#ifndef SPADE_H_
#define SPADE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SPADE_OK = 0,
  SPADE_ERR_INVALID_ARG = -1,     /* null pointer, non-positive size, bad mode / value, misaligned pointer */
  SPADE_ERR_UNSUPPORTED = -2,     /* d != 128, block size not in {64,128}, more than 2048 blocks, > 8 candidates, B*heads > 4096 */
  SPADE_ERR_WORKSPACE = -3,       /* workspace pointer null or misaligned */
  SPADE_ERR_CUDA = -4,            /* a CUDA runtime / driver call failed (message holds the CUDA error) */
  SPADE_ERR_DEVICE_TIMEOUT = -5,  /* a bounded device-side wait ran out (reported by spade_status) */
  SPADE_ERR_ORDER = -6,           /* stage called before the stage it depends on */
  SPADE_ERR_DEBUG_CHECK = -7      /* debug build only: an index check inside a kernel failed, or a guard word behind a
                                     workspace region was overwritten (reported by spade_status) */
} spade_error_t;

typedef struct spade_plan_s spade_plan_t;   /* opaque; created and destroyed by the library */

typedef struct { int32_t T, H, W; int32_t n_text; } spade_grid_t;
typedef struct { int32_t bt, bh, bw; } spade_blocking_t;

typedef enum { SPADE_TOPK = 0, SPADE_TOPP = 1, SPADE_SPARSITY = 2, SPADE_POLICY_AS = 3 } spade_mode_t;

/* Budget of the index search (the "inter-top value" of Sec. 3.1).
 *   SPADE_TOPK      value = k: keep the k highest-scoring video KV blocks per query block
 *                   (clamped to [1, number of video KV blocks]); ties -> lower block id.
 *   SPADE_TOPP      value = p in (0, 1]: keep the shortest prefix of the descending order whose
 *                   softmax mass reaches p (at least one block).
 *   SPADE_SPARSITY  value = s in [0, 1): Top-K with k_h = clamp(ceil((1-s)*NKB_h - 1e-9), 1, NKB_h),
 *                   NKB_h = video KV blocks under head h's scheme.
 *   SPADE_POLICY_AS an example policy function (Sec. 3.1: the budget follows the head's Selected Aggregation
 *                   Score, negatively correlated, Sec. 4.4): value = mean target sparsity s, `gain` >= 0; with
 *                   a_h the selected normalised score and a_bar its mean over all heads, head h keeps the
 *                   fraction f_h = clamp((1-s) * (1 - gain*(a_h - a_bar)/a_bar), 1/NKB_h, 1) of its video KV
 *                   blocks (Top-K with k_h = ceil(f_h*NKB_h - 1e-9)).  Computed on the device in spade_plan;
 *                   with forced schemes the Aggregation Scores are still computed.
 * per_head: optional HOST array of B*heads values overriding `value` per head (copied at create; not used
 * by SPADE_POLICY_AS).  gain: only read in SPADE_POLICY_AS mode. */
typedef struct { int32_t mode; float value; const float* per_head; float gain; } spade_budget_t;

/* Create a plan for a fixed problem shape.  `cands` is a HOST array of n_cands (1..8) candidates.
 * `device` is the CUDA device ordinal the plan (and all later calls with it) works on. */
int spade_plan_create(spade_plan_t** out, int32_t B, int32_t heads, int32_t d, const spade_grid_t* grid,
                      const spade_blocking_t* cands, int32_t n_cands, const spade_budget_t* budget, int32_t device);
int spade_plan_destroy(spade_plan_t* plan);

/* Static and intra-block masks united with the dynamic selection (Sec. 3.3: intra scores are OR-combined
 * with the inter scores, the result is united with local-window and attention-sink masks).
 *   intra_threshold  a block whose mean pairwise cosine SICS / n^2 is below it is never pruned: as a KV
 *                    block it is kept by every query block, as a query block it keeps every block
 *                    (<= 0 disables).  Uses the SICS of K resp. Q under the head's chosen scheme.
 *   window           query block i keeps KV block j when their block-grid coordinates differ by at most
 *                    `window` along every axis (< 0 disables).
 *   sink_tokens      KV blocks that hold any of the first `sink_tokens` tokens are kept by every query block.
 * Call before spade_workspace_bytes(): with any mask enabled a row can list every block, so the index
 * lists get full capacity and the workspace grows.  NULL or all-disabled restores the plain selection. */
typedef struct { float intra_threshold; int32_t window; int32_t sink_tokens; } spade_static_mask_t;
int spade_plan_set_masks(spade_plan_t* plan, const spade_static_mask_t* masks);

/* Summarizer and Estimator Expressions (Sec. 3.1, Fig. 4): which block summaries the inter-block
 * estimator of spade_select works on.
 *   SPADE_EST_MEAN  mean summaries, S[i,j] = <q_mean_i, k_mean_j> / sqrt(d)  (Fig. 4c; the default)
 *   SPADE_EST_DSA   channel-wise max / min summaries, q~ = (q_max + q_min) / 2,
 *                   S[i,j] = sum_c max(q~_c kmax_jc, q~_c kmin_jc) / sqrt(d)   (Fig. 4a)
 *   SPADE_EST_DSA2  S[i,j] = sum_c max over {qmax_ic, qmin_ic} x {kmax_jc, kmin_jc} of the product / sqrt(d) (Fig. 4b)
 * The figure's equations are not part of the paper's text; the two max/min forms are this library's
 * reading: the dot product of two vectors picked channel by channel from the summaries, an upper bound
 * of q.k / sqrt(d) over the boxes the summaries span.  spade_summarize then also leaves the max / min
 * summaries of the video blocks in the workspace, and spade_select scores with them; softmax, Top-K /
 * Top-P, the static masks and the attention stage are unchanged.  Call before spade_workspace_bytes():
 * the workspace grows by 4 * B * heads * 128 * ld floats (ld = the largest video block count, rounded up to 64).  Unknown values: SPADE_ERR_INVALID_ARG. */
typedef enum { SPADE_EST_MEAN = 0, SPADE_EST_DSA = 1, SPADE_EST_DSA2 = 2 } spade_estimator_t;
int spade_plan_set_estimator(spade_plan_t* plan, int32_t estimator);

/* Bytes of device workspace the stages need for this plan (0 if plan is NULL). */
size_t spade_workspace_bytes(const spade_plan_t* plan);

/* Stage 1 (Eq. 3-5, Algorithm 1; Sec. 3.2).  forced_scheme: optional HOST array of B*heads
 * candidate indices; if non-NULL the Aggregation Scores are not computed and each head takes
 * the given candidate.  The array is read before the call returns and never afterwards, pinned or
 * not: the schemes travel as an argument of the launch, so a launch captured in a CUDA graph replays
 * the schemes it was captured with. */
int spade_plan(spade_plan_t* plan, const void* Q, const void* K, void* ws, void* stream, const int32_t* forced_scheme);
/* Stage 2 (Sec. 3.1, 3.3).  Needs spade_plan on the same workspace first. */
int spade_summarize(spade_plan_t* plan, const void* Q, const void* K, void* ws, void* stream);
/* Stage 3 (Sec. 3.1, 3.3).  Needs spade_summarize first. */
int spade_select(spade_plan_t* plan, void* ws, void* stream);
/* Stage 4 (Eq. 2; Sec. 3.3).  Needs spade_select first, or lists written by the caller into the
 * kv_idx / kv_cnt tables (see spade_get_tables) after spade_plan. */
int spade_attn(spade_plan_t* plan, const void* Q, const void* K, const void* V, void* O, void* ws, void* stream);

/* All four stages back to back on `stream`. */
int spade_forward(spade_plan_t* plan, const void* Q, const void* K, const void* V, void* O, void* ws, void* stream,
                  const int32_t* forced_scheme);

/* End-to-end call with HOST tensors: copies hQ, hK, hV (host, same layout as the device tensors) into the
 * caller-provided device buffers dQ, dK, dV, runs the four stages, copies dO back into hO and returns
 * when all of it is done.  Heads are independent, so the call works on up to 12 chunks of heads (shrinking in size) and
 * overlaps the copies of one chunk with the kernels of another (two internal copy streams; the host
 * tensors must be pinned for the overlap, pageable memory still gives correct results).  Results are
 * identical to spade_forward on the same tensors.  SPADE_POLICY_AS budgets couple the heads and run as one
 * chunk.  On return the workspace tables describe only the last chunk: call spade_plan again before
 * spade_get_tables or a stage call.  Work already queued on `stream` finishes before the first copy. */
int spade_forward_host(spade_plan_t* plan, const void* hQ, const void* hK, const void* hV, void* hO,
                       void* dQ, void* dK, void* dV, void* dO, void* ws, void* stream, const int32_t* forced_scheme);

/* Device tables inside the workspace (valid while `ws` lives), for tests and benchmarks.
 * BH = B*heads, C = n_cands, NBmax = max over candidates of (video + text blocks). */
typedef struct {
  int32_t BH, C, NBmax, cap;      /* cap = row capacity of kv_idx */
  int32_t* scheme;                /* [BH]            chosen candidate per head */
  int32_t* keep;                  /* [BH]            Top-K keep count per head (0 in Top-P mode) */
  float*   as;                    /* [BH][C][2]      raw Aggregation Score of Q and of K */
  float*   score;                 /* [BH][C]         (AS(Q)+AS(K)) / (2*sum_i n_i^2) */
  float*   sics;                  /* [BH][C][2][NBvmax] per-block SICS (video blocks) */
  int32_t  NBvmax;
  float*   qsum;                  /* [BH][NBmax][128] Q' */
  float*   ksum;                  /* [BH][NBmax][128] K' */
  int32_t* kv_idx;                /* [BH][NBmax][cap] ascending kept KV block ids per query block */
  int32_t* kv_cnt;                /* [BH][NBmax] */
  int32_t* head_order;            /* [BH]            order in which the attention stage takes the heads: grouped by scheme after
                                     spade_plan, by decreasing list length per query tile after spade_select */
  int32_t* group_count;           /* [C]             heads per scheme */
  int32_t* item_start;            /* [BH+1]          prefix of attention work items over head_order */
  uint8_t* cell_axis;             /* [BH][cell_ld]   64-token schemes: axis (0 t, 1 h, 2 w) along which the query blocks of a 2 x 2 x 2 cell of
                                     the block grid pair into 128-row tiles (see spade_get_pair_table) */
  uint32_t* status;               /* [4]             device status words (0 = ok) */
  float*   minmax;                /* [4][BH][128][ld] channel-major max/min summaries of the video blocks, ld = block_scores_ld
                                     (NULL with SPADE_EST_MEAN): plane 0 = q_max (SPADE_EST_DSA2) or (q_max + q_min) / 2
                                     (SPADE_EST_DSA), 1 = q_min, 2 = (k_max + k_min) / 2, 3 = (k_max - k_min) / 2 */
  float*   block_scores;          /* [BH][NBvmax][ld] estimator output S of the chosen scheme, ld = block_scores_ld */
  int32_t  block_scores_ld;
  int32_t  cell_ld;
} spade_tables_t;
int spade_get_tables(const spade_plan_t* plan, void* ws, spade_tables_t* out);

/* Per-candidate geometry as the library sees it: out[0..5] = blocks along T, H, W, video blocks,
 * text blocks, block size. */
int spade_get_geometry(const spade_plan_t* plan, int32_t cand, int32_t* out6);

/* How the attention stage pairs the 64-token query blocks of candidate `cand` into 128-row tiles (Sec. 3.3: the
 * kernel's tile is 128 rows).  The block grid is cut into cells of 2 x 2 x 2 blocks (fewer at an odd end); after the
 * index search every head picks, per cell, the axis along which its blocks pair so that the merged lists are shortest
 * (cell_axis of spade_tables_t).  For video tile t: tile_cell[t] = its cell; pairs[3 t + a] = qb0 | qb1 << 16 are its
 * blocks when the cell pairs along axis a (qb1 = 0xffff: a lone block).  Host arrays of the returned length (and three
 * times it), either may be NULL.  Returns the number of video tiles, 0 for a 128-token candidate, or a negative code. */
int spade_get_pair_table(const spade_plan_t* plan, int32_t cand, int32_t* tile_cell, uint32_t* pairs);

/* Synchronises `stream` and returns SPADE_OK, SPADE_ERR_DEVICE_TIMEOUT (a bounded wait inside a
 * kernel gave up; the output of that call is invalid) or SPADE_ERR_CUDA. */
int spade_status(spade_plan_t* plan, void* ws, void* stream);

/* Failure-detection self-test (no paper counterpart; Sec. 3.3's kernels have device-side waits, and every
 * such wait in this library is bounded).  Launches one warp that waits, with the library's bounded wait
 * and a limit of `limit_us` microseconds (1 .. 1 000 000), on a barrier that nothing completes.
 * out4: DEVICE pointer to 4 uint32: [0] = 1 if the wait gave up, [1] = 1 if it raised the abort flag the
 * attention kernel's other roles poll, [2..3] = elapsed SM cycles (low, high).  Asynchronous on `stream`;
 * the context stays usable afterwards. */
int spade_selftest_bounded_wait(void* out4, int32_t limit_us, void* stream);

/* Number of kernels launched by the last spade_forward / stage sequence on this plan. */
int spade_launch_count(const spade_plan_t* plan);

/* Aggregation Scores without any allocation (the paper has no counterpart: this entry point
 * exists for callers, not for the method).
 *
 * Some code that wants the per-candidate Aggregation Scores cannot obtain device memory at the
 * moment it runs: a plugin living inside another framework whose caching allocator owns the whole
 * device, a service with a fixed, pre-reserved memory budget, or a latency-critical loop where a
 * cudaMalloc (which may synchronise the device) is off the table.  For them this call computes what
 * spade_plan leaves in its `as` table -- AS(Q|c) and AS(K|c) for every head and candidate -- but
 * needs no workspace: the per-block SICS values, which the other path keeps in the caller's
 * workspace, go to a fixed array that is part of the library image itself.  The two entry points
 * agree to fp32 rounding, not bit for bit: this one always reduces each block from its token rows,
 * spade_plan usually adds up per-cell sums shared by all candidates, a different summation order.
 *
 *   as_out   DEVICE pointer, float [B*heads][n_cands][2] (Q then K), written by the call.
 *   Q, K     as for spade_plan.
 *
 * Limit: B*heads * n_cands * 2 * (largest video-block count of any candidate) must not exceed
 * SPADE_NOALLOC_MAX_FLOATS (1 Mi floats = 4 MiB); larger plans get SPADE_ERR_UNSUPPORTED and
 * nothing is launched.  Every GPU that loads the library carries those 4 MiB until the process exits.
 * The call performs no cudaMalloc / cudaFree and calls no allocating library routine.  The first
 * call on a device looks up the array's device address (once per device, with that device
 * current); make that first call outside any stream capture.  That look-up is also the moment the
 * CUDA runtime loads this library's device code on that GPU, the 4 MiB included, if nothing of the
 * library ran there before: on a device another allocator has filled to the brim this is where
 * SPADE_ERR_CUDA (out of memory) can still come from, so make the first call at start-up.  The
 * address is remembered for the life of the device's primary context; after cudaDeviceReset the
 * process must not call this entry point again.  All calls on one device share the
 * array and it keeps whatever the previous call left in it; every value a call reads it has
 * written itself first, so nothing has to be cleared -- but two calls whose kernels overlap in
 * time on the same GPU (different streams, different plans, different threads) race on it:
 * serialise them.  Asynchronous on `stream` like the other stages. */
#define SPADE_NOALLOC_MAX_FLOATS (1u << 20)
int spade_aggregation_scores_noalloc(spade_plan_t* plan, const void* Q, const void* K, float* as_out, void* stream);

/* Thread-local message of the last failing call; never NULL. */
const char* spade_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* SPADE_H_ */
