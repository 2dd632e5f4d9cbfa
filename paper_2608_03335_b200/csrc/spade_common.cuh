// Shared declarations of the SPADE CUDA library (sm_100a): geometry of the blocking candidates,
// the workspace tables and the kernel launchers the C-ABI layer calls.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#define SPADE_MAX_CANDS 8
#define SPADE_MAX_NB 2048          // blocks per head (video + text) the kernels are sized for
#define SPADE_D 128

// One blocking candidate (bt, bh, bw), order (T, H, W) as in Fig. 3, on the plan's grid.
struct CandGeo {
  int bt, bh, bw;
  int nbt, nbh, nbw;     // blocks along each axis (ceil division: edge blocks are partial)
  int NBv, NBt, NB, BS;  // video blocks, text blocks, total, nominal block size (64 or 128)
  int pair;              // 1 when BS == 64: two consecutive query blocks share one 128-row tile
  int tiles;             // upper bound of attention work items per head
  int ctiles;            // pair schemes: video query tiles (blocks are paired inside 2 x 2 x 2 cells of the block grid, along an axis chosen per cell)
  int ncell;             // pair schemes: cells of the block grid = ceil(nbt/2) * ceil(nbh/2) * ceil(nbw/2)
  int pt_off, pc_off;    // pair schemes: offsets of this candidate's rows in the tile tables (pair_tab, tile_cell) and in cell_tile0
  int ttiles;            // pair schemes: text query tiles = ceil(NBt / 2)
  int unit_off;          // prefix of NBv over candidates (unit decoding of the SICS pass)
  int tab_off;           // offset of this candidate's rows in the per-block tables (nvalid, kvalid)
  float inv_z;           // 1 / (2 * sum_i n_i^2): normaliser of the Aggregation Score
  int kt, kh, kw;        // extents of a 64-row K/V box: the block itself (BS 64) or its first half (BS 128)
  int ht, hh, hw;        // origin offset of the second half of a 128-token block (0 for BS 64)
  uint32_t mag_w, mag_hw; // floor(2^32 / nbw) + 1 and floor(2^32 / (nbw * nbh)) + 1: block id -> (it, ih, iw) with two high
                         // multiplies (exact for ids below 2^16) instead of three divisions
};

// Block id -> block coordinates along (t, h, w), for ids below 2^16.
__host__ __device__ __forceinline__ void block_coords(const CandGeo& g, int blk, int& it, int& ih, int& iw) {
#ifdef __CUDA_ARCH__
  it = g.mag_hw ? (int)__umulhi((unsigned)blk, g.mag_hw) : blk;          // 0 stands for a divisor of 1
  const int rem = blk - it * (g.nbw * g.nbh);
  ih = g.mag_w ? (int)__umulhi((unsigned)rem, g.mag_w) : rem;
  iw = rem - ih * g.nbw;
#else
  iw = blk % g.nbw; ih = (blk / g.nbw) % g.nbh; it = blk / (g.nbw * g.nbh);
#endif
}

struct Shape {
  int BH, N, Nv, n_text, T, H, W, C;
  int NBmax, NBvmax, cap;   // max blocks over candidates, max video blocks, kv_idx row capacity
  int units_per_ht;         // sum over candidates of NBv
  int mode;                 // spade_mode_t
  float value;
  float gain;               // SPADE_POLICY_AS: strength of the (negative) coupling of the budget to the score
  // Cell decomposition: the common refinement of all candidates (per-axis gcd of their extents).
  // Every block of every candidate is a union of whole cells, so one pass over the tokens that
  // leaves per-cell sums serves all candidates.  use_cells = 0 when a cell would hold < 4 tokens.
  int use_cells;
  int ct, ch, cw;           // cell extents (powers of two)
  int lcw, lch;             // log2(cw), log2(ch)
  int nct, nch, ncw, NCELL; // cells along each axis, cells per head
  int CS;                   // tokens per full cell
  int ld_scores;            // row length of the block-score scratch (NBvmax rounded up to 64)
  int bits_ld;              // 32-bit words per row of the list bitmaps (ld_scores / 32)
  int cell_ld;              // bytes per head of the cell-axis table (largest cell count over the pair candidates, rounded up to 16)
  // static / intra-block masks united with the dynamic selection (masks_on = any of them enabled)
  int masks_on, window, sink;
  float intra_thr;
  int estimator;            // spade_estimator_t: 0 mean*mean, 1 / 2 the max/min-summary estimators
};

// Read-only per-candidate tables owned by the plan (device memory).
struct StaticTables {
  const uint32_t* rowoff;   // [C][128]  in-block row r -> dt<<20 | dh<<10 | dw
  const int* nvalid;        // [sum NB_c] valid tokens per block
  const uint64_t* kvalid;   // [sum NB_c][2] bit r set <=> in-block row r is a real token
  const float* budget;      // [BH] per-head budget value (k, p or sparsity)
  // pair schemes (64-token blocks): the video tiles of a cell are consecutive; a tile's two blocks depend on the cell's axis
  const uint32_t* pair_tab; // [sum ctiles][3] tile, axis (0 t, 1 h, 2 w) -> qb0 | qb1 << 16 (0xffff: lone block); an axis along which the
                            // cell is one block wide repeats the entry of one that is not
  const int* tile_cell;     // [sum ctiles] tile -> cell
  const int* cell_tile0;    // [sum (ncell + 1)] cell -> its first tile
};

// Pointers into the caller's workspace.
struct WsTables {
  uint32_t* status;     // [64]
  int* scheme;          // [BH]
  int* keep;            // [BH]
  float* pthr;          // [BH]
  float* as;            // [BH][C][2]
  float* score;         // [BH][C]
  float* sics;          // [BH][C][2][NBvmax]
  float* qsum;          // [BH][NBmax][128]
  float* ksum;          // [BH][NBmax][128]
  float* ksplit;        // [BH][2][NBmax][128] K' split for the tensor-core estimator: nearest TF32 value, remainder
  int* kv_idx;          // [BH][NBmax][cap]
  int* kv_cnt;          // [BH][NBmax]
  int* head_order;      // [BH] order in which the attention kernel takes the heads
  float* head_work;     // [BH] sort key behind head_order
  int* group_count;     // [C]
  int* item_start;      // [BH+1]
  int* text_start;      // [BH+1] prefix of the text query tiles over head_order (they are scheduled first)
  float* cells;         // [BH][2 tensors][NCELL][2 (sum of q/|q|, sum of q)][128]
  float* csum;          // [BH][2 tensors][C][NBmax][128] mean summaries of every candidate
  float* nsum;          // same shape: sum over a block's tokens of q / |q| (one-pass scheme generation only)
  uint8_t* cell_axis;   // [BH][cell_ld] axis (0 t, 1 h, 2 w) along which the 64-token query blocks of a cell are paired into 128-row tiles
  int* pair_union;      // [BH][4] total merged-list length for each pairing axis; [3] = blocks listed over the head's video query rows
  uint32_t* rowbits;    // [BH][NBvmax][bits_ld] the video part of every video query block's list as a bitmap (bit j = KV block j kept)
  uint8_t* colkeep;     // [BH][NBmax] KV block kept by every query block (intra rule on K, sink)
  uint8_t* rowfull;     // [BH][NBmax] query block keeps every block (intra rule on Q)
  float* scores;        // [BH][NBvmax][ld_scores] block scores S = Q'K'^T / sqrt(d) of the chosen scheme
  uint32_t* att_scratch; // [2 * #SMs CTAs][2][SPADE_MAX_NB] merged index lists of the attention kernel's work items
  float* mm;            // [4][BH][128][ld_scores] channel-major max / min summaries (planes: see k_minmax)
  float* qmid;          // [BH][NBmax][128] (q_max + q_min) / 2 row-major (SPADE_EST_DSA: operand A of the tensor-core estimator)
  float* kdsa;          // [BH][4][NBmax][128] k_mid and k_half, each split into nearest TF32 value and remainder
};

struct GeoPack { CandGeo g[SPADE_MAX_CANDS]; };

// Forced schemes travel as a kernel argument (4 bits per head), so a launch -- also one captured in a
// CUDA graph -- holds its own copy and no host array has to outlive the call.
#define SPADE_MAX_BH 4096                        // B * heads a plan may have
struct ForcedPack {
  int on;                                        // 0: argmax of the Aggregation Score, 1: schemes packed below
  uint32_t w[SPADE_MAX_BH / 8];
};

enum : uint32_t {
  SPADE_ST_OK = 0,
  SPADE_ST_TIMEOUT = 1,     // status[0]: a bounded wait gave up; status[1] = where, status[2] = item
};
// Status words: [0..2] as above, [4] number of failed index checks of the debug build, [5] site of the first
// one, [6] the offending value, [8] work-item counter of the attention kernel, [9] / [10] tickets by which the last CTA
// of the scheme-choice / pairing-axis kernel finds out that it is the last (left at zero by that CTA).

// Debug build (-DSPADE_DEBUG): every index taken from a list, a histogram or a table is checked before use.
// A failed check never traps: it is counted in the status words, the first site and value are kept, and the
// access is skipped; spade_status reports it.  In the release build the macro is the constant `true`.
#ifdef SPADE_DEBUG
__device__ __forceinline__ bool spade_dbg_check(bool ok, uint32_t* status, uint32_t site, uint32_t value) {
  if (!ok && atomicAdd(status + 4, 1u) == 0u) { status[5] = site; status[6] = value; }
  return ok;
}
#define SPADE_CHECK(cond, status, site, value) spade_dbg_check((cond), (status), (site), (uint32_t)(value))
#else
#define SPADE_CHECK(cond, status, site, value) (true)
#endif

// Configuration of the one-pass scheme-generation kernel (plan.cu); on = 0 when the candidate set does not
// fit it (a block footprint above 128 tokens in the (h, w) plane, more than 64 blocks of all candidates in one
// column slice) and the cell tables serve instead.
struct PlanFusedCand {
  int lbt, bt_mask;        // log2(bt), bt - 1
  int lbh, lbw;            // log2 of the block extents along h and w
  int cbw, lcbw, nblk;     // blocks per column along w (and its log2), blocks per column slice
  int slot_base;           // first slot of this candidate's blocks among the slots of a slice
};
struct PlanFusedCfg {
  int on;
  int colH, colW, lcolW;   // column footprint in the (h, w) plane: 128 tokens, a multiple of every candidate's (bh, bw)
  int ncol_h, ncol_w;      // columns over the grid
  int tchunk, nchunks;     // slices per work item (a multiple of every candidate's bt) and chunks over T
  int stages;              // ring of slices in shared memory
  int nblk;                // slots: blocks of all candidates in one column slice
  int cpw;                 // 32-column chunks (8 slots each) per epilogue warpgroup; rows of the weight matrix = 64 * cpw
  int nrows;
  int text_blocks;         // text blocks over all candidates
  PlanFusedCand cand[SPADE_MAX_CANDS];
  unsigned char slot_cand[64];   // slot -> candidate
};

// ---- launchers (definitions in the .cu files) ------------------------------------------------
cudaError_t launch_sics(const void* Q, const void* K, const Shape& sh, const GeoPack& gp, const StaticTables& st,
                        const WsTables& ws, int num_sms, cudaStream_t s);
cudaError_t launch_cells(const void* Q, const void* K, const Shape& sh, const WsTables& ws, int num_sms, cudaStream_t s);
cudaError_t launch_blocks(const void* Q, const void* K, const Shape& sh, const GeoPack& gp, const StaticTables& st,
                          const WsTables& ws, int num_sms, cudaStream_t s);
cudaError_t launch_static(const Shape& sh, const GeoPack& gp, const StaticTables& st, const WsTables& ws, cudaStream_t s);
cudaError_t launch_gather(const Shape& sh, const GeoPack& gp, const WsTables& ws, int num_sms, int split, cudaStream_t s);
cudaError_t launch_split_k(const Shape& sh, const GeoPack& gp, const WsTables& ws, int num_sms, cudaStream_t s);
cudaError_t launch_choose(const Shape& sh, const GeoPack& gp, const StaticTables& st, const WsTables& ws,
                          const ForcedPack& forced, int have_sics, cudaStream_t s);
cudaError_t launch_pair_axis(const Shape& sh, const GeoPack& gp, const StaticTables& st, const WsTables& ws, int num_sms, cudaStream_t s);
cudaError_t launch_groups_after_select(const Shape& sh, const GeoPack& gp, const WsTables& ws, cudaStream_t s);
cudaError_t launch_summarize(const void* Q, const void* K, const Shape& sh, const GeoPack& gp, const StaticTables& st,
                             const WsTables& ws, int num_sms, cudaStream_t s);
cudaError_t launch_minmax(const void* Q, const void* K, const Shape& sh, const GeoPack& gp, const StaticTables& st,
                          const WsTables& ws, int num_sms, cudaStream_t s);
cudaError_t launch_scores_minmax(const Shape& sh, const GeoPack& gp, const WsTables& ws, cudaStream_t s);
cudaError_t launch_select(const Shape& sh, const GeoPack& gp, const StaticTables& st, const WsTables& ws,
                          cudaStream_t s);

struct PlanMaps;   // tensor maps of Q and K for the one-pass scheme generation, defined in plan.cu
size_t plan_maps_bytes();
void plan_fused_configure(PlanFusedCfg* cfg, const Shape& sh, const GeoPack& gp, int num_sms);
int plan_encode_maps(PlanMaps* out, const void* Q, const void* K, const Shape& sh, const PlanFusedCfg& cfg, char* err,
                     size_t errlen);
void plan_fused_tables(const PlanFusedCfg& cfg, const Shape& sh, const GeoPack& gp, std::vector<int>& e,
                       std::vector<float>& inv, std::vector<uint32_t>& ends);
cudaError_t launch_plan_fused(const PlanMaps* maps, const void* Q, const void* K, const Shape& sh, const GeoPack& gp,
                              const StaticTables& st, const WsTables& ws, const PlanFusedCfg& cfg, int num_sms,
                              const int* tab_e, const float* tab_inv, const uint32_t* tab_m, cudaStream_t s);

struct ScoreMaps;  // tensor map of the K' summaries, defined in scores.cu
size_t score_maps_bytes();
int scores_encode_maps(ScoreMaps* out, const Shape& sh, const WsTables& ws, char* err, size_t errlen);
cudaError_t launch_scores(const ScoreMaps* maps, const Shape& sh, const GeoPack& gp, const WsTables& ws, int num_sms,
                          int term, cudaStream_t s);
cudaError_t launch_dsa_rows(const Shape& sh, const GeoPack& gp, const WsTables& ws, int num_sms, cudaStream_t s);

struct AttnMaps;   // tensor maps of one (Q, K, V, O) quadruple, defined in attn.cu
cudaError_t launch_attn(const AttnMaps* maps, const Shape& sh, const GeoPack& gp, const StaticTables& st,
                        const WsTables& ws, int num_sms, cudaStream_t s);
size_t attn_maps_bytes();
cudaError_t launch_selftest_wait(uint32_t* out, unsigned long long limit_ns, cudaStream_t s);
// Encodes the TMA descriptors for the given device pointers; returns 0 or a CUresult-like code.
int attn_encode_maps(AttnMaps* out, const void* Q, const void* K, const void* V, void* O, const Shape& sh,
                     const GeoPack& gp, char* err, size_t errlen);

// Query tile -> its one or two query blocks.  128-token schemes: the block itself.  64-token schemes: two blocks of one
// 2 x 2 x 2 cell of the block grid, adjacent along the cell's axis (a lone block where the cell is a single block); text
// blocks are paired among themselves after the video tiles.
__device__ __forceinline__ void tile_blocks(const CandGeo& g, const StaticTables& st, const uint8_t* cell_axis, int tile, int& qb0, int& qb1) {
  if (!g.pair) { qb0 = tile; qb1 = -1; return; }
  if (tile >= g.ctiles) {
    qb0 = g.NBv + 2 * (tile - g.ctiles);
    qb1 = qb0 + 1 < g.NB ? qb0 + 1 : -1;
    return;
  }
  int axis = cell_axis[__ldg(st.tile_cell + g.pt_off + tile)];
  axis = axis > 2 ? 2 : axis;
  const uint32_t e = __ldg(st.pair_tab + (size_t)(g.pt_off + tile) * 3 + axis);
  qb0 = (int)(e & 0xffffu);
  qb1 = (e >> 16) == 0xffffu ? -1 : (int)(e >> 16);
}
__host__ __device__ inline int head_tiles(const CandGeo& g) { return g.pair ? g.ctiles + g.ttiles : g.NB; }

__device__ __forceinline__ void bf16x8_to_float(const uint4& v, float* x) {
  x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
  x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
  x[4] = __uint_as_float(v.z << 16); x[5] = __uint_as_float(v.z & 0xffff0000u);
  x[6] = __uint_as_float(v.w << 16); x[7] = __uint_as_float(v.w & 0xffff0000u);
}
