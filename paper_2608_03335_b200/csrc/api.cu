// C-ABI layer of the SPADE CUDA library: argument checks, plan construction (per-candidate
// geometry tables), workspace carving and stage launches.  No stage synchronises the host.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <vector>

#include "../../include/spade.h"
#include "spade_common.cuh"

namespace {

thread_local char g_err[512] = "";

int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

#define CUDA_TRY(expr)                                                                        \
  do {                                                                                        \
    cudaError_t e__ = (expr);                                                                 \
    if (e__ != cudaSuccess) return fail(SPADE_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__)); \
  } while (0)

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Makes the plan's device current for the duration of a call and puts the caller's device back.
struct DeviceGuard {
  int prev = -1, want = -1;
  cudaError_t err = cudaSuccess;
  explicit DeviceGuard(int device) : want(device) {
    err = cudaGetDevice(&prev);
    if (err == cudaSuccess && prev != device) err = cudaSetDevice(device);
  }
  ~DeviceGuard() { if (prev >= 0 && prev != want) cudaSetDevice(prev); }
};
#define ON_PLAN_DEVICE(p)              \
  DeviceGuard guard__((p)->device);    \
  CUDA_TRY(guard__.err)

struct WsLayout {
  size_t status, scheme, keep, pthr, as, score, sics, qsum, ksum, ksplit, kv_idx, kv_cnt, head_order, group_count, item_start, cells, csum, nsum, scores, colkeep, rowfull, cell_axis, pair_union, rowbits, mm, qmid, kdsa, text_start, head_work, att_scratch;
  size_t bytes;
  size_t canary[40];     // debug build: offsets of the 256-byte guard words after each region
  int n_canary;
};

}  // namespace

#define SPADE_HOST_CHUNKS 12  // most head chunks spade_forward_host pipelines

struct spade_plan_s {
  int device, B, heads, num_sms;
  Shape sh;
  GeoPack gp;
  StaticTables st;
  void* d_static;        // one allocation holding rowoff, nvalid, kvalid, budget and the tile tables of the pair schemes
  uint32_t* h_pair_tab;  // host copies of those tile tables (spade_get_pair_table)
  int* h_tile_cell;
  WsLayout lay;
  PlanFusedCfg pf;       // one-pass scheme generation (plan.cu), when the candidate set fits it
  PlanMaps* pmaps;       // its tensor maps for the last (Q, K) seen
  void* d_pf;            // its output tables (device): int rows, then float reciprocals of the block sizes
  size_t pf_entries;
  const void *pq, *pk;
  ScoreMaps* smaps;      // tensor map of the K' summaries inside `smaps_ws`
  const void* smaps_ws;
  AttnMaps* maps;        // host copy of the TMA descriptors for the last (Q,K,V,O) seen
  const void *mq, *mk, *mv, *mo;
  const void* stage_ws;
  int base_cap;          // list capacity without static masks
  int have_csum;         // the last spade_plan left every candidate's summaries in the workspace
  int stage;             // 0 none, 1 planned, 2 summarised, 3 selected
  int launches;
  int keep_status;       // spade_plan leaves the device status words alone (later head chunks of one host call)
  // copy streams and events of spade_forward_host, created on first use
  cudaStream_t copy_in, copy_out;
  cudaEvent_t ev_in[SPADE_HOST_CHUNKS], ev_done[SPADE_HOST_CHUNKS], ev_edge;
  int host_ready;
};

namespace {

WsTables tables_at(const spade_plan_s* p, void* ws) {
  char* b = (char*)ws;
  const WsLayout& l = p->lay;
  WsTables t;
  t.status = (uint32_t*)(b + l.status);
  t.scheme = (int*)(b + l.scheme);
  t.keep = (int*)(b + l.keep);
  t.pthr = (float*)(b + l.pthr);
  t.as = (float*)(b + l.as);
  t.score = (float*)(b + l.score);
  t.sics = (float*)(b + l.sics);
  t.qsum = (float*)(b + l.qsum);
  t.ksum = (float*)(b + l.ksum);
  t.ksplit = (float*)(b + l.ksplit);
  t.kv_idx = (int*)(b + l.kv_idx);
  t.kv_cnt = (int*)(b + l.kv_cnt);
  t.head_order = (int*)(b + l.head_order);
  t.head_work = (float*)(b + l.head_work);
  t.group_count = (int*)(b + l.group_count);
  t.item_start = (int*)(b + l.item_start);
  t.text_start = (int*)(b + l.text_start);
  t.cells = (float*)(b + l.cells);
  t.csum = (float*)(b + l.csum);
  t.nsum = (float*)(b + l.nsum);
  t.scores = (float*)(b + l.scores);
  t.cell_axis = (uint8_t*)(b + l.cell_axis);
  t.pair_union = (int*)(b + l.pair_union);
  t.rowbits = (uint32_t*)(b + l.rowbits);
  t.colkeep = (uint8_t*)(b + l.colkeep);
  t.rowfull = (uint8_t*)(b + l.rowfull);
  t.mm = (float*)(b + l.mm);
  t.qmid = (float*)(b + l.qmid);
  t.kdsa = (float*)(b + l.kdsa);
  t.att_scratch = (uint32_t*)(b + l.att_scratch);
  return t;
}

int check_call(const spade_plan_s* p, const void* ws) {
  if (!p) return fail(SPADE_ERR_INVALID_ARG, "plan is NULL");
  if (!ws || ((uintptr_t)ws & 255)) return fail(SPADE_ERR_WORKSPACE, "workspace is NULL or not 256-byte aligned");
  return SPADE_OK;
}

int check_tensor(const void* x, const char* name) {
  if (!x) return fail(SPADE_ERR_INVALID_ARG, "%s is NULL", name);
  if ((uintptr_t)x & 15) return fail(SPADE_ERR_INVALID_ARG, "%s is not 16-byte aligned", name);
  return SPADE_OK;
}

// Carves the workspace; the list capacity is full when a static mask is enabled.
void compute_layout(spade_plan_s* p) {
  Shape& sh = p->sh;
  const int BH = sh.BH, n_cands = sh.C;
  sh.cap = sh.masks_on ? ((sh.NBmax + 3) & ~3) : p->base_cap;
  WsLayout& l = p->lay;
  size_t o = 0;
  l.n_canary = 0;
  auto take = [&](size_t bytes) {
    size_t at = o;
    o = align_up(o + bytes, 256);
#ifdef SPADE_DEBUG
    if (l.n_canary < 40) l.canary[l.n_canary++] = o;       // a guard word behind every region
    o += 256;
#endif
    return at;
  };
  l.status = take(64 * 4);
  l.scheme = take((size_t)BH * 4);
  l.keep = take((size_t)BH * 4);
  l.pthr = take((size_t)BH * 4);
  l.as = take((size_t)BH * n_cands * 2 * 4);
  l.score = take((size_t)BH * n_cands * 4);
  l.sics = take((size_t)BH * n_cands * 2 * sh.NBvmax * 4);
  l.head_order = take((size_t)BH * 4);
  l.head_work = take((size_t)BH * 4);
  l.group_count = take((size_t)SPADE_MAX_CANDS * 4);
  l.item_start = take((size_t)(BH + 1) * 4);
  l.text_start = take((size_t)(BH + 1) * 4);
  l.kv_cnt = take((size_t)BH * sh.NBmax * 4);
  l.cell_axis = take((size_t)BH * sh.cell_ld);
  l.pair_union = take((size_t)BH * 4 * 4);
  l.colkeep = take((size_t)BH * sh.NBmax);
  l.rowfull = take((size_t)BH * sh.NBmax);
  l.qsum = take((size_t)BH * sh.NBmax * SPADE_D * 4);
  l.ksum = take((size_t)BH * sh.NBmax * SPADE_D * 4);
  l.ksplit = take((size_t)BH * 2 * sh.NBmax * SPADE_D * 4);
  l.kv_idx = take((size_t)BH * sh.NBmax * sh.cap * 4);
  l.cells = take(sh.use_cells && !p->pf.on ? (size_t)BH * 2 * sh.NCELL * 2 * SPADE_D * 4 : 0);
  l.csum = take(sh.use_cells || p->pf.on ? (size_t)BH * 2 * n_cands * sh.NBmax * SPADE_D * 4 : 0);
  l.nsum = take(p->pf.on ? (size_t)BH * 2 * n_cands * sh.NBmax * SPADE_D * 4 : 0);
  sh.ld_scores = (sh.NBvmax + 63) & ~63;
  sh.bits_ld = sh.ld_scores / 32;
  l.rowbits = take((size_t)BH * sh.NBvmax * sh.bits_ld * 4);
  l.scores = take((size_t)BH * sh.NBvmax * sh.ld_scores * 4);
  l.mm = take(sh.estimator ? (size_t)4 * BH * SPADE_D * sh.ld_scores * 4 : 0);
  l.qmid = take(sh.estimator == 1 ? (size_t)BH * sh.NBmax * SPADE_D * 4 : 0);
  l.kdsa = take(sh.estimator == 1 ? (size_t)BH * 4 * sh.NBmax * SPADE_D * 4 : 0);
  l.att_scratch = take((size_t)2 * p->num_sms * 2 * SPADE_MAX_NB * 4);
  l.bytes = o;
}

// Valid-row mask of block `b` under geometry g (bit r <=> in-block row r is a real token).
void block_mask(const CandGeo& g, const Shape& sh, int b, uint64_t m[2], int* n) {
  m[0] = m[1] = 0;
  *n = 0;
  for (int r = 0; r < g.BS; ++r) {
    bool ok;
    if (b >= g.NBv) {
      ok = (b - g.NBv) * g.BS + r < sh.n_text;
    } else {
      const int iw = b % g.nbw, ih = (b / g.nbw) % g.nbh, it = b / (g.nbw * g.nbh);
      const int dw = r % g.bw, dh = (r / g.bw) % g.bh, dt = r / (g.bw * g.bh);
      ok = it * g.bt + dt < sh.T && ih * g.bh + dh < sh.H && iw * g.bw + dw < sh.W;
    }
    if (ok) { m[r >> 6] |= 1ull << (r & 63); ++*n; }
  }
}

}  // namespace

extern "C" {

const char* spade_last_error(void) { return g_err; }

int spade_plan_create(spade_plan_t** out, int32_t B, int32_t heads, int32_t d, const spade_grid_t* grid,
                      const spade_blocking_t* cands, int32_t n_cands, const spade_budget_t* budget, int32_t device) {
  if (!out) return fail(SPADE_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  if (!grid || !cands || !budget) return fail(SPADE_ERR_INVALID_ARG, "grid, cands or budget is NULL");
  if (B < 1 || heads < 1) return fail(SPADE_ERR_INVALID_ARG, "B and heads must be positive");
  if (d != SPADE_D) return fail(SPADE_ERR_UNSUPPORTED, "head dimension %d (only 128 is built)", d);
  if (grid->T < 1 || grid->H < 1 || grid->W < 1 || grid->n_text < 0)
    return fail(SPADE_ERR_INVALID_ARG, "bad grid %dx%dx%d + %d text", grid->T, grid->H, grid->W, grid->n_text);
  if (n_cands < 1) return fail(SPADE_ERR_INVALID_ARG, "n_cands must be at least 1");
  if (n_cands > SPADE_MAX_CANDS) return fail(SPADE_ERR_UNSUPPORTED, "more than %d candidates", SPADE_MAX_CANDS);
  // the head ordering of the plan and select stages ranks the heads pairwise in one CTA
  if ((long)B * heads > SPADE_MAX_BH) return fail(SPADE_ERR_UNSUPPORTED, "B*heads above %d", SPADE_MAX_BH);
  if (budget->mode < 0 || budget->mode > 3) return fail(SPADE_ERR_INVALID_ARG, "unknown budget mode %d", budget->mode);
  const int BH = B * heads;
  for (int i = 0; i < BH; ++i) {
    const float v = budget->per_head ? budget->per_head[i] : budget->value;
    const bool ok = budget->mode == SPADE_TOPK ? (v >= 1.f) : budget->mode == SPADE_TOPP ? (v > 0.f && v <= 1.f)
                                                                                         : (v >= 0.f && v < 1.f);
    if (budget->mode == SPADE_POLICY_AS && !(budget->gain >= 0.f)) return fail(SPADE_ERR_INVALID_ARG, "policy gain %g must be >= 0", budget->gain);
    if (!ok || v != v) return fail(SPADE_ERR_INVALID_ARG, "budget value %g out of range for mode %d", v, budget->mode);
  }
  const long Nv = (long)grid->T * grid->H * grid->W;
  if (Nv + grid->n_text > (1l << 24)) return fail(SPADE_ERR_UNSUPPORTED, "more than 2^24 tokens");
  if (grid->T > 1023 || grid->H > 1023 || grid->W > 1023) return fail(SPADE_ERR_UNSUPPORTED, "grid axis above 1023");

  spade_plan_s* p = (spade_plan_s*)calloc(1, sizeof(spade_plan_s));
  if (!p) return fail(SPADE_ERR_INVALID_ARG, "out of host memory");
  p->device = device; p->B = B; p->heads = heads;
  Shape& sh = p->sh;
  sh.BH = BH; sh.Nv = (int)Nv; sh.n_text = grid->n_text; sh.N = (int)Nv + grid->n_text;
  sh.T = grid->T; sh.H = grid->H; sh.W = grid->W; sh.C = n_cands;
  sh.mode = budget->mode; sh.value = budget->value; sh.gain = budget->mode == SPADE_POLICY_AS ? budget->gain : 0.f;
  int units = 0, tab = 0;
  sh.NBmax = 0; sh.NBvmax = 0;
  for (int c = 0; c < n_cands; ++c) {
    CandGeo& g = p->gp.g[c];
    g.bt = cands[c].bt; g.bh = cands[c].bh; g.bw = cands[c].bw;
    if (g.bt < 1 || g.bh < 1 || g.bw < 1) { free(p); return fail(SPADE_ERR_INVALID_ARG, "candidate %d has a non-positive extent", c); }
    g.BS = g.bt * g.bh * g.bw;
    if (g.BS != 64 && g.BS != 128) { const int bs = g.BS; free(p); return fail(SPADE_ERR_UNSUPPORTED, "candidate %d has %d tokens per block (64 or 128 needed)", c, bs); }
    if (g.bt > 128 || g.bh > 128 || g.bw > 128) { free(p); return fail(SPADE_ERR_UNSUPPORTED, "candidate %d: extent above 128", c); }
    g.nbt = (sh.T + g.bt - 1) / g.bt; g.nbh = (sh.H + g.bh - 1) / g.bh; g.nbw = (sh.W + g.bw - 1) / g.bw;
    g.mag_w = g.nbw > 1 ? (uint32_t)(0x100000000ull / (unsigned long long)g.nbw) + 1u : 0u;
    g.mag_hw = g.nbw * g.nbh > 1 ? (uint32_t)(0x100000000ull / ((unsigned long long)g.nbw * g.nbh)) + 1u : 0u;
    g.NBv = g.nbt * g.nbh * g.nbw;
    g.NBt = (sh.n_text + g.BS - 1) / g.BS;
    g.NB = g.NBv + g.NBt;
    if (g.NB > SPADE_MAX_NB) { const int nb = g.NB; free(p); return fail(SPADE_ERR_UNSUPPORTED, "candidate %d gives %d blocks per head (max %d)", c, nb, SPADE_MAX_NB); }
    g.pair = g.BS == 64;
    g.ttiles = (g.NBt + 1) / 2;
    g.tiles = g.NB;              // pair schemes: set with the tile tables below
    g.ctiles = 0; g.ncell = 0; g.pt_off = 0; g.pc_off = 0;
    // K/V travel in 64-row boxes: a 128-token block is split along its outermost extended axis
    g.kt = g.bt; g.kh = g.bh; g.kw = g.bw; g.ht = g.hh = g.hw = 0;
    if (!g.pair) {
      if (g.bt > 1) { g.kt = g.bt / 2; g.ht = g.kt; }
      else if (g.bh > 1) { g.kh = g.bh / 2; g.hh = g.kh; }
      else { g.kw = g.bw / 2; g.hw = g.kw; }
    }
    g.unit_off = units; units += g.NBv;
    g.tab_off = tab; tab += g.NB;
    if (g.NB > sh.NBmax) sh.NBmax = g.NB;
    if (g.NBv > sh.NBvmax) sh.NBvmax = g.NBv;
  }
  sh.units_per_ht = units;
  {
    auto gcd = [](int a, int b) { while (b) { int t = a % b; a = b; b = t; } return a; };
    int ct = p->gp.g[0].bt, ch = p->gp.g[0].bh, cw = p->gp.g[0].bw;
    for (int c = 1; c < n_cands; ++c) { ct = gcd(ct, p->gp.g[c].bt); ch = gcd(ch, p->gp.g[c].bh); cw = gcd(cw, p->gp.g[c].bw); }
    sh.ct = ct; sh.ch = ch; sh.cw = cw; sh.CS = ct * ch * cw;
    sh.lcw = 0; while ((1 << sh.lcw) < cw) ++sh.lcw;
    sh.lch = 0; while ((1 << sh.lch) < ch) ++sh.lch;
    sh.nct = (sh.T + ct - 1) / ct; sh.nch = (sh.H + ch - 1) / ch; sh.ncw = (sh.W + cw - 1) / cw;
    sh.NCELL = sh.nct * sh.nch * sh.ncw;
    sh.use_cells = sh.CS >= 4;          // extents are powers of two because every block has 64 or 128 tokens
  }

  // Row capacity of the index lists: the longest list any head can get.
  int cap = 0;
  for (int c = 0; c < n_cands; ++c) {
    const CandGeo& g = p->gp.g[c];
    int kmax = g.NBv;
    if (budget->mode != SPADE_TOPP && budget->mode != SPADE_POLICY_AS) {
      kmax = 1;
      for (int i = 0; i < BH; ++i) {
        const float v = budget->per_head ? budget->per_head[i] : budget->value;
        int k = budget->mode == SPADE_TOPK ? (int)v : (int)ceil((1.0 - (double)v) * (double)g.NBv - 1e-9);
        k = k < 1 ? 1 : (k > g.NBv ? g.NBv : k);
        if (k > kmax) kmax = k;
      }
    }
    int need = kmax + g.NBt;
    if (g.NBt > 0) need = g.NB;            // text query blocks list every block
    if (need > cap) cap = need;
  }
  sh.cap = (cap + 3) & ~3;

  // ---- static tables ---------------------------------------------------------------------------
  std::vector<uint32_t> rowoff((size_t)n_cands * 128, 0);
  std::vector<int> nvalid(tab);
  std::vector<uint64_t> kvalid((size_t)tab * 2);
  std::vector<float> bud(BH);
  for (int i = 0; i < BH; ++i) bud[i] = budget->per_head ? budget->per_head[i] : budget->value;
  for (int c = 0; c < n_cands; ++c) {
    CandGeo& g = p->gp.g[c];
    for (int r = 0; r < g.BS; ++r) {
      const int dw = r % g.bw, dh = (r / g.bw) % g.bh, dt = r / (g.bw * g.bh);
      rowoff[(size_t)c * 128 + r] = ((uint32_t)dt << 20) | ((uint32_t)dh << 10) | (uint32_t)dw;
    }
    double z = 0.0;
    for (int b = 0; b < g.NB; ++b) {
      int n;
      block_mask(g, sh, b, &kvalid[(size_t)(g.tab_off + b) * 2], &n);
      nvalid[g.tab_off + b] = n;
      if (b < g.NBv) z += (double)n * (double)n;
    }
    g.inv_z = (float)(1.0 / (2.0 * z));
  }

  // Tile tables of the 64-token schemes.  The block grid is cut into cells of 2 x 2 x 2 blocks (fewer at an odd end); the
  // blocks of a cell are paired along one axis, chosen per head and cell after the index search.  A cell's tiles are the
  // blocks with offset 0 along that axis, in raster order; an axis along which the cell is one block wide stands for the
  // first one along which it is two (a cell of one block is a lone tile), so every choice gives the same number of tiles.
  std::vector<uint32_t> pair_tab;
  std::vector<int> tile_cell, cell_tile0;
  sh.cell_ld = 16;
  for (int c = 0; c < n_cands; ++c) {
    CandGeo& g = p->gp.g[c];
    if (!g.pair) continue;
    g.pt_off = (int)tile_cell.size();
    g.pc_off = (int)cell_tile0.size();
    const int nb[3] = {g.nbt, g.nbh, g.nbw}, stride[3] = {g.nbh * g.nbw, g.nbw, 1};
    const int nc[3] = {(g.nbt + 1) / 2, (g.nbh + 1) / 2, (g.nbw + 1) / 2};
    g.ncell = nc[0] * nc[1] * nc[2];
    int tiles = 0;
    for (int cell = 0; cell < g.ncell; ++cell) {
      const int cc[3] = {cell / (nc[1] * nc[2]), (cell / nc[2]) % nc[1], cell % nc[2]};
      int ext[3], first_wide = -1;
      for (int a = 0; a < 3; ++a) {
        ext[a] = nb[a] - 2 * cc[a] >= 2 ? 2 : 1;
        if (ext[a] == 2 && first_wide < 0) first_wide = a;
      }
      cell_tile0.push_back(tiles);
      const int origin = 2 * cc[0] * stride[0] + 2 * cc[1] * stride[1] + 2 * cc[2] * stride[2];
      const int ntile = first_wide < 0 ? 1 : ext[0] * ext[1] * ext[2] / 2;
      const size_t at = pair_tab.size();
      pair_tab.resize(at + (size_t)ntile * 3);
      for (int a = 0; a < 3; ++a) {
        const int ax = first_wide < 0 ? -1 : (ext[a] == 2 ? a : first_wide);
        int k = 0;
        for (int o0 = 0; o0 < ext[0]; ++o0)
          for (int o1 = 0; o1 < ext[1]; ++o1)
            for (int o2 = 0; o2 < ext[2]; ++o2) {
              const int off[3] = {o0, o1, o2};
              if (ax >= 0 && off[ax] != 0) continue;
              const int qb0 = origin + o0 * stride[0] + o1 * stride[1] + o2 * stride[2];
              const uint32_t qb1 = ax >= 0 ? (uint32_t)(qb0 + stride[ax]) : 0xffffu;
              pair_tab[at + (size_t)k * 3 + a] = (uint32_t)qb0 | (qb1 << 16);
              ++k;
            }
      }
      for (int k = 0; k < ntile; ++k) tile_cell.push_back(cell);
      tiles += ntile;
    }
    cell_tile0.push_back(tiles);
    g.ctiles = tiles;
    g.tiles = g.ctiles + g.ttiles;
    if (((g.ncell + 15) & ~15) > sh.cell_ld) sh.cell_ld = (g.ncell + 15) & ~15;
  }

  cudaError_t e = cudaSetDevice(device);
  cudaDeviceProp prop;
  if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, device);
  if (e != cudaSuccess) { free(p); return fail(SPADE_ERR_CUDA, "device %d: %s", device, cudaGetErrorString(e)); }
  if (prop.major != 10) { free(p); return fail(SPADE_ERR_UNSUPPORTED, "device %d is sm_%d%d; this library is built for sm_100a only", device, prop.major, prop.minor); }
  p->num_sms = prop.multiProcessorCount;

  const size_t o_rowoff = 0;
  const size_t o_nvalid = align_up(o_rowoff + rowoff.size() * 4, 256);
  const size_t o_kvalid = align_up(o_nvalid + nvalid.size() * 4, 256);
  const size_t o_budget = align_up(o_kvalid + kvalid.size() * 8, 256);
  const size_t o_ptab = align_up(o_budget + bud.size() * 4, 256);
  const size_t o_tcell = align_up(o_ptab + pair_tab.size() * 4, 256);
  const size_t o_ctile = align_up(o_tcell + tile_cell.size() * 4, 256);
  const size_t total = align_up(o_ctile + cell_tile0.size() * 4, 256);
  e = cudaMalloc(&p->d_static, total);
  if (e != cudaSuccess) { free(p); return fail(SPADE_ERR_CUDA, "cudaMalloc(%zu): %s", total, cudaGetErrorString(e)); }
  char* base = (char*)p->d_static;
  e = cudaMemcpy(base + o_rowoff, rowoff.data(), rowoff.size() * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(base + o_nvalid, nvalid.data(), nvalid.size() * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(base + o_kvalid, kvalid.data(), kvalid.size() * 8, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(base + o_budget, bud.data(), bud.size() * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess && !pair_tab.empty()) e = cudaMemcpy(base + o_ptab, pair_tab.data(), pair_tab.size() * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess && !tile_cell.empty()) e = cudaMemcpy(base + o_tcell, tile_cell.data(), tile_cell.size() * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess && !cell_tile0.empty()) e = cudaMemcpy(base + o_ctile, cell_tile0.data(), cell_tile0.size() * 4, cudaMemcpyHostToDevice);
  if (e != cudaSuccess) { cudaFree(p->d_static); free(p); return fail(SPADE_ERR_CUDA, "table upload: %s", cudaGetErrorString(e)); }
  p->st.rowoff = (const uint32_t*)(base + o_rowoff);
  p->st.nvalid = (const int*)(base + o_nvalid);
  p->st.kvalid = (const uint64_t*)(base + o_kvalid);
  p->st.budget = (const float*)(base + o_budget);
  p->st.pair_tab = (const uint32_t*)(base + o_ptab);
  p->st.tile_cell = (const int*)(base + o_tcell);
  p->st.cell_tile0 = (const int*)(base + o_ctile);

  p->base_cap = sh.cap;
  plan_fused_configure(&p->pf, sh, p->gp, p->num_sms);
  if (p->pf.on) {
    std::vector<int> pe;
    std::vector<float> pi;
    std::vector<uint32_t> pm;
    plan_fused_tables(p->pf, sh, p->gp, pe, pi, pm);
    p->pf_entries = pe.size();
    e = cudaMalloc(&p->d_pf, pe.size() * 8 + pm.size() * 4);
    if (e == cudaSuccess) e = cudaMemcpy(p->d_pf, pe.data(), pe.size() * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy((char*)p->d_pf + pe.size() * 4, pi.data(), pi.size() * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy((char*)p->d_pf + pe.size() * 8, pm.data(), pm.size() * 4, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) { cudaFree(p->d_pf); cudaFree(p->d_static); free(p); return fail(SPADE_ERR_CUDA, "table upload: %s", cudaGetErrorString(e)); }
  }
  compute_layout(p);

  p->maps = (AttnMaps*)calloc(1, attn_maps_bytes());
  p->smaps = (ScoreMaps*)calloc(1, score_maps_bytes());
  p->pmaps = (PlanMaps*)calloc(1, plan_maps_bytes());
  p->h_pair_tab = (uint32_t*)malloc(pair_tab.size() * 4 + 4);
  p->h_tile_cell = (int*)malloc(tile_cell.size() * 4 + 4);
  if (!p->maps || !p->smaps || !p->pmaps || !p->h_pair_tab || !p->h_tile_cell) {
    cudaFree(p->d_pf); cudaFree(p->d_static); free(p->maps); free(p->smaps); free(p->pmaps); free(p->h_pair_tab); free(p->h_tile_cell); free(p);
    return fail(SPADE_ERR_INVALID_ARG, "out of host memory");
  }
  if (!pair_tab.empty()) memcpy(p->h_pair_tab, pair_tab.data(), pair_tab.size() * 4);
  if (!tile_cell.empty()) memcpy(p->h_tile_cell, tile_cell.data(), tile_cell.size() * 4);
  *out = p;
  return SPADE_OK;
}

int spade_plan_destroy(spade_plan_t* p) {
  if (!p) return SPADE_OK;
  cudaFree(p->d_static);
  cudaFree(p->d_pf);
  if (p->host_ready) {
    cudaStreamDestroy(p->copy_in);
    cudaStreamDestroy(p->copy_out);
    for (int i = 0; i < SPADE_HOST_CHUNKS; ++i) { cudaEventDestroy(p->ev_in[i]); cudaEventDestroy(p->ev_done[i]); }
    cudaEventDestroy(p->ev_edge);
  }
  free(p->maps);
  free(p->smaps);
  free(p->pmaps);
  free(p->h_pair_tab);
  free(p->h_tile_cell);
  free(p);
  return SPADE_OK;
}

int spade_plan_set_masks(spade_plan_t* p, const spade_static_mask_t* m) {
  if (!p) return fail(SPADE_ERR_INVALID_ARG, "plan is NULL");
  Shape& sh = p->sh;
  sh.intra_thr = 0.f; sh.window = -1; sh.sink = 0;
  if (m) {
    if (m->intra_threshold != m->intra_threshold) return fail(SPADE_ERR_INVALID_ARG, "intra_threshold is NaN");
    if (m->sink_tokens < 0) return fail(SPADE_ERR_INVALID_ARG, "sink_tokens is negative");
    sh.intra_thr = m->intra_threshold > 0.f ? m->intra_threshold : 0.f;
    sh.window = m->window < 0 ? -1 : m->window;
    sh.sink = m->sink_tokens;
  }
  sh.masks_on = (sh.intra_thr > 0.f || sh.window >= 0 || sh.sink > 0) ? 1 : 0;
  compute_layout(p);
  p->stage = 0; p->stage_ws = nullptr; p->smaps_ws = nullptr;      // tables moved: stages start over
  return SPADE_OK;
}

int spade_plan_set_estimator(spade_plan_t* p, int32_t estimator) {
  if (!p) return fail(SPADE_ERR_INVALID_ARG, "plan is NULL");
  if (estimator != SPADE_EST_MEAN && estimator != SPADE_EST_DSA && estimator != SPADE_EST_DSA2)
    return fail(SPADE_ERR_INVALID_ARG, "estimator %d is not one of SPADE_EST_MEAN, SPADE_EST_DSA, SPADE_EST_DSA2", estimator);
  p->sh.estimator = estimator;
  compute_layout(p);
  p->stage = 0; p->stage_ws = nullptr; p->smaps_ws = nullptr;      // tables moved: stages start over
  return SPADE_OK;
}

size_t spade_workspace_bytes(const spade_plan_t* p) { return p ? p->lay.bytes : 0; }

int spade_get_geometry(const spade_plan_t* p, int32_t c, int32_t* out6) {
  if (!p || !out6) return fail(SPADE_ERR_INVALID_ARG, "plan or out is NULL");
  if (c < 0 || c >= p->sh.C) return fail(SPADE_ERR_INVALID_ARG, "candidate %d out of range", c);
  const CandGeo& g = p->gp.g[c];
  out6[0] = g.nbt; out6[1] = g.nbh; out6[2] = g.nbw; out6[3] = g.NBv; out6[4] = g.NBt; out6[5] = g.BS;
  return SPADE_OK;
}

int spade_get_pair_table(const spade_plan_t* p, int32_t c, int32_t* tile_cell, uint32_t* pairs) {
  if (!p) return fail(SPADE_ERR_INVALID_ARG, "plan is NULL");
  if (c < 0 || c >= p->sh.C) return fail(SPADE_ERR_INVALID_ARG, "candidate %d out of range", c);
  const CandGeo& g = p->gp.g[c];
  if (!g.pair) return 0;
  if (tile_cell) memcpy(tile_cell, p->h_tile_cell + g.pt_off, (size_t)g.ctiles * 4);
  if (pairs) memcpy(pairs, p->h_pair_tab + (size_t)g.pt_off * 3, (size_t)g.ctiles * 3 * 4);
  return g.ctiles;
}

int spade_get_tables(const spade_plan_t* p, void* ws, spade_tables_t* out) {
  int rc = check_call(p, ws);
  if (rc) return rc;
  if (!out) return fail(SPADE_ERR_INVALID_ARG, "out is NULL");
  WsTables t = tables_at(p, ws);
  out->BH = p->sh.BH; out->C = p->sh.C; out->NBmax = p->sh.NBmax; out->cap = p->sh.cap;
  out->scheme = t.scheme; out->keep = t.keep; out->as = t.as; out->score = t.score; out->sics = t.sics;
  out->NBvmax = p->sh.NBvmax;
  out->qsum = t.qsum; out->ksum = t.ksum; out->kv_idx = t.kv_idx; out->kv_cnt = t.kv_cnt;
  out->head_order = t.head_order; out->group_count = t.group_count; out->item_start = t.item_start;
  out->cell_axis = t.cell_axis;
  out->cell_ld = p->sh.cell_ld;
  out->status = t.status;
  out->minmax = p->sh.estimator ? t.mm : nullptr;
  out->block_scores = t.scores;
  out->block_scores_ld = p->sh.ld_scores;
  return SPADE_OK;
}

int spade_plan(spade_plan_t* p, const void* Q, const void* K, void* ws, void* stream, const int32_t* forced) {
  int rc = check_call(p, ws);
  if (rc) return rc;
  if ((rc = check_tensor(Q, "Q")) || (rc = check_tensor(K, "K"))) return rc;
  if (forced)
    for (int i = 0; i < p->sh.BH; ++i)
      if (forced[i] < 0 || forced[i] >= p->sh.C) return fail(SPADE_ERR_INVALID_ARG, "forced_scheme[%d] = %d out of range", i, forced[i]);
  cudaStream_t s = (cudaStream_t)stream;
  ON_PLAN_DEVICE(p);
  WsTables t = tables_at(p, ws);
  p->launches = 0;
  if (!p->keep_status) CUDA_TRY(cudaMemsetAsync(t.status, 0, 64 * 4, s));
#ifdef SPADE_DEBUG
  for (int i = 0; i < p->lay.n_canary; ++i) CUDA_TRY(cudaMemsetAsync((char*)ws + p->lay.canary[i], 0xC5, 256, s));
#endif
  const bool skip_sics = forced != nullptr && !(p->sh.masks_on && p->sh.intra_thr > 0.f) && p->sh.mode != SPADE_POLICY_AS;
  // The caller's array is read here and never again: the schemes travel inside the launch itself
  // (4 bits per head), so a captured launch replays the values it was captured with.
  ForcedPack fpack;
  memset(&fpack, 0, sizeof(fpack));
  if (forced) {
    fpack.on = 1;
    for (int i = 0; i < p->sh.BH; ++i) fpack.w[i >> 3] |= (uint32_t)forced[i] << ((i & 7) * 4);
  }
  p->have_csum = 0;
  if (!skip_sics) {
    if (p->pf.on) {
      if (Q != p->pq || K != p->pk) {
        char msg[256];
        if (plan_encode_maps(p->pmaps, Q, K, p->sh, p->pf, msg, sizeof(msg))) return fail(SPADE_ERR_CUDA, "tensor map: %s", msg);
        p->pq = Q; p->pk = K;
      }
      CUDA_TRY(launch_plan_fused(p->pmaps, Q, K, p->sh, p->gp, p->st, t, p->pf, p->num_sms, (const int*)p->d_pf,
                                 (const float*)((const char*)p->d_pf + p->pf_entries * 4),
                                 (const uint32_t*)((const char*)p->d_pf + p->pf_entries * 8), s));
      p->launches += 2;
      p->have_csum = 1;
    } else if (p->sh.use_cells) {
      CUDA_TRY(launch_cells(Q, K, p->sh, t, p->num_sms, s));
      CUDA_TRY(launch_blocks(Q, K, p->sh, p->gp, p->st, t, p->num_sms, s));
      p->launches += 2;
      p->have_csum = 1;
    } else {
      CUDA_TRY(launch_sics(Q, K, p->sh, p->gp, p->st, t, p->num_sms, s));
      p->launches += 1;
    }
  }
  CUDA_TRY(launch_choose(p->sh, p->gp, p->st, t, fpack, skip_sics ? 0 : 1, s));
  p->launches += 1;
  if (p->sh.masks_on) {
    CUDA_TRY(launch_static(p->sh, p->gp, p->st, t, s));
    p->launches += 1;
  }
  p->stage = 1; p->stage_ws = ws;
  return SPADE_OK;
}

int spade_summarize(spade_plan_t* p, const void* Q, const void* K, void* ws, void* stream) {
  int rc = check_call(p, ws);
  if (rc) return rc;
  if ((rc = check_tensor(Q, "Q")) || (rc = check_tensor(K, "K"))) return rc;
  if (p->stage < 1 || p->stage_ws != ws) return fail(SPADE_ERR_ORDER, "spade_summarize needs spade_plan on this workspace first");
  ON_PLAN_DEVICE(p);
  // the copy of the chosen candidate's sums also writes the estimator's split K'; the token pass needs a kernel for it
  if (p->have_csum) CUDA_TRY(launch_gather(p->sh, p->gp, tables_at(p, ws), p->num_sms, p->sh.estimator == 0, (cudaStream_t)stream));
  else CUDA_TRY(launch_summarize(Q, K, p->sh, p->gp, p->st, tables_at(p, ws), p->num_sms, (cudaStream_t)stream));
  p->launches += 1;
  if (!p->sh.estimator && !p->have_csum) {
    CUDA_TRY(launch_split_k(p->sh, p->gp, tables_at(p, ws), p->num_sms, (cudaStream_t)stream));
    p->launches += 1;
  }
  if (p->sh.estimator) {
    CUDA_TRY(launch_minmax(Q, K, p->sh, p->gp, p->st, tables_at(p, ws), p->num_sms, (cudaStream_t)stream));
    p->launches += 1;
    if (p->sh.estimator == 1) {
      CUDA_TRY(launch_dsa_rows(p->sh, p->gp, tables_at(p, ws), p->num_sms, (cudaStream_t)stream));
      p->launches += 1;
    }
  }
  p->stage = 2;
  return SPADE_OK;
}

int spade_select(spade_plan_t* p, void* ws, void* stream) {
  int rc = check_call(p, ws);
  if (rc) return rc;
  if (p->stage < 2 || p->stage_ws != ws) return fail(SPADE_ERR_ORDER, "spade_select needs spade_summarize on this workspace first");
  ON_PLAN_DEVICE(p);
  WsTables t = tables_at(p, ws);
  if (p->sh.estimator == 2) {
    CUDA_TRY(launch_scores_minmax(p->sh, p->gp, t, (cudaStream_t)stream));
  } else {
    if (p->smaps_ws != ws) {
      char msg[256];
      if (scores_encode_maps(p->smaps, p->sh, t, msg, sizeof(msg))) return fail(SPADE_ERR_CUDA, "tensor map: %s", msg);
      p->smaps_ws = ws;
    }
    if (p->sh.estimator == 1) {       // Fig. 4a as two tensor-core passes over the same score table
      CUDA_TRY(launch_scores(p->smaps, p->sh, p->gp, t, p->num_sms, 1, (cudaStream_t)stream));
      CUDA_TRY(launch_scores(p->smaps, p->sh, p->gp, t, p->num_sms, 2, (cudaStream_t)stream));
      p->launches += 1;
    } else {
      CUDA_TRY(launch_scores(p->smaps, p->sh, p->gp, t, p->num_sms, 0, (cudaStream_t)stream));
    }
  }
  CUDA_TRY(launch_select(p->sh, p->gp, p->st, t, (cudaStream_t)stream));
  p->launches += 2;
  bool any_pair = false;
  for (int c = 0; c < p->sh.C; ++c) any_pair = any_pair || p->gp.g[c].pair;
  if (any_pair) {
    // pair the 64-token query blocks along the axis that gives the shortest merged lists, per head (the totals start
    // at zero: the plan stage and the previous use leave them so); the kernel's last CTA then orders the heads
    CUDA_TRY(launch_pair_axis(p->sh, p->gp, p->st, t, p->num_sms, (cudaStream_t)stream));
  } else {
    CUDA_TRY(launch_groups_after_select(p->sh, p->gp, t, (cudaStream_t)stream));
  }
  p->launches += 1;
  p->stage = 3;
  return SPADE_OK;
}

int spade_attn(spade_plan_t* p, const void* Q, const void* K, const void* V, void* O, void* ws, void* stream) {
  int rc = check_call(p, ws);
  if (rc) return rc;
  if ((rc = check_tensor(Q, "Q")) || (rc = check_tensor(K, "K")) || (rc = check_tensor(V, "V")) || (rc = check_tensor(O, "O"))) return rc;
  if (p->stage < 1 || p->stage_ws != ws) return fail(SPADE_ERR_ORDER, "spade_attn needs spade_plan (and index lists) on this workspace first");
  ON_PLAN_DEVICE(p);
  if (Q != p->mq || K != p->mk || V != p->mv || O != p->mo) {
    char msg[256];
    if (attn_encode_maps(p->maps, Q, K, V, O, p->sh, p->gp, msg, sizeof(msg))) return fail(SPADE_ERR_CUDA, "tensor map: %s", msg);
    p->mq = Q; p->mk = K; p->mv = V; p->mo = O;
  }
  CUDA_TRY(cudaMemsetAsync(tables_at(p, ws).status + 8, 0, 4, (cudaStream_t)stream));     // work-item counter of k_attn
  CUDA_TRY(launch_attn(p->maps, p->sh, p->gp, p->st, tables_at(p, ws), p->num_sms, (cudaStream_t)stream));
  p->launches += 1;
  return SPADE_OK;
}

int spade_forward(spade_plan_t* p, const void* Q, const void* K, const void* V, void* O, void* ws, void* stream,
                  const int32_t* forced) {
  int rc;
  if ((rc = spade_plan(p, Q, K, ws, stream, forced))) return rc;
  if ((rc = spade_summarize(p, Q, K, ws, stream))) return rc;
  if ((rc = spade_select(p, ws, stream))) return rc;
  return spade_attn(p, Q, K, V, O, ws, stream);
}

// Heads are independent (Sec. 3.2: per-head schemes; Sec. 3.3: per-head lists), so the host call works
// on chunks of heads: the copies of chunk g+1 (own stream) run under the kernels of chunk g, and the
// output of chunk g goes back (third stream) under the kernels of chunk g+1.  Every chunk runs the
// four stages through a view of the plan with fewer heads, on the same workspace.
int spade_forward_host(spade_plan_t* p, const void* hQ, const void* hK, const void* hV, void* hO, void* dQ, void* dK,
                       void* dV, void* dO, void* ws, void* stream, const int32_t* forced) {
  if (!p) return fail(SPADE_ERR_INVALID_ARG, "plan is NULL");
  if (!hQ || !hK || !hV || !hO) return fail(SPADE_ERR_INVALID_ARG, "a host tensor is NULL");
  cudaStream_t s = (cudaStream_t)stream;
  ON_PLAN_DEVICE(p);
  int rc;
  if ((rc = check_call(p, ws))) return rc;
  if ((rc = check_tensor(dQ, "dQ")) || (rc = check_tensor(dK, "dK")) || (rc = check_tensor(dV, "dV")) || (rc = check_tensor(dO, "dO"))) return rc;
  if (!p->host_ready) {
    CUDA_TRY(cudaStreamCreateWithFlags(&p->copy_in, cudaStreamNonBlocking));
    CUDA_TRY(cudaStreamCreateWithFlags(&p->copy_out, cudaStreamNonBlocking));
    for (int i = 0; i < SPADE_HOST_CHUNKS; ++i) {
      CUDA_TRY(cudaEventCreateWithFlags(&p->ev_in[i], cudaEventDisableTiming));
      CUDA_TRY(cudaEventCreateWithFlags(&p->ev_done[i], cudaEventDisableTiming));
    }
    CUDA_TRY(cudaEventCreateWithFlags(&p->ev_edge, cudaEventDisableTiming));
    p->host_ready = 1;
  }
  const int BH = p->sh.BH;
  // The AS-coupled budget needs the scores of all heads at once; everything else is per head.
  int chunks = p->sh.mode == SPADE_POLICY_AS ? 1 : (BH >= 32 ? 12 : BH >= 12 ? 8 : BH >= 4 ? 4 : 1);
  if (chunks > SPADE_HOST_CHUNKS) chunks = SPADE_HOST_CHUNKS;
  // The input copies are the slower side (about 1.1 ms per Wan-14B head against 0.9 ms of kernels), so the call ends one
  // chunk's kernels and output copy after the last input byte, provided the kernels of chunk g are done by the time chunk
  // g + 1 has arrived.  Chunk sizes therefore shrink geometrically, by a fifth from one chunk to the next.
  int size[SPADE_HOST_CHUNKS], first[SPADE_HOST_CHUNKS + 1];
  {
    double w[SPADE_HOST_CHUNKS], total = 0.0, run = 0.0;
    for (int k = 0; k < chunks; ++k) { w[k] = pow(1.25, (double)(chunks - 1 - k)); total += w[k]; }
    first[0] = 0;
    for (int k = 0; k < chunks; ++k) {
      run += w[k];
      int end = k + 1 == chunks ? BH : (int)floor((double)BH * run / total + 0.5);
      const int lo = first[k] + 1, hi = BH - (chunks - 1 - k);       // every chunk holds at least one head
      end = end < lo ? lo : (end > hi ? hi : end);
      first[k + 1] = end;
      size[k] = end - first[k];
    }
  }
  const size_t head_bytes = (size_t)p->sh.N * SPADE_D * 2;
  // copies start after the work already queued on `stream` (it may still read the device buffers)
  CUDA_TRY(cudaEventRecord(p->ev_edge, s));
  CUDA_TRY(cudaStreamWaitEvent(p->copy_in, p->ev_edge, 0));
  CUDA_TRY(cudaStreamWaitEvent(p->copy_out, p->ev_edge, 0));
  int n_chunks = 0;
  for (; n_chunks < chunks; ++n_chunks) {
    const int h0 = first[n_chunks], nh = size[n_chunks];
    const size_t off = (size_t)h0 * head_bytes, bytes = (size_t)nh * head_bytes;
    CUDA_TRY(cudaMemcpyAsync((char*)dQ + off, (const char*)hQ + off, bytes, cudaMemcpyHostToDevice, p->copy_in));
    CUDA_TRY(cudaMemcpyAsync((char*)dK + off, (const char*)hK + off, bytes, cudaMemcpyHostToDevice, p->copy_in));
    CUDA_TRY(cudaMemcpyAsync((char*)dV + off, (const char*)hV + off, bytes, cudaMemcpyHostToDevice, p->copy_in));
    CUDA_TRY(cudaEventRecord(p->ev_in[n_chunks], p->copy_in));
  }
  int launches = 0;
  rc = SPADE_OK;
  for (int g = 0; g < n_chunks && rc == SPADE_OK; ++g) {
    const int h0 = first[g], nh = size[g];
    const size_t off = (size_t)h0 * head_bytes, bytes = (size_t)nh * head_bytes;
    spade_plan_s view = *p;                           // shares the static tables and the descriptor scratch
    view.sh.BH = nh;
    view.st.budget = p->st.budget + h0;
    view.keep_status = g > 0;
    view.stage = 0; view.stage_ws = nullptr; view.smaps_ws = nullptr;
    view.mq = view.mk = view.mv = view.mo = nullptr;
    view.pq = view.pk = nullptr;
    compute_layout(&view);
    CUDA_TRY(cudaStreamWaitEvent(s, p->ev_in[g], 0));
    rc = spade_forward(&view, (char*)dQ + off, (char*)dK + off, (char*)dV + off, (char*)dO + off, ws, stream,
                       forced ? forced + h0 : nullptr);
    launches += view.launches;
    if (rc) break;
    CUDA_TRY(cudaEventRecord(p->ev_done[g], s));
    CUDA_TRY(cudaStreamWaitEvent(p->copy_out, p->ev_done[g], 0));
    CUDA_TRY(cudaMemcpyAsync((char*)hO + off, (const char*)dO + off, bytes, cudaMemcpyDeviceToHost, p->copy_out));
  }
  // the views overwrote the shared descriptors and laid the workspace out for fewer heads
  p->mq = p->mk = p->mv = p->mo = nullptr;
  p->pq = p->pk = nullptr;
  p->smaps_ws = nullptr;
  p->stage = 0; p->stage_ws = nullptr;
  p->launches = launches;
  cudaError_t e1 = cudaEventRecord(p->ev_edge, p->copy_out);
  cudaError_t e2 = cudaStreamWaitEvent(s, p->ev_edge, 0);
  cudaError_t e3 = cudaStreamSynchronize(s);
  cudaError_t e4 = cudaStreamSynchronize(p->copy_in);       // nothing of this call is in flight on return
  if (rc) return rc;
  CUDA_TRY(e1); CUDA_TRY(e2); CUDA_TRY(e3); CUDA_TRY(e4);
  return SPADE_OK;
}

int spade_status(spade_plan_t* p, void* ws, void* stream) {
  int rc = check_call(p, ws);
  if (rc) return rc;
  ON_PLAN_DEVICE(p);
  uint32_t st[4] = {0, 0, 0, 0};
  CUDA_TRY(cudaMemcpyAsync(st, tables_at(p, ws).status, sizeof(st), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
  if (st[0] == SPADE_ST_TIMEOUT)
    return fail(SPADE_ERR_DEVICE_TIMEOUT, "a device-side wait gave up (site %u, work item %u)", st[1], st[2]);
  if (st[0] != 0) return fail(SPADE_ERR_CUDA, "device status %u", st[0]);
#ifdef SPADE_DEBUG
  {
    uint32_t dbg[4] = {0, 0, 0, 0};
    CUDA_TRY(cudaMemcpyAsync(dbg, tables_at(p, ws).status + 4, sizeof(dbg), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    if (dbg[0] != 0)
      return fail(SPADE_ERR_DEBUG_CHECK, "%u index checks failed; first at site %u with value %u", dbg[0], dbg[1], dbg[2]);
    if (p->stage > 0 && p->stage_ws == ws) {               // the workspace is laid out as this plan describes
      std::vector<unsigned char> guard((size_t)p->lay.n_canary * 256);
      for (int i = 0; i < p->lay.n_canary; ++i)
        CUDA_TRY(cudaMemcpyAsync(guard.data() + (size_t)i * 256, (const char*)ws + p->lay.canary[i], 256, cudaMemcpyDeviceToHost,
                                 (cudaStream_t)stream));
      CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
      for (size_t i = 0; i < guard.size(); ++i)
        if (guard[i] != 0xC5)
          return fail(SPADE_ERR_DEBUG_CHECK, "guard word behind workspace region %zu was overwritten (byte %zu)", i / 256, i % 256);
    }
  }
#endif
  return SPADE_OK;
}

int spade_launch_count(const spade_plan_t* p) { return p ? p->launches : 0; }

int spade_selftest_bounded_wait(void* out4, int32_t limit_us, void* stream) {
  if (!out4 || ((uintptr_t)out4 & 3)) return fail(SPADE_ERR_INVALID_ARG, "out4 is NULL or misaligned");
  if (limit_us < 1 || limit_us > 1000000) return fail(SPADE_ERR_INVALID_ARG, "limit_us must be in [1, 1000000]");
  CUDA_TRY(launch_selftest_wait((uint32_t*)out4, (unsigned long long)limit_us * 1000ull, (cudaStream_t)stream));
  return SPADE_OK;
}

}  // extern "C"

// ================================================================================================
// Allocation-free Aggregation Scores.  The per-block SICS table lives in a fixed array inside the
// library image instead of the caller's workspace, for callers that cannot get device memory when
// they need the scores (see spade.h).  The array is shared by every call on a device.
// ================================================================================================
#include <mutex>

namespace {

static __device__ __align__(256) float g_noalloc_sics[SPADE_NOALLOC_MAX_FLOATS];

constexpr int NOALLOC_MAX_DEVICES = 64;
std::mutex g_noalloc_mutex;
float* g_noalloc_ptr[NOALLOC_MAX_DEVICES];      // device address of the array, per device ordinal

// AS(X|c) = sum of the per-block SICS (Eq. 3), added in the fixed order the planning stage uses
// (lane-strided partial sums, then a butterfly).  The block values themselves come from the
// per-candidate token pass here; the planning stage usually builds them from shared cell sums, so the
// two entry points agree to fp32 summation order, not bit for bit.
__global__ void __launch_bounds__(32)
k_as_from_scratch(const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp,
                  const float* __restrict__ sics, float* __restrict__ as_out) {
  const int bh = blockIdx.x, lane = threadIdx.x;
  for (int c = 0; c < sh.C; ++c)
    for (int t = 0; t < 2; ++t) {
      const float* p = sics + (((size_t)bh * sh.C + c) * 2 + t) * sh.NBvmax;
      float s = 0.f;
      for (int b = lane; b < gp.g[c].NBv; b += 32) s += p[b];
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (lane == 0) as_out[((size_t)bh * sh.C + c) * 2 + t] = s;
    }
}

}  // namespace

extern "C" int spade_aggregation_scores_noalloc(spade_plan_t* p, const void* Q, const void* K, float* as_out,
                                                void* stream) {
  if (!p) return fail(SPADE_ERR_INVALID_ARG, "plan is NULL");
  int rc;
  if ((rc = check_tensor(Q, "Q")) || (rc = check_tensor(K, "K"))) return rc;
  if (!as_out || ((uintptr_t)as_out & 3)) return fail(SPADE_ERR_INVALID_ARG, "as_out is NULL or misaligned");
  const size_t need = (size_t)p->sh.BH * p->sh.C * 2 * p->sh.NBvmax;
  if (need > SPADE_NOALLOC_MAX_FLOATS)
    return fail(SPADE_ERR_UNSUPPORTED,
                "this plan needs %zu scratch floats (B*heads=%d x candidates=%d x 2 x %d blocks); the built-in array "
                "holds %u -- use spade_plan with a workspace instead",
                need, p->sh.BH, p->sh.C, p->sh.NBvmax, (unsigned)SPADE_NOALLOC_MAX_FLOATS);
  if (p->device < 0 || p->device >= NOALLOC_MAX_DEVICES) return fail(SPADE_ERR_UNSUPPORTED, "device ordinal %d", p->device);
  ON_PLAN_DEVICE(p);
  float* scratch;
  {
    // Once per device: in host code the array's name is only a handle, so ask the runtime for the
    // address the kernels must be given (this device is current here).
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[p->device]) {
      void* addr = nullptr;
      cudaError_t e = cudaGetSymbolAddress(&addr, g_noalloc_sics);
      if (e != cudaSuccess || !addr) return fail(SPADE_ERR_CUDA, "cudaGetSymbolAddress(scratch): %s", cudaGetErrorString(e));
      g_noalloc_ptr[p->device] = (float*)addr;
    }
    scratch = g_noalloc_ptr[p->device];
  }
  WsTables t;
  memset(&t, 0, sizeof(t));
  t.sics = scratch;                       // the SICS pass touches no other table
  cudaStream_t s = (cudaStream_t)stream;
  CUDA_TRY(launch_sics(Q, K, p->sh, p->gp, p->st, t, p->num_sms, s));
  k_as_from_scratch<<<p->sh.BH, 32, 0, s>>>(p->sh, p->gp, scratch, as_out);
  CUDA_TRY(cudaGetLastError());
  p->launches = 2;
  return SPADE_OK;
}
