// Flash block-sparse attention for sm_100a (Eq. 2; Sec. 3.3, optimisation 3).
//
// One persistent CTA walks work items (head, 128-row query tile), head by head, longest items first.
// A query tile is one 128-token block, or two consecutive 64-token
// blocks whose index lists are merged (union) with a per-half column mask.  The 3-D blocks are
// never re-laid-out in memory: every Q/K/V tile is a 5-D TMA box (d, w, h, t, head) of the
// original [B,H,N,d] tensor that lands in shared memory already in the 128-byte-swizzled
// operand layout of the tensor core; out-of-grid positions of edge blocks are zero-filled on
// load, masked to -inf as keys and clipped on store.
//
// K and V travel in units of 64 keys (a 64-token block, or half of a 128-token block): K in a ring of
// three stages, V of two.  Warp roles (256 threads): warps 0-3 softmax + epilogue (one query row per
// thread, TMEM lane = row), warp 4 producer (builds the item's list, loads Q and every K unit), warp 5
// issuer of S = Q K^T, warp 6 issuer of O += P V (one thread each), warp 7 loader of V.
// Per 64-key unit h: S = Q K^T into TMEM (128x64 fp32, one buffer); the softmax warps copy it into
// registers and free the buffer at once, so S of unit h+1 is issued while the softmax of unit h runs
// (its only other condition is that K has arrived, hence the deeper K ring); online max / sum with lazy
// rescale; P as bf16 into a TMEM buffer of its own; O += P V and the row sums L += P 1 (a second, 16-column
// product against a block of ones) with P read from TMEM.  The
// lists of the work items live in a per-CTA scratch of the workspace (shared memory is full of tiles)
// and are read a unit or two ahead.  All waits are bounded; on expiry the CTA records the site in the
// status words and leaves.
#include <cuda.h>
#include <stdio.h>
#include <string.h>

#include "sm100_ptx.cuh"
#include "spade_common.cuh"

struct CandMaps { CUtensorMap q, k, v, o; };   // q, o: box of one block; k, v: box of 64 rows
struct AttnMaps {
  CandMaps c[SPADE_MAX_CANDS];     // 5-D maps (d, W, H, T, head)
  CandMaps text[2];                // 3-D maps (d, N, head) for the text rows: [0] 64-token, [1] 128-token blocks
};

namespace {

constexpr int ATT_THREADS = 256;
constexpr int REGS_SOFTMAX = 168;           // 128*168 + 128*88 = 32768 registers = half an SM
constexpr int REGS_OTHER = 88;
constexpr int SUB_BYTES = 16384;            // Q / O tile: 128 rows x 128 B per 64-channel half
constexpr int TILE_BYTES = 2 * SUB_BYTES;
constexpr int KSUB_BYTES = 8192;            // K / V unit: 64 rows x 128 B per 64-channel half
constexpr int KV_BYTES = 2 * KSUB_BYTES;
constexpr uint64_t WAIT_NS = 2000000000ull; // bound of every device-side wait
constexpr uint32_t TMEM_COLS = 256;         // S: columns 0..63, P (bf16 pairs): 64..95, row sums L: 96..111, Q channels 0..31: 112..127, O: 128..255
#ifndef ATT_CODE_PAD
#define ATT_CODE_PAD 256    // instructions; see the softmax role.  Attention time repeats with a period of 512 (8 KB): fastest at 192..320
#endif
constexpr int Q_TS_STEPS = 2;                // 16-channel steps of S = Q K^T that take Q from tensor memory (what the 16 spare columns hold)
constexpr unsigned FULL = 0xffffffffu;

// One work item as the producer warp publishes it to the other roles.  The (merged) list itself lives in
// a per-CTA scratch in the workspace (shared memory is taken by the tiles): entry e = KV block id in bits
// 0..15, bit 16 + q set <=> query half q wants that block; ascending block ids.
struct ItemSlot {
  int bh, c, qb0, qb1, n_entries, H, item, pad1;   // H = number of 64-key units; H < 0: no more work
};
constexpr int K_STAGES = 3;                 // K needs the longest look-ahead: S = Q K^T of unit j+1 is issued as soon
constexpr int V_STAGES = 2;                 // as the scores of unit j are in registers

struct Ctl {
  uint64_t list_full[2], list_empty[2];
  uint64_t q_full, q_empty, qt_full;
  uint64_t k_full[K_STAGES], k_empty[K_STAGES], v_full[V_STAGES], v_empty[V_STAGES], s_full, s_free, p_full, pv_done;
  uint32_t tmem_base;
  volatile uint32_t abort;
  __align__(128) uint16_t ones[64];  // one 8 x 8 core matrix of bf16 1.0: operand B of the row-sum product
  uint32_t bm[2][SPADE_MAX_NB / 32];
  ItemSlot slot[2];
};

constexpr size_t ATT_SMEM = TILE_BYTES + (K_STAGES + V_STAGES) * KV_BYTES + sizeof(Ctl);
static_assert(ATT_SMEM <= 113 * 1024, "two CTAs per SM");

template <int N> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// Loads one Q block (BS rows, both 64-channel halves) into a 128-row tile at `dst`.
__device__ __forceinline__ void load_q_block(uint8_t* dst, const CandMaps& vm, const CandMaps& tm, uint64_t* bar,
                                             const CandGeo& g, const Shape& sh, int blk, int bh) {
  if (blk >= g.NBv) {
    const int row = sh.Nv + (blk - g.NBv) * g.BS;
    ptx::tma_load_3d(dst, &tm.q, bar, 0, row, bh);
    ptx::tma_load_3d(dst + SUB_BYTES, &tm.q, bar, 64, row, bh);
  } else {
    int it, ih, iw;
    block_coords(g, blk, it, ih, iw);
    ptx::tma_load_5d(dst, &vm.q, bar, 0, iw * g.bw, ih * g.bh, it * g.bt, bh);
    ptx::tma_load_5d(dst + SUB_BYTES, &vm.q, bar, 64, iw * g.bw, ih * g.bh, it * g.bt, bh);
  }
}

// Loads one 64-key unit of K (which = 0) or V (which = 1): block `blk`, half `half` (0 for 64-token blocks).
__device__ __forceinline__ void load_kv_unit(uint8_t* dst, const CandMaps& vm, const CandMaps& tm, int which,
                                             uint64_t* bar, const CandGeo& g, const Shape& sh, int blk, int half, int bh) {
  const CUtensorMap* vmap = which == 0 ? &vm.k : &vm.v;
  const CUtensorMap* tmap = which == 0 ? &tm.k : &tm.v;
  if (blk >= g.NBv) {
    const int row = sh.Nv + (blk - g.NBv) * g.BS + half * 64;
    ptx::tma_load_3d(dst, tmap, bar, 0, row, bh);
    ptx::tma_load_3d(dst + KSUB_BYTES, tmap, bar, 64, row, bh);
  } else {
    int it, ih, iw;
    block_coords(g, blk, it, ih, iw);          // two high multiplies: this runs per unit in a thread that shares a scheduler with a softmax warp
    const int w0 = iw * g.bw + half * g.hw, h0 = ih * g.bh + half * g.hh, t0 = it * g.bt + half * g.ht;
    ptx::tma_load_5d(dst, vmap, bar, 0, w0, h0, t0, bh);
    ptx::tma_load_5d(dst + KSUB_BYTES, vmap, bar, 64, w0, h0, t0, bh);
  }
}

__device__ __forceinline__ void store_o_block(const uint8_t* src, const CandMaps& vm, const CandMaps& tm,
                                              const CandGeo& g, const Shape& sh, int blk, int bh) {
  if (blk >= g.NBv) {
    const int row = sh.Nv + (blk - g.NBv) * g.BS;
    ptx::tma_store_3d(&tm.o, src, 0, row, bh);
    ptx::tma_store_3d(&tm.o, src + SUB_BYTES, 64, row, bh);
  } else {
    const int iw = blk % g.nbw, ih = (blk / g.nbw) % g.nbh, it = blk / (g.nbw * g.nbh);   // once per item: the divisions stay (nothing to win here; the 14 % once measured against the multiply form was code placement, see ATT_CODE_PAD)
    ptx::tma_store_5d(&vm.o, src, 0, iw * g.bw, ih * g.bh, it * g.bt, bh);
    ptx::tma_store_5d(&vm.o, src + SUB_BYTES, 64, iw * g.bw, ih * g.bh, it * g.bt, bh);
  }
}

__device__ __forceinline__ void report_timeout(const WsTables& ws, Ctl& ctl, uint32_t site, uint32_t item) {
  ctl.abort = 1;
  if (atomicCAS(ws.status, 0u, (uint32_t)SPADE_ST_TIMEOUT) == 0u) { ws.status[1] = site; ws.status[2] = item; }
}

__global__ void __launch_bounds__(ATT_THREADS, 2)
k_attn(const __grid_constant__ AttnMaps maps, const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp,
       const StaticTables st, const WsTables ws, const float scale_log2) {
  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* sQ = smem;                         // also the staging buffer of the output tile
  uint8_t* sK = smem + TILE_BYTES;            // K_STAGES stages of KV_BYTES
  uint8_t* sV = sK + K_STAGES * KV_BYTES;     // V_STAGES stages of KV_BYTES
  Ctl& ctl = *reinterpret_cast<Ctl*>(sV + V_STAGES * KV_BYTES);
  if (ptx::smem_u32(smem) & 1023u) {          // the swizzled tiles need 1024-byte alignment; never seen otherwise
    if (threadIdx.x == 0 && atomicCAS(ws.status, 0u, (uint32_t)SPADE_ST_TIMEOUT) == 0u) { ws.status[1] = 99; ws.status[2] = 0; }
    return;
  }
  uint32_t* const scratch = ws.att_scratch + (size_t)blockIdx.x * 2 * SPADE_MAX_NB;     // two lists of SPADE_MAX_NB entries

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // ---- one-time set-up -----------------------------------------------------------------------
  for (int i = tid; i < (TILE_BYTES + (K_STAGES + V_STAGES) * KV_BYTES) / 16; i += ATT_THREADS)        // buffers start finite: rows that a
    reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);      // partly filled tile never loads multiply p = 0
  if (tid == 0) {
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(&ctl.list_full[b], 1);
      ptx::mbar_init(&ctl.list_empty[b], 4);      // both issuers, the V loader and the epilogue thread
    }
    for (int b = 0; b < K_STAGES; ++b) { ptx::mbar_init(&ctl.k_full[b], 1); ptx::mbar_init(&ctl.k_empty[b], 1); }
    for (int b = 0; b < V_STAGES; ++b) { ptx::mbar_init(&ctl.v_full[b], 1); ptx::mbar_init(&ctl.v_empty[b], 1); }
    ptx::mbar_init(&ctl.p_full, 4);             // one arrival per softmax warp
    ptx::mbar_init(&ctl.pv_done, 1);
    ptx::mbar_init(&ctl.s_full, 1);
    ptx::mbar_init(&ctl.s_free, 4);             // the four softmax warps hold the scores in registers
    ptx::mbar_init(&ctl.q_full, 1);
    ptx::mbar_init(&ctl.q_empty, 2);          // epilogue thread + MMA issuer
    ptx::mbar_init(&ctl.qt_full, 4);          // one arrival per softmax warp: the first channels of Q are in tensor memory
    ctl.abort = 0;
    for (int i = 0; i < 64; ++i) ctl.ones[i] = 0x3f80;
    ptx::fence_mbar_init();
  }
  if (warp == 5) {
    ptx::tmem_alloc(&ctl.tmem_base, TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::fence_proxy_async_smem();
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_S = ctl.tmem_base;
  const uint32_t tmem_P = tmem_S + 64;
  const uint32_t tmem_L = tmem_S + 96;        // 16 equal columns: sum over the keys of the bf16 weights, kept by the tensor core
  const uint32_t tmem_Q = tmem_S + 112;       // Q channels 0..31 as bf16 pairs (operand A of the first two steps of S)
  const uint32_t tmem_O = tmem_S + 128;
  const int total_items = ws.item_start[sh.BH];
  const int total_text = ws.text_start[sh.BH];

  if (warp >= 4) {
    reg_dec<REGS_OTHER>();
    if (warp == 4) {
      // ================= producer: decode item, build its list, issue every TMA load ================
      uint32_t it = 0, hc = 0;        // items and 64-key units so far
      // The two prefix tables of the work-item order, two entries per lane (up to 63 heads): finding the head
      // of an item is then two ballots instead of a chain of dependent global loads.
      const bool cached = sh.BH + 1 <= 64;
      int ts_c[2], vs_c[2];
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int i = lane + 32 * k;
        ts_c[k] = (cached && i <= sh.BH) ? ws.text_start[i] : 0x7fffffff;
        vs_c[k] = (cached && i <= sh.BH) ? ws.item_start[i] - ws.text_start[i] : 0x7fffffff;
      }
      for (;; ++it) {
        ItemSlot& sl = ctl.slot[it & 1];
        uint32_t* const list = scratch + (it & 1) * SPADE_MAX_NB;
        bool ok = ptx::mbar_wait(&ctl.list_empty[it & 1], ((it >> 1) & 1) ^ 1, &ctl.abort, WAIT_NS);
        if (ok && *reinterpret_cast<volatile uint32_t*>(ws.status) != 0) { ctl.abort = 1; ok = false; }   // another CTA gave up
        if (!__all_sync(FULL, ok)) { if (lane == 0) report_timeout(ws, ctl, 1, it); break; }
        // work items are handed out dynamically (list lengths differ a lot between query tiles)
        int w = 0;
        if (lane == 0) w = (int)atomicAdd(ws.status + 8, 1u);
        w = __shfl_sync(FULL, w, 0);
        if (w >= total_items) {
          if (lane == 0) { sl.H = -1; ptx::mbar_arrive(&ctl.list_full[it & 1]); }
          break;
        }
        // longest items first: the text query tiles of all heads (they attend every block), then the
        // video tiles head by head.  lo_i = largest i whose prefix is <= the index within its section.
        const bool text_item = w < total_text;
        const int wi = text_item ? w : w - total_text;
        int lo_i = 0, t_lo, t_hi, v_lo, v_hi;      // the two prefixes at lo_i and lo_i + 1
        if (cached) {
          int below = 0;                            // entries i < BH whose start is <= wi (entry 0 always is)
#pragma unroll
          for (int k = 0; k < 2; ++k) {
            const bool le = lane + 32 * k < sh.BH && (text_item ? ts_c[k] : vs_c[k]) <= wi;
            below += __popc(__ballot_sync(FULL, le));
          }
          lo_i = below - 1;
          const int a = lo_i, b2 = lo_i + 1;
          const int ta0 = __shfl_sync(FULL, ts_c[0], a & 31), ta1 = __shfl_sync(FULL, ts_c[1], a & 31);
          const int tb0 = __shfl_sync(FULL, ts_c[0], b2 & 31), tb1 = __shfl_sync(FULL, ts_c[1], b2 & 31);
          const int va0 = __shfl_sync(FULL, vs_c[0], a & 31), va1 = __shfl_sync(FULL, vs_c[1], a & 31);
          const int vb0 = __shfl_sync(FULL, vs_c[0], b2 & 31), vb1 = __shfl_sync(FULL, vs_c[1], b2 & 31);
          t_lo = a < 32 ? ta0 : ta1; t_hi = b2 < 32 ? tb0 : tb1;
          v_lo = a < 32 ? va0 : va1; v_hi = b2 < 32 ? vb0 : vb1;
        } else {
          int hi_i = sh.BH;
          while (hi_i - lo_i > 1) {
            const int mid = (lo_i + hi_i) >> 1;
            const int start = text_item ? ws.text_start[mid] : ws.item_start[mid] - ws.text_start[mid];
            if (start <= wi) lo_i = mid; else hi_i = mid;
          }
          t_lo = ws.text_start[lo_i]; t_hi = ws.text_start[lo_i + 1];
          v_lo = ws.item_start[lo_i] - t_lo; v_hi = ws.item_start[lo_i + 1] - t_hi;
        }
        const int bh = ws.head_order[lo_i];
        const int c = ws.scheme[bh];
        const CandGeo& g = gp.g[c];
        const int n_video_tiles = v_hi - v_lo;
        const int tile = text_item ? n_video_tiles + (wi - t_lo) : wi - v_lo;
        int qb0, qb1;
        tile_blocks(g, st, ws.cell_axis + (size_t)bh * sh.cell_ld, tile, qb0, qb1);
        int n_entries;
        if (g.pair) {
          // merged (union) list of the two 64-token query blocks, via a bitmap over KV block ids
          for (int i = lane; i < 2 * (SPADE_MAX_NB / 32); i += 32) (&ctl.bm[0][0])[i] = 0;
          __syncwarp();
          // both rows at once, two entries of each per lane in flight (the loads are the slow part)
          const int* row0 = ws.kv_idx + ((size_t)bh * sh.NBmax + qb0) * sh.cap;
          const int* row1 = ws.kv_idx + ((size_t)bh * sh.NBmax + (qb1 >= 0 ? qb1 : qb0)) * sh.cap;
          int cnt0 = ws.kv_cnt[(size_t)bh * sh.NBmax + qb0];
          int cnt1 = qb1 >= 0 ? ws.kv_cnt[(size_t)bh * sh.NBmax + qb1] : 0;
          (void)SPADE_CHECK(cnt0 >= 0 && cnt0 <= sh.cap && cnt1 >= 0 && cnt1 <= sh.cap, ws.status, 403, cnt0);
          cnt0 = cnt0 < 0 ? 0 : (cnt0 > sh.cap ? sh.cap : cnt0);
          cnt1 = cnt1 < 0 ? 0 : (cnt1 > sh.cap ? sh.cap : cnt1);
          const int cmax = cnt0 > cnt1 ? cnt0 : cnt1;
          for (int e = lane; e < cmax; e += 64) {
            const int a0 = e < cnt0 ? row0[e] : -1, a1 = e + 32 < cnt0 ? row0[e + 32] : -1;
            const int c0 = e < cnt1 ? row1[e] : -1, c1 = e + 32 < cnt1 ? row1[e + 32] : -1;
            if (a0 >= 0 && a0 < g.NB) atomicOr(&ctl.bm[0][a0 >> 5], 1u << (a0 & 31));
            if (a1 >= 0 && a1 < g.NB) atomicOr(&ctl.bm[0][a1 >> 5], 1u << (a1 & 31));
            if (c0 >= 0 && c0 < g.NB) atomicOr(&ctl.bm[1][c0 >> 5], 1u << (c0 & 31));
            if (c1 >= 0 && c1 < g.NB) atomicOr(&ctl.bm[1][c1 >> 5], 1u << (c1 & 31));
          }
          __syncwarp();
          const int nw = (g.NB + 31) >> 5;         // <= 64 words: two per lane
          const uint32_t a0 = lane < nw ? ctl.bm[0][lane] : 0u, b0 = lane < nw ? ctl.bm[1][lane] : 0u;
          const uint32_t a1 = lane + 32 < nw ? ctl.bm[0][lane + 32] : 0u, b1 = lane + 32 < nw ? ctl.bm[1][lane + 32] : 0u;
          const int c0 = __popc(a0 | b0), c1 = __popc(a1 | b1);
          int i0 = c0, i1 = c1;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const int x = __shfl_up_sync(FULL, i0, o), y = __shfl_up_sync(FULL, i1, o);
            if (lane >= o) { i0 += x; i1 += y; }
          }
          const int tot0 = __shfl_sync(FULL, i0, 31), tot1 = __shfl_sync(FULL, i1, 31);
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const uint32_t wa = half ? a1 : a0, wb = half ? b1 : b0;
            uint32_t u = wa | wb;
            int pos = half ? tot0 + i1 - c1 : i0 - c0;
            const int wi = lane + 32 * half;
            while (u) {
              const int bit = __ffs(u) - 1;
              u &= u - 1;
              if (SPADE_CHECK(pos < SPADE_MAX_NB && wi * 32 + bit < g.NB, ws.status, 401, pos))
                list[pos] = (uint32_t)(wi * 32 + bit) | (((wa >> bit) & 1u) << 16) | (((wb >> bit) & 1u) << 17);
              ++pos;
            }
          }
          n_entries = tot0 + tot1;
        } else {
          const int* row = ws.kv_idx + ((size_t)bh * sh.NBmax + qb0) * sh.cap;
          int cnt = ws.kv_cnt[(size_t)bh * sh.NBmax + qb0];
          (void)SPADE_CHECK(cnt >= 0 && cnt <= sh.cap, ws.status, 404, cnt);
          cnt = cnt < 0 ? 0 : (cnt > sh.cap ? sh.cap : cnt);
          cnt = cnt > SPADE_MAX_NB ? SPADE_MAX_NB : cnt;
          for (int e = lane; e < cnt; e += 32) {
            int id = row[e];
            (void)SPADE_CHECK(id >= 0 && id < g.NB, ws.status, 402, id);
            list[e] = (uint32_t)((id >= 0 && id < g.NB) ? id : 0) | (3u << 16);
          }
          n_entries = cnt;
        }
        const int H = g.pair ? n_entries : 2 * n_entries;
        if (lane == 0) { sl.bh = bh; sl.c = c; sl.qb0 = qb0; sl.qb1 = qb1; sl.n_entries = n_entries; sl.H = H; sl.item = w; }
        __syncwarp();
        if (lane == 0) {
          ptx::mbar_arrive(&ctl.list_full[it & 1]);
          const CandMaps& vm = maps.c[c];
          const CandMaps& tm = maps.text[g.pair ? 0 : 1];
          uint32_t site = 0;
          if (!ptx::mbar_wait(&ctl.q_empty, (it & 1) ^ 1, &ctl.abort, WAIT_NS)) site = 2;
          if (!site) {
            ptx::mbar_expect_tx(&ctl.q_full, g.pair ? (qb1 >= 0 ? TILE_BYTES : TILE_BYTES / 2) : TILE_BYTES);
            load_q_block(sQ, vm, tm, &ctl.q_full, g, sh, qb0, bh);
            if (qb1 >= 0) load_q_block(sQ + SUB_BYTES / 2, vm, tm, &ctl.q_full, g, sh, qb1, bh);
          }
          // K units (V has a loader of its own so that a full V ring never holds back the K look-ahead)
          uint32_t e_next = H > 0 ? __ldcg(list) : 0u;
          for (int j = 0; j < H && !site; ++j, ++hc) {
            const int blk = (int)(e_next & 0xffffu);
            (void)SPADE_CHECK(blk < g.NB, ws.status, 405, blk);
            const int half = g.pair ? 0 : (j & 1);
            const int jn = j + 1 < H ? j + 1 : j;
            e_next = __ldcg(list + (g.pair ? jn : (jn >> 1)));          // fetched one unit ahead
            const uint32_t b = hc % K_STAGES, par = ((hc / K_STAGES) & 1) ^ 1;
            if (!ptx::mbar_wait(&ctl.k_empty[b], par, &ctl.abort, WAIT_NS)) { site = 3; break; }
            ptx::mbar_expect_tx(&ctl.k_full[b], KV_BYTES);
            load_kv_unit(sK + b * KV_BYTES, vm, tm, 0, &ctl.k_full[b], g, sh, blk, half, bh);
          }
          if (site) report_timeout(ws, ctl, site, (uint32_t)w);
        }
        __syncwarp();
        if (__any_sync(FULL, ctl.abort != 0)) break;
      }
    } else if (warp == 7 && lane == 0) {
      // ================= loader of V ======================================================================
      uint32_t it = 0, hc = 0;
      for (;; ++it) {
        uint32_t site = 0;
        if (!ptx::mbar_wait(&ctl.list_full[it & 1], (it >> 1) & 1, &ctl.abort, WAIT_NS)) site = 18;
        const ItemSlot& sl = ctl.slot[it & 1];
        const int H = site ? 0 : sl.H;
        const int w = sl.item;
        if (H < 0) break;
        const CandGeo& g = gp.g[site ? 0 : sl.c];
        const CandMaps& vm = maps.c[site ? 0 : sl.c];
        const CandMaps& tm = maps.text[g.pair ? 0 : 1];
        const uint32_t* list = scratch + (it & 1) * SPADE_MAX_NB;
        const int bh = sl.bh;
        uint32_t e_next = H > 0 ? __ldcg(list) : 0u;
        for (int j = 0; j < H && !site; ++j, ++hc) {
          const int blk = (int)(e_next & 0xffffu);
          const int half = g.pair ? 0 : (j & 1);
          const int jn = j + 1 < H ? j + 1 : j;
          e_next = __ldcg(list + (g.pair ? jn : (jn >> 1)));
          const uint32_t b = hc % V_STAGES, par = ((hc / V_STAGES) & 1) ^ 1;
          if (!ptx::mbar_wait(&ctl.v_empty[b], par, &ctl.abort, WAIT_NS)) { site = 4; break; }
          ptx::mbar_expect_tx(&ctl.v_full[b], KV_BYTES);
          load_kv_unit(sV + b * KV_BYTES, vm, tm, 1, &ctl.v_full[b], g, sh, blk, half, bh);
        }
        if (site) { report_timeout(ws, ctl, site, (uint32_t)w); break; }
        ptx::mbar_arrive(&ctl.list_empty[it & 1]);
      }
    } else if (warp == 5 && lane == 0) {
      // ================= issuer of S = Q K^T ============================================================
      // (two issuing threads: a tcgen05.mma issue blocks while the tensor pipe is busy, so one thread
      //  doing both products would hold back O += P V of unit j behind the issue of S of unit j+1)
      const uint32_t idesc_s = ptx::idesc_bf16(128, 64, false);
      const uint32_t aQ = ptx::smem_u32(sQ), aK = ptx::smem_u32(sK);
      // Descriptors differ from a base only in the 16-byte address units of their low bits (shared-memory addresses stay
      // below 2^18, so nothing carries): the eight of Q are fixed, K's are a base per stage plus a constant per step.
      uint64_t qd[8];
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) qd[ks] = ptx::smem_desc_sw128(aQ + (ks >> 2) * SUB_BYTES + (ks & 3) * 32, 16, 1024);
      const uint64_t kd0 = ptx::smem_desc_sw128(aK, 16, 1024);
      uint32_t it = 0, hc = 0;
      for (;; ++it) {
        uint32_t site = 0;
        if (!ptx::mbar_wait(&ctl.list_full[it & 1], (it >> 1) & 1, &ctl.abort, WAIT_NS)) site = 5;
        const int H = site ? 0 : ctl.slot[it & 1].H;
        const int w = ctl.slot[it & 1].item;
        if (H < 0) break;
        if (!site && !ptx::mbar_wait(&ctl.q_full, it & 1, &ctl.abort, WAIT_NS)) site = 6;
        if (!site && !ptx::mbar_wait(&ctl.qt_full, it & 1, &ctl.abort, WAIT_NS)) site = 19;
        if (!site) ptx::mbar_arrive(&ctl.q_empty);      // this role has seen the tile; the epilogue frees it
        for (int j = 0; j < H && !site; ++j) {
          const uint32_t h = hc + j, b = h % K_STAGES, u = (h / K_STAGES) & 1;
          if (!ptx::mbar_wait(&ctl.k_full[b], u, &ctl.abort, WAIT_NS) ||
              !ptx::mbar_wait(&ctl.s_free, (h & 1) ^ 1, &ctl.abort, WAIT_NS)) { site = 7; break; }   // S of unit h-1 is in registers
          ptx::tc_fence_after();
          const uint64_t kdb = kd0 + (uint64_t)((b * KV_BYTES) >> 4);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {          // both operands K-major, 16 channels per step
            const uint64_t kd = kdb + (uint64_t)(((ks >> 2) * KSUB_BYTES + (ks & 3) * 32) >> 4);
            // A product with Q in shared memory reads 6 KB per step and takes 48 clk for 32 clk of arithmetic; with Q in
            // tensor memory it reads K alone and takes the 32
            if (ks < Q_TS_STEPS) ptx::umma_ts(tmem_S, tmem_Q + ks * 8, kd, idesc_s, ks > 0);
            else ptx::umma_ss(tmem_S, qd[ks], kd, idesc_s, ks > 0);
          }
          ptx::umma_commit(&ctl.s_full);
          ptx::umma_commit(&ctl.k_empty[b]);
        }
        hc += (uint32_t)H;
        if (site) { report_timeout(ws, ctl, site, (uint32_t)w); break; }
        ptx::mbar_arrive(&ctl.list_empty[it & 1]);
      }
    } else if (warp == 6 && lane == 0) {
      // ================= issuer of O += P V =============================================================
      const uint32_t idesc_o = ptx::idesc_bf16(128, 128, true);
      const uint32_t idesc_l = ptx::idesc_bf16(128, 16, false);
      const uint32_t aV = ptx::smem_u32(sV);
      // every 8 x 8 core matrix of the 16 x 16 ones operand is the same 128 bytes: strides 0, no swizzle
      const uint64_t desc_ones = (uint64_t)((ptx::smem_u32(ctl.ones) & 0x3ffffu) >> 4) | ((uint64_t)1 << 46);
      const uint64_t vd0 = ptx::smem_desc_sw128(aV, KSUB_BYTES, 1024);
      uint32_t it = 0, hc = 0;
      for (;; ++it) {
        uint32_t site = 0;
        if (!ptx::mbar_wait(&ctl.list_full[it & 1], (it >> 1) & 1, &ctl.abort, WAIT_NS)) site = 16;
        const int H = site ? 0 : ctl.slot[it & 1].H;
        const int w = ctl.slot[it & 1].item;
        if (H < 0) break;
        for (int j = 0; j < H && !site; ++j) {
          const uint32_t h = hc + j, b = h & 1, u = (h >> 1) & 1;          // V stage and its phase
          if (!ptx::mbar_wait(&ctl.p_full, h & 1, &ctl.abort, WAIT_NS) ||
              !ptx::mbar_wait(&ctl.v_full[b], u, &ctl.abort, WAIT_NS)) { site = 8; break; }
          ptx::tc_fence_after();
          const uint64_t vdb = vd0 + (uint64_t)((b * KV_BYTES) >> 4);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)            // P from TMEM (bf16 pairs), V MN-major, 16 keys per step
            ptx::umma_ts(tmem_O, tmem_P + ks * 8, vdb + (uint64_t)((ks * 2048) >> 4), idesc_o, (j > 0 || ks > 0) ? 1u : 0u);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)            // L += P 1: the row sums of the weights as the tensor core sees them
            ptx::umma_ts(tmem_L, tmem_P + ks * 8, desc_ones, idesc_l, (j > 0 || ks > 0) ? 1u : 0u);
          ptx::umma_commit(&ctl.pv_done);
          ptx::umma_commit(&ctl.v_empty[b]);
        }
        hc += (uint32_t)H;
        if (site) { report_timeout(ws, ctl, site, (uint32_t)w); break; }
        ptx::mbar_arrive(&ctl.list_empty[it & 1]);
      }
    }
  } else {
    // ================= softmax + epilogue (warps 0..3, one query row per thread) ======================
    reg_inc<REGS_SOFTMAX>();
    // Never taken (BH is positive).  The instructions it keeps in the binary shift the loop below against the loops of the
    // helper roles in the instruction cache.  Measured over paddings of 0..2048 instructions: attention time repeats every
    // 512 instructions (8 KB), 2.02-2.04 ms at 0, 512, 1024, ... and 1.80 ms at 192..320 and 768 on the Wan-1.3B shape, with
    // the same instructions executed and instruction-fetch stalls per issue of 1.5 against 0.7: the loops evict one another
    // when they fall on the same cache sets.
    if (sh.BH < 0) {
#pragma unroll
      for (int i = 0; i < ATT_CODE_PAD; ++i) asm volatile("nanosleep.u32 1;");
    }
    const int row = warp * 32 + lane;
    const int qhalf = row >> 6;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    const uint64_t sc2 = pack2(scale_log2, scale_log2);
    uint32_t it = 0, hc = 0;
    for (;; ++it) {
      uint32_t site = 0;
      if (!__all_sync(FULL, ptx::mbar_wait(&ctl.list_full[it & 1], (it >> 1) & 1, &ctl.abort, WAIT_NS))) site = 9;
      const ItemSlot& sl = ctl.slot[it & 1];
      if (!site && sl.H < 0) break;                  // the producer has run out of work items
      const int H = site ? 0 : sl.H, bh = sl.bh, w = sl.item;
      const CandGeo& g = gp.g[site ? 0 : sl.c];
      const uint64_t* kvalid = st.kvalid + (size_t)g.tab_off * 2;
      if (!site) {
        // the row's first 32 channels go to tensor memory (the S products of the previous item are complete: their
        // last scores have been read)
        if (!__all_sync(FULL, ptx::mbar_wait(&ctl.q_full, it & 1, &ctl.abort, WAIT_NS))) site = 20;
        if (!site) {
          uint32_t qa[16];
#pragma unroll
          for (int c16 = 0; c16 < 4; ++c16) {
            const uint4 v = *reinterpret_cast<const uint4*>(sQ + row * 128 + ((c16 ^ (row & 7)) << 4));
            qa[c16 * 4 + 0] = v.x; qa[c16 * 4 + 1] = v.y; qa[c16 * 4 + 2] = v.z; qa[c16 * 4 + 3] = v.w;
          }
          ptx::tmem_st16(tmem_Q + lane_base, qa);
          ptx::tmem_wait_st();
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&ctl.qt_full);
        }
      }
      float m = -INFINITY;
      // List entries are fetched two units ahead and the valid-key masks one unit ahead, each touched only
      // an iteration after its load was issued, so neither latency sits on the critical path.
      const uint32_t* list = scratch + (it & 1) * SPADE_MAX_NB;
      auto entry_at = [&](int j) -> uint32_t {           // entry of unit j (the last unit's again past the end)
        const int jj = j < H ? j : (H > 0 ? H - 1 : 0);
        return __ldcg(list + (g.pair ? jj : (jj >> 1)));
      };
      auto mask_ptr = [&](uint32_t e, int j) -> const uint64_t* {
        return g.pair ? kvalid + 2 * (size_t)(e & 0xffffu) : kvalid + 2 * (size_t)(e & 0xffffu) + (j & 1);
      };
      uint32_t e_cur = (site || H == 0) ? 0u : entry_at(0);
      uint32_t e_nxt = (site || H == 0) ? 0u : entry_at(1);
      uint64_t mk_next = (site || H == 0) ? 0ull : __ldg(mask_ptr(e_cur, 0));
      for (int j = 0; j < H && !site; ++j) {
        const uint32_t h = hc + j;
        // the mask fetched one unit ahead is only touched now, so its latency is off the critical path
        const uint64_t mk = mk_next;
        const uint32_t e = e_cur;
        e_cur = e_nxt;                                    // unit j + 1: loaded an iteration ago
        e_nxt = entry_at(j + 2);
        mk_next = __ldg(mask_ptr(e_cur, j + 1 < H ? j + 1 : j));
        const uint64_t mask = (!g.pair || ((e >> (16 + qhalf)) & 1)) ? mk : 0ull;
        const bool all_valid = __all_sync(FULL, mask == ~0ull);
        if (!__all_sync(FULL, ptx::mbar_wait(&ctl.s_full, h & 1, &ctl.abort, WAIT_NS))) { site = 10; break; }
        ptx::tc_fence_after();
        if (__builtin_expect(__all_sync(FULL, mask == 0ull), 0)) {
          // None of this warp's 32 rows takes part in the unit (the other half of a paired tile listed it, or the
          // unit holds no real key): its weights are exact zeros, no score is read and no exponential is taken.
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&ctl.s_free);
          if (!__all_sync(FULL, ptx::mbar_wait(&ctl.pv_done, (h & 1) ^ 1, &ctl.abort, WAIT_NS))) { site = 15; break; }
          ptx::tc_fence_after();
          uint32_t zero[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) zero[i] = 0u;
          ptx::tmem_st32(tmem_P + lane_base, zero);
          ptx::tmem_wait_st();
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&ctl.p_full);
          continue;
        }
        uint32_t sr[2][32];
        ptx::tmem_ld32(tmem_S + lane_base, sr[0]);
        ptx::tmem_ld32(tmem_S + lane_base + 32, sr[1]);
        ptx::tmem_wait_ld();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&ctl.s_free);      // the scores are in registers: S of the next unit may be issued
        if (__builtin_expect(!all_valid, 0)) {
#pragma unroll
          for (int ch = 0; ch < 2; ++ch) {
            const uint32_t bits = (uint32_t)(mask >> (ch * 32));
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (!((bits >> i) & 1u)) sr[ch][i] = 0xff800000u;          // -inf: outside the mask of Eq. 2
          }
        }
        float mxa = -INFINITY, mxb = -INFINITY;
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          mxa = max3(mxa, __uint_as_float(sr[0][i]), __uint_as_float(sr[0][i + 1]));
          mxb = max3(mxb, __uint_as_float(sr[1][i]), __uint_as_float(sr[1][i + 1]));
        }
        const float m_new = max3(m, mxa, mxb);
        // lazy rescale: move the reference maximum only when it grew by more than 2^8
        const bool grow = (m_new - m) * scale_log2 > 8.f;     // also true the first time a finite score appears
        if (__builtin_expect(__any_sync(FULL, grow), 0)) {      // rare: laid out away from the loop, like the other unlikely branches
          if (j > 0) {
            const uint32_t hp = h - 1;                          // O must hold every product issued so far
            if (!__all_sync(FULL, ptx::mbar_wait(&ctl.pv_done, hp & 1, &ctl.abort, WAIT_NS))) { site = 11; break; }
            ptx::tc_fence_after();
            const float alpha = grow ? ptx::ex2((m - m_new) * scale_log2) : 1.f;
#pragma unroll 1                                  // rare, and the unit loop has to stay short for the instruction cache
            for (int ch = 0; ch < 4; ++ch) {
              uint32_t o[32];
              ptx::tmem_ld32(tmem_O + lane_base + ch * 32, o);
              ptx::tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
              ptx::tmem_st32(tmem_O + lane_base + ch * 32, o);
            }
            {                                                   // the row sums (and the 16 unused columns next to them)
              uint32_t o[32];
              ptx::tmem_ld32(tmem_L + lane_base, o);
              ptx::tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
              ptx::tmem_st32(tmem_L + lane_base, o);
            }
          }
          if (grow) m = m_new;
        }
        const float mb = m == -INFINITY ? 0.f : m * scale_log2;
        const uint64_t nb2 = pack2(-mb, -mb);
        uint32_t pk[32];
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          // a chunk of 32 scores at a time: 16 packed scalings, 32 exponentials, 16 packings (independent work next to every exponential)
          float x[32];
#pragma unroll
          for (int i = 0; i < 16; ++i)
            unpack2(fma2(pack2(__uint_as_float(sr[ch][2 * i]), __uint_as_float(sr[ch][2 * i + 1])), sc2, nb2), x[2 * i], x[2 * i + 1]);
#pragma unroll
          for (int i = 0; i < 32; ++i) x[i] = ptx::ex2(x[i]);
#pragma unroll
          for (int i = 0; i < 16; ++i)
            pk[ch * 16 + i] = ptx::pack_bf16(x[2 * i], x[2 * i + 1]);    // their row sum is taken by the tensor core (L += P 1) from these rounded values
        }
        // P was last read by the products of unit h - 1 (issued about one softmax ago)
        if (!__all_sync(FULL, ptx::mbar_wait(&ctl.pv_done, (h & 1) ^ 1, &ctl.abort, WAIT_NS))) { site = 14; break; }
        ptx::tc_fence_after();
        ptx::tmem_st32(tmem_P + lane_base, pk);                // P (bf16 pairs) in a buffer of its own
        ptx::tmem_wait_st();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&ctl.p_full);
      }
      hc += (uint32_t)H;
      // ---- epilogue: O / l -> bf16 -> swizzled staging tile -> TMA store -------------------------------
      if (!site) {
        if (H > 0) {
          const uint32_t hl = hc - 1;
          if (!__all_sync(FULL, ptx::mbar_wait(&ctl.pv_done, hl & 1, &ctl.abort, WAIT_NS))) site = 12;
        } else {
          if (!__all_sync(FULL, ptx::mbar_wait(&ctl.q_full, it & 1, &ctl.abort, WAIT_NS))) site = 13;
        }
      }
      if (!site) {
        ptx::tc_fence_after();
        float l = 0.f;
        if (H > 0) {
          uint32_t o[32];
          ptx::tmem_ld32(tmem_L + lane_base, o);
          ptx::tmem_wait_ld();
          l = __uint_as_float(o[0]);
        }
        const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          uint32_t o[32];
          if (H > 0) {
            ptx::tmem_ld32(tmem_O + lane_base + ch * 32, o);
            ptx::tmem_wait_ld();
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = 0u;
          }
          uint8_t* dst = sQ + (ch >> 1) * SUB_BYTES + row * 128;
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint4 v;
            v.x = ptx::pack_bf16(__uint_as_float(o[q4 * 8 + 0]) * inv, __uint_as_float(o[q4 * 8 + 1]) * inv);
            v.y = ptx::pack_bf16(__uint_as_float(o[q4 * 8 + 2]) * inv, __uint_as_float(o[q4 * 8 + 3]) * inv);
            v.z = ptx::pack_bf16(__uint_as_float(o[q4 * 8 + 4]) * inv, __uint_as_float(o[q4 * 8 + 5]) * inv);
            v.w = ptx::pack_bf16(__uint_as_float(o[q4 * 8 + 6]) * inv, __uint_as_float(o[q4 * 8 + 7]) * inv);
            const int c16 = (ch & 1) * 4 + q4;
            *reinterpret_cast<uint4*>(dst + ((c16 ^ (row & 7)) << 4)) = v;
          }
        }
        ptx::tc_fence_before();
        ptx::fence_proxy_async_smem();
      } else if (lane == 0) {
        report_timeout(ws, ctl, site, (uint32_t)w);
      }
      if (ptx::named_bar_or(1, 128, ctl.abort)) break;      // uniform over the four warps
      if (tid == 0) {
        const CandMaps& vm = maps.c[sl.c];
        const CandMaps& tm = maps.text[g.pair ? 0 : 1];
        store_o_block(sQ, vm, tm, g, sh, sl.qb0, bh);
        if (sl.qb1 >= 0) store_o_block(sQ + SUB_BYTES / 2, vm, tm, g, sh, sl.qb1, bh);
        ptx::tma_store_commit();
        ptx::tma_store_wait_read();
        ptx::mbar_arrive(&ctl.q_empty);
        ptx::mbar_arrive(&ctl.list_empty[it & 1]);
      }
    }
    if (tid == 0) ptx::tma_store_wait_all();
  }

  // ---- teardown --------------------------------------------------------------------------------
  __syncwarp();
  if (ctl.abort) {                      // let copies still in flight land before the CTA goes away
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 5) ptx::tmem_dealloc(tmem_S, TMEM_COLS);
}

// Exercises the bounded wait on a barrier that nothing ever completes: the wait must give up after
// the limit, raise the CTA's abort flag and leave the context usable.  out[0] = 1 when it gave up,
// out[1] = 1 when the abort flag was raised, out[2..3] = elapsed SM cycles.
__global__ void __launch_bounds__(32) k_selftest_wait(uint32_t* out, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ volatile uint32_t abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bar, 1);
    abort_flag = 0;
    ptx::fence_mbar_init();
    const long long t0 = clock64();
    const bool ok = ptx::mbar_wait(&bar, 0, &abort_flag, limit_ns);
    const long long dt = clock64() - t0;
    out[0] = ok ? 0u : 1u;
    out[1] = abort_flag;
    out[2] = (uint32_t)dt;
    out[3] = (uint32_t)(dt >> 32);
  }
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
  static EncodeFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeFn)p;
  }
  return fn;
}

}  // namespace

size_t attn_maps_bytes() { return sizeof(AttnMaps); }

cudaError_t launch_selftest_wait(uint32_t* out, unsigned long long limit_ns, cudaStream_t s) {
  k_selftest_wait<<<1, 32, 0, s>>>(out, limit_ns);
  return cudaGetLastError();
}

int attn_encode_maps(AttnMaps* out, const void* Q, const void* K, const void* V, void* O, const Shape& sh,
                     const GeoPack& gp, char* err, size_t errlen) {
  EncodeFn enc = encode_fn();
  if (!enc) { snprintf(err, errlen, "cuTensorMapEncodeTiled is not available from this driver"); return 1; }
  const void* ptrs[4] = {Q, K, V, O};
  const cuuint32_t es[5] = {1, 1, 1, 1, 1};
  for (int c = 0; c < sh.C; ++c) {
    const CandGeo& g = gp.g[c];
    CUtensorMap* dst[4] = {&out->c[c].q, &out->c[c].k, &out->c[c].v, &out->c[c].o};
    const cuuint64_t dims[5] = {SPADE_D, (cuuint64_t)sh.W, (cuuint64_t)sh.H, (cuuint64_t)sh.T, (cuuint64_t)sh.BH};
    const cuuint64_t str[4] = {256, 256ull * sh.W, 256ull * sh.W * sh.H, 256ull * sh.N};
    const cuuint32_t box_blk[5] = {64, (cuuint32_t)g.bw, (cuuint32_t)g.bh, (cuuint32_t)g.bt, 1};
    const cuuint32_t box_kv[5] = {64, (cuuint32_t)g.kw, (cuuint32_t)g.kh, (cuuint32_t)g.kt, 1};
    for (int t = 0; t < 4; ++t) {
      const cuuint32_t* box = (t == 1 || t == 2) ? box_kv : box_blk;
      CUresult r = enc(dst[t], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(ptrs[t]), dims, str, box, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) { snprintf(err, errlen, "cuTensorMapEncodeTiled (candidate %d, tensor %d) failed with %d", c, t, (int)r); return 1; }
    }
  }
  for (int v = 0; v < 2; ++v) {
    CUtensorMap* dst[4] = {&out->text[v].q, &out->text[v].k, &out->text[v].v, &out->text[v].o};
    const cuuint64_t dims[3] = {SPADE_D, (cuuint64_t)sh.N, (cuuint64_t)sh.BH};
    const cuuint64_t str[2] = {256, 256ull * sh.N};
    const cuuint32_t box_blk[3] = {64, v == 0 ? 64u : 128u, 1};
    const cuuint32_t box_kv[3] = {64, 64u, 1};
    for (int t = 0; t < 4; ++t) {
      const cuuint32_t* box = (t == 1 || t == 2) ? box_kv : box_blk;
      CUresult r = enc(dst[t], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptrs[t]), dims, str, box, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) { snprintf(err, errlen, "cuTensorMapEncodeTiled (text, tensor %d) failed with %d", t, (int)r); return 1; }
    }
  }
  return 0;
}

cudaError_t launch_attn(const AttnMaps* maps, const Shape& sh, const GeoPack& gp, const StaticTables& st,
                        const WsTables& ws, int num_sms, cudaStream_t s) {
  cudaError_t e = cudaFuncSetAttribute(k_attn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ATT_SMEM);
  if (e != cudaSuccess) return e;
  int max_tiles = 0;
  for (int c = 0; c < sh.C; ++c) max_tiles = gp.g[c].tiles > max_tiles ? gp.g[c].tiles : max_tiles;
  long items = (long)sh.BH * max_tiles;             // upper bound; the kernel reads the exact count
  long grid = 2L * num_sms;
  if (grid > items) grid = items;
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)SPADE_D);
  k_attn<<<(unsigned)grid, ATT_THREADS, ATT_SMEM, s>>>(*maps, sh, gp, st, ws, scale_log2);
  return cudaGetLastError();
}
