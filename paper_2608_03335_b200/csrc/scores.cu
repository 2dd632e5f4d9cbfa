// Inter-block estimator on the tensor cores (Sec. 3.1, Fig. 4c; Sec. 3.3): S = Q' K'^T / sqrt(d) for
// the video blocks of every head, written to a scratch table that the index search reads.
//
// The summaries are fp32 and the selection must agree with an fp64 evaluation to 1e-4 in the logits,
// so a plain TF32 product (10-bit mantissa) is not enough.  Each operand is split x = hi + lo with
// hi = x rounded to the nearest TF32 value and lo = x - hi (exact in fp32); the product uses the three terms
// hi*hi + hi*lo + lo*hi (the dropped lo*lo term is at most 2^-22 relative, of either sign), all accumulated in one fp32
// TMEM tile by tcgen05.mma kind::tf32.
//
// One CTA per SM walks work items (head, 128-row tile of query blocks, a range of 128-column tiles of KV blocks).
// Everything reaches shared memory through one ring of 32 KB entries filled by a loader warp that runs ahead
// across items: two entries carry the item's A rows (fp32, 64 channels each), then four per column tile carry a
// 32-channel slice of B, hi and lo planes as k_split_k wrote them.  Warps 0-3 split A into TMEM (256 columns),
// one thread issues the products (measured: a 128 x 128 x 8 TF32 product takes 64 clk, a 128 x 64 x 8 one 56),
// D is double-buffered in the other 256 columns, and warps 0-3 move finished tiles out through per-warp
// swizzled staging buffers and TMA stores (a thread owns a row, so direct stores would touch 32 rows per
// instruction).  The epilogue of an item's last tile is postponed until the next item's A is in TMEM.
#include <cuda.h>
#include <stdio.h>

#include "sm100_ptx.cuh"
#include "spade_common.cuh"

struct ScoreMaps {
  CUtensorMap k;      // 4-D (128 floats, NBmax rows, hi | lo, head) over the split K' means, box (32 floats, 128 rows, 1, 1)
  CUtensorMap kd;     // same with four planes: hi | lo of k_mid, hi | lo of k_half (the max/min estimator of Fig. 4a)
  CUtensorMap q;      // 3-D (128 floats, NBmax rows, head) over the Q' means, box (32 floats, 128 rows, 1)
  CUtensorMap qd;     // same over q~ of the max/min estimator
  CUtensorMap s;      // 3-D (ld, NBvmax rows, head) over the score table, box (32 floats, 32 rows, 1): stores
};

namespace {

constexpr int SC_THREADS = 192;                  // warps 0-3: A split + epilogue, warp 4: MMA issue, warp 5: TMA loads
constexpr int SC_N = 128;                        // KV blocks per column tile
constexpr int SC_BOX = 128 * 128;                // bytes of one TMA box: 128 rows x 32 floats
constexpr int SC_ENTRY = 2 * SC_BOX;             // ring entry: two boxes (A: two channel groups; B: hi and lo of one group)
constexpr int SC_NST = 6;                        // ring entries
constexpr int SC_OBUF = 32 * 128;                // staging buffer of one warp: 32 rows x 32 floats
constexpr uint64_t SC_WAIT_NS = 2000000000ull;
constexpr size_t SC_SMEM = SC_NST * SC_ENTRY + 8 * SC_OBUF + 1024 + 256;

__host__ __device__ constexpr uint32_t idesc_tf32(int M, int N) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_ts_tf32(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc)
      : "memory");
}

struct ScCtl {
  uint64_t full[SC_NST];   // TMA landed a ring entry                         (copy engine -> consumer)
  uint64_t empty[SC_NST];  // the entry has been consumed, one arrival        (issuer -> loader)
  uint64_t mma_done[2];    // products of the tile are complete               (issuer -> compute warps)
  uint64_t d_free[2];      // the D tile has been read                        (compute warps -> issuer), 4 arrivals
  uint64_t a_ready;        // A is split into TMEM                            (compute warps -> issuer), 4 arrivals
  uint32_t tmem_base;
  volatile uint32_t abort;
  int seg_bh, seg_rem, seg_count;   // this CTA's range: first head, tile offset inside it, tiles
};

// The tiles of all heads form one sequence (head, row tile, column tile); CTA b takes the b-th of gridDim.x equal
// ranges of it and walks its range in segments that stay inside one row tile (one A).
struct ScSeg { int bh, rt, ct0, n_ct, nbv; };
struct ScWalk { int bh, rt, ct, n, nbv, left; };

__device__ __forceinline__ int sc_side(const GeoPack& gp, const int* scheme, int bh) { return (gp.g[scheme[bh]].NBv + SC_N - 1) / SC_N; }

__device__ __forceinline__ ScWalk sc_walk_init(int bh, int rem, int count, const GeoPack& gp, const int* scheme, int BH) {
  ScWalk w;
  w.bh = bh; w.left = count; w.nbv = 0; w.n = 0; w.rt = 0; w.ct = 0;
  if (count > 0 && bh < BH) {
    w.nbv = gp.g[scheme[bh]].NBv;
    w.n = (w.nbv + SC_N - 1) / SC_N;
    w.rt = rem / w.n; w.ct = rem % w.n;       // count > 0 puts the range's first tile inside this head: n > 0
  }
  return w;
}
__device__ __forceinline__ bool sc_next(ScWalk& w, ScSeg& s, const GeoPack& gp, const int* scheme, int BH) {
  if (w.left <= 0) return false;
  while (w.rt >= w.n) {                        // on to the next head that has video blocks
    if (++w.bh >= BH) return false;
    w.nbv = gp.g[scheme[w.bh]].NBv;
    w.n = (w.nbv + SC_N - 1) / SC_N; w.rt = 0; w.ct = 0;
  }
  s.bh = w.bh; s.rt = w.rt; s.ct0 = w.ct; s.nbv = w.nbv;
  s.n_ct = min(w.left, w.n - w.ct);
  w.left -= s.n_ct; w.ct += s.n_ct;
  if (w.ct == w.n) { w.ct = 0; ++w.rt; }
  return true;
}

__global__ void __launch_bounds__(SC_THREADS, 1)
k_scores(const __grid_constant__ ScoreMaps maps, const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp,
         const WsTables ws, const float scale, const int a_abs, const int term) {
  // term 0: S = A K'^T with the mean summaries.  terms 1, 2: the two halves of the max/min estimator,
  // S = q~ k_mid^T (written) and S += |q~| k_half^T (added to what term 1 left).
  const CUtensorMap* const kmap = term == 0 ? &maps.k : &maps.kd;
  const CUtensorMap* const qmap = term == 0 ? &maps.q : &maps.qd;
  const int plane0 = term == 2 ? 2 : 0;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* obuf = smem + SC_NST * SC_ENTRY;
  ScCtl& ctl = *reinterpret_cast<ScCtl*>(obuf + 8 * SC_OBUF);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int b = 0; b < SC_NST; ++b) {
      ptx::mbar_init(&ctl.full[b], 1);
      ptx::mbar_init(&ctl.empty[b], 1);
    }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(&ctl.mma_done[b], 1);
      ptx::mbar_init(&ctl.d_free[b], 4);
    }
    ptx::mbar_init(&ctl.a_ready, 4);
    ctl.abort = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 4) { ptx::tmem_alloc(&ctl.tmem_base, 512); ptx::tmem_relinquish(); }
  if (warp == 0) {
    // tiles of all heads, then the head in which this CTA's range starts (warp scan over the heads, 32 at a time)
    int total = 0;
    for (int base = 0; base < sh.BH; base += 32) {
      const int h = base + lane, n = h < sh.BH ? sc_side(gp, ws.scheme, h) : 0;
      total += n * n;
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    const int lo = (int)((long long)blockIdx.x * total / gridDim.x), hi = (int)((long long)(blockIdx.x + 1) * total / gridDim.x);
    int acc = 0, s_bh = sh.BH, s_rem = 0;
    for (int base = 0; base < sh.BH && hi > lo; base += 32) {
      const int h = base + lane, n = h < sh.BH ? sc_side(gp, ws.scheme, h) : 0;
      int incl = n * n;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
      }
      const uint32_t hit = __ballot_sync(0xffffffffu, acc + incl > lo);
      if (hit) {
        const int first = __ffs(hit) - 1;
        const int incl_f = __shfl_sync(0xffffffffu, incl, first), nn_f = __shfl_sync(0xffffffffu, n * n, first);
        s_bh = base + first; s_rem = lo - (acc + incl_f - nn_f);
        break;
      }
      acc += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) { ctl.seg_bh = s_bh; ctl.seg_rem = s_rem; ctl.seg_count = hi - lo; }
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tm = ctl.tmem_base;                 // A hi: cols 0..127, A lo: 128..255, D: 256..383 and 384..511
  ScWalk walk = sc_walk_init(ctl.seg_bh, ctl.seg_rem, ctl.seg_count, gp, ws.scheme, sh.BH);
  ScSeg it;
  uint32_t ent = 0;                                   // ring entries so far (the same sequence in every role)
  uint32_t tiles = 0;                                 // column tiles so far
  uint32_t items_done = 0;                            // segments so far
  uint32_t site = 0;
  int site_item = 0;

  if (warp == 5) {
    // ================= loader: A rows and B slices by TMA, as far ahead as the ring allows ================
    if (lane == 0) {
      while (!site && sc_next(walk, it, gp, ws.scheme, sh.BH)) {
        site_item = it.bh * 4096 + it.rt;
        for (int e = 0; e < 2 + 4 * it.n_ct; ++e, ++ent) {
          const uint32_t st = ent % SC_NST;
          if (!ptx::mbar_wait(&ctl.empty[st], ((ent / SC_NST) & 1) ^ 1, &ctl.abort, SC_WAIT_NS)) { site = 101; break; }
          uint8_t* dst = smem + st * SC_ENTRY;
          ptx::mbar_expect_tx(&ctl.full[st], SC_ENTRY);
          if (e < 2) {
            ptx::tma_load_3d(dst, qmap, &ctl.full[st], 64 * e, it.rt * 128, it.bh);
            ptx::tma_load_3d(dst + SC_BOX, qmap, &ctl.full[st], 64 * e + 32, it.rt * 128, it.bh);
          } else {
            const int ct = (e - 2) >> 2, ksl = (e - 2) & 3;
            ptx::tma_load_4d(dst, kmap, &ctl.full[st], 32 * ksl, (it.ct0 + ct) * SC_N, plane0, it.bh);
            ptx::tma_load_4d(dst + SC_BOX, kmap, &ctl.full[st], 32 * ksl, (it.ct0 + ct) * SC_N, plane0 + 1, it.bh);
          }
        }
      }
      if (site || ctl.abort) {
        // giving up: let the copies already issued land before the CTA leaves (short, bounded waits)
        volatile uint32_t dummy = 0;
        for (uint32_t e = ent > SC_NST ? ent - SC_NST : 0; e < ent; ++e)
          ptx::mbar_wait(&ctl.full[e % SC_NST], (e / SC_NST) & 1, &dummy, 1000000ull);
      }
    }
  } else if (warp == 4) {
    // ================= issuer: products and commits ======================================================
    if (lane == 0) {
      const uint32_t idesc = idesc_tf32(128, SC_N);
      const uint32_t sB = ptx::smem_u32(smem);
      while (!site && sc_next(walk, it, gp, ws.scheme, sh.BH)) {
        site_item = it.bh * 4096 + it.rt;
        // the A entries are read by the compute warps; once A is in TMEM they go back to the loader
        if (!ptx::mbar_wait(&ctl.a_ready, items_done & 1, &ctl.abort, SC_WAIT_NS)) { site = 102; break; }
        ptx::mbar_arrive(&ctl.empty[ent % SC_NST]);
        ptx::mbar_arrive(&ctl.empty[(ent + 1) % SC_NST]);
        ent += 2;
        ptx::tc_fence_after();
        for (int ct = 0; ct < it.n_ct && !site; ++ct, ++tiles) {
          const uint32_t db = tiles & 1;
          if (!ptx::mbar_wait(&ctl.d_free[db], ((tiles >> 1) & 1) ^ 1, &ctl.abort, SC_WAIT_NS)) { site = 103; break; }
          const uint32_t d = tm + 256 + db * SC_N;
          for (int ksl = 0; ksl < 4; ++ksl, ++ent) {
            const uint32_t st = ent % SC_NST;
            if (!ptx::mbar_wait(&ctl.full[st], (ent / SC_NST) & 1, &ctl.abort, SC_WAIT_NS)) { site = 104; break; }
            ptx::tc_fence_after();
            const uint32_t bhi = sB + st * SC_ENTRY, blo = bhi + SC_BOX;
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4) {            // 8 channels per product
              const uint32_t ac = (uint32_t)(ksl * 4 + k4) * 8;
              const uint64_t dh = ptx::smem_desc_sw128(bhi + k4 * 32, 16, 1024), dl = ptx::smem_desc_sw128(blo + k4 * 32, 16, 1024);
              umma_ts_tf32(d, tm + ac, dh, idesc, (ksl | k4) != 0);
              umma_ts_tf32(d, tm + ac, dl, idesc, 1);
              umma_ts_tf32(d, tm + 128 + ac, dh, idesc, 1);
            }
            ptx::umma_commit(&ctl.empty[st]);           // the slice returns to the loader when its products are complete
          }
          if (!site) ptx::umma_commit(&ctl.mma_done[db]);
        }
        items_done += 1;
      }
    }
  } else {
    // ================= compute warps: A into TMEM, epilogue ===============================================
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    const int trow = warp * 32 + lane;                // row of the tile = TMEM lane
    uint8_t* const my_obuf = obuf + warp * 2 * SC_OBUF;
    uint32_t ochunks = 0;                             // staging chunks written so far by this warp
    int pend_bh = -1, pend_rt = 0, pend_ct = 0, pend_nbv = 0;      // epilogue of the previous item's last tile
    uint32_t pend_tile = 0;

    auto epilogue = [&](int bh, int rt, int ctile, int nbv, uint32_t tt) -> bool {
      const uint32_t sp = tt & 1;
      if (!__all_sync(0xffffffffu, ptx::mbar_wait(&ctl.mma_done[sp], (tt >> 1) & 1, &ctl.abort, SC_WAIT_NS))) return false;
      ptx::tc_fence_after();
      const bool rows_live = rt * 128 + warp * 32 < nbv;      // none of this warp's 32 rows is a video block otherwise
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t r[32];
        ptx::tmem_ld32(tm + lane_base + 256 + sp * SC_N + ch * 32, r);
        ptx::tmem_wait_ld();
        if (ch == 3) {                                  // D is in registers: the issuer may overwrite it
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&ctl.d_free[sp]);
        }
        if (!rows_live || ctile * SC_N + ch * 32 >= sh.ld_scores) continue;
        uint8_t* buf = my_obuf + (ochunks & 1) * SC_OBUF;
        if (lane == 0) ptx::tma_store_wait_read1();     // the store that last read this buffer is two chunks back
        __syncwarp();
#pragma unroll
        for (int q = 0; q < 8; ++q)
          *reinterpret_cast<float4*>(buf + lane * 128 + ((q ^ (lane & 7)) << 4)) =
              make_float4(__uint_as_float(r[4 * q]) * scale, __uint_as_float(r[4 * q + 1]) * scale,
                          __uint_as_float(r[4 * q + 2]) * scale, __uint_as_float(r[4 * q + 3]) * scale);
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          if (term == 2) ptx::tma_reduce_add_3d(&maps.s, buf, ctile * SC_N + ch * 32, rt * 128 + warp * 32, bh);
          else ptx::tma_store_3d(&maps.s, buf, ctile * SC_N + ch * 32, rt * 128 + warp * 32, bh);
          ptx::tma_store_commit();
        }
        ++ochunks;
      }
      return true;
    };

    while (!site && sc_next(walk, it, gp, ws.scheme, sh.BH)) {
      site_item = it.bh * 4096 + it.rt;
      // ---- A: this thread's row, 128 channels, from the two ring entries into TMEM as hi and lo --------------
      const uint32_t st0 = ent % SC_NST, st1 = (ent + 1) % SC_NST;
      if (!ptx::mbar_wait_warp(&ctl.full[st0], (ent / SC_NST) & 1, &ctl.abort, SC_WAIT_NS) ||
          !ptx::mbar_wait_warp(&ctl.full[st1], ((ent + 1) / SC_NST) & 1, &ctl.abort, SC_WAIT_NS)) { site = 105; break; }
      // every product that reads the previous A is complete once the previous item's last tile is
      if (pend_bh >= 0 && !__all_sync(0xffffffffu, ptx::mbar_wait(&ctl.mma_done[pend_tile & 1], (pend_tile >> 1) & 1, &ctl.abort, SC_WAIT_NS))) { site = 106; break; }
      ptx::tc_fence_after();
#pragma unroll 1
      for (int g = 0; g < 4; ++g) {                     // 32 channels per step
        const uint8_t* box = smem + ((g >> 1) ? st1 : st0) * SC_ENTRY + (g & 1) * SC_BOX + trow * 128;
        uint32_t hi[32], lo[32];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          float4 w = *reinterpret_cast<const float4*>(box + ((q ^ (trow & 7)) << 4));
          if (a_abs) { w.x = fabsf(w.x); w.y = fabsf(w.y); w.z = fabsf(w.z); w.w = fabsf(w.w); }
          const float x[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const uint32_t h = (__float_as_uint(x[e]) + 0x1000u) & 0xffffe000u;      // nearest TF32 value
            hi[q * 4 + e] = h;
            lo[q * 4 + e] = __float_as_uint(x[e] - __uint_as_float(h));
          }
        }
        ptx::tmem_st32(tm + lane_base + g * 32, hi);
        ptx::tmem_st32(tm + lane_base + 128 + g * 32, lo);
      }
      ptx::tmem_wait_st();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&ctl.a_ready);
      ent += 2 + 4 * (uint32_t)it.n_ct;
      // ---- epilogues: the previous item's last tile first, then all but the last of this item ---------------
      if (pend_bh >= 0 && !epilogue(pend_bh, pend_rt, pend_ct, pend_nbv, pend_tile)) { site = 107; break; }
      pend_bh = -1;
      for (int ct = 0; ct + 1 < it.n_ct; ++ct)
        if (!epilogue(it.bh, it.rt, it.ct0 + ct, it.nbv, tiles + ct)) { site = 108; break; }
      if (site) break;
      pend_bh = it.bh; pend_rt = it.rt; pend_ct = it.ct0 + it.n_ct - 1; pend_nbv = it.nbv; pend_tile = tiles + it.n_ct - 1;
      tiles += (uint32_t)it.n_ct;
    }
    if (!site && pend_bh >= 0 && !epilogue(pend_bh, pend_rt, pend_ct, pend_nbv, pend_tile)) site = 109;
    if (lane == 0) ptx::tma_store_wait_all();           // the staging buffers and the table are final before the CTA leaves
  }
  // a role that gave up reports it (the bounded waits of the others see ctl.abort and leave as well)
  if (site && lane == 0 && atomicCAS(ws.status, 0u, (uint32_t)SPADE_ST_TIMEOUT) == 0u) { ws.status[1] = site; ws.status[2] = (uint32_t)site_item; }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 4) ptx::tmem_dealloc(tm, 512);
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

size_t score_maps_bytes() { return sizeof(ScoreMaps); }

int scores_encode_maps(ScoreMaps* out, const Shape& sh, const WsTables& ws, char* err, size_t errlen) {
  EncodeFn enc = encode_fn();
  if (!enc) { snprintf(err, errlen, "cuTensorMapEncodeTiled is not available from this driver"); return 1; }
  const cuuint32_t es[4] = {1, 1, 1, 1};
  auto tiled = [&](CUtensorMap* m, void* base, int rank, const cuuint64_t* dims, const cuuint64_t* str, const cuuint32_t* box,
                   const char* what) {
    const CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, (cuuint32_t)rank, base, dims, str, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { snprintf(err, errlen, "cuTensorMapEncodeTiled (%s) failed with %d", what, (int)r); return 1; }
    return 0;
  };
  const cuuint32_t kbox[4] = {32, SC_N, 1, 1};
  const cuuint64_t kdims[4] = {SPADE_D, (cuuint64_t)sh.NBmax, 2, (cuuint64_t)sh.BH};
  const cuuint64_t kstr[3] = {512, 512ull * sh.NBmax, 1024ull * sh.NBmax};
  const cuuint32_t qbox[3] = {32, 128, 1};
  const cuuint64_t qdims[3] = {SPADE_D, (cuuint64_t)sh.NBmax, (cuuint64_t)sh.BH};
  const cuuint64_t qstr[2] = {512, 512ull * sh.NBmax};
  const cuuint32_t sbox[3] = {32, 32, 1};
  const cuuint64_t sdims[3] = {(cuuint64_t)sh.ld_scores, (cuuint64_t)sh.NBvmax, (cuuint64_t)sh.BH};
  const cuuint64_t sstr[2] = {4ull * sh.ld_scores, 4ull * sh.ld_scores * sh.NBvmax};
  if (tiled(&out->s, ws.scores, 3, sdims, sstr, sbox, "score table")) return 1;
  if (sh.estimator == 0) {
    if (tiled(&out->k, ws.ksplit, 4, kdims, kstr, kbox, "K' summaries")) return 1;
    if (tiled(&out->q, ws.qsum, 3, qdims, qstr, qbox, "Q' summaries")) return 1;
  }
  if (sh.estimator == 1) {
    const cuuint64_t dims4[4] = {SPADE_D, (cuuint64_t)sh.NBmax, 4, (cuuint64_t)sh.BH};
    const cuuint64_t str4[3] = {512, 512ull * sh.NBmax, 2048ull * sh.NBmax};
    if (tiled(&out->kd, ws.kdsa, 4, dims4, str4, kbox, "max/min summaries of K")) return 1;
    if (tiled(&out->qd, ws.qmid, 3, qdims, qstr, qbox, "max/min summaries of Q")) return 1;
  }
  return 0;
}

cudaError_t launch_scores(const ScoreMaps* maps, const Shape& sh, const GeoPack& gp, const WsTables& ws, int num_sms,
                          int term, cudaStream_t s) {
  cudaError_t e = cudaFuncSetAttribute(k_scores, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SC_SMEM);
  if (e != cudaSuccess) return e;
  const int side = (sh.NBvmax + SC_N - 1) / SC_N;
  const long long most = (long long)sh.BH * side * side;       // tiles if every head took the finest candidate
  const int grid = most < num_sms ? (int)(most > 0 ? most : 1) : num_sms;
  k_scores<<<grid, SC_THREADS, SC_SMEM, s>>>(*maps, sh, gp, ws, 1.0f / sqrtf((float)SPADE_D), term == 2 ? 1 : 0, term);
  return cudaGetLastError();
}
