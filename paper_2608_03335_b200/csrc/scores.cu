// Inter-block estimator on the tensor cores (Sec. 3.1, Fig. 4c; Sec. 3.3): S = Q' K'^T / sqrt(d) for
// the video blocks of every head, written to a scratch table that the index search reads.
//
// The summaries are fp32 and the selection must agree with an fp64 evaluation to 1e-4 in the logits,
// so a plain TF32 product (10-bit mantissa) is not enough.  Each operand is split x = hi + lo with
// hi = x rounded to the nearest TF32 value and lo = x - hi (exact in fp32); the product uses the three terms
// hi*hi + hi*lo + lo*hi (the dropped lo*lo term is at most 2^-22 relative, of either sign), all accumulated in one fp32
// TMEM tile by tcgen05.mma kind::tf32.  A (128 query blocks x 128 channels, hi and lo) lives in TMEM,
// B (64 KV blocks x 128 channels, hi and lo planes written by k_split_k) arrives by TMA through a ring of
// stages.  Warp 4 issues the TMA loads and the products; warps 0-3 stage A and write the scores, so the
// epilogue of tile j-1 runs while the tensor pipe works on tile j.
#include <cuda.h>
#include <stdio.h>

#include "sm100_ptx.cuh"
#include "spade_common.cuh"

struct ScoreMaps {
  CUtensorMap k;      // 4-D (128 floats, NBmax rows, hi | lo, head) over the split K' means, box (32 floats, 64 rows, 1, 1)
  CUtensorMap kd;     // same with four planes: hi | lo of k_mid, hi | lo of k_half (the max/min estimator of Fig. 4a)
};

namespace {

constexpr int SC_THREADS = 160;                  // warps 0-3: operand split + epilogue, warp 4: TMA + MMA issue
constexpr int SC_N = 64;                         // KV blocks per column tile
constexpr int SC_SUB = SC_N * 128;               // bytes of one 32-channel sub-tile (64 rows x 128 B)
constexpr int SC_STAGE = 8 * SC_SUB;             // hi (4 sub-tiles) + lo (4 sub-tiles) = 64 KB
constexpr uint64_t SC_WAIT_NS = 2000000000ull;
constexpr int SC_PARTS = 3;                      // work items per row tile (balance over the SMs)
constexpr int SC_NST = 3;                        // shared-memory stages of B (D stays double-buffered in TMEM)
constexpr size_t SC_SMEM = SC_NST * SC_STAGE + 1024 + 256;

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
  uint64_t b_full[SC_NST]; // TMA landed a K' tile, hi and lo planes (copy engine -> issuer)
  uint64_t mma_done[2];    // products of the tile are complete   (issuer -> compute warps and itself)
  uint64_t d_free[2];      // the D tile has been read            (compute warps -> issuer), 4 arrivals
  uint64_t a_ready;        // A is staged in TMEM                 (compute warps -> issuer), 4 arrivals
  uint32_t tmem_base;
  volatile uint32_t abort;
};

__global__ void __launch_bounds__(SC_THREADS, 1)
k_scores(const __grid_constant__ ScoreMaps maps, const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp,
         const WsTables ws, const float scale, const float* __restrict__ a_rows, const int a_abs, const int term) {
  // term 0: S = A K'^T with the mean summaries.  terms 1, 2: the two halves of the max/min estimator,
  // S = q~ k_mid^T (written) and S += |q~| k_half^T (added to what term 1 left).
  const CUtensorMap* const kmap = term == 0 ? &maps.k : &maps.kd;
  const int plane0 = term == 2 ? 2 : 0;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  ScCtl& ctl = *reinterpret_cast<ScCtl*>(smem + SC_NST * SC_STAGE);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    for (int b = 0; b < SC_NST; ++b) {
      ptx::mbar_init(&ctl.b_full[b], 1);
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
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tm = ctl.tmem_base;                 // A hi: cols 0..127, A lo: 128..255, D: 256..319 and 320..383
  const int row_tiles = (sh.NBvmax + 127) / 128;
  const int items = sh.BH * row_tiles * SC_PARTS;     // a row tile's column tiles are split over SC_PARTS work items
  uint32_t tiles_done = 0;                            // column tiles so far (same in every role)
  uint32_t items_done = 0;
  uint32_t site = 0;

  for (int item = blockIdx.x; item < items && !site; item += gridDim.x) {
    const int part = item % SC_PARTS, rt = (item / SC_PARTS) % row_tiles, bh = item / (SC_PARTS * row_tiles);
    const int nbv = gp.g[ws.scheme[bh]].NBv;
    if (rt * 128 >= nbv) continue;
    const int n_ct_all = (nbv + SC_N - 1) / SC_N, per_part = (n_ct_all + SC_PARTS - 1) / SC_PARTS;
    const int ct0 = part * per_part;
    const int n_ct = min(per_part, n_ct_all - ct0);
    if (n_ct <= 0) continue;
    if (warp == 4) {
      // ================= issuer: K' tiles by TMA, products, commits ===================================
      if (lane == 0) {
        const uint32_t idesc = idesc_tf32(128, SC_N);
        const uint32_t sB = ptx::smem_u32(smem);
        auto load_tile = [&](int ct) {                 // the stage of tile ct must be free
          const uint32_t st = (tiles_done + ct) % SC_NST;
          ptx::mbar_expect_tx(&ctl.b_full[st], 8 * SC_SUB);
          for (int s = 0; s < 8; ++s)       // four 32-channel sub-tiles of the hi plane, then of the lo plane
            ptx::tma_load_4d(smem + st * SC_STAGE + s * SC_SUB, kmap, &ctl.b_full[st], 32 * (s & 3), (ct0 + ct) * SC_N, plane0 + (s >> 2), bh);
        };
        // every stage is free here: all products of the previous item were waited for below
        for (int ct = 0; ct < SC_NST && ct < n_ct; ++ct) load_tile(ct);
        if (!ptx::mbar_wait(&ctl.a_ready, items_done & 1, &ctl.abort, SC_WAIT_NS)) site = 101;
        for (int ct = 0; ct < n_ct && !site; ++ct) {
          const uint32_t t = tiles_done + ct, st = t % SC_NST, db = t & 1;
          if (!ptx::mbar_wait(&ctl.b_full[st], (t / SC_NST) & 1, &ctl.abort, SC_WAIT_NS) ||
              !ptx::mbar_wait(&ctl.d_free[db], ((t >> 1) & 1) ^ 1, &ctl.abort, SC_WAIT_NS)) { site = 102; break; }
          ptx::tc_fence_after();
          const uint32_t d = tm + 256 + db * SC_N;
          const uint32_t bhi = sB + st * SC_STAGE, blo = bhi + 4 * SC_SUB;
#pragma unroll
          for (int ks = 0; ks < 16; ++ks) {             // 8 channels per step; sub-tile of 32 channels = 4 steps
            const uint32_t off = (ks >> 2) * SC_SUB + (ks & 3) * 32;
            const uint64_t dh = ptx::smem_desc_sw128(bhi + off, 16, 1024), dl = ptx::smem_desc_sw128(blo + off, 16, 1024);
            umma_ts_tf32(d, tm + ks * 8, dh, idesc, ks > 0);
            umma_ts_tf32(d, tm + ks * 8, dl, idesc, 1);
            umma_ts_tf32(d, tm + 128 + ks * 8, dh, idesc, 1);
          }
          ptx::umma_commit(&ctl.mma_done[db]);
          // the stage of tile ct-1 is free once its products are complete: it takes tile ct-1+SC_NST
          if (ct >= 1 && ct - 1 + SC_NST < n_ct) {
            const uint32_t tp = t - 1;
            if (!ptx::mbar_wait(&ctl.mma_done[tp & 1], (tp >> 1) & 1, &ctl.abort, SC_WAIT_NS)) { site = 103; break; }
            load_tile(ct - 1 + SC_NST);
          }
        }
        // all products of this item complete before A (and the stages) are reused
        for (int back = 0; back < 2 && back < n_ct && !site; ++back) {
          const uint32_t tp = tiles_done + n_ct - 1 - back;
          if (!ptx::mbar_wait(&ctl.mma_done[tp & 1], (tp >> 1) & 1, &ctl.abort, SC_WAIT_NS)) site = 104;
        }
      }
      site = __shfl_sync(0xffffffffu, site, 0);
    } else {
      // ================= compute warps: A into TMEM, split of B, epilogue ===============================
      const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
      const int row = rt * 128 + warp * 32 + lane;
      {
        const float4* src = reinterpret_cast<const float4*>(a_rows + ((size_t)bh * sh.NBmax + (row < sh.NBmax ? row : 0)) * SPADE_D);
#pragma unroll 1
        for (int ch = 0; ch < 4; ++ch) {
          uint32_t hi[32], lo[32];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            float4 v = row < sh.NBmax ? __ldg(src + ch * 8 + q) : make_float4(0.f, 0.f, 0.f, 0.f);
            if (a_abs) { v.x = fabsf(v.x); v.y = fabsf(v.y); v.z = fabsf(v.z); v.w = fabsf(v.w); }
            const float x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const uint32_t h = (__float_as_uint(x[e]) + 0x1000u) & 0xffffe000u;      // nearest TF32 value
              hi[q * 4 + e] = h;
              lo[q * 4 + e] = __float_as_uint(x[e] - __uint_as_float(h));
            }
          }
          ptx::tmem_st32(tm + lane_base + ch * 32, hi);
          ptx::tmem_st32(tm + lane_base + 128 + ch * 32, lo);
        }
        ptx::tmem_wait_st();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&ctl.a_ready);
      }
      for (int ct = 0; ct <= n_ct && !site; ++ct) {
        const uint32_t t = tiles_done + ct;
        if (ct >= 1) {
          // epilogue of tile ct-1 (the issuer is already on tile ct)
          const uint32_t tp = t - 1, sp = tp & 1;
          if (!__all_sync(0xffffffffu, ptx::mbar_wait(&ctl.mma_done[sp], (tp >> 1) & 1, &ctl.abort, SC_WAIT_NS))) { site = 106; break; }
          ptx::tc_fence_after();
          float* dst = ws.scores + ((size_t)bh * sh.NBvmax + row) * sh.ld_scores + (ct0 + ct - 1) * SC_N;
#pragma unroll
          for (int ch = 0; ch < 2; ++ch) {
            uint32_t r[32];
            ptx::tmem_ld32(tm + lane_base + 256 + sp * SC_N + ch * 32, r);
            ptx::tmem_wait_ld();
            if (row < nbv) {
#pragma unroll
              for (int q = 0; q < 8; ++q) {
                float4 o = make_float4(__uint_as_float(r[4 * q]) * scale, __uint_as_float(r[4 * q + 1]) * scale,
                                       __uint_as_float(r[4 * q + 2]) * scale, __uint_as_float(r[4 * q + 3]) * scale);
                if (term == 2) {
                  const float4 old = reinterpret_cast<const float4*>(dst + ch * 32)[q];
                  o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                }
                reinterpret_cast<float4*>(dst + ch * 32)[q] = o;
              }
            }
          }
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&ctl.d_free[sp]);
        }
      }
    }
    tiles_done += (uint32_t)n_ct;
    items_done += 1;
    // a role that gave up reports it; everybody leaves at the same item boundary
    if (site && lane == 0 && atomicCAS(ws.status, 0u, (uint32_t)SPADE_ST_TIMEOUT) == 0u) { ws.status[1] = site; ws.status[2] = (uint32_t)item; }
    if (__syncthreads_or(site != 0 || ctl.abort != 0)) { site = site ? site : 199; break; }
  }
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
  const cuuint64_t dims[4] = {SPADE_D, (cuuint64_t)sh.NBmax, 2, (cuuint64_t)sh.BH};
  const cuuint64_t str[3] = {512, 512ull * sh.NBmax, 1024ull * sh.NBmax};
  const cuuint32_t box[4] = {32, SC_N, 1, 1};
  const cuuint32_t es[4] = {1, 1, 1, 1};
  CUresult r = enc(&out->k, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, ws.ksplit, dims, str, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { snprintf(err, errlen, "cuTensorMapEncodeTiled (K' summaries) failed with %d", (int)r); return 1; }
  if (sh.estimator == 1) {
    const cuuint64_t dims4[4] = {SPADE_D, (cuuint64_t)sh.NBmax, 4, (cuuint64_t)sh.BH};
    const cuuint64_t str4[3] = {512, 512ull * sh.NBmax, 2048ull * sh.NBmax};
    r = enc(&out->kd, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, ws.kdsa, dims4, str4, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { snprintf(err, errlen, "cuTensorMapEncodeTiled (max/min summaries) failed with %d", (int)r); return 1; }
  }
  return 0;
}

cudaError_t launch_scores(const ScoreMaps* maps, const Shape& sh, const GeoPack& gp, const WsTables& ws, int num_sms,
                          int term, cudaStream_t s) {
  cudaError_t e = cudaFuncSetAttribute(k_scores, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SC_SMEM);
  if (e != cudaSuccess) return e;
  const int items = sh.BH * ((sh.NBvmax + 127) / 128) * SC_PARTS;
  const int grid = items < num_sms ? items : num_sms;
  k_scores<<<grid, SC_THREADS, SC_SMEM, s>>>(*maps, sh, gp, ws, 1.0f / sqrtf((float)SPADE_D), term == 0 ? ws.qsum : ws.qmid,
                                             term == 2 ? 1 : 0, term);
  return cudaGetLastError();
}
