// Scheme generation in one pass over Q and K (Eq. 3-5, Algorithm 1; Sec. 3.1 Summarizer Expression):
// per-block SICS and mean summaries of EVERY blocking candidate, with nothing but the results written.
//
// Both quantities are sums over the tokens of a block: SICS = |sum_t q_t / |q_t||^2 (what Algorithm 1 returns
// as 2*sigma + n) and the mean = sum_t q_t / n.  With several candidates every token belongs to one block of
// each, and adding a token row into four or more accumulators on the SIMT pipes is issue-bound, three times
// slower than the read of Q and K.  A sum over tokens with 0/1 membership is a matrix product, so the tensor
// core takes it:
//
//   D[channel, (block, piece)] = sum_token X[token, channel] * Wt[(block, piece), token]
//
// over one t-slice of a "column" of the grid (128 tokens: colH x colW, a common multiple of the candidates'
// (bh, bw) footprints; block extents are powers of two).  X is the slice as TMA delivers it (two 64-channel
// boxes, 128-byte swizzle; positions outside the grid are zero-filled and add nothing), used as the
// MN-major operand A.  Wt has four rows per block of every candidate present in the slice ("slot"): three
// bf16 pieces r1 + r2 + r3 of 1/|q_t| (24 mantissa bits together; bf16 x bf16 products are exact in the fp32
// accumulator) and one row of ones for the plain sum, non-zero only where the token belongs to the block.
// The zero pattern and the ones never change; per slice only 3 values per token and candidate are rewritten.
//
// Warp roles: warps 0-3 one thread per token (|q_t|^2 straight from shared memory, no shuffle; the three
// pieces into Wt), warps 4-11 the epilogue, one channel per thread (TMEM lane): add the pieces, accumulate a
// block over its bt slices in registers, and when the block ends write the mean (coalesced) and the SICS
// (warp sums over 32 channels, the last of the four warps to arrive adds the four partials in a fixed
// order); warp 12 loads slices (ring of stages, running ahead across work items), warp 13 issues the
// products (D double-buffered in TMEM).  All waits are bounded.  HBM traffic: Q and K once, the tables once.
#include <cuda.h>
#include <stdio.h>
#include <string.h>

#include <vector>

#include "sm100_ptx.cuh"
#include "spade_common.cuh"

struct PlanMaps { CUtensorMap q, k; };      // 5-D (d, W, H, T, head), box (64, colW, colH, 1, 1), 128-byte swizzle

namespace {

constexpr unsigned FULL = 0xffffffffu;
constexpr uint64_t PF_WAIT_NS = 2000000000ull;
constexpr int PF_MAX_STAGES = 4;
constexpr int PF_SLICE_BYTES = 32768;        // 128 tokens x 256 bytes
constexpr int PF_HALF_BYTES = 16384;         // one 64-channel half of a slice
constexpr int PF_NG = 2;                     // epilogue warpgroups
constexpr int PF_THREADS = (4 + 4 * PF_NG + 2) * 32;        // 4 token warps, the epilogue warps, loader, issuer
constexpr int PF_WARP_LOAD = 4 + 4 * PF_NG, PF_WARP_MMA = PF_WARP_LOAD + 1;

struct PfCtl {
  uint64_t full[PF_MAX_STAGES], empty[PF_MAX_STAGES];
  uint64_t w_full[2], w_empty[2], d_full[2], d_empty[2];
  uint64_t tab_full[2], tab_empty[2];      // the output table rows of a work item in shared memory (loader -> epilogue warps)
  uint32_t tmem_base;
  volatile uint32_t abort;
  float sp[2][64][4];        // SICS partials of the four warps of a warpgroup, per slice parity and slot
  int cnt[2][64];            // arrivals on a slot's partials
};

__host__ __device__ constexpr uint32_t pf_idesc(int M, int N) {      // bf16 x bf16 -> fp32, A MN-major, B K-major
  return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ uint16_t pf_bf16(float x) {
  return __bfloat16_as_ushort(__float2bfloat16_rn(x));
}
__device__ __forceinline__ float pf_bf16_to_float(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }

// Byte offset of (row n, token) inside one weight-matrix buffer: two 64-token halves of nrows x 128 bytes,
// 16-byte chunks swizzled with the row index as the tensor core expects of a K-major operand.
__device__ __forceinline__ uint32_t pf_w_offset(int nrows, int n, int tok) {
  return (uint32_t)((tok >> 6) * nrows * 128 + n * 128 + ((((tok & 63) >> 3) ^ (n & 7)) << 4) + (tok & 7) * 2);
}

// Row of the weight matrix (= column of D) of (slot, piece).  Slots go round the four epilogue warpgroups
// (slot mod 4), so that the candidates whose blocks end most often are shared by all; a warpgroup's slots
// sit in CPW chunks of 32 columns, 8 slots of 4 pieces each.
// Two slots share eight columns, piece by piece: [r1 a, r1 b, r2 a, r2 b, r3 a, r3 b, ones a, ones b], so that the
// epilogue adds the pieces of both with packed fp32 instructions on adjacent registers.
__device__ __forceinline__ int pf_row(int cpw, int slot, int piece) {
  const int k = slot / PF_NG;
  return 32 * ((slot % PF_NG) * cpw + (k >> 3)) + 8 * ((k & 7) >> 1) + 2 * piece + (k & 1);
}
__device__ __forceinline__ uint64_t pf_pack2(uint32_t lo, uint32_t hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ uint64_t pf_add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ float pf_half(uint64_t v, int hi) {
  float a, b;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
  return hi ? b : a;
}

template <int CPW>
__global__ void __launch_bounds__(PF_THREADS, 1)
k_plan_fused(const __grid_constant__ PlanMaps maps, const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp,
             const WsTables ws, const __grid_constant__ PlanFusedCfg cfg,
             const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
             const int* __restrict__ tab_e, const float* __restrict__ tab_inv, const uint32_t* __restrict__ tab_m) {
  extern __shared__ __align__(1024) uint8_t pf_smem[];
  constexpr int NROWS = 32 * PF_NG * CPW;    // rows of the weight matrix = columns of D
  uint8_t* slices = pf_smem;                                            // cfg.stages x 32 KB
  uint8_t* wmat = pf_smem + cfg.stages * PF_SLICE_BYTES;                // 2 buffers x (2 halves x NROWS x 128 B)
  constexpr int W_BYTES = 2 * NROWS * 128;
  constexpr uint32_t TMEM_COLS = 2 * NROWS <= 128 ? 128 : 2 * NROWS <= 256 ? 256 : 512;     // a power of two
  // per work item: tchunk rows of the row table, of the 1/n table and of the end masks (16 bytes per slice), two buffers
  constexpr int PER = PF_NG * 8 * CPW;
  const int TAB_BYTES = cfg.tchunk * (PER * 8 + 16);
  uint8_t* tabs = wmat + 2 * W_BYTES;
  PfCtl& ctl = *reinterpret_cast<PfCtl*>(tabs + 2 * TAB_BYTES);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int col_items = cfg.ncol_h * cfg.ncol_w;
  const int items = sh.BH * 2 * cfg.nchunks * col_items;

  // ---- one-time set-up: barriers, TMEM, the constant part of the weight matrix -------------------------
  if (tid == 0) {
    for (int s = 0; s < cfg.stages; ++s) { ptx::mbar_init(&ctl.full[s], 1); ptx::mbar_init(&ctl.empty[s], 5); }
    for (int b = 0; b < 2; ++b) {
      ptx::mbar_init(&ctl.w_full[b], 4); ptx::mbar_init(&ctl.w_empty[b], 1);
      ptx::mbar_init(&ctl.d_full[b], 1); ptx::mbar_init(&ctl.d_empty[b], 4 * PF_NG);
      ptx::mbar_init(&ctl.tab_full[b], 1); ptx::mbar_init(&ctl.tab_empty[b], 4 * PF_NG);
    }
    ctl.abort = 0;
    ptx::fence_mbar_init();
  }
  for (int i = tid; i < 2 * 64; i += PF_THREADS) (&ctl.cnt[0][0])[i] = 0;
  for (int i = tid; i < 2 * W_BYTES / 16; i += PF_THREADS) reinterpret_cast<uint4*>(wmat)[i] = make_uint4(0, 0, 0, 0);
  if (ptx::smem_u32(pf_smem) & 1023u) {        // the swizzled tiles need 1024-byte alignment; never seen otherwise
    if (tid == 0 && atomicCAS(ws.status, 0u, (uint32_t)SPADE_ST_TIMEOUT) == 0u) { ws.status[1] = 299; ws.status[2] = 0; }
    return;
  }
  if (warp == PF_WARP_MMA) { ptx::tmem_alloc(&ctl.tmem_base, TMEM_COLS); ptx::tmem_relinquish(); }
  __syncthreads();
  if (tid < 128) {                           // the row of ones of every block this token belongs to (both buffers)
    const int dh = tid >> cfg.lcolW, dw = tid & (cfg.colW - 1);
    for (int c = 0; c < sh.C; ++c) {
      const PlanFusedCand& pc = cfg.cand[c];
      const int slot = pc.slot_base + ((dh >> pc.lbh) << pc.lcbw) + (dw >> pc.lbw);
      const uint32_t off = pf_w_offset(NROWS, pf_row(CPW, slot, 3), tid);
      *reinterpret_cast<uint16_t*>(wmat + off) = 0x3f80;
      *reinterpret_cast<uint16_t*>(wmat + W_BYTES + off) = 0x3f80;
    }
  }
  ptx::fence_proxy_async_smem();
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_D = ctl.tmem_base;
  uint32_t site = 0;

  if (warp == PF_WARP_LOAD) {
    // ================= loader: slices of this CTA's work items through the ring ==========================
    if (lane == 0) {
      uint32_t nit = 0, s = 0, sph = 0;          // ring stage of the next slice and its phase (kept by hand: a division per slice costs a single thread hundreds of cycles)
      for (int item = blockIdx.x; item < items && !site; item += gridDim.x) {
        const int col = item % col_items, chunk = (item / col_items) % cfg.nchunks, ht = item / (col_items * cfg.nchunks);
        const int h0 = (col / cfg.ncol_w) * cfg.colH, w0 = (col % cfg.ncol_w) * cfg.colW;
        const int t0 = chunk * cfg.tchunk, t1 = min(sh.T, t0 + cfg.tchunk);
        const CUtensorMap* map = (ht & 1) ? &maps.k : &maps.q;
        {                                         // the item's rows of the output tables, ahead of its slices
          const uint32_t tb = nit & 1, nsl = (uint32_t)(t1 - t0);
          if (!ptx::mbar_wait_sleepy(&ctl.tab_empty[tb], ((nit >> 1) & 1) ^ 1, &ctl.abort, PF_WAIT_NS)) { site = 203; break; }
          uint8_t* dst = tabs + tb * TAB_BYTES;
          const size_t r0 = (size_t)col * sh.T + t0;
          ptx::mbar_expect_tx(&ctl.tab_full[tb], nsl * (PER * 8 + 16));
          ptx::bulk_load(dst, tab_e + r0 * PER, nsl * PER * 4, &ctl.tab_full[tb]);
          ptx::bulk_load(dst + cfg.tchunk * PER * 4, tab_inv + r0 * PER, nsl * PER * 4, &ctl.tab_full[tb]);
          ptx::bulk_load(dst + cfg.tchunk * PER * 8, tab_m + r0 * 4, nsl * 16, &ctl.tab_full[tb]);
          ++nit;
        }
        for (int t = t0; t < t1; ++t) {
          if (!ptx::mbar_wait_sleepy(&ctl.empty[s], sph ^ 1, &ctl.abort, PF_WAIT_NS)) { site = 201; break; }
          ptx::mbar_expect_tx(&ctl.full[s], PF_SLICE_BYTES);
          ptx::tma_load_5d(slices + s * PF_SLICE_BYTES, map, &ctl.full[s], 0, w0, h0, t, ht >> 1);
          ptx::tma_load_5d(slices + s * PF_SLICE_BYTES + PF_HALF_BYTES, map, &ctl.full[s], 64, w0, h0, t, ht >> 1);
          if (++s == (uint32_t)cfg.stages) { s = 0; sph ^= 1; }
        }
      }
    }
  } else if (warp == PF_WARP_MMA) {
    // ================= issuer: D[channel, row] = X^T Wt^T per slice ======================================
    if (lane == 0) {
      const uint32_t idesc = pf_idesc(128, NROWS);
      const uint32_t aS = ptx::smem_u32(slices), aW = ptx::smem_u32(wmat);
      uint32_t i = 0, s = 0, sph = 0;        // slice count; ring stage and its phase
      for (int item = blockIdx.x; item < items && !site; item += gridDim.x) {
        const int chunk = (item / col_items) % cfg.nchunks;
        const int t0 = chunk * cfg.tchunk, t1 = min(sh.T, t0 + cfg.tchunk);
        for (int t = t0; t < t1; ++t, ++i) {
          const uint32_t b = i & 1, ph = (i >> 1) & 1;
          if (!ptx::mbar_wait(&ctl.full[s], sph, &ctl.abort, PF_WAIT_NS) ||
              !ptx::mbar_wait(&ctl.w_full[b], ph, &ctl.abort, PF_WAIT_NS) ||
              !ptx::mbar_wait(&ctl.d_empty[b], ph ^ 1, &ctl.abort, PF_WAIT_NS)) { site = 205; break; }
          ptx::tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {        // 16 tokens per step
            const uint64_t ad = ptx::smem_desc_sw128(aS + s * PF_SLICE_BYTES + ks * 2048, PF_HALF_BYTES, 1024);
            const uint64_t bd = ptx::smem_desc_sw128(aW + b * W_BYTES + (ks >> 2) * (NROWS * 128) + (ks & 3) * 32, 16, 1024);
            ptx::umma_ss(tmem_D + b * NROWS, ad, bd, idesc, ks > 0);
          }
          ptx::umma_commit(&ctl.d_full[b]);
          ptx::umma_commit(&ctl.w_empty[b]);
          ptx::umma_commit(&ctl.empty[s]);
          if (++s == (uint32_t)cfg.stages) { s = 0; sph ^= 1; }
        }
      }
    }
  } else if (warp < 4) {
    // ================= token warps: |q_t|^2 and the three pieces of 1/|q_t| into the weight matrix ========
    const int tok = tid;
    const int dh = tok >> cfg.lcolW, dw = tok & (cfg.colW - 1);
    uint32_t woff[4][3];                       // where this token's three pieces go, per candidate
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const PlanFusedCand& pc = cfg.cand[c < sh.C ? c : 0];
      const int slot = pc.slot_base + ((dh >> pc.lbh) << pc.lcbw) + (dw >> pc.lbw);
#pragma unroll
      for (int pce = 0; pce < 3; ++pce) woff[c][pce] = pf_w_offset(NROWS, pf_row(CPW, slot, pce), tok);
    }
    uint32_t i = 0, s = 0, sph = 0;
    for (int item = blockIdx.x; item < items && !site; item += gridDim.x) {
      const int chunk = (item / col_items) % cfg.nchunks;
      const int t0 = chunk * cfg.tchunk, t1 = min(sh.T, t0 + cfg.tchunk);
      for (int t = t0; t < t1 && !site; ++t, ++i) {
        const uint32_t b = i & 1, ph = (i >> 1) & 1;
        if (!ptx::mbar_wait_warp(&ctl.full[s], sph, &ctl.abort, PF_WAIT_NS)) { site = 202; break; }
        const uint8_t* row = slices + s * PF_SLICE_BYTES + tok * 128;
        uint64_t acc2[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          uint4 v[8];
#pragma unroll
          for (int u = 0; u < 8; ++u)            // the chunk order does not matter for a sum: take the bank-friendly one
            v[u] = *reinterpret_cast<const uint4*>(row + h * PF_HALF_BYTES + ((u ^ (tok & 7)) << 4));
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const uint32_t wv[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              uint64_t x;
              asm("mov.b64 %0, {%1, %2};" : "=l"(x) : "r"(wv[e] << 16), "r"(wv[e] & 0xffff0000u));
              asm("fma.rn.f32x2 %0, %1, %1, %0;" : "+l"(acc2[e]) : "l"(x));
            }
          }
        }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&ctl.empty[s]);                 // this warp has read the slice
        float ss = 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float sa, sb;
          asm("mov.b64 {%0, %1}, %2;" : "=f"(sa), "=f"(sb) : "l"(acc2[e]));
          ss += sa + sb;
        }
        const float rn = ss > 0.f ? rsqrtf(ss) : 0.f;
        const uint16_t r1 = pf_bf16(rn);
        const float e1 = rn - pf_bf16_to_float(r1);
        const uint16_t r2 = pf_bf16(e1);
        const uint16_t r3 = pf_bf16(e1 - pf_bf16_to_float(r2));
        if (!ptx::mbar_wait_warp(&ctl.w_empty[b], ph ^ 1, &ctl.abort, PF_WAIT_NS)) { site = 206; break; }
        uint8_t* wb = wmat + b * W_BYTES;
#pragma unroll
        for (int c = 0; c < 4; ++c) {                                    // the first four candidates: offsets kept in registers
          if (c >= sh.C) break;
          if (!SPADE_CHECK(woff[c][2] < (uint32_t)W_BYTES && woff[c][0] < (uint32_t)W_BYTES, ws.status, 602, woff[c][0])) continue;
          *reinterpret_cast<uint16_t*>(wb + woff[c][0]) = r1;
          *reinterpret_cast<uint16_t*>(wb + woff[c][1]) = r2;
          *reinterpret_cast<uint16_t*>(wb + woff[c][2]) = r3;
        }
        for (int c = 4; c < sh.C; ++c) {
          const PlanFusedCand& pc = cfg.cand[c];
          const int slot = pc.slot_base + ((dh >> pc.lbh) << pc.lcbw) + (dw >> pc.lbw);
          const int n0 = pf_row(CPW, slot, 0);
          *reinterpret_cast<uint16_t*>(wb + pf_w_offset(NROWS, n0 + 0, tok)) = r1;
          *reinterpret_cast<uint16_t*>(wb + pf_w_offset(NROWS, n0 + 1, tok)) = r2;
          *reinterpret_cast<uint16_t*>(wb + pf_w_offset(NROWS, n0 + 2, tok)) = r3;
        }
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&ctl.w_full[b]);
        if (++s == (uint32_t)cfg.stages) { s = 0; sph ^= 1; }
      }
    }
    // ---- text blocks (outside the 3-D grid: no SICS, mean summaries only), straight from their rows ------
    if (!site) {
      const int hw = lane >> 4, l16 = lane & 15;
      const long total = (long)sh.BH * 2 * cfg.text_blocks;
      for (long u = (long)blockIdx.x * 4 + warp; u < total; u += (long)gridDim.x * 4) {
        const int ht = (int)(u / cfg.text_blocks);
        int rem = (int)(u % cfg.text_blocks), c = 0;
        while (rem >= gp.g[c].NBt) { rem -= gp.g[c].NBt; ++c; }
        const CandGeo& g = gp.g[c];
        const __nv_bfloat16* src = ((ht & 1) ? K : Q) + (size_t)(ht >> 1) * sh.N * SPADE_D;
        const int first = sh.Nv + rem * g.BS;
        float acc[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = 0.f;
        int nval = 0;
        for (int r = hw; r < g.BS; r += 2) {
          const int tk = first + r;
          if (tk >= sh.N) break;
          ++nval;
          float x[8];
          bf16x8_to_float(__ldg(reinterpret_cast<const uint4*>(src + (size_t)tk * SPADE_D) + l16), x);
#pragma unroll
          for (int k = 0; k < 8; ++k) acc[k] += x[k];
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] += __shfl_xor_sync(FULL, acc[k], 16);
        nval += __shfl_xor_sync(FULL, nval, 16);
        if (hw == 0) {
          const float inv = nval > 0 ? 1.f / (float)nval : 0.f;
          float* mean = ws.csum + ((((size_t)ht * sh.C + c) * sh.NBmax) + g.NBv + rem) * SPADE_D + l16 * 8;
          reinterpret_cast<float4*>(mean)[0] = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
          reinterpret_cast<float4*>(mean)[1] = make_float4(acc[4] * inv, acc[5] * inv, acc[6] * inv, acc[7] * inv);
        }
      }
    }
  } else {
    // ================= epilogue: one channel per thread, 8 * CPW slots per warpgroup ======================
    // The warpgroup index is a compile-time constant of the code each warp runs, so that every branch on
    // slot ranges is provably uniform (no reconvergence bookkeeping around the 8 * CPW slot tests).
    {
      const int grp = (warp - 4) >> 2;
      const int wq = warp & 3;
      const int ch = wq * 32 + lane;
      const uint32_t lane_base = (uint32_t)(wq * 32) << 16;
      uint64_t an[4 * CPW], ar[4 * CPW];       // per pair of slots (2p, 2p + 1): summed q / |q| and summed q of this channel, packed fp32 x 2
#pragma unroll
      for (int k = 0; k < 4 * CPW; ++k) an[k] = ar[k] = 0ull;
      uint32_t i = 0, nit = 0;
      for (int item = blockIdx.x; item < items && !site; item += gridDim.x, ++nit) {
        const int chunk = (item / col_items) % cfg.nchunks, ht = item / (col_items * cfg.nchunks);
        const int t0 = chunk * cfg.tchunk, t1 = min(sh.T, t0 + cfg.tchunk);
        // the item's rows of the output tables arrive in shared memory (a row is used once: from global memory every
        // slice paid two trips to the L2 in the middle of its output step)
        const uint32_t tb = nit & 1;
        if (!__all_sync(FULL, ptx::mbar_wait(&ctl.tab_full[tb], (nit >> 1) & 1, &ctl.abort, PF_WAIT_NS))) { site = 209; break; }
        const int* const s_e = reinterpret_cast<const int*>(tabs + tb * TAB_BYTES) + grp * (8 * CPW);
        const float* const s_inv = reinterpret_cast<const float*>(tabs + tb * TAB_BYTES + cfg.tchunk * PER * 4) + grp * (8 * CPW);
        const uint32_t* const s_m = reinterpret_cast<const uint32_t*>(tabs + tb * TAB_BYTES + cfg.tchunk * PER * 8) + grp;
        for (int t = t0; t < t1 && !site; ++t, ++i) {
          const uint32_t b = i & 1, ph = (i >> 1) & 1;
          if (!__all_sync(FULL, ptx::mbar_wait(&ctl.d_full[b], ph, &ctl.abort, PF_WAIT_NS))) { site = 207; break; }
          ptx::tc_fence_after();
#pragma unroll
          for (int q = 0; q < CPW; ++q) {
            uint32_t r[32];
            ptx::tmem_ld32(tmem_D + lane_base + b * NROWS + (grp * CPW + q) * 32, r);
            ptx::tmem_wait_ld();
#pragma unroll
            for (int pr = 0; pr < 4; ++pr) {
              const uint64_t p12 = pf_add2(pf_pack2(r[8 * pr], r[8 * pr + 1]), pf_pack2(r[8 * pr + 2], r[8 * pr + 3]));
              an[q * 4 + pr] = pf_add2(an[q * 4 + pr], pf_add2(p12, pf_pack2(r[8 * pr + 4], r[8 * pr + 5])));
              ar[q * 4 + pr] = pf_add2(ar[q * 4 + pr], pf_pack2(r[8 * pr + 6], r[8 * pr + 7]));
            }
          }
          // D is in the accumulators: the issuer may overwrite the buffer while the outputs below are written
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&ctl.d_empty[b]);
          // Blocks that end at this slice are written.  Which of the warpgroup's slots end at (column, t), where
          // their rows sit in the tables and the 1 / n of each block were worked out on the host: the output
          // step is a table look-up and two predicated stores per slot; a group of four slots none of which ends
          // here (a bit mask per column, slice and warpgroup, the same for every thread) is skipped as a whole.
          {
            const int row = (t - t0) * PER;
            const uint32_t ends = s_m[(t - t0) * 4];
            float* const cs = ws.csum + ((size_t)ht * sh.C * sh.NBmax) * SPADE_D + ch;
            float* const ns = ws.nsum + ((size_t)ht * sh.C * sh.NBmax) * SPADE_D + ch;
#pragma unroll
            for (int k4 = 0; k4 < 8 * CPW; k4 += 4) {
              if (!((ends >> k4) & 0xfu)) continue;
              const int4 e4 = *reinterpret_cast<const int4*>(s_e + row + k4);
              const float4 i4 = *reinterpret_cast<const float4*>(s_inv + row + k4);
              const int e[4] = {e4.x, e4.y, e4.z, e4.w};
              const float iv[4] = {i4.x, i4.y, i4.z, i4.w};
#pragma unroll
              for (int u = 0; u < 4; ++u) {
                const int k = k4 + u;
                const float anv = pf_half(an[k >> 1], k & 1), arv = pf_half(ar[k >> 1], k & 1);
                if (e[u] >= 0 && SPADE_CHECK(e[u] < sh.C * sh.NBmax, ws.status, 601, e[u])) {
                  cs[(size_t)e[u] * SPADE_D] = arv * iv[u];            // mean summary, this channel
                  ns[(size_t)e[u] * SPADE_D] = anv;                    // sum of q / |q|; SICS = its squared norm
                }
                if (e[u] >= 0) {                                       // the block is done: its half of the pair starts again at zero
                  an[k >> 1] = (k & 1) ? pf_pack2(__float_as_uint(pf_half(an[k >> 1], 0)), 0u) : pf_pack2(0u, __float_as_uint(pf_half(an[k >> 1], 1)));
                  ar[k >> 1] = (k & 1) ? pf_pack2(__float_as_uint(pf_half(ar[k >> 1], 0)), 0u) : pf_pack2(0u, __float_as_uint(pf_half(ar[k >> 1], 1)));
                }
              }
            }
          }
        }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&ctl.tab_empty[tb]);          // the table buffer may take the item after next
      }
    }
  }
  site = __shfl_sync(FULL, site, 0) | site;
  if (site && lane == 0 && atomicCAS(ws.status, 0u, (uint32_t)SPADE_ST_TIMEOUT) == 0u) { ws.status[1] = site; ws.status[2] = 0; }

  // ---- teardown ------------------------------------------------------------------------------------------
  __syncwarp();
  if (ctl.abort) {                      // let copies still in flight land before the CTA goes away
    for (int k = 0; k < 200; ++k) __nanosleep(1000);
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == PF_WARP_MMA) ptx::tmem_dealloc(tmem_D, TMEM_COLS);
}

// SICS(block) = |sum_t q_t / |q_t||^2 (Eq. 4 / Algorithm 1) from the summed unit vectors the one-pass kernel left:
// one warp per (head, tensor, candidate, video block), channels in a fixed order.
template <class Index>      // int when the number of blocks fits (64-bit division costs a call per block), long otherwise
__global__ void __launch_bounds__(256)
k_sics_from_sums(const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp, const WsTables ws) {
  const int lane = threadIdx.x & 31;
  const Index gw = (Index)blockIdx.x * 8 + (threadIdx.x >> 5), nw = (Index)gridDim.x * 8;
  const Index total = (Index)sh.BH * 2 * sh.units_per_ht;
  for (Index u0 = gw * 4; u0 < total; u0 += nw * 4) {           // four blocks per warp and step: four loads in flight
    float4 v[4];
    size_t out[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const Index u = u0 + q < total ? u0 + q : total - 1;
      const int ht = (int)(u / (Index)sh.units_per_ht), rem = (int)(u % (Index)sh.units_per_ht);
      int c = 0;
#pragma unroll
      for (int i = 1; i < SPADE_MAX_CANDS; ++i)
        if (i < sh.C && rem >= gp.g[i].unit_off) c = i;
      const int b = rem - gp.g[c].unit_off;
      v[q] = __ldcs(reinterpret_cast<const float4*>(ws.nsum + ((((size_t)ht * sh.C + c) * sh.NBmax) + b) * SPADE_D) + lane);
      out[q] = (((size_t)(ht >> 1) * sh.C + c) * 2 + (ht & 1)) * sh.NBvmax + b;
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float s = (v[q].x * v[q].x + v[q].y * v[q].y) + (v[q].z * v[q].z + v[q].w * v[q].w);
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(FULL, s, o);
      if (lane == 0 && u0 + q < total) ws.sics[out[q]] = s;
    }
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

size_t plan_fused_smem(const PlanFusedCfg& cfg) {
  return (size_t)cfg.stages * PF_SLICE_BYTES + (size_t)2 * (2 * cfg.nrows * 128) + (size_t)2 * cfg.tchunk * (PF_NG * 8 * cfg.cpw * 8 + 16) + sizeof(PfCtl);
}

int ilog2(int x) { int l = 0; while ((1 << l) < x) ++l; return l; }

}  // namespace

size_t plan_maps_bytes() { return sizeof(PlanMaps); }

// Decides whether the one-pass kernel serves this candidate set and fills its configuration.
void plan_fused_configure(PlanFusedCfg* cfg, const Shape& sh, const GeoPack& gp, int num_sms) {
  (void)num_sms;
  memset(cfg, 0, sizeof(*cfg));
  int maxbh = 1, maxbw = 1, maxbt = 1;
  for (int c = 0; c < sh.C; ++c) {
    const CandGeo& g = gp.g[c];
    maxbh = g.bh > maxbh ? g.bh : maxbh; maxbw = g.bw > maxbw ? g.bw : maxbw; maxbt = g.bt > maxbt ? g.bt : maxbt;
  }
  if (maxbh * maxbw > 128) return;                             // a column slice is one product over 128 tokens
  int colW = maxbw > 16 ? maxbw : 16;                          // wide rows keep the box copies long
  if (128 / colW < maxbh) colW = maxbw;
  const int colH = 128 / colW;
  cfg->colH = colH; cfg->colW = colW; cfg->lcolW = ilog2(colW);
  cfg->ncol_h = (sh.H + colH - 1) / colH; cfg->ncol_w = (sh.W + colW - 1) / colW;
  cfg->tchunk = maxbt > 4 ? maxbt : 4;
  cfg->nchunks = (sh.T + cfg->tchunk - 1) / cfg->tchunk;
  int slots = 0;
  for (int c = 0; c < sh.C; ++c) {
    const CandGeo& g = gp.g[c];
    PlanFusedCand& pc = cfg->cand[c];
    pc.lbt = ilog2(g.bt); pc.bt_mask = g.bt - 1; pc.lbh = ilog2(g.bh); pc.lbw = ilog2(g.bw);
    pc.cbw = colW / g.bw; pc.lcbw = ilog2(pc.cbw); pc.nblk = (colH / g.bh) * pc.cbw;
    pc.slot_base = slots;
    for (int j = 0; j < pc.nblk && slots + j < 64; ++j) cfg->slot_cand[slots + j] = (unsigned char)c;
    slots += pc.nblk;
    cfg->text_blocks += g.NBt;
  }
  if (slots > 64) return;                                      // 4 rows per slot, at most 256 columns of D
  cfg->nblk = slots;
  cfg->cpw = (slots + 8 * PF_NG - 1) / (8 * PF_NG);            // 8 slots per 32-column chunk of a warpgroup
  cfg->nrows = 32 * PF_NG * cfg->cpw;
  cfg->stages = PF_MAX_STAGES;
  const size_t budget = 226 * 1024;
  while (cfg->stages > 2 && plan_fused_smem(*cfg) > budget) --cfg->stages;
  if (plan_fused_smem(*cfg) > budget) return;
  cfg->on = 1;
}

int plan_encode_maps(PlanMaps* out, const void* Q, const void* K, const Shape& sh, const PlanFusedCfg& cfg, char* err,
                     size_t errlen) {
  EncodeFn enc = encode_fn();
  if (!enc) { snprintf(err, errlen, "cuTensorMapEncodeTiled is not available from this driver"); return 1; }
  const void* ptrs[2] = {Q, K};
  CUtensorMap* dst[2] = {&out->q, &out->k};
  const cuuint64_t dims[5] = {SPADE_D, (cuuint64_t)sh.W, (cuuint64_t)sh.H, (cuuint64_t)sh.T, (cuuint64_t)sh.BH};
  const cuuint64_t str[4] = {256, 256ull * sh.W, 256ull * sh.W * sh.H, 256ull * sh.N};
  const cuuint32_t box[5] = {64, (cuuint32_t)cfg.colW, (cuuint32_t)cfg.colH, 1, 1};
  const cuuint32_t es[5] = {1, 1, 1, 1, 1};
  for (int t = 0; t < 2; ++t) {
    CUresult r = enc(dst[t], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(ptrs[t]), dims, str, box, es,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { snprintf(err, errlen, "cuTensorMapEncodeTiled (plan stage, tensor %d) failed with %d", t, (int)r); return 1; }
  }
  return 0;
}

// The epilogue's output table: for every (column, t, slot) the row the slot's block has in the per-candidate
// tables (candidate * NBmax + block id) if the block ends at slice t and lies inside the grid, else -1, and the
// reciprocal of the block's valid-token count.  Slots are ordered [warpgroup][position] as the kernel reads them.
void plan_fused_tables(const PlanFusedCfg& cfg, const Shape& sh, const GeoPack& gp, std::vector<int>& e,
                       std::vector<float>& inv, std::vector<uint32_t>& ends) {
  const int ncol = cfg.ncol_h * cfg.ncol_w, per = PF_NG * 8 * cfg.cpw;
  e.assign((size_t)ncol * sh.T * per, -1);
  inv.assign((size_t)ncol * sh.T * per, 0.f);
  ends.assign((size_t)ncol * sh.T * 4, 0u);              // per (column, slice): one word per warpgroup (16 bytes per slice), bit k <=> the slot at position k ends here
  for (int col = 0; col < ncol; ++col) {
    const int ch0 = (col / cfg.ncol_w) * cfg.colH, cw0 = (col % cfg.ncol_w) * cfg.colW;
    for (int t = 0; t < sh.T; ++t)
      for (int j = 0; j < cfg.nblk; ++j) {
        const int c = cfg.slot_cand[j];
        const PlanFusedCand& pc = cfg.cand[c];
        const CandGeo& g = gp.g[c];
        if (((t + 1) & pc.bt_mask) != 0 && t + 1 != sh.T) continue;
        const int jl = j - pc.slot_base;
        const int it = t >> pc.lbt, ih = (ch0 >> pc.lbh) + (jl >> pc.lcbw), iw = (cw0 >> pc.lbw) + (jl & (pc.cbw - 1));
        if (ih >= g.nbh || iw >= g.nbw) continue;
        const int nt = g.bt < sh.T - it * g.bt ? g.bt : sh.T - it * g.bt;
        const int nh = g.bh < sh.H - ih * g.bh ? g.bh : sh.H - ih * g.bh;
        const int nw = g.bw < sh.W - iw * g.bw ? g.bw : sh.W - iw * g.bw;
        const size_t at = ((size_t)col * sh.T + t) * per + (j % PF_NG) * (8 * cfg.cpw) + j / PF_NG;
        e[at] = c * sh.NBmax + (it * g.nbh + ih) * g.nbw + iw;
        ends[((size_t)col * sh.T + t) * 4 + j % PF_NG] |= 1u << (j / PF_NG);
        inv[at] = 1.f / (float)(nt * nh * nw);
      }
  }
}

cudaError_t launch_plan_fused(const PlanMaps* maps, const void* Q, const void* K, const Shape& sh, const GeoPack& gp,
                              const StaticTables& st, const WsTables& ws, const PlanFusedCfg& cfg, int num_sms,
                              const int* tab_e, const float* tab_inv, const uint32_t* tab_m, cudaStream_t s) {
  (void)st;
  const size_t smem = plan_fused_smem(cfg);
  const long items = (long)sh.BH * 2 * cfg.nchunks * cfg.ncol_h * cfg.ncol_w;
  long grid = num_sms;
  if (grid > items) grid = items;
  cudaError_t e = cudaErrorInvalidValue;
#define PF_LAUNCH(CPW_)                                                                                              \
  if (cfg.cpw == CPW_) {                                                                                             \
    e = cudaFuncSetAttribute(k_plan_fused<CPW_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);            \
    if (e != cudaSuccess) return e;                                                                                  \
    k_plan_fused<CPW_><<<(unsigned)grid, PF_THREADS, smem, s>>>(*maps, sh, gp, ws, cfg, (const __nv_bfloat16*)Q,     \
                                                                (const __nv_bfloat16*)K, tab_e, tab_inv, tab_m);    \
  }
  PF_LAUNCH(1) PF_LAUNCH(2) PF_LAUNCH(3) PF_LAUNCH(4)
#undef PF_LAUNCH
  if (e != cudaSuccess) return e;
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const long blocks = (long)sh.BH * 2 * sh.units_per_ht;
  long ctas = (blocks + 31) / 32;
  if (ctas > (long)num_sms * 8) ctas = (long)num_sms * 8;
  if (blocks + 4l * num_sms * 64 < 0x7fffffffl) k_sics_from_sums<int><<<(unsigned)ctas, 256, 0, s>>>(sh, gp, ws);
  else k_sics_from_sums<long><<<(unsigned)ctas, 256, 0, s>>>(sh, gp, ws);
  return cudaGetLastError();
}
