// Selection stages of the SPADE hot path (sm_100a, SIMT kernels):
//   k_sics       SICS of every block of every candidate (Eq. 4 / Algorithm 1, as ||sum q_hat||^2)
//   k_choose     Aggregation Score (Eq. 3), per-head argmax candidate (Sec. 3.2), keep counts
//   k_groups     heads ordered by chosen scheme + attention work-item prefix (Sec. 3.3, head grouping)
//   k_summarize  mean summaries Q', K' of the chosen scheme (Sec. 3.1 Summarizer Expression)
//   k_minmax     channel-wise max / min summaries; k_scores_minmax: the estimators built on them (Fig. 4a, 4b)
//   k_select_reg index search on the block scores: softmax over KV blocks, Top-K / Top-P, ascending lists
//                (the scores S = <Q'_i,K'_j>/sqrt(d) come from k_scores in scores.cu)
#include "spade_common.cuh"

namespace {

constexpr int WARPS_PER_CTA = 8;
constexpr unsigned FULL = 0xffffffffu;

// ------------------------------------------------------------------------------------------------
// One warp reduces one block: each half-warp reads one token row per step (16 lanes x 16 bytes
// = the 256-byte bf16 row), four row pairs in flight.  NORMALISE = true accumulates q/||q||
// (for SICS), false accumulates q (for the mean).  Result: lanes 0..15 hold 8 channels each
// (channel 8*l16 + i), already summed over both half-warps.
template <bool NORMALISE>
__device__ __forceinline__ void reduce_block(const __nv_bfloat16* __restrict__ base, const CandGeo& g,
                                             const uint32_t* __restrict__ rowoff, int b, bool full,
                                             const Shape& sh, int lane, float (&acc)[8]) {
  const int hw = lane >> 4, l16 = lane & 15;
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.f;
  int t0 = 0, h0 = 0, w0 = 0, text_first = -1;
  if (b >= g.NBv) {
    text_first = sh.Nv + (b - g.NBv) * g.BS;
  } else {
    int iw = b % g.nbw, ih = (b / g.nbw) % g.nbh, it = b / (g.nbw * g.nbh);
    t0 = it * g.bt; h0 = ih * g.bh; w0 = iw * g.bw;
  }
  for (int r0 = 0; r0 < g.BS; r0 += 8) {
    uint4 v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int r = r0 + 2 * i + hw;
      int tok; bool ok;
      if (text_first >= 0) {
        tok = text_first + r; ok = tok < sh.N;
      } else {
        const uint32_t code = __ldg(rowoff + r);
        const int t = t0 + (int)(code >> 20), h = h0 + (int)((code >> 10) & 1023), w = w0 + (int)(code & 1023);
        ok = full || (t < sh.T && h < sh.H && w < sh.W);
        tok = (t * sh.H + h) * sh.W + w;
      }
      v[i] = ok ? __ldg(reinterpret_cast<const uint4*>(base + (size_t)tok * SPADE_D) + l16) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float x[8];
      bf16x8_to_float(v[i], x);
      if (NORMALISE) {
        float ss = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) ss = fmaf(x[c], x[c], ss);
#pragma unroll
        for (int o = 8; o >= 1; o >>= 1) ss += __shfl_xor_sync(FULL, ss, o);
        const float rn = ss > 0.f ? rsqrtf(ss) : 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[c] = fmaf(x[c], rn, acc[c]);
      } else {
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[c] += x[c];
      }
    }
  }
#pragma unroll
  for (int c = 0; c < 8; ++c) acc[c] += __shfl_xor_sync(FULL, acc[c], 16);
}

// SICS(block) = sum over all token pairs of cos(q_a, q_b) = || sum_k q_hat_k ||^2, which is what
// Algorithm 1 returns as 2*sigma + BS (second line of Eq. 5 with the diagonal folded back in).
__global__ void __launch_bounds__(WARPS_PER_CTA * 32)
k_sics(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K, const __grid_constant__ Shape sh,
       const __grid_constant__ GeoPack gp,
       StaticTables st, WsTables ws) {
  const int lane = threadIdx.x & 31;
  const int gw = blockIdx.x * WARPS_PER_CTA + (threadIdx.x >> 5);
  const int nw = gridDim.x * WARPS_PER_CTA;
  const long total = (long)sh.BH * 2 * sh.units_per_ht;
  for (long u = gw; u < total; u += nw) {
    const int ht = (int)(u / sh.units_per_ht), rem = (int)(u % sh.units_per_ht);
    const int bh = ht >> 1, tensor = ht & 1;
    int c = 0;
#pragma unroll
    for (int i = 1; i < SPADE_MAX_CANDS; ++i)
      if (i < sh.C && rem >= gp.g[i].unit_off) c = i;
    const CandGeo& g = gp.g[c];
    const int b = rem - g.unit_off;
    const __nv_bfloat16* base = (tensor ? K : Q) + (size_t)bh * sh.N * SPADE_D;
    const bool full = __ldg(st.nvalid + g.tab_off + b) == g.BS;
    float acc[8];
    reduce_block<true>(base, g, st.rowoff + c * 128, b, full, sh, lane, acc);
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) s = fmaf(acc[i], acc[i], s);
#pragma unroll
    for (int o = 8; o >= 1; o >>= 1) s += __shfl_xor_sync(FULL, s, o);
    if (lane == 0) ws.sics[(((size_t)bh * sh.C + c) * 2 + tensor) * sh.NBvmax + b] = s;
  }
}

// ------------------------------------------------------------------------------------------------
// Cell pass: ONE read of Q and K.  Each half-warp owns one cell (the common refinement of all
// candidates) and leaves two 128-vectors per cell: sum of q/||q|| and sum of q over the cell's
// valid tokens.  Lane l16 holds channels 8*l16 .. 8*l16+7.
__global__ void __launch_bounds__(WARPS_PER_CTA * 32)
k_cells(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K, const __grid_constant__ Shape sh,
        float* __restrict__ cells) {
  const int lane = threadIdx.x & 31, hw = lane >> 4, l16 = lane & 15;
  const long gw = (long)blockIdx.x * WARPS_PER_CTA + (threadIdx.x >> 5);
  const long nw = (long)gridDim.x * WARPS_PER_CTA;
  const int pairs = (sh.NCELL + 1) >> 1;
  const long total = (long)sh.BH * 2 * pairs;
  for (long u = gw; u < total; u += nw) {
    const int ht = (int)(u / pairs), cell = 2 * (int)(u % pairs) + hw;
    const int bh = ht >> 1, tensor = ht & 1;
    const bool live = cell < sh.NCELL;
    const __nv_bfloat16* base = (tensor ? K : Q) + (size_t)bh * sh.N * SPADE_D;
    const int iw = cell % sh.ncw, ih = (cell / sh.ncw) % sh.nch, it = cell / (sh.ncw * sh.nch);
    const int t0 = it * sh.ct, h0 = ih * sh.ch, w0 = iw * sh.cw;
    float an[8], ar[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) an[i] = ar[i] = 0.f;
    for (int r0 = 0; r0 < sh.CS; r0 += 4) {
      uint4 v[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int r = r0 + i;
        const int t = t0 + (r >> (sh.lcw + sh.lch)), h = h0 + ((r >> sh.lcw) & (sh.ch - 1)), w = w0 + (r & (sh.cw - 1));
        const bool ok = live && r < sh.CS && t < sh.T && h < sh.H && w < sh.W;
        const int tok = (t * sh.H + h) * sh.W + w;
        v[i] = ok ? __ldg(reinterpret_cast<const uint4*>(base + (size_t)tok * SPADE_D) + l16) : make_uint4(0, 0, 0, 0);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float x[8];
        bf16x8_to_float(v[i], x);
        float ss = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) ss = fmaf(x[c], x[c], ss);
#pragma unroll
        for (int o = 8; o >= 1; o >>= 1) ss += __shfl_xor_sync(FULL, ss, o);
        const float rn = ss > 0.f ? rsqrtf(ss) : 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) { an[c] = fmaf(x[c], rn, an[c]); ar[c] += x[c]; }
      }
    }
    if (live) {
      float* out = cells + (((size_t)ht * sh.NCELL + cell) * 2) * SPADE_D + l16 * 8;
      reinterpret_cast<float4*>(out)[0] = make_float4(an[0], an[1], an[2], an[3]);
      reinterpret_cast<float4*>(out)[1] = make_float4(an[4], an[5], an[6], an[7]);
      reinterpret_cast<float4*>(out + SPADE_D)[0] = make_float4(ar[0], ar[1], ar[2], ar[3]);
      reinterpret_cast<float4*>(out + SPADE_D)[1] = make_float4(ar[4], ar[5], ar[6], ar[7]);
    }
  }
}

// Block pass: one warp per (head, tensor, candidate, block) adds up the block's cells.
//   SICS(block) = || sum q_hat ||^2 (Eq. 4 / Algorithm 1), mean summary = sum q / n (Sec. 3.1).
// Text blocks (not part of the 3-D grid) are reduced from their token rows directly.
__global__ void __launch_bounds__(WARPS_PER_CTA * 32)
k_blocks(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K, const __grid_constant__ Shape sh,
         const __grid_constant__ GeoPack gp, StaticTables st, WsTables ws) {
  const int lane = threadIdx.x & 31;
  const long gw = (long)blockIdx.x * WARPS_PER_CTA + (threadIdx.x >> 5);
  const long nw = (long)gridDim.x * WARPS_PER_CTA;
  int per_ht = 0;
  for (int c = 0; c < sh.C; ++c) per_ht += gp.g[c].NB;
  const long total = (long)sh.BH * 2 * per_ht;
  for (long u = gw; u < total; u += nw) {
    const int ht = (int)(u / per_ht);
    int rem = (int)(u % per_ht), c = 0;
    while (rem >= gp.g[c].NB) { rem -= gp.g[c].NB; ++c; }
    const CandGeo& g = gp.g[c];
    const int b = rem, bh = ht >> 1, tensor = ht & 1;
    const int nval = __ldg(st.nvalid + g.tab_off + b);
    const float inv = nval > 0 ? 1.f / (float)nval : 0.f;
    float* mean = ws.csum + ((((size_t)ht * sh.C + c) * sh.NBmax) + b) * SPADE_D;
    if (b >= g.NBv) {
      const __nv_bfloat16* base = (tensor ? K : Q) + (size_t)bh * sh.N * SPADE_D;
      float acc[8];
      reduce_block<false>(base, g, st.rowoff + c * 128, b, false, sh, lane, acc);
      if (lane < 16) {
        reinterpret_cast<float4*>(mean + lane * 8)[0] = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
        reinterpret_cast<float4*>(mean + lane * 8)[1] = make_float4(acc[4] * inv, acc[5] * inv, acc[6] * inv, acc[7] * inv);
      }
      continue;
    }
    const int iw = b % g.nbw, ih = (b / g.nbw) % g.nbh, it = b / (g.nbw * g.nbh);
    const int c_t0 = it * (g.bt / sh.ct), c_h0 = ih * (g.bh / sh.ch), c_w0 = iw * (g.bw / sh.cw);
    const int n_t = g.bt / sh.ct, n_h = g.bh / sh.ch, n_w = g.bw / sh.cw;
    const float* cell0 = ws.cells + (size_t)ht * sh.NCELL * 2 * SPADE_D + lane * 4;
    float4 an = make_float4(0, 0, 0, 0), ar = make_float4(0, 0, 0, 0);
    for (int dt = 0; dt < n_t; ++dt) {
      if (c_t0 + dt >= sh.nct) break;
      for (int dh = 0; dh < n_h; ++dh) {
        if (c_h0 + dh >= sh.nch) break;
        const int rowc = ((c_t0 + dt) * sh.nch + c_h0 + dh) * sh.ncw + c_w0;
        for (int dw = 0; dw < n_w && c_w0 + dw < sh.ncw; ++dw) {
          if (!SPADE_CHECK(rowc + dw < sh.NCELL, ws.status, 501, rowc + dw)) continue;
          const float* p = cell0 + (size_t)(rowc + dw) * 2 * SPADE_D;
          const float4 a = *reinterpret_cast<const float4*>(p);
          const float4 r = *reinterpret_cast<const float4*>(p + SPADE_D);
          an.x += a.x; an.y += a.y; an.z += a.z; an.w += a.w;
          ar.x += r.x; ar.y += r.y; ar.z += r.z; ar.w += r.w;
        }
      }
    }
    float s = an.x * an.x + an.y * an.y + an.z * an.z + an.w * an.w;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(FULL, s, o);
    if (lane == 0) ws.sics[(((size_t)bh * sh.C + c) * 2 + tensor) * sh.NBvmax + b] = s;
    *reinterpret_cast<float4*>(mean + lane * 4) = make_float4(ar.x * inv, ar.y * inv, ar.z * inv, ar.w * inv);
  }
}

// Per-head tables of the static part of the mask (Sec. 3.3): KV blocks every query block keeps (mean
// pairwise cosine of K below the threshold, or holding one of the first `sink` tokens) and query blocks
// that keep everything (mean pairwise cosine of Q below the threshold).
__global__ void __launch_bounds__(256)
k_static(const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp, StaticTables st, WsTables ws) {
  const int bh = blockIdx.y;
  const int c = ws.scheme[bh];
  const CandGeo& g = gp.g[c];
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < g.NBv; j += gridDim.x * blockDim.x) {
    const float n = (float)__ldg(st.nvalid + g.tab_off + j);
    const float nn = n * n;
    bool col = false, row = false;
    if (sh.intra_thr > 0.f) {
      col = ws.sics[(((size_t)bh * sh.C + c) * 2 + 1) * sh.NBvmax + j] < sh.intra_thr * nn;
      row = ws.sics[(((size_t)bh * sh.C + c) * 2 + 0) * sh.NBvmax + j] < sh.intra_thr * nn;
    }
    const int iw = j % g.nbw, ih = (j / g.nbw) % g.nbh, it = j / (g.nbw * g.nbh);
    const int origin = ((it * g.bt) * sh.H + ih * g.bh) * sh.W + iw * g.bw;      // the block's smallest token index
    col = col || origin < sh.sink;
    ws.colkeep[(size_t)bh * sh.NBmax + j] = col ? 1 : 0;
    ws.rowfull[(size_t)bh * sh.NBmax + j] = row ? 1 : 0;
  }
}

// Summaries of the chosen scheme, picked out of the all-candidate table of the block pass.
__global__ void __launch_bounds__(256)
k_gather(const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp, WsTables ws, const int split) {
  const unsigned total = (unsigned)sh.BH * 2u * (unsigned)sh.NBmax * 32u;       // float4 elements: at most 4096 * 2 * 2048 * 32 = 2^29
  for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    const int c4 = (int)(i & 31u);
    const unsigned rowi = i >> 5;
    const int b = (int)(rowi % (unsigned)sh.NBmax), ht = (int)(rowi / (unsigned)sh.NBmax);
    const int bh = ht >> 1, tensor = ht & 1;
    const int c = ws.scheme[bh];
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (b < gp.g[c].NB) {
      v = reinterpret_cast<const float4*>(ws.csum + ((((size_t)ht * sh.C + c) * sh.NBmax) + b) * SPADE_D)[c4];
      reinterpret_cast<float4*>((tensor ? ws.ksum : ws.qsum) + ((size_t)bh * sh.NBmax + b) * SPADE_D)[c4] = v;
    }
    if (split && tensor) {
      // the estimator's operand B as k_split_k writes it: K' of the video blocks as TF32 value and remainder, zero rows behind them
      if (b >= gp.g[c].NBv) v = make_float4(0.f, 0.f, 0.f, 0.f);
      float4 h, l;
      h.x = __uint_as_float((__float_as_uint(v.x) + 0x1000u) & 0xffffe000u); l.x = v.x - h.x;
      h.y = __uint_as_float((__float_as_uint(v.y) + 0x1000u) & 0xffffe000u); l.y = v.y - h.y;
      h.z = __uint_as_float((__float_as_uint(v.z) + 0x1000u) & 0xffffe000u); l.z = v.z - h.z;
      h.w = __uint_as_float((__float_as_uint(v.w) + 0x1000u) & 0xffffe000u); l.w = v.w - h.w;
      reinterpret_cast<float4*>(ws.ksplit + (((size_t)bh * 2 + 0) * sh.NBmax + b) * SPADE_D)[c4] = h;
      reinterpret_cast<float4*>(ws.ksplit + (((size_t)bh * 2 + 1) * sh.NBmax + b) * SPADE_D)[c4] = l;
    }
  }
}

// Max/min estimator of Fig. 4a on the tensor cores: S = q~ k_mid^T + |q~| k_half^T is a contraction over 256
// channels.  The channel-major planes k_minmax leaves (what the SIMT estimator kernel reads) are turned into the
// row-major operands of k_scores: q~ rows, and k_mid / k_half rows split into nearest TF32 value and remainder.
// A CTA transposes a 32-channel x 32-block patch of one plane through shared memory.
__global__ void __launch_bounds__(256)
k_dsa_rows(const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp, WsTables ws) {
  __shared__ float tile[32][33];
  const int bh = blockIdx.z / 3, which = blockIdx.z % 3;            // 0: q~, 1: k_mid, 2: k_half
  const int nbv = gp.g[ws.scheme[bh]].NBv;
  const int b0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
  if (b0 >= ((nbv + 63) & ~63)) return;
  const size_t plane = (size_t)sh.BH * SPADE_D * sh.ld_scores;
  const float* src = ws.mm + (size_t)(which == 0 ? 0 : which + 1) * plane + ((size_t)bh * SPADE_D + c0) * sh.ld_scores + b0;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
#pragma unroll
  for (int r = ty; r < 32; r += 8) tile[r][tx] = b0 + tx < sh.ld_scores ? src[(size_t)r * sh.ld_scores + tx] : 0.f;
  __syncthreads();
#pragma unroll
  for (int r = ty; r < 32; r += 8) {
    const int b = b0 + r;
    if (b >= sh.NBmax) continue;
    const float v = b < nbv ? tile[tx][r] : 0.f;
    if (which == 0) {
      ws.qmid[((size_t)bh * sh.NBmax + b) * SPADE_D + c0 + tx] = v;
    } else {
      const float h = __uint_as_float((__float_as_uint(v) + 0x1000u) & 0xffffe000u);
      float* dst = ws.kdsa + (((size_t)bh * 4 + 2 * (which - 1)) * sh.NBmax + b) * SPADE_D + c0 + tx;
      dst[0] = h;
      dst[(size_t)sh.NBmax * SPADE_D] = v - h;
    }
  }
}

// K' of the chosen scheme, split for the tensor-core estimator (scores.cu): hi = the nearest TF32 value,
// lo = the exact remainder, as two planes the estimator's TMA copies read directly.
__global__ void __launch_bounds__(256)
k_split_k(const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp, WsTables ws) {
  const long total = (long)sh.BH * sh.NBmax * 32;          // float4 elements
  for (long i = (long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
    const int c4 = (int)(i & 31);
    const long rowi = i >> 5;
    const int b = (int)(rowi % sh.NBmax), bh = (int)(rowi / sh.NBmax);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (b < gp.g[ws.scheme[bh]].NBv) v = reinterpret_cast<const float4*>(ws.ksum + ((size_t)bh * sh.NBmax + b) * SPADE_D)[c4];
    float4 h, l;
    h.x = __uint_as_float((__float_as_uint(v.x) + 0x1000u) & 0xffffe000u); l.x = v.x - h.x;
    h.y = __uint_as_float((__float_as_uint(v.y) + 0x1000u) & 0xffffe000u); l.y = v.y - h.y;
    h.z = __uint_as_float((__float_as_uint(v.z) + 0x1000u) & 0xffffe000u); l.z = v.z - h.z;
    h.w = __uint_as_float((__float_as_uint(v.w) + 0x1000u) & 0xffffe000u); l.w = v.w - h.w;
    reinterpret_cast<float4*>(ws.ksplit + (((size_t)bh * 2 + 0) * sh.NBmax + b) * SPADE_D)[c4] = h;
    reinterpret_cast<float4*>(ws.ksplit + (((size_t)bh * 2 + 1) * sh.NBmax + b) * SPADE_D)[c4] = l;
  }
}

// One CTA per head: AS(X|c) = sum_b SICS (Eq. 3; fixed lane-strided order, one warp per (candidate, tensor)),
// then warp 0: normalised score, argmax (ties -> lowest candidate) unless forced, and the head's keep count /
// threshold.
__device__ __forceinline__ void groups_body(const Shape& sh, const GeoPack& gp, const WsTables& ws, int mode);
__device__ __forceinline__ bool last_cta_done(uint32_t* status, int word);

__global__ void __launch_bounds__(256)
k_choose(const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp, StaticTables st, WsTables ws,
         const __grid_constant__ ForcedPack fp, int have_sics) {
  __shared__ float as_sm[SPADE_MAX_CANDS * 2];
  const int bh = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (have_sics) {
    for (int ct = warp; ct < sh.C * 2; ct += 8) {
      const int c = ct >> 1, t = ct & 1;
      const float* p = ws.sics + (((size_t)bh * sh.C + c) * 2 + t) * sh.NBvmax;
      float s = 0.f;
      for (int b = lane; b < gp.g[c].NBv; b += 32) s += p[b];
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(FULL, s, o);
      if (lane == 0) as_sm[ct] = s;
    }
  }
  __syncthreads();
  if (warp == 0) {
  int best = 0;
  if (have_sics) {
    float best_score = -1e30f;
    for (int c = 0; c < sh.C; ++c) {
      const float a0 = as_sm[2 * c], a1 = as_sm[2 * c + 1];
      const float sc = (a0 + a1) * gp.g[c].inv_z;
      if (lane == 0) {
        ws.as[((size_t)bh * sh.C + c) * 2 + 0] = a0;
        ws.as[((size_t)bh * sh.C + c) * 2 + 1] = a1;
        ws.score[(size_t)bh * sh.C + c] = sc;
      }
      if (sc > best_score) { best_score = sc; best = c; }
    }
  }
  if (fp.on) best = (int)((fp.w[bh >> 3] >> ((bh & 7) * 4)) & 15u);
  if (lane == 0) {
    ws.scheme[bh] = best;
    const int nkb = gp.g[best].NBv;
    const float v = st.budget[bh];
    int keep = 0;
    float p = 0.f;
    if (sh.mode == 0) {
      keep = (int)v;
    } else if (sh.mode == 2) {
      keep = (int)ceil((1.0 - (double)v) * (double)nkb - 1e-9);
    } else if (sh.mode == 1) {
      p = v;
    }                                           // mode 3: k_groups sets the keep count (needs all heads' scores)
    if (sh.mode != 1) keep = keep < 1 ? 1 : (keep > nkb ? nkb : keep);
    ws.keep[bh] = keep;
    ws.pthr[bh] = p;
  }
  }
  // the last CTA to get here orders the heads for the attention kernel (what k_groups does in a launch of its own)
  if (last_cta_done(ws.status, 9)) groups_body(sh, gp, ws, 0);
}

// Order in which the attention kernel takes the heads, heads per scheme, and the prefixes of attention
// work items (all query tiles, and the text query tiles alone: those attend every block and are handed
// out first).
// mode 0 (plan stage, lists unknown): heads grouped by scheme (Sec. 3.3), every cell's pairing axis reset to w.
// mode 1 (after the index search): heads by decreasing list length per query tile, so that the longest
// work items start first and the last ones are short (k_pair_axis has set the cells' axes).
// Runs in ONE CTA (every thread of it): k_groups, or the last CTA to finish of k_choose (mode 0) / k_pair_axis (mode 1).
__device__ __forceinline__ void groups_body(const Shape& sh, const GeoPack& gp, const WsTables& ws, int mode) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nthreads = blockDim.x, nwarps = blockDim.x >> 5;
  if (tid == 0 && mode == 0 && sh.mode == 3) {
    // example policy function: keep fraction negatively correlated with the Selected Aggregation Score
    double abar = 0.0;
    for (int bh = 0; bh < sh.BH; ++bh) abar += (double)__ldcg(ws.score + (size_t)bh * sh.C + __ldcg(ws.scheme + bh));
    abar /= (double)sh.BH;
    for (int bh = 0; bh < sh.BH; ++bh) {
      const int nkb = gp.g[__ldcg(ws.scheme + bh)].NBv;
      const double a = (double)__ldcg(ws.score + (size_t)bh * sh.C + __ldcg(ws.scheme + bh));
      double f = (1.0 - (double)sh.value) * (1.0 - (double)sh.gain * (a - abar) / abar);
      f = f < 1.0 / nkb ? 1.0 / nkb : (f > 1.0 ? 1.0 : f);
      int k = (int)ceil(f * (double)nkb - 1e-9);
      ws.keep[bh] = k < 1 ? 1 : (k > nkb ? nkb : k);
    }
  }
  if (tid < SPADE_MAX_CANDS) ws.group_count[tid] = 0;
  // sort key per head (larger = earlier) and its pairing axis
  for (int bh = warp; bh < sh.BH; bh += nwarps) {
    const int c = __ldcg(ws.scheme + bh);
    const CandGeo& g = gp.g[c];
    float key = -(float)c;
    if (mode == 1) {
      const int sum = __ldcg(ws.pair_union + bh * 4 + 3);       // listed blocks over the head's video query rows (added up by the index search)
      // 64-key units per query tile, roughly: two per listed 128-token block; the merged list of two
      // 64-token query blocks is somewhat shorter than both lists together
      key = (float)sum / (float)g.NBv * (g.pair ? 1.7f : 2.0f);
    }
    if (mode == 0 && g.pair)
      for (int i = lane; i < sh.cell_ld; i += 32) ws.cell_axis[(size_t)bh * sh.cell_ld + i] = 2;
    if (lane == 0) ws.head_work[bh] = key;
  }
  __syncthreads();
  for (int i = tid; i < sh.BH; i += nthreads) {                  // rank = heads that come before head i
    const float ki = ws.head_work[i];
    int rank = 0;
    for (int j = 0; j < sh.BH; ++j) {
      const float kj = ws.head_work[j];
      rank += (kj > ki || (kj == ki && j < i)) ? 1 : 0;
    }
    const int c = __ldcg(ws.scheme + i);
    ws.head_order[rank] = i;
    ws.item_start[rank + 1] = head_tiles(gp.g[c]);      // counts; scanned below
    ws.text_start[rank + 1] = gp.g[c].pair ? gp.g[c].ttiles : gp.g[c].NBt;
    atomicAdd(&ws.group_count[c], 1);
  }
  __syncthreads();
  if (warp == 0) {                                           // inclusive scan of the two count arrays
    int carry_i = 0, carry_t = 0;
    if (lane == 0) { ws.item_start[0] = 0; ws.text_start[0] = 0; }
    for (int base = 0; base < sh.BH; base += 32) {
      const int pos = base + lane;
      int vi = pos < sh.BH ? ws.item_start[pos + 1] : 0, vt = pos < sh.BH ? ws.text_start[pos + 1] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int xi = __shfl_up_sync(FULL, vi, o), xt = __shfl_up_sync(FULL, vt, o);
        if (lane >= o) { vi += xi; vt += xt; }
      }
      vi += carry_i; vt += carry_t;
      if (pos < sh.BH) { ws.item_start[pos + 1] = vi; ws.text_start[pos + 1] = vt; }
      carry_i = __shfl_sync(FULL, vi, 31); carry_t = __shfl_sync(FULL, vt, 31);
    }
  }
  // the per-head totals have been used (mode 1) or are not measured yet (mode 0): the index search and k_pair_axis add into zeros
  __syncthreads();
  for (int i = tid; i < sh.BH * 4; i += nthreads) ws.pair_union[i] = 0;
}

__global__ void __launch_bounds__(1024) k_groups(const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp, WsTables ws, int mode) {
  groups_body(sh, gp, ws, mode);
}

// True in every thread of the CTA that finishes last (a ticket in status word `word`, which the last CTA leaves at zero).
// What the other CTAs wrote before their ticket is visible to it.
__device__ __forceinline__ bool last_cta_done(uint32_t* status, int word) {
  __shared__ int last_sm;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned ticket = atomicAdd(status + word, 1u);
    last_sm = ticket == gridDim.x - 1 ? 1 : 0;
    if (last_sm) status[word] = 0u;
  }
  __syncthreads();
  if (last_sm) __threadfence();
  return last_sm != 0;
}

// Pairing axis of every cell of a head's block grid (64-token schemes): one warp per (head, cell) adds up, for each of the
// three axes, the merged-list lengths |L_i u L_j| of the cell's tiles (|L_i| of a lone block) -- popcounts over the bitmaps
// the index search leaves next to the lists; the text blocks every list ends with do not change the ranking -- and keeps
// the axis with the smallest total (ties -> w, then h, then t).
__global__ void __launch_bounds__(WARPS_PER_CTA * 32)
k_pair_axis(const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp, StaticTables st, WsTables ws) {
  const int lane = threadIdx.x & 31;
  const int gw = blockIdx.x * WARPS_PER_CTA + (threadIdx.x >> 5);
  const int nw = gridDim.x * WARPS_PER_CTA;
  const int total = sh.BH * sh.cell_ld;               // at most 4096 * 2048
  for (int u = gw; u < total; u += nw) {
    const int cell = u % sh.cell_ld, bh = u / sh.cell_ld;
    const CandGeo& g = gp.g[ws.scheme[bh]];
    if (!g.pair || cell >= g.ncell) continue;
    const int t0 = __ldg(st.cell_tile0 + g.pc_off + cell), t1 = __ldg(st.cell_tile0 + g.pc_off + cell + 1);
    const uint32_t* rows = ws.rowbits + (size_t)bh * sh.NBvmax * sh.bits_ld;
    const int words = (g.NBv + 31) >> 5;
    int cost[3] = {0, 0, 0};
    for (int t = t0; t < t1; ++t) {
#pragma unroll
      for (int a = 0; a < 3; ++a) {
        const uint32_t e = __ldg(st.pair_tab + (size_t)(g.pt_off + t) * 3 + a);
        const uint32_t qb0 = e & 0xffffu, qb1 = (e >> 16) == 0xffffu ? qb0 : (e >> 16);
        if (!SPADE_CHECK(qb0 < (uint32_t)g.NBv && qb1 < (uint32_t)g.NBv, ws.status, 501, (int)e)) continue;
        const uint32_t* Bi = rows + (size_t)qb0 * sh.bits_ld;
        const uint32_t* Bj = rows + (size_t)qb1 * sh.bits_ld;
        for (int wd = lane; wd < words; wd += 32) cost[a] += __popc(Bi[wd] | Bj[wd]);
      }
    }
#pragma unroll
    for (int a = 0; a < 3; ++a)
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) cost[a] += __shfl_xor_sync(FULL, cost[a], o);
    if (lane == 0) {
      int axis = 2;
      if (cost[1] < cost[2]) axis = 1;
      if (cost[0] < cost[axis]) axis = 0;
      ws.cell_axis[(size_t)bh * sh.cell_ld + cell] = (uint8_t)axis;
    }
  }
  // the last CTA to get here orders the heads by list length
  if (last_cta_done(ws.status, 10)) groups_body(sh, gp, ws, 1);
}

// Mean summaries of the chosen scheme: one warp per (head, tensor, block).
__global__ void __launch_bounds__(WARPS_PER_CTA * 32)
k_summarize(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K,
            const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp,
            StaticTables st, WsTables ws) {
  const int lane = threadIdx.x & 31;
  const int gw = blockIdx.x * WARPS_PER_CTA + (threadIdx.x >> 5);
  const int nw = gridDim.x * WARPS_PER_CTA;
  const long total = (long)sh.BH * 2 * sh.NBmax;
  for (long u = gw; u < total; u += nw) {
    const int ht = (int)(u / sh.NBmax), b = (int)(u % sh.NBmax);
    const int bh = ht >> 1, tensor = ht & 1;
    const int c = ws.scheme[bh];
    const CandGeo& g = gp.g[c];
    if (b >= g.NB) continue;
    const int nval = __ldg(st.nvalid + g.tab_off + b);
    const __nv_bfloat16* base = (tensor ? K : Q) + (size_t)bh * sh.N * SPADE_D;
    float acc[8];
    reduce_block<false>(base, g, st.rowoff + c * 128, b, nval == g.BS, sh, lane, acc);
    if (lane < 16) {
      const float inv = nval > 0 ? 1.f / (float)nval : 0.f;
      float* out = (tensor ? ws.ksum : ws.qsum) + ((size_t)bh * sh.NBmax + b) * SPADE_D + lane * 8;
      reinterpret_cast<float4*>(out)[0] = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
      reinterpret_cast<float4*>(out)[1] = make_float4(acc[4] * inv, acc[5] * inv, acc[6] * inv, acc[7] * inv);
    }
  }
}

// Channel-wise max and min summaries of the chosen scheme's video blocks (Sec. 3.1, Summarizer
// Expression), stored the way the estimator kernel consumes them: channel-major planes
//   mm[plane][head][channel][block],  row length ld_scores,
//   plane 0 = q_max (estimator 2) or the midpoint (q_max + q_min) / 2 (estimator 1), plane 1 = q_min,
//   plane 2 = k_mid = (k_max + k_min) / 2, plane 3 = k_half = (k_max - k_min) / 2.
// A CTA takes eight consecutive blocks of one (head, tensor), one warp per block (each half-warp reads
// one token row per step, lane l16 holds channels 8*l16 .. 8*l16+7), and writes 32-byte runs through
// shared memory.  Blocks past the scheme's last video block get zeros.
constexpr int MMS_T_PAD = 64;       // tile edge of k_scores_minmax: blocks up to the next multiple are zero-filled
__global__ void __launch_bounds__(WARPS_PER_CTA * 32)
k_minmax(const __nv_bfloat16* __restrict__ Q, const __nv_bfloat16* __restrict__ K, const __grid_constant__ Shape sh,
         const __grid_constant__ GeoPack gp, StaticTables st, WsTables ws) {
  __shared__ __align__(16) float stage[2][SPADE_D][WARPS_PER_CTA];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, hw = lane >> 4, l16 = lane & 15;
  const int groups = sh.ld_scores / WARPS_PER_CTA;
  const long total = (long)sh.BH * 2 * groups;
  const float INF = __int_as_float(0x7f800000);
  const size_t plane = (size_t)sh.BH * SPADE_D * sh.ld_scores;
  for (long u = blockIdx.x; u < total; u += gridDim.x) {
    const int ht = (int)(u / groups), b0 = (int)(u % groups) * WARPS_PER_CTA, b = b0 + warp;
    const int bh = ht >> 1, tensor = ht & 1;
    const int c = ws.scheme[bh];
    const CandGeo& g = gp.g[c];
    if (b0 >= ((g.NBv + MMS_T_PAD - 1) & ~(MMS_T_PAD - 1))) continue;   // past the last score tile of this head
    float hi[8], lo[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) { hi[i] = 0.f; lo[i] = 0.f; }
    if (b < g.NBv) {
#pragma unroll
      for (int i = 0; i < 8; ++i) { hi[i] = -INF; lo[i] = INF; }
      const bool full = __ldg(st.nvalid + g.tab_off + b) == g.BS;
      const __nv_bfloat16* base = (tensor ? K : Q) + (size_t)bh * sh.N * SPADE_D;
      const uint32_t* rowoff = st.rowoff + c * 128;
      const int iw = b % g.nbw, ih = (b / g.nbw) % g.nbh, it = b / (g.nbw * g.nbh);
      const int t0 = it * g.bt, h0 = ih * g.bh, w0 = iw * g.bw;
      for (int r0 = 0; r0 < g.BS; r0 += 8) {
        uint4 v[4];
        bool ok[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t code = __ldg(rowoff + r0 + 2 * i + hw);
          const int t = t0 + (int)(code >> 20), h = h0 + (int)((code >> 10) & 1023), w = w0 + (int)(code & 1023);
          ok[i] = full || (t < sh.T && h < sh.H && w < sh.W);
          const int tok = (t * sh.H + h) * sh.W + w;
          v[i] = ok[i] ? __ldg(reinterpret_cast<const uint4*>(base + (size_t)tok * SPADE_D) + l16) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          if (!ok[i]) continue;
          float x[8];
          bf16x8_to_float(v[i], x);
#pragma unroll
          for (int k = 0; k < 8; ++k) { hi[k] = fmaxf(hi[k], x[k]); lo[k] = fminf(lo[k], x[k]); }
        }
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        hi[k] = fmaxf(hi[k], __shfl_xor_sync(FULL, hi[k], 16));
        lo[k] = fminf(lo[k], __shfl_xor_sync(FULL, lo[k], 16));
      }
    }
    if (hw == 0) {
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        float p0, p1;
        if (tensor) { p0 = 0.5f * (hi[k] + lo[k]); p1 = 0.5f * (hi[k] - lo[k]); }
        else { p0 = sh.estimator == 1 ? 0.5f * (hi[k] + lo[k]) : hi[k]; p1 = lo[k]; }
        stage[0][l16 * 8 + k][warp] = p0;
        stage[1][l16 * 8 + k][warp] = p1;
      }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 2 * SPADE_D * 2; i += WARPS_PER_CTA * 32) {
      const int half = i & 1, ch = (i >> 1) & (SPADE_D - 1), pl = i >> 8;
      const float4 v = *reinterpret_cast<const float4*>(&stage[pl][ch][half * 4]);
      float* dst = ws.mm + (size_t)(2 * tensor + pl) * plane + ((size_t)bh * SPADE_D + ch) * sh.ld_scores + b0 + half * 4;
      *reinterpret_cast<float4*>(dst) = v;
    }
    __syncthreads();
  }
}

// Inter-block estimators on the max / min summaries (Sec. 3.1, Fig. 4a / 4b).  The block importance is
// the dot product of two vectors picked channel by channel from the summaries so that every channel
// contributes its largest product:
//   VARIANT 1: q~ = (q_max + q_min) / 2,  S[i,j] = sum_c max(q~_c kmax_jc, q~_c kmin_jc) / sqrt(d)
//   VARIANT 2: S[i,j] = sum_c max over {qmax_ic, qmin_ic} x {kmax_jc, kmin_jc} of the product / sqrt(d)
// computed as max(q kmax, q kmin) = q k_mid + |q| k_half.  The per-channel max keeps VARIANT 2 off the
// tensor cores.  A CTA computes a 128 x 64 tile of S, a thread an 8 x 4 patch held as row pairs for the
// packed f32x2 pipe; the channel-major summary planes arrive 16 channels at a time through a two-deep
// cp.async pipeline.  A ragged last row tile reads past the q row of a channel into memory that still
// belongs to the table (the k planes follow the q planes); those rows are never stored.
constexpr int MMS_TR = 128, MMS_TC = MMS_T_PAD, MMS_CH = 16;
constexpr int MMS_STAGE = (2 * MMS_TR + 2 * MMS_TC) * MMS_CH;      // floats per pipeline stage
constexpr int MMS_SMEM = 2 * MMS_STAGE * (int)sizeof(float);

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
               : "memory");
}
__device__ __forceinline__ uint64_t pk2(float a, float b) { uint64_t r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b)); return r; }
__device__ __forceinline__ void upk2(uint64_t v, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t max2(uint64_t a, uint64_t b) {
  float a0, a1, b0, b1;
  upk2(a, a0, a1); upk2(b, b0, b1);
  return pk2(fmaxf(a0, b0), fmaxf(a1, b1));
}

template <int VARIANT>
__global__ void __launch_bounds__(256)
k_scores_minmax(const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp, WsTables ws, float scale) {
  extern __shared__ __align__(16) float mms[];      // [2 stages]{q0 [CH][TR], q1 [CH][TR], kmid [CH][TC], khalf [CH][TC]}
  const int bh = blockIdx.z;
  const CandGeo& g = gp.g[ws.scheme[bh]];
  const int n = g.NBv;
  const int row0 = blockIdx.y * MMS_TR, col0 = blockIdx.x * MMS_TC;
  if (row0 >= n || col0 >= n) return;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const size_t plane = (size_t)sh.BH * SPADE_D * sh.ld_scores;
  const float* head = ws.mm + (size_t)bh * SPADE_D * sh.ld_scores;
  auto issue = [&](int chunk) {
    float* dst = mms + (size_t)(chunk & 1) * MMS_STAGE;
    const size_t ch_off = (size_t)(chunk * MMS_CH) * sh.ld_scores;
#pragma unroll
    for (int t = 0; t < 2; ++t) {                   // q planes: 32 segments of 16 bytes per channel row
      if (VARIANT == 1 && t == 1) continue;
      const float* src = head + t * plane + ch_off + row0;
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int e = tid + i * 256, ch = e >> 5, seg = e & 31;
        cp_async16(dst + (t * MMS_CH + ch) * MMS_TR + seg * 4, src + (size_t)ch * sh.ld_scores + seg * 4);
      }
    }
#pragma unroll
    for (int t = 0; t < 2; ++t) {                   // k planes: 16 segments per channel row
      const float* src = head + (2 + t) * plane + ch_off + col0;
      const int ch = tid >> 4, seg = tid & 15;
      cp_async16(dst + 2 * MMS_CH * MMS_TR + (t * MMS_CH + ch) * MMS_TC + seg * 4, src + (size_t)ch * sh.ld_scores + seg * 4);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  uint64_t acc[4][4];                               // acc[ip][j] = rows (2 ip, 2 ip + 1) of column j
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0ull;
  issue(0);
  for (int chunk = 0; chunk < SPADE_D / MMS_CH; ++chunk) {
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();                     // this chunk has landed; everyone is done with the other stage
    if (chunk + 1 < SPADE_D / MMS_CH) issue(chunk + 1);
    const float* sq = mms + (size_t)(chunk & 1) * MMS_STAGE;
    const float* sk = sq + 2 * MMS_CH * MMS_TR;
#pragma unroll 2
    for (int ch = 0; ch < MMS_CH; ++ch) {
      const ulonglong2 qa = *reinterpret_cast<const ulonglong2*>(sq + ch * MMS_TR + ty * 8);
      const ulonglong2 qb = *reinterpret_cast<const ulonglong2*>(sq + ch * MMS_TR + ty * 8 + 4);
      const float4 km = *reinterpret_cast<const float4*>(sk + ch * MMS_TC + tx * 4);
      const float4 kh = *reinterpret_cast<const float4*>(sk + (MMS_CH + ch) * MMS_TC + tx * 4);
      const uint64_t q0[4] = {qa.x, qa.y, qb.x, qb.y};
      const uint64_t kmid[4] = {pk2(km.x, km.x), pk2(km.y, km.y), pk2(km.z, km.z), pk2(km.w, km.w)};
      const uint64_t khalf[4] = {pk2(kh.x, kh.x), pk2(kh.y, kh.y), pk2(kh.z, kh.z), pk2(kh.w, kh.w)};
      const uint64_t ABS = 0x7fffffff7fffffffull;
      if (VARIANT == 1) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint64_t qabs = q0[i] & ABS;
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = fma2(q0[i], kmid[j], fma2(qabs, khalf[j], acc[i][j]));
        }
      } else {
        const ulonglong2 qc = *reinterpret_cast<const ulonglong2*>(sq + (MMS_CH + ch) * MMS_TR + ty * 8);
        const ulonglong2 qd = *reinterpret_cast<const ulonglong2*>(sq + (MMS_CH + ch) * MMS_TR + ty * 8 + 4);
        const uint64_t q1[4] = {qc.x, qc.y, qd.x, qd.y};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint64_t a0 = q0[i] & ABS, a1 = q1[i] & ABS;
#pragma unroll
          for (int j = 0; j < 4; ++j)
            acc[i][j] = add2(acc[i][j], max2(fma2(q0[i], kmid[j], mul2(a0, khalf[j])), fma2(q1[i], kmid[j], mul2(a1, khalf[j]))));
        }
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float lo[4], hi[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) upk2(acc[i][j], lo[j], hi[j]);
    const int row = row0 + ty * 8 + 2 * i;
    float* dst = ws.scores + ((size_t)bh * sh.NBvmax + row) * sh.ld_scores + col0 + tx * 4;
    if (row < n) *reinterpret_cast<float4*>(dst) = make_float4(lo[0] * scale, lo[1] * scale, lo[2] * scale, lo[3] * scale);
    if (row + 1 < n)
      *reinterpret_cast<float4*>(dst + sh.ld_scores) = make_float4(hi[0] * scale, hi[1] * scale, hi[2] * scale, hi[3] * scale);
  }
}

// ------------------------------------------------------------------------------------------------
// Estimator + index search.
constexpr int SEL_R = 8;        // query-block rows per CTA; one warp per row
// Scan a 256-bin histogram from the top bin down; find the first NON-EMPTY bin at which
// `above + cumulative >= need`.  Lane l owns bins 255-8l .. 248-8l.  Returns the bin (or -1 when the
// total never reaches `need`) and adds the weight of the bins above it to `above`.  All lanes get the
// same result.  The crossing is only ever placed in a bin that holds something: an empty bin would
// leave the next pass without a single value.
template <class T>
__device__ __forceinline__ int find_bin(const T* hist, T need, T& above, int lane) {
  T v[8], tot = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) { v[i] = hist[255 - (8 * lane + i)]; tot += v[i]; }
  T incl = tot;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    T n = __shfl_up_sync(FULL, incl, o);
    if (lane >= o) incl += n;
  }
  const T excl = incl - tot;
  const unsigned hit = __ballot_sync(FULL, tot > 0 && above + incl >= need);
  int bin = -1;
  T add = 0;
  if (hit) {
    const int src = __ffs(hit) - 1;
    int my_bin = -1;
    T run = excl;
    if (lane == src) {
      int last = -1;                       // last non-empty bin of the lane seen so far
      T run_last = excl;                   // weight above it
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (my_bin < 0 && v[i] > 0) {
          if (above + run + v[i] >= need) { my_bin = 255 - (8 * lane + i); }
          else { last = 255 - (8 * lane + i); run_last = run; run += v[i]; }
        }
      }
      if (my_bin < 0) { my_bin = last; run = run_last; }     // rounding: the lane's last non-empty bin (tot > 0: there is one)
    }
    bin = __shfl_sync(FULL, my_bin, src);
    add = __shfl_sync(FULL, run, src);
  }
  above += add;
  return bin;
}

// Index search (Sec. 3.1, 3.3) with the row held in registers (rows of up to NV * 128 blocks; a plan takes at most 2048).  The scores are read once
// into NV float4 per lane.  The k-th largest value is found by histogram passes that are LINEAR in the value
// between the smallest and largest score still in the race (250 bins), so that a row of roughly bell-shaped
// scores leaves a dozen values in the bin the cut falls in; up to 64 of them are then ranked directly (every
// lane counts how many are larger than its own).  A bin with more than 64 is split again between its own
// minimum and maximum.  Binning only decides which values are ranked: the kept set is the exact top-k of the
// fp32 scores, ties by lower id; text KV blocks are appended, text query rows list every block.  Lane l holds blocks 128 u + 4 l .. + 3 of vector u, so a lane's four keep bits
// are consecutive ids: eight lanes' nibbles make a word of the row's bitmap, and the ascending id list is written
// from the bitmap words.
//
// Top-P (TOPP) runs the same passes on softmax mass: exp(s - max) in 2^-40 fixed point (integer sums do not
// depend on the order the lanes add them in, and a bin's mass equals the sum of its values' masses exactly); the ranking
// loop then also adds up the mass of the values above each candidate.
constexpr int SELR_CAND = 64;
constexpr int SELR_WORDS = 296 + SELR_CAND + 8 + 64;   // per warp: 256 bin counts, 32 dump slots, list counter (word 288); candidates (+ 8 of padding); bitmap words
constexpr int SELR_WORDS_P = SELR_WORDS + 512 + 2 * (SELR_CAND + 8);     // Top-P: + 256 bin masses and the candidates' masses (64-bit)

template <int NV, bool TOPP>
__global__ void __launch_bounds__(SEL_R * 32, TOPP ? 2 : 3)
k_select_reg(const __grid_constant__ Shape sh, const __grid_constant__ GeoPack gp, StaticTables st, WsTables ws) {
  constexpr int WORDS = TOPP ? SELR_WORDS_P : SELR_WORDS;
  __shared__ __align__(16) int sel_sm[SEL_R * WORDS];
  const int bh = blockIdx.y;
  const CandGeo& g = gp.g[ws.scheme[bh]];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row = blockIdx.x * SEL_R + warp;
  if (row >= g.NB) return;
  const int n = g.NBv;
  int* out = ws.kv_idx + ((size_t)bh * sh.NBmax + row) * sh.cap;
  if (row >= n) {                               // text query block: every block
    for (int j = lane; j < g.NB; j += 32)
      if (SPADE_CHECK(j < sh.cap, ws.status, 301, j)) out[j] = j;
    if (lane == 0) ws.kv_cnt[(size_t)bh * sh.NBmax + row] = g.NB;
    return;
  }
  uint32_t* bits = ws.rowbits + ((size_t)bh * sh.NBvmax + row) * sh.bits_ld;      // the same list as a bitmap, for k_pair_axis
  if ((!TOPP && ws.keep[bh] >= n) || (sh.masks_on && ws.rowfull[(size_t)bh * sh.NBmax + row])) {
    // every video block is kept: nothing to search, the scores are not read
    for (int j = lane; j < n; j += 32)
      if (SPADE_CHECK(j < sh.cap, ws.status, 302, j)) out[j] = j;
    for (int wd = lane; wd * 32 < n; wd += 32) bits[wd] = n - wd * 32 >= 32 ? 0xffffffffu : (1u << (n - wd * 32)) - 1u;
    for (int j = lane; j < g.NBt; j += 32)
      if (SPADE_CHECK(n + j < sh.cap, ws.status, 306, n + j)) out[n + j] = n + j;
    if (lane == 0) { ws.kv_cnt[(size_t)bh * sh.NBmax + row] = n + g.NBt; atomicAdd(&ws.pair_union[bh * 4 + 3], n + g.NBt); }
    return;
  }
  int* hcnt = sel_sm + warp * WORDS;                             // [256] bins, [256 + lane] dump slots, [288] list counter
  float* cand = reinterpret_cast<float*>(hcnt + 296);            // [SELR_CAND + 8]
  uint32_t* words = reinterpret_cast<uint32_t*>(hcnt + 296 + SELR_CAND + 8);     // [64] the row's keep bitmap
  unsigned long long* hmass = reinterpret_cast<unsigned long long*>(hcnt + SELR_WORDS);      // Top-P: [256] mass per bin
  unsigned long long* cand_w = hmass + 256;                                                   // Top-P: [SELR_CAND + 8]
  const int ldc = sh.ld_scores;

  // ---- the row: NV float4 per lane; slots past the row's end hold NaN, which fails every comparison below ----------
  float v[NV][4];
  {
    const float4* src = reinterpret_cast<const float4*>(ws.scores + ((size_t)bh * sh.NBvmax + row) * ldc);
    const float qnan = __int_as_float(0x7fffffff);
#pragma unroll
    for (int u = 0; u < NV; ++u) {
      const int i = u * 32 + lane, left = n - 4 * i;
      const float4 f = left > 0 ? __ldcs(src + i) : make_float4(qnan, qnan, qnan, qnan);      // rows are ld_scores long (a multiple of 64)
      v[u][0] = f.x; v[u][1] = left > 1 ? f.y : qnan; v[u][2] = left > 2 ? f.z : qnan; v[u][3] = left > 3 ? f.w : qnan;
    }
  }
  float lo_v = INFINITY, hi_v = -INFINITY;
#pragma unroll
  for (int u = 0; u < NV; ++u)
#pragma unroll
    for (int e = 0; e < 4; ++e) { lo_v = fminf(lo_v, v[u][e]); hi_v = fmaxf(hi_v, v[u][e]); }     // NaN operands are ignored
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) {
    lo_v = fminf(lo_v, __shfl_xor_sync(FULL, lo_v, o));
    hi_v = fmaxf(hi_v, __shfl_xor_sync(FULL, hi_v, o));
  }

  // ---- the cut: keep v > T_hi, and need_t of the cnt_T blocks with T_lo <= v <= T_hi (lowest ids first) ---------------
  int need_r = TOPP ? 1 : ws.keep[bh];                            // Top-K: blocks still to keep among those in [lo_v, hi_v]
  bool all = false;                                               // set only if a pass finds its own histogram short (kept as a guard)
  int m = n;                                                      // blocks in [lo_v, hi_v]
  float T_lo = 0.f, T_hi = 0.f;
  int need_t = 0, cnt_T = 0;
  // Top-P: mass still to cover is target - above, both in 2^-40 fixed point of exp(s - max)
  const float mx = hi_v;
  auto weight = [&](float x) -> unsigned long long { return __float2ull_rn(expf(x - mx) * 1099511627776.f); };
  unsigned long long target = 0ull, above_m = 0ull;
  auto ties_for_mass = [&](unsigned long long above_T, unsigned long long wT, int cnt) -> int {
    // every block at the cut value carries the same mass: how many of them (lowest ids first) the target still needs
    unsigned long long t = wT > 0ull ? (target - above_T + wT - 1ull) / wT : (unsigned long long)cnt;
    if (target <= above_T) t = 1ull;
    return (int)(t < 1ull ? 1ull : (t > (unsigned long long)cnt ? (unsigned long long)cnt : t));
  };
  if constexpr (TOPP) {
    unsigned long long z = 0ull;
#pragma unroll
    for (int u = 0; u < NV; ++u) {
      if (u * 128 >= n) break;
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (v[u][e] >= lo_v) z += weight(v[u][e]);                // NaN (past the row's end) fails the test
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) z += __shfl_xor_sync(FULL, z, o);
    target = (unsigned long long)ceil((double)ws.pthr[bh] * (double)z);
    if (target > z) target = z;
    if (target == 0ull) target = 1ull;
  }
  for (int level = 0; !all; ++level) {
    const float range = hi_v - lo_v;
    if (!(range > 1e-30f) || level >= 40) {                       // one value left (or values no fp32 arithmetic tells apart): ties
      T_lo = lo_v; T_hi = hi_v; cnt_T = m;
      need_t = TOPP ? ties_for_mass(above_m, weight(hi_v), m) : need_r;
      break;
    }
    const float a = 250.f / range;
    for (int i = lane; i < 256; i += 32) {
      hcnt[i] = 0;
      if constexpr (TOPP) hmass[i] = 0ull;
    }
    __syncwarp();
#pragma unroll
    for (int u = 0; u < NV; ++u) {
      if (u * 128 >= n) break;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float d = v[u][e] - lo_v;
        const bool in = d >= 0.f && d <= range;
        const uint32_t bin = __float_as_uint(fmaf(d, a, 8388610.f)) & 255u;        // 2 .. 252, monotone in the value
        if constexpr (TOPP) {
          if (in) { atomicAdd(&hcnt[bin], 1); atomicAdd(&hmass[bin], weight(v[u][e])); }
        } else {
          atomicAdd(&hcnt[in ? bin : 256u + lane], 1);                           // misses go to the lane's own dump slot
        }
      }
    }
    __syncwarp();
    int cut;
    if constexpr (TOPP) {
      cut = find_bin<unsigned long long>(hmass, target, above_m, lane);
    } else {
      int above = 0;
      cut = find_bin<int>(hcnt, need_r, above, lane);
      need_r -= above;
    }
    if (cut < 0) { all = true; break; }          // cannot happen (the target is within what the range holds); keep the row whole if it does
    m = hcnt[cut];
    __syncwarp();
    // one more pass over the registers: the cut bin's own range, and (when it is short) its values
    const bool collect = m <= SELR_CAND;
    if (lane == 0) hcnt[288] = 0;
    __syncwarp();
    float lo_n = INFINITY, hi_n = -INFINITY;
#pragma unroll
    for (int u = 0; u < NV; ++u) {
      if (u * 128 >= n) break;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float x = v[u][e], d = x - lo_v;
        const bool in = d >= 0.f && d <= range;
        const uint32_t bin = __float_as_uint(fmaf(d, a, 8388610.f)) & 255u;
        if (in && bin == (uint32_t)cut) {
          lo_n = fminf(lo_n, x); hi_n = fmaxf(hi_n, x);
          if (collect) {
            const int at = atomicAdd(&hcnt[288], 1);
            if (SPADE_CHECK(at < SELR_CAND, ws.status, 305, at)) {
              cand[at] = x;
              if constexpr (TOPP) cand_w[at] = weight(x);
            }
          }
        }
      }
    }
    __syncwarp();
    if (!collect) {
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) {
        lo_n = fminf(lo_n, __shfl_xor_sync(FULL, lo_n, o));
        hi_n = fmaxf(hi_n, __shfl_xor_sync(FULL, hi_n, o));
      }
      lo_v = lo_n; hi_v = hi_n;
      continue;
    }
    // rank the m <= 64 values: lane l owns cand[l] and cand[32 + l]
    const float qnan = __int_as_float(0x7fffffff);
    const float a0 = lane < m ? cand[lane] : qnan, a1 = lane + 32 < m ? cand[lane + 32] : qnan;
    __syncwarp();
    if (lane < 8) cand[m + lane] = qnan;          // the loop below reads eight at a time; NaN counts for nothing
    unsigned long long wa0 = 0ull, wa1 = 0ull, G0 = 0ull, G1 = 0ull;       // Top-P: own mass, mass of the values above
    if constexpr (TOPP) {
      wa0 = lane < m ? cand_w[lane] : 0ull; wa1 = lane + 32 < m ? cand_w[lane + 32] : 0ull;
    }
    __syncwarp();
    int gt0 = 0, ge0 = 0, gt1 = 0, ge1 = 0;
    for (int j0 = 0; j0 < m; j0 += 8) {
      const float4 ba = *reinterpret_cast<const float4*>(cand + j0), bb = *reinterpret_cast<const float4*>(cand + j0 + 4);
      const float b[8] = {ba.x, ba.y, ba.z, ba.w, bb.x, bb.y, bb.z, bb.w};
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        gt0 += b[k] > a0 ? 1 : 0; ge0 += b[k] >= a0 ? 1 : 0;
        gt1 += b[k] > a1 ? 1 : 0; ge1 += b[k] >= a1 ? 1 : 0;
        if constexpr (TOPP) {
          const unsigned long long wb = cand_w[j0 + k];          // past the end: unused, the comparison with NaN fails
          G0 += b[k] > a0 ? wb : 0ull; G1 += b[k] > a1 ? wb : 0ull;
        }
      }
    }
    bool c0, c1;
    if constexpr (TOPP) {
      const unsigned long long lo0 = above_m + G0, lo1 = above_m + G1;
      c0 = lane < m && lo0 < target && target <= lo0 + (unsigned long long)(ge0 - gt0) * wa0;
      c1 = lane + 32 < m && lo1 < target && target <= lo1 + (unsigned long long)(ge1 - gt1) * wa1;
    } else {
      c0 = lane < m && gt0 < need_r && need_r <= ge0;
      c1 = lane + 32 < m && gt1 < need_r && need_r <= ge1;
    }
    const unsigned h0 = __ballot_sync(FULL, c0), h1 = __ballot_sync(FULL, c1);
    if (!(h0 | h1)) { all = true; break; }       // cannot happen (the cut lies inside this bin)
    const int src = h0 ? __ffs(h0) - 1 : __ffs(h1) - 1;
    const float Tv = __shfl_sync(FULL, h0 ? a0 : a1, src);
    const int gt = __shfl_sync(FULL, h0 ? gt0 : gt1, src), ge = __shfl_sync(FULL, h0 ? ge0 : ge1, src);
    T_lo = Tv; T_hi = Tv; cnt_T = ge - gt;
    if constexpr (TOPP) {
      const unsigned long long G = __shfl_sync(FULL, h0 ? G0 : G1, src), wT = __shfl_sync(FULL, h0 ? wa0 : wa1, src);
      need_t = ties_for_mass(above_m + G, wT, cnt_T);
    } else {
      need_t = need_r - gt;
    }
    break;
  }

  // ---- the keep bitmap, then the ascending id list ----------------------------------------------------------
  const int nw = (n + 31) >> 5;                  // <= NV * 4 <= 64 words
  if (all) {
    for (int wd = lane; wd < nw; wd += 32) words[wd] = n - wd * 32 >= 32 ? 0xffffffffu : (1u << (n - wd * 32)) - 1u;
  } else if (need_t >= cnt_T) {
    // every block at the cut value is kept: keep <=> v >= T_lo
#pragma unroll
    for (int u = 0; u < NV; ++u) {
      if (u * 128 >= n) break;
      uint32_t kn = 0u;
#pragma unroll
      for (int e = 0; e < 4; ++e) kn |= (v[u][e] >= T_lo ? 1u : 0u) << e;
      uint32_t w = kn << (4 * (lane & 7));
      w |= __shfl_xor_sync(FULL, w, 1);
      w |= __shfl_xor_sync(FULL, w, 2);
      w |= __shfl_xor_sync(FULL, w, 4);
      if ((lane & 7) == 0) words[u * 4 + (lane >> 3)] = w;
    }
  } else {
    // only need_t of the cnt_T blocks at the cut are kept: rank them by id
    unsigned long long knp = 0ull, eqp = 0ull;
#pragma unroll
    for (int u = 0; u < NV; ++u) {
      if (u * 128 >= n) break;
      uint32_t kn = 0u, eqn = 0u;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        kn |= (v[u][e] > T_hi ? 1u : 0u) << e;
        eqn |= (v[u][e] >= T_lo && v[u][e] <= T_hi ? 1u : 0u) << e;
      }
      knp |= (unsigned long long)kn << (4 * u);
      eqp |= (unsigned long long)eqn << (4 * u);
    }
    int ties_seen = 0;
#pragma unroll 1
    for (int u = 0; u * 128 < n; ++u) {
      uint32_t kn = (uint32_t)(knp >> (4 * u)) & 15u;
      const uint32_t eqn = (uint32_t)(eqp >> (4 * u)) & 15u;
      const int c = __popc(eqn);
      int incl = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(FULL, incl, o);
        if (lane >= o) incl += up;
      }
      int r = ties_seen + incl - c;
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if ((eqn >> e) & 1u) { if (r < need_t) kn |= 1u << e; ++r; }
      ties_seen += __shfl_sync(FULL, incl, 31);
      uint32_t w = kn << (4 * (lane & 7));
      w |= __shfl_xor_sync(FULL, w, 1);
      w |= __shfl_xor_sync(FULL, w, 2);
      w |= __shfl_xor_sync(FULL, w, 4);
      if ((lane & 7) == 0) words[u * 4 + (lane >> 3)] = w;
    }
  }
  __syncwarp();
  // lane l owns words l and 32 + l: static masks, the bitmap row, and the ids of its set bits
  uint32_t w0 = lane < nw ? words[lane] : 0u, w1 = lane + 32 < nw ? words[lane + 32] : 0u;
  if (sh.masks_on && !all) {
    const uint8_t* colkeep = ws.colkeep + (size_t)bh * sh.NBmax;
    const int r_w = row % g.nbw, r_h = (row / g.nbw) % g.nbh, r_t = row / (g.nbw * g.nbh);
#pragma unroll 1
    for (int half = 0; half < 2; ++half) {
      const int wi = lane + 32 * half;
      if (wi >= nw) continue;
      uint32_t add = 0u;
      for (int bit = 0; bit < 32; ++bit) {
        const int j = wi * 32 + bit;
        if (j >= n) break;
        bool k = colkeep[j] != 0;
        if (sh.window >= 0) {
          const int dw = j % g.nbw - r_w, dh = (j / g.nbw) % g.nbh - r_h, dt = j / (g.nbw * g.nbh) - r_t;
          k = k || (abs(dw) <= sh.window && abs(dh) <= sh.window && abs(dt) <= sh.window);
        }
        add |= (k ? 1u : 0u) << bit;
      }
      if (half) w1 |= add; else w0 |= add;
    }
  }
  if (lane < nw) bits[lane] = w0;
  if (lane + 32 < nw) bits[lane + 32] = w1;
  const int c0 = __popc(w0), c1 = __popc(w1);
  int i0 = c0, i1 = c1;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int x = __shfl_up_sync(FULL, i0, o), y = __shfl_up_sync(FULL, i1, o);
    if (lane >= o) { i0 += x; i1 += y; }
  }
  const int tot0 = __shfl_sync(FULL, i0, 31), tot1 = __shfl_sync(FULL, i1, 31);
#pragma unroll 1
  for (int half = 0; half < 2; ++half) {
    uint32_t w = half ? w1 : w0;
    int pos = half ? tot0 + i1 - c1 : i0 - c0;
    const int base = (lane + 32 * half) * 32;
    while (w) {
      const int bit = __ffs(w) - 1;
      w &= w - 1;
      if (SPADE_CHECK(pos < sh.cap, ws.status, 303, pos)) out[pos] = base + bit;
      ++pos;
    }
  }
  const int count = tot0 + tot1;
  for (int j = lane; j < g.NBt; j += 32)
    if (SPADE_CHECK(count + j < sh.cap, ws.status, 306, count + j)) out[count + j] = n + j;     // text KV blocks are always kept
  if (lane == 0) { ws.kv_cnt[(size_t)bh * sh.NBmax + row] = count + g.NBt; atomicAdd(&ws.pair_union[bh * 4 + 3], count + g.NBt); }
}

}  // namespace

cudaError_t launch_sics(const void* Q, const void* K, const Shape& sh, const GeoPack& gp, const StaticTables& st,
                        const WsTables& ws, int num_sms, cudaStream_t s) {
  const long total = (long)sh.BH * 2 * sh.units_per_ht;
  long ctas = (total + WARPS_PER_CTA - 1) / WARPS_PER_CTA;
  const long cap = (long)num_sms * 8;                        // 8 resident CTAs of 8 warps per SM
  if (ctas > cap) ctas = cap;
  k_sics<<<(unsigned)ctas, WARPS_PER_CTA * 32, 0, s>>>((const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, sh, gp, st, ws);
  return cudaGetLastError();
}

cudaError_t launch_cells(const void* Q, const void* K, const Shape& sh, const WsTables& ws, int num_sms, cudaStream_t s) {
  const long total = (long)sh.BH * 2 * ((sh.NCELL + 1) / 2);
  long ctas = (total + WARPS_PER_CTA - 1) / WARPS_PER_CTA;
  const long cap = (long)num_sms * 8;
  if (ctas > cap) ctas = cap;
  k_cells<<<(unsigned)ctas, WARPS_PER_CTA * 32, 0, s>>>((const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, sh, ws.cells);
  return cudaGetLastError();
}

cudaError_t launch_blocks(const void* Q, const void* K, const Shape& sh, const GeoPack& gp, const StaticTables& st,
                          const WsTables& ws, int num_sms, cudaStream_t s) {
  long per_ht = 0;
  for (int c = 0; c < sh.C; ++c) per_ht += gp.g[c].NB;
  const long total = (long)sh.BH * 2 * per_ht;
  long ctas = (total + WARPS_PER_CTA - 1) / WARPS_PER_CTA;
  const long cap = (long)num_sms * 8;
  if (ctas > cap) ctas = cap;
  k_blocks<<<(unsigned)ctas, WARPS_PER_CTA * 32, 0, s>>>((const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, sh, gp, st, ws);
  return cudaGetLastError();
}

cudaError_t launch_static(const Shape& sh, const GeoPack& gp, const StaticTables& st, const WsTables& ws, cudaStream_t s) {
  dim3 grid((sh.NBvmax + 255) / 256, sh.BH);
  k_static<<<grid, 256, 0, s>>>(sh, gp, st, ws);
  return cudaGetLastError();
}

cudaError_t launch_gather(const Shape& sh, const GeoPack& gp, const WsTables& ws, int num_sms, int split, cudaStream_t s) {
  const long total = (long)sh.BH * 2 * sh.NBmax * 32;
  long ctas = (total + 255) / 256;
  if (ctas > (long)num_sms * 16) ctas = (long)num_sms * 16;
  k_gather<<<(unsigned)ctas, 256, 0, s>>>(sh, gp, ws, split);
  return cudaGetLastError();
}

cudaError_t launch_dsa_rows(const Shape& sh, const GeoPack& gp, const WsTables& ws, int num_sms, cudaStream_t s) {
  (void)num_sms;
  dim3 grid((sh.ld_scores + 31) / 32, SPADE_D / 32, sh.BH * 3);
  k_dsa_rows<<<grid, 256, 0, s>>>(sh, gp, ws);
  return cudaGetLastError();
}

cudaError_t launch_split_k(const Shape& sh, const GeoPack& gp, const WsTables& ws, int num_sms, cudaStream_t s) {
  const long total = (long)sh.BH * sh.NBmax * 32;
  long ctas = (total + 255) / 256;
  if (ctas > (long)num_sms * 16) ctas = (long)num_sms * 16;
  k_split_k<<<(unsigned)ctas, 256, 0, s>>>(sh, gp, ws);
  return cudaGetLastError();
}

cudaError_t launch_choose(const Shape& sh, const GeoPack& gp, const StaticTables& st, const WsTables& ws,
                          const ForcedPack& forced, int have_sics, cudaStream_t s) {
  k_choose<<<sh.BH, 256, 0, s>>>(sh, gp, st, ws, forced, have_sics);      // its last CTA also orders the heads (k_groups, mode 0)
  return cudaGetLastError();
}

cudaError_t launch_groups_after_select(const Shape& sh, const GeoPack& gp, const WsTables& ws, cudaStream_t s) {
  k_groups<<<1, 1024, 0, s>>>(sh, gp, ws, 1);
  return cudaGetLastError();
}

cudaError_t launch_pair_axis(const Shape& sh, const GeoPack& gp, const StaticTables& st, const WsTables& ws, int num_sms, cudaStream_t s) {
  const long total = (long)sh.BH * sh.cell_ld;
  long ctas = (total + WARPS_PER_CTA - 1) / WARPS_PER_CTA;
  if (ctas > (long)num_sms * 8) ctas = (long)num_sms * 8;
  k_pair_axis<<<(unsigned)ctas, WARPS_PER_CTA * 32, 0, s>>>(sh, gp, st, ws);
  return cudaGetLastError();
}

cudaError_t launch_summarize(const void* Q, const void* K, const Shape& sh, const GeoPack& gp, const StaticTables& st,
                             const WsTables& ws, int num_sms, cudaStream_t s) {
  const long total = (long)sh.BH * 2 * sh.NBmax;
  long ctas = (total + WARPS_PER_CTA - 1) / WARPS_PER_CTA;
  const long cap = (long)num_sms * 8;
  if (ctas > cap) ctas = cap;
  k_summarize<<<(unsigned)ctas, WARPS_PER_CTA * 32, 0, s>>>((const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, sh, gp, st, ws);
  return cudaGetLastError();
}

cudaError_t launch_minmax(const void* Q, const void* K, const Shape& sh, const GeoPack& gp, const StaticTables& st,
                          const WsTables& ws, int num_sms, cudaStream_t s) {
  const long total = (long)sh.BH * 2 * (sh.ld_scores / WARPS_PER_CTA);
  long ctas = total;
  const long cap = (long)num_sms * 8;
  if (ctas > cap) ctas = cap;
  k_minmax<<<(unsigned)ctas, WARPS_PER_CTA * 32, 0, s>>>((const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, sh, gp, st, ws);
  return cudaGetLastError();
}

cudaError_t launch_scores_minmax(const Shape& sh, const GeoPack& gp, const WsTables& ws, cudaStream_t s) {
  dim3 grid((sh.NBvmax + MMS_TC - 1) / MMS_TC, (sh.NBvmax + MMS_TR - 1) / MMS_TR, sh.BH);
  const float scale = 1.0f / sqrtf((float)SPADE_D);
  cudaError_t e;
  if (sh.estimator == 1) {
    e = cudaFuncSetAttribute(k_scores_minmax<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, MMS_SMEM);
    if (e != cudaSuccess) return e;
    k_scores_minmax<1><<<grid, 256, MMS_SMEM, s>>>(sh, gp, ws, scale);
  } else {
    e = cudaFuncSetAttribute(k_scores_minmax<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, MMS_SMEM);
    if (e != cudaSuccess) return e;
    k_scores_minmax<2><<<grid, 256, MMS_SMEM, s>>>(sh, gp, ws, scale);
  }
  return cudaGetLastError();
}

cudaError_t launch_select(const Shape& sh, const GeoPack& gp, const StaticTables& st, const WsTables& ws,
                          cudaStream_t s) {
  static_assert(SPADE_MAX_NB <= 16 * 128, "k_select_reg holds a row of at most 16 float4 per lane");
  dim3 grid((sh.NBmax + SEL_R - 1) / SEL_R, sh.BH);
  if (sh.mode != 1) {
    if (sh.NBvmax <= 4 * 128) k_select_reg<4, false><<<grid, SEL_R * 32, 0, s>>>(sh, gp, st, ws);
    else if (sh.NBvmax <= 8 * 128) k_select_reg<8, false><<<grid, SEL_R * 32, 0, s>>>(sh, gp, st, ws);
    else if (sh.NBvmax <= 12 * 128) k_select_reg<12, false><<<grid, SEL_R * 32, 0, s>>>(sh, gp, st, ws);
    else k_select_reg<16, false><<<grid, SEL_R * 32, 0, s>>>(sh, gp, st, ws);
  } else {
    if (sh.NBvmax <= 4 * 128) k_select_reg<4, true><<<grid, SEL_R * 32, 0, s>>>(sh, gp, st, ws);
    else if (sh.NBvmax <= 8 * 128) k_select_reg<8, true><<<grid, SEL_R * 32, 0, s>>>(sh, gp, st, ws);
    else if (sh.NBvmax <= 12 * 128) k_select_reg<12, true><<<grid, SEL_R * 32, 0, s>>>(sh, gp, st, ws);
    else k_select_reg<16, true><<<grid, SEL_R * 32, 0, s>>>(sh, gp, st, ws);
  }
  return cudaGetLastError();
}
