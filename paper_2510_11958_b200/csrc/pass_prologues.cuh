// Stage prologues of the pass kernel: each puts the activations this block's share of a
// projection multiplies into shared memory as bf16 hi/lo columns (the B operand of the MMA).
// Every prologue issues all of its global loads before it uses any of them, and loops instead
// of unrolling so that its code stays small.
#pragma once

#include "pass_stream.cuh"

namespace dmtd {

constexpr int PK_MERGE_BATCH = 16;   // partial outputs (float4 per lane) in flight per warp in the merge
constexpr int PK_SPAN_UNITS = 3;     // float4 units of a block's k-slab span per thread: span <= 3072 values

// Inputs of a prologue come into shared memory as bulk copies issued by one thread: no load
// instruction waits in a register, and the whole input costs one trip to L2.  stage_begin
// (thread 0) arms the barrier, stage_copy adds a copy, stage_wait (all threads) waits for them.
// fence: the thread that calls this also issues the copies (the copies must see what other blocks wrote before
// the grid barrier: a proxy fence by every thread that issues some, once).
__device__ __forceinline__ void stage_begin(const PassShared &S, uint32_t bytes, bool fence = true) {
  if (fence) fence_proxy_async_global();
  mbar_expect_tx(smem_u32(S.stage_bar), bytes);
}
__device__ __forceinline__ void stage_copy(const PassShared &S, void *dst, const void *src, uint32_t bytes) {
  bulk_g2s(smem_u32(dst), src, bytes, smem_u32(S.stage_bar));
}
__device__ __forceinline__ bool stage_wait(const PassParams &P, const PassShared &S) {
  const unsigned uses = *S.stage_uses;
  const uint32_t bar = smem_u32(S.stage_bar);
  bool ok = mbar_try_wait(bar, uses & 1u) || pipe_wait_slow(P, bar, uses & 1u);
  pk_sync();
  if (threadIdx.x == 0) *S.stage_uses = uses + 1;
  return ok;
}

// RMSNorm of M rows (row r at x + r * row_stride), written as bf16 hi/lo columns for the
// k-slabs this block needs of matrix W (steps a2 / a6 / a9, first half).
__device__ __noinline__ void norm_prologue(const PassParams &P, const float *x, size_t row_stride, int M,
                                           const float *w_norm, const PackedMat &W, int kind) {
  const PassShared S = pass_shared();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, H = P.H;
  PK_PROSTAMP(0);
  // one copy per row, each issued by its own lane of the first warp
  if (threadIdx.x == 0) stage_begin(S, (uint32_t)(M * H * 4), false);
  if (warp == 0) {
    __syncwarp();
    if (lane < M) {
      fence_proxy_async_global();
      stage_copy(S, S.xs + lane * H, x + (size_t)lane * row_stride, (uint32_t)(H * 4));
    }
  }
  const SlabSpan sp = slab_span(S, W, kind);
  const int ks4 = sp.KS / 4, nu = sp.count * ks4;
  float4 wv[PK_SPAN_UNITS];
#pragma unroll
  for (int j = 0; j < PK_SPAN_UNITS; ++j) {
    const int u = threadIdx.x + j * PK_THREADS;
    wv[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (u < nu) wv[j] = __ldg(reinterpret_cast<const float4 *>(w_norm + sp.first * sp.KS) + u);
  }
  PK_PROSTAMP(1);
  stage_wait(P, S);
  PK_PROSTAMP(2);
  // the rows' sums of squares side by side (independent chains through the loads and the warp reductions)
  {
    float ss[PK_MAX_ROWS];
#pragma unroll
    for (int m = 0; m < PK_MAX_ROWS; ++m) ss[m] = 0.f;
#pragma unroll 1
    for (int k4 = threadIdx.x; k4 < H / 4; k4 += PK_THREADS) {
#pragma unroll
      for (int m = 0; m < PK_MAX_ROWS; ++m) {
        if (m < M) {
          const float4 v = reinterpret_cast<const float4 *>(S.xs)[m * (H / 4) + k4];
          ss[m] += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
      for (int m = 0; m < PK_MAX_ROWS; ++m) ss[m] += __shfl_xor_sync(0xffffffffu, ss[m], o);
    }
    if (lane < PK_MAX_ROWS) {
      float mine = ss[0];
#pragma unroll
      for (int m = 1; m < PK_MAX_ROWS; ++m) mine = lane == m ? ss[m] : mine;
      S.red[warp * PK_MAX_ROWS + lane] = mine;
    }
  }
  pk_sync();
  PK_PROSTAMP(3);
  const float inv_h = 1.f / (float)H;
#pragma unroll 1
  for (int m = 0; m < M; ++m) {
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < PK_WARPS; ++w) v += S.red[w * PK_MAX_ROWS + m];
    const float inv = rsqrtf(v * inv_h + P.eps);
#pragma unroll
    for (int j = 0; j < PK_SPAN_UNITS; ++j) {
      const int u = threadIdx.x + j * PK_THREADS;
      if (u < nu) {
        const int sl = u >= ks4 ? 1 : 0, kl = (u - sl * ks4) * 4;         // a block's share touches at most two slabs
        float4 a = reinterpret_cast<const float4 *>(S.xs)[(m * H + (sp.first + sl) * sp.KS + kl) / 4];
        a.x *= inv * wv[j].x; a.y *= inv * wv[j].y; a.z *= inv * wv[j].z; a.w *= inv * wv[j].w;
        store_act4(S.bstage + (size_t)sl * 8 * sp.row_bytes, sp.row_bytes, m, kl, a);
      }
    }
  }
  PK_PROSTAMP(4);
  pk_sync();
  PK_PROSTAMP(5);
}

// SwiGLU gate (step a6, second half) for the k-slabs this block needs of the down projection.
__device__ __noinline__ void swiglu_prologue(const PassParams &P, int M, const PackedMat &W, int kind = PK_MAT_DOWN) {
  const PassShared S = pass_shared();
  const SlabSpan sp = slab_span(S, W, kind);
  const int ks4 = sp.KS / 4, ldgu = 2 * P.I, total = sp.count * M * ks4;
  // two copies (gate values, up values) per (slab, row) i = sl * M + m, spread over the lanes of the first warp
  if (threadIdx.x == 0) stage_begin(S, (uint32_t)(sp.count * M * 2 * sp.KS * 4), false);
  if (threadIdx.x < 32) {
    __syncwarp();
    fence_proxy_async_global();
#pragma unroll 1
    for (int c = threadIdx.x; c < 2 * sp.count * M; c += 32) {
      const int i = c >> 1, up = c & 1;
      const float *src = P.gu + (size_t)(i % M) * ldgu + (sp.first + i / M) * sp.KS + up * P.I;
      stage_copy(S, S.xs + (size_t)i * 2 * sp.KS + up * sp.KS, src, (uint32_t)(sp.KS * 4));
    }
  }
  stage_wait(P, S);
#pragma unroll 1
  for (int idx = threadIdx.x; idx < total; idx += PK_THREADS) {
    const int i = idx / ks4, u4 = idx - i * ks4;
    const float4 g = reinterpret_cast<const float4 *>(S.xs + (size_t)i * 2 * sp.KS)[u4];
    const float4 u = reinterpret_cast<const float4 *>(S.xs + (size_t)i * 2 * sp.KS + sp.KS)[u4];
    float4 a;
    a.x = g.x / (1.f + __expf(-g.x)) * u.x;
    a.y = g.y / (1.f + __expf(-g.y)) * u.y;
    a.z = g.z / (1.f + __expf(-g.z)) * u.z;
    a.w = g.w / (1.f + __expf(-g.w)) * u.w;
    store_act4(S.bstage + (size_t)(i / M) * 8 * sp.row_bytes, sp.row_bytes, i % M, u4 * 4, a);
  }
  pk_sync();
}

// Online-softmax merge of the key slices (step a4, second half) for the heads this block's share
// of the O projection multiplies, written as bf16 hi/lo columns: one warp per (row, head), one
// lane per 4 output values, every slice's partial output loaded before any is used.
__device__ __noinline__ void merge_prologue(const PassParams &P, int M, int nsplit, const PackedMat &W, int kind = PK_MAT_O) {
  const PassShared S = pass_shared();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const SlabSpan sp = slab_span(S, W, kind);
  const int heads_per_slab = sp.KS / PK_D, n_heads = sp.count * heads_per_slab;
#pragma unroll 1
  for (int pair = warp; pair < M * n_heads; pair += PK_WARPS) {
    const int m = pair / n_heads, hh = pair - m * n_heads;
    const int sl = hh / heads_per_slab, h = sp.first * heads_per_slab + hh;
    const size_t slot0 = ((size_t)m * P.nq + h) * PK_NSPLIT_CAP;
    float2 ml = make_float2(-INFINITY, 0.f);
    if (lane < nsplit) ml = __ldcg(reinterpret_cast<const float2 *>(P.part_ml) + slot0 + lane);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float wgt = 0.f;
#pragma unroll 1
    for (int s0 = 0; s0 < nsplit; s0 += PK_MERGE_BATCH) {
      float4 po[PK_MERGE_BATCH];
#pragma unroll
      for (int s = 0; s < PK_MERGE_BATCH; ++s)
        if (s0 + s < nsplit) po[s] = __ldcg(reinterpret_cast<const float4 *>(P.part_o + (slot0 + s0 + s) * PK_D) + lane);
      if (s0 == 0) {
        const float mxx = warp_max(ml.y > 0.f ? ml.x : -INFINITY);
        wgt = ml.y > 0.f ? __expf(ml.x - mxx) : 0.f;
        wgt /= warp_sum(wgt * ml.y);
      }
#pragma unroll
      for (int s = 0; s < PK_MERGE_BATCH; ++s) {
        const float w = __shfl_sync(0xffffffffu, wgt, (s0 + s) & 31);
        if (s0 + s < nsplit) { acc.x += w * po[s].x; acc.y += w * po[s].y; acc.z += w * po[s].z; acc.w += w * po[s].w; }
      }
    }
    store_act4(S.bstage + (size_t)sl * 8 * sp.row_bytes, sp.row_bytes, m, (hh - sl * heads_per_slab) * PK_D + lane * 4, acc);
  }
  pk_sync();
}

// Step a1 for the first layer of a pass: x[m][:] = E[token of row m], the rows spread over the
// grid (row m = b*R + r sits at position pos0 + r).  Readers wait for the next grid barrier.
__device__ __noinline__ void embed_rows(const PassParams &P, float *x, int M, int R, int pos0) {
  const int units = P.H / 8;
#pragma unroll 1
  for (int i = blockIdx.x * PK_THREADS + threadIdx.x; i < M * units; i += gridDim.x * PK_THREADS) {
    const int m = i / units, u = i - m * units;
    int tok = P.tokens[(size_t)(m / R) * P.max_seq + pos0 + m % R];
    if (tok < 0 || tok >= P.embed.N) {
      atomicMax(P.error, PK_ERR_TOKEN);
      tok = min(max(tok, 0), P.embed.N - 1);
    }
    float f[8];
    embed8(P.embed, tok, u, f);
    float *dst = x + (size_t)m * P.H + u * 8;
    *reinterpret_cast<float4 *>(dst) = make_float4(f[0], f[1], f[2], f[3]);
    *reinterpret_cast<float4 *>(dst + 4) = make_float4(f[4], f[5], f[6], f[7]);
  }
}

// Step a8: the newest row of every sequence leaves the lower stack and becomes the residual
// row of the decoding layers (Section 2.2: only that row goes on); spread over the grid.
__device__ __forceinline__ void select_rows(const PassParams &P) {
  const int h4 = P.H / 4;
#pragma unroll 1
  for (int i = blockIdx.x * PK_THREADS + threadIdx.x; i < P.B * h4; i += gridDim.x * PK_THREADS) {
    const int b = i / h4, k4 = i - b * h4;
    reinterpret_cast<float4 *>(P.x_up)[(size_t)b * h4 + k4] =
        __ldcg(reinterpret_cast<const float4 *>(P.x_lo + ((size_t)b * P.R_lo + P.R_lo - 1) * P.H) + k4);
  }
}

}  // namespace dmtd
