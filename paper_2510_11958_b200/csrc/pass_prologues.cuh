// Stage prologues of the pass kernel: each puts the activations this block's share of a
// projection multiplies into shared memory as bf16 hi/lo columns (the B operand of the MMA).
// Every prologue issues all of its global loads before it uses any of them, and loops instead
// of unrolling so that its code stays small.
#pragma once

#include "pass_stream.cuh"

namespace dmtd {

constexpr int PK_BATCH = 4;          // float4 loads a thread keeps in flight in an elementwise prologue
constexpr int PK_STAGE_BATCH = 8;    // float4 loads a thread keeps in flight while staging rows
constexpr int PK_SPAN_UNITS = 3;     // float4 units of a block's k-slab span per thread: span <= 3072 values

// Copy M rows of H floats (row r at src + r * row_stride) into shared memory.
__device__ __forceinline__ void stage_rows(float *xs, const float *src, size_t row_stride, int M, int H) {
  const int h4 = H / 4, n4 = M * h4;
  for (int base = 0; base < n4; base += PK_STAGE_BATCH * PK_THREADS) {
    float4 tmp[PK_STAGE_BATCH];
#pragma unroll
    for (int j = 0; j < PK_STAGE_BATCH; ++j) {
      const int i = base + j * PK_THREADS + threadIdx.x;
      if (i < n4) tmp[j] = __ldcg(reinterpret_cast<const float4 *>(src + (size_t)(i / h4) * row_stride) + i % h4);
    }
#pragma unroll
    for (int j = 0; j < PK_STAGE_BATCH; ++j) {
      const int i = base + j * PK_THREADS + threadIdx.x;
      if (i < n4) reinterpret_cast<float4 *>(xs)[i] = tmp[j];
    }
  }
}

// RMSNorm of M rows (row r at x + r * row_stride), written as bf16 hi/lo columns for the
// k-slabs this block needs of matrix W (steps a2 / a6 / a9, first half).
__device__ __noinline__ void norm_prologue(const PassParams &P, const float *x, size_t row_stride, int M,
                                           const float *w_norm, const PackedMat &W) {
  const PassShared S = pass_shared();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, H = P.H;
  const SlabSpan sp = slab_span(W);
  const int ks4 = sp.KS / 4, nu = sp.count * ks4;
  float4 wv[PK_SPAN_UNITS];
#pragma unroll
  for (int j = 0; j < PK_SPAN_UNITS; ++j) {
    const int u = threadIdx.x + j * PK_THREADS;
    wv[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (u < nu) wv[j] = __ldg(reinterpret_cast<const float4 *>(w_norm + sp.first * sp.KS) + u);
  }
  stage_rows(S.xs, x, row_stride, M, H);
  pk_sync();
  for (int m = 0; m < M; ++m) {
    float ss = 0.f;
    for (int k4 = threadIdx.x; k4 < H / 4; k4 += PK_THREADS) {
      const float4 v = reinterpret_cast<const float4 *>(S.xs)[m * (H / 4) + k4];
      ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    ss = warp_sum(ss);
    if (lane == 0) S.red[warp * PK_MAX_ROWS + m] = ss;
  }
  pk_sync();
  for (int m = 0; m < M; ++m) {
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < PK_WARPS; ++w) v += S.red[w * PK_MAX_ROWS + m];
    const float inv = rsqrtf(v / (float)H + P.eps);
#pragma unroll
    for (int j = 0; j < PK_SPAN_UNITS; ++j) {
      const int u = threadIdx.x + j * PK_THREADS;
      if (u < nu) {
        const int sl = u / ks4, kl = (u - sl * ks4) * 4;
        float4 a = reinterpret_cast<const float4 *>(S.xs)[(m * H + (sp.first + sl) * sp.KS + kl) / 4];
        a.x *= inv * wv[j].x; a.y *= inv * wv[j].y; a.z *= inv * wv[j].z; a.w *= inv * wv[j].w;
        store_act4(S.bstage + (size_t)sl * 8 * sp.row_bytes, sp.row_bytes, m, kl, a);
      }
    }
  }
  pk_sync();
}

// SwiGLU gate (step a6, second half) for the k-slabs this block needs of the down projection.
__device__ __noinline__ void swiglu_prologue(const PassParams &P, int M, const PackedMat &W) {
  const PassShared S = pass_shared();
  const SlabSpan sp = slab_span(W);
  const int ks4 = sp.KS / 4, ldgu = 2 * P.I, total = sp.count * M * ks4;
  for (int base = 0; base < total; base += PK_BATCH * PK_THREADS) {
    float4 g[PK_BATCH], u[PK_BATCH];
#pragma unroll
    for (int j = 0; j < PK_BATCH; ++j) {
      const int idx = base + j * PK_THREADS + threadIdx.x;
      if (idx < total) {
        const int u4 = idx % ks4, m = (idx / ks4) % M, sl = idx / (ks4 * M);
        const float *src = P.gu + (size_t)m * ldgu + (sp.first + sl) * sp.KS + u4 * 4;
        g[j] = __ldcg(reinterpret_cast<const float4 *>(src));
        u[j] = __ldcg(reinterpret_cast<const float4 *>(src + P.I));
      }
    }
#pragma unroll
    for (int j = 0; j < PK_BATCH; ++j) {
      const int idx = base + j * PK_THREADS + threadIdx.x;
      if (idx < total) {
        const int u4 = idx % ks4, m = (idx / ks4) % M, sl = idx / (ks4 * M);
        float4 a;
        a.x = g[j].x / (1.f + __expf(-g[j].x)) * u[j].x;
        a.y = g[j].y / (1.f + __expf(-g[j].y)) * u[j].y;
        a.z = g[j].z / (1.f + __expf(-g[j].z)) * u[j].z;
        a.w = g[j].w / (1.f + __expf(-g[j].w)) * u[j].w;
        store_act4(S.bstage + (size_t)sl * 8 * sp.row_bytes, sp.row_bytes, m, u4 * 4, a);
      }
    }
  }
  pk_sync();
}

// Rows of `src` [M][ld] as bf16 hi/lo columns for the k-slabs this block needs of W (the merged
// attention output entering the O projection).
__device__ __noinline__ void plain_prologue(const float *src, int ld, int M, const PackedMat &W) {
  const PassShared S = pass_shared();
  const SlabSpan sp = slab_span(W);
  const int ks4 = sp.KS / 4, total = sp.count * M * ks4;
  for (int base = 0; base < total; base += PK_BATCH * PK_THREADS) {
    float4 v[PK_BATCH];
#pragma unroll
    for (int j = 0; j < PK_BATCH; ++j) {
      const int idx = base + j * PK_THREADS + threadIdx.x;
      if (idx < total) {
        const int u4 = idx % ks4, m = (idx / ks4) % M, sl = idx / (ks4 * M);
        v[j] = __ldcg(reinterpret_cast<const float4 *>(src + (size_t)m * ld + (sp.first + sl) * sp.KS + u4 * 4));
      }
    }
#pragma unroll
    for (int j = 0; j < PK_BATCH; ++j) {
      const int idx = base + j * PK_THREADS + threadIdx.x;
      if (idx < total) {
        const int u4 = idx % ks4, m = (idx / ks4) % M, sl = idx / (ks4 * M);
        store_act4(S.bstage + (size_t)sl * 8 * sp.row_bytes, sp.row_bytes, m, u4 * 4, v[j]);
      }
    }
  }
  pk_sync();
}

// Step a1 for the first layer of a pass: x[m][:] = E[token of row m], the rows spread over the
// grid (row m = b*R + r sits at position pos0 + r).  Readers wait for the next grid barrier.
__device__ __noinline__ void embed_rows(const PassParams &P, float *x, int M, int R, int pos0) {
  const int units = P.H / 8;
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
  for (int i = blockIdx.x * PK_THREADS + threadIdx.x; i < P.B * h4; i += gridDim.x * PK_THREADS) {
    const int b = i / h4, k4 = i - b * h4;
    reinterpret_cast<float4 *>(P.x_up)[(size_t)b * h4 + k4] =
        __ldcg(reinterpret_cast<const float4 *>(P.x_lo + ((size_t)b * P.R_lo + P.R_lo - 1) * P.H) + k4);
  }
}

}  // namespace dmtd
