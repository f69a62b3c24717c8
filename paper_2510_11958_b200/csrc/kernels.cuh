// Per-step kernels of the DMTD decode path (one launch per step of the layer).
// Every projection accumulates into its output with fp32 reductions, so split-K work
// division needs no second pass; the buffers that start at zero are cleared by the
// preceding "prep" kernel.
#pragma once

#include "common.cuh"

namespace dmtd {

constexpr int GEMV_THREADS = 256;
constexpr int GEMV_WARPS = GEMV_THREADS / 32;

// ------------------------------------------------------------------------------------
// Weight repacking (runs once, at create)
// ------------------------------------------------------------------------------------

// src [N][K] bf16 row-major -> atoms of tiles [tile0, tile0 + ceil(N/16)) of a stream that
// has n_tiles_total row tiles.  One thread per 16-byte chunk.
__global__ void pack_bf16_kernel(const __nv_bfloat16 *__restrict__ src, int N, int K,
                                 uint4 *__restrict__ dst, int tile0, int n_tiles_total, int aps,
                                 int n_slabs) {
  int tiles_local = (N + 15) / 16;
  long long total = (long long)n_slabs * tiles_local * aps * 64;
  for (long long c = (long long)blockIdx.x * blockDim.x + threadIdx.x; c < total;
       c += (long long)gridDim.x * blockDim.x) {
    int lane_pos = (int)(c % 64);
    long long atom_idx = c / 64;
    int a = (int)(atom_idx % aps);
    int tl = (int)((atom_idx / aps) % tiles_local);
    int s = (int)(atom_idx / aps / tiles_local);
    int half = lane_pos >> 5, lane = lane_pos & 31, g = lane >> 2, t = lane & 3;
    int row = tl * 16 + half * 8 + g;
    int k = (s * aps + a) * 32 + t * 8;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (row < N) v = *reinterpret_cast<const uint4 *>(src + (size_t)row * K + k);
    dst[(((long long)s * n_tiles_total + tile0 + tl) * aps + a) * 64 + half * 32 + lane] = v;
  }
}

template <typename T>
__global__ void to_float_kernel(const T *__restrict__ src, float *__restrict__ dst, int n) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = (float)src[i];
}

// ------------------------------------------------------------------------------------
// a1: embedding gather.  x[m][:] = E[token of row m]; row m = b*R + r sits at position
// *pos0 + r of sequence b.
// ------------------------------------------------------------------------------------
__global__ void embed_kernel(PackedMat E, const int *__restrict__ tokens, int max_seq,
                             const int *__restrict__ pos0, int R, float *__restrict__ x, int ldx,
                             int accumulate, DevState *st) {
  int m = blockIdx.x, b = m / R, r = m % R;
  int tok = tokens[(size_t)b * max_seq + *pos0 + r];
  if (tok < 0 || tok >= E.N) {
    if (threadIdx.x == 0) atomicMax(&st->error, 1);
    tok = min(max(tok, 0), E.N - 1);
  }
  float *xr = x + (size_t)m * ldx;
  if (E.wf) {
    const float *e = E.wf + (size_t)tok * E.K;
    for (int k = threadIdx.x; k < E.K; k += blockDim.x) xr[k] = accumulate ? xr[k] + e[k] : e[k];
    return;
  }
  int T = tok >> 4, half = (tok >> 3) & 1, g = tok & 7;
  for (int c = threadIdx.x; c < E.K / 8; c += blockDim.x) {   // one 16-byte chunk = 8 values
    int k = c * 8, atom = k >> 5, t = (k >> 3) & 3;
    int s = atom / E.aps, a = atom % E.aps;
    uint4 v = E.w[(((long long)s * E.n_tiles + T) * E.aps + a) * 64 + half * 32 + g * 4 + t];
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float lo = bf16_bits_to_float(w[j] & 0xffffu), hi = bf16_bits_to_float(w[j] >> 16);
      if (accumulate) { lo += xr[k + 2 * j]; hi += xr[k + 2 * j + 1]; }
      xr[k + 2 * j] = lo;
      xr[k + 2 * j + 1] = hi;
    }
  }
}

// ------------------------------------------------------------------------------------
// Activation preparation for a projection: act[m][:] = x[m][:] / rms(x[m]) * w, and clear
// the accumulator row the projection will add into.  Grid (rows, slices): every block clears
// PREP_ZERO_COLS columns of its row's accumulator, the first block of a row also does the norm.
// ------------------------------------------------------------------------------------
constexpr int PREP_ZERO_COLS = 4096;
__global__ void prep_norm_kernel(const float *__restrict__ x, int ldx, const float *__restrict__ w,
                                 int K, float eps, float *__restrict__ act, int lda,
                                 float *__restrict__ zero_buf, int zero_ld, int zero_cols) {
  const int m = blockIdx.x;
  if (zero_buf) {
    const int c0 = blockIdx.y * PREP_ZERO_COLS, c1 = min(zero_cols, c0 + PREP_ZERO_COLS);
    float *row = zero_buf + (size_t)m * zero_ld;
    const bool aligned = (zero_ld & 3) == 0;              // then every row starts on a 16-byte boundary
    for (int k = c0 + threadIdx.x * 4; k < c1; k += blockDim.x * 4) {
      if (aligned && k + 4 <= c1) *reinterpret_cast<float4 *>(row + k) = make_float4(0.f, 0.f, 0.f, 0.f);
      else for (int j = k; j < c1; ++j) row[j] = 0.f;
    }
  }
  if (blockIdx.y != 0) return;
  const float *xr = x + (size_t)m * ldx;
  float ss = 0.f;
  for (int k = threadIdx.x; k < K; k += blockDim.x) ss += xr[k] * xr[k];
  __shared__ float red[32];
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x < 32) {
    float v = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.f;
    v = warp_sum(v);
    if (threadIdx.x == 0) red[0] = v;
  }
  __syncthreads();
  float inv = rsqrtf(red[0] / (float)K + eps);
  for (int k = threadIdx.x; k < K; k += blockDim.x) act[(size_t)m * lda + k] = xr[k] * inv * w[k];
}

// act[m][i] = silu(g) * u with g = gu[m][i], u = gu[m][I + i]  (the SwiGLU gate).
__global__ void prep_swiglu_kernel(const float *__restrict__ gu, int ldgu, int I,
                                   float *__restrict__ act, int lda) {
  int m = blockIdx.y;
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= I) return;
  float g = gu[(size_t)m * ldgu + i], u = gu[(size_t)m * ldgu + I + i];
  act[(size_t)m * lda + i] = g / (1.f + expf(-g)) * u;
}

// ------------------------------------------------------------------------------------
// Projection, bf16 weights: out[m][n] += sum_k W[n][k] * act[m][k].
//
// The atom stream is cut into equal contiguous ranges, one per warp of the grid, so every
// warp streams the same number of bytes whatever N and K are.  A warp walks its range
// segment by segment (a segment = atoms of one row tile inside one k-slab), accumulates with
// mma.m16n8k16 (weights = A operand straight from global memory in register order,
// activations = B operand from shared memory as bf16 hi/lo column pairs), and adds each
// finished segment into `out` with fp32 reductions.  NT n8-tiles cover 4*NT activation rows
// per sweep; more rows are swept in turn.
// ------------------------------------------------------------------------------------
template <int NT>
__global__ void __launch_bounds__(GEMV_THREADS)
gemv_bf16_kernel(PackedMat W, const float *__restrict__ act, int lda, int M,
                 float *__restrict__ out, int ldo) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int KS = W.aps * 32;
  const int row_bytes = ((KS * 2) % 128 == 64) ? KS * 2 : KS * 2 + 64;   // conflict-free LDS.128
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;

  const long long A = packed_atoms(W);
  const long long c0 = A * blockIdx.x / gridDim.x, c1 = A * (blockIdx.x + 1) / gridDim.x;
  const long long w0 = c0 + (c1 - c0) * warp / GEMV_WARPS, w1 = c0 + (c1 - c0) * (warp + 1) / GEMV_WARPS;
  if (c0 >= c1) return;
  const long long slab_atoms = (long long)W.n_tiles * W.aps;
  const int s_first = (int)(c0 / slab_atoms), s_last = (int)((c1 - 1) / slab_atoms);

  for (int m0 = 0; m0 < M; m0 += 4 * NT) {
    for (int s = s_first; s <= s_last; ++s) {
      __syncthreads();
      // stage rows m0 .. m0+4NT-1, k in slab s, as columns (2r: hi, 2r+1: lo)
      for (int idx = threadIdx.x; idx < 4 * NT * (KS / 4); idx += GEMV_THREADS) {
        int r = idx / (KS / 4), k4 = (idx % (KS / 4)) * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (m0 + r < M) v = *reinterpret_cast<const float4 *>(act + (size_t)(m0 + r) * lda + s * KS + k4);
        __nv_bfloat16 h[4], l[4];
        split_bf16(v.x, h[0], l[0]); split_bf16(v.y, h[1], l[1]);
        split_bf16(v.z, h[2], l[2]); split_bf16(v.w, h[3], l[3]);
        *reinterpret_cast<uint2 *>(smem_raw + (size_t)(2 * r) * row_bytes + k4 * 2) =
            *reinterpret_cast<uint2 *>(h);
        *reinterpret_cast<uint2 *>(smem_raw + (size_t)(2 * r + 1) * row_bytes + k4 * 2) =
            *reinterpret_cast<uint2 *>(l);
      }
      __syncthreads();
      long long a_lo = max(w0, (long long)s * slab_atoms), a_hi = min(w1, (long long)(s + 1) * slab_atoms);
      while (a_lo < a_hi) {
        long long in_slab = a_lo - (long long)s * slab_atoms;
        int T = (int)(in_slab / W.aps), a_begin = (int)(in_slab % W.aps);
        int a_end = (int)min((long long)W.aps, a_begin + (a_hi - a_lo));
        float acc[NT][4];
#pragma unroll
        for (int i = 0; i < NT; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
        const uint4 *wp = W.w + (a_lo - a_begin) * 64 + lane;
        const unsigned char *bp = smem_raw + (size_t)g * row_bytes + t * 16;
        int a = a_begin;
        for (; a + 4 <= a_end; a += 4) {
          uint4 A0[4], A1[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            A0[u] = ldg_stream(wp + (size_t)(a + u) * 64);
            A1[u] = ldg_stream(wp + (size_t)(a + u) * 64 + 32);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
#pragma unroll
            for (int i = 0; i < NT; ++i) {
              uint4 Bv = *reinterpret_cast<const uint4 *>(bp + (size_t)(8 * i) * row_bytes + (a + u) * 64);
              mma_bf16_16816(acc[i], A0[u].x, A1[u].x, A0[u].y, A1[u].y, Bv.x, Bv.y);
              mma_bf16_16816(acc[i], A0[u].z, A1[u].z, A0[u].w, A1[u].w, Bv.z, Bv.w);
            }
          }
        }
        for (; a < a_end; ++a) {
          uint4 A0 = ldg_stream(wp + (size_t)a * 64), A1 = ldg_stream(wp + (size_t)a * 64 + 32);
#pragma unroll
          for (int i = 0; i < NT; ++i) {
            uint4 Bv = *reinterpret_cast<const uint4 *>(bp + (size_t)(8 * i) * row_bytes + a * 64);
            mma_bf16_16816(acc[i], A0.x, A1.x, A0.y, A1.y, Bv.x, Bv.y);
            mma_bf16_16816(acc[i], A0.z, A1.z, A0.w, A1.w, Bv.z, Bv.w);
          }
        }
        // accumulator columns 2t (hi) and 2t+1 (lo) belong to activation row 4i+t
        int n_lo = T * 16 + g;
#pragma unroll
        for (int i = 0; i < NT; ++i) {
          int m = m0 + 4 * i + t;
          if (m < M) {
            if (n_lo < W.N) atomicAdd(out + (size_t)m * ldo + n_lo, acc[i][0] + acc[i][1]);
            if (n_lo + 8 < W.N) atomicAdd(out + (size_t)m * ldo + n_lo + 8, acc[i][2] + acc[i][3]);
          }
        }
        a_lo += a_end - a_begin;
      }
    }
  }
}

// Projection, fp32 weights (small verification models only): one warp per output row.
__global__ void gemv_f32_kernel(PackedMat W, const float *__restrict__ act, int lda, int M,
                                float *__restrict__ out, int ldo) {
  int lane = threadIdx.x & 31;
  int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, n_warps = (gridDim.x * blockDim.x) >> 5;
  for (int n = warp; n < W.N; n += n_warps) {
    const float *wr = W.wf + (size_t)n * W.K;
    for (int m0 = 0; m0 < M; m0 += 4) {
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      for (int k = lane * 4; k < W.K; k += 128) {
        float4 w = *reinterpret_cast<const float4 *>(wr + k);
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (m0 + i < M) {
            float4 a = *reinterpret_cast<const float4 *>(act + (size_t)(m0 + i) * lda + k);
            acc[i] += w.x * a.x + w.y * a.y + w.z * a.z + w.w * a.w;
          }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float v = warp_sum(acc[i]);
        if (lane == 0 && m0 + i < M) out[(size_t)(m0 + i) * ldo + n] += v;
      }
    }
  }
}

// ------------------------------------------------------------------------------------
// a3: per-head QK-norm, rotary embedding, KV append.
// ------------------------------------------------------------------------------------

// cos/sin of pos * theta^(-2i/d) for the R positions of this pass, computed in double so
// that long contexts do not lose angle precision.  table [R][d/2] of (cos, sin).
__global__ void rope_table_kernel(const int *__restrict__ pos0, int R, int half,
                                  const double *__restrict__ inv_freq, float2 *__restrict__ table) {
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= R * half) return;
  int r = idx / half, i = idx % half;
  double s, c;
  sincos((double)(*pos0 + r) * inv_freq[i], &s, &c);
  table[idx] = make_float2((float)c, (float)s);
}

template <typename KVT> __device__ __forceinline__ KVT to_kv(float v);
template <> __device__ __forceinline__ float to_kv<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 to_kv<__nv_bfloat16>(float v) {
  return __float2bfloat16_rn(v);
}
template <> __device__ __forceinline__ __half to_kv<__half>(float v) { return __float2half_rn(v); }

// One warp per (row, head); heads are q heads, then k heads, then v heads.  q is normalised
// and rotated in place (fp32); k is normalised, rotated and stored in the cache; v is stored.
// qkv [M][ldq] = (q | k | v) per row.  Cache layout [b][kv head][max_seq][D].
template <int D, typename KVT>
__global__ void qk_norm_rope_append_kernel(float *__restrict__ qkv, int ldq, int nq, int nkv, int R,
                                           const float *__restrict__ w_qn, const float *__restrict__ w_kn,
                                           float eps, const float2 *__restrict__ table,
                                           const int *__restrict__ pos0, KVT *__restrict__ kc,
                                           KVT *__restrict__ vc, int max_seq) {
  constexpr int E = D / 32;                 // values per lane; value j pairs with j + E/2
  int lane = threadIdx.x & 31;
  int head = blockIdx.y * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (head >= nq + 2 * nkv) return;
  int m = blockIdx.x, b = m / R, r = m % R, pos = *pos0 + r;
  float *src = qkv + (size_t)m * ldq + (size_t)head * D;
  float v[E];
#pragma unroll
  for (int j = 0; j < E; ++j) v[j] = src[lane + 32 * j];
  if (head >= nq + nkv) {                   // v head: plain append
    int h = head - nq - nkv;
    KVT *dst = vc + (((size_t)b * nkv + h) * max_seq + pos) * D;
#pragma unroll
    for (int j = 0; j < E; ++j) dst[lane + 32 * j] = to_kv<KVT>(v[j]);
    return;
  }
  float ss = 0.f;
#pragma unroll
  for (int j = 0; j < E; ++j) ss += v[j] * v[j];
  ss = warp_sum(ss);
  float inv = rsqrtf(ss / (float)D + eps);
  const float *w = head < nq ? w_qn : w_kn;
#pragma unroll
  for (int j = 0; j < E; ++j) v[j] = v[j] * inv * w[lane + 32 * j];
  float o[E];
#pragma unroll
  for (int j = 0; j < E / 2; ++j) {
    float2 cs = table[(size_t)r * (D / 2) + lane + 32 * j];
    float a = v[j], bb = v[j + E / 2];
    o[j] = a * cs.x - bb * cs.y;
    o[j + E / 2] = bb * cs.x + a * cs.y;
  }
  if (head < nq) {
#pragma unroll
    for (int j = 0; j < E; ++j) src[lane + 32 * j] = o[j];
  } else {
    int h = head - nq;
    KVT *dst = kc + (((size_t)b * nkv + h) * max_seq + pos) * D;
#pragma unroll
    for (int j = 0; j < E; ++j) dst[lane + 32 * j] = to_kv<KVT>(o[j]);
  }
}

// ------------------------------------------------------------------------------------
// a4: split-KV attention.  Each block handles one (sequence, kv head, block of RB new
// positions, slice of CH keys): the G query heads of that kv head for those positions form
// up to 16 query rows that share every key/value it reads.  Blocks write unnormalised
// partial outputs with their running max and sum; attn_merge_kernel combines the slices.
// ------------------------------------------------------------------------------------
constexpr int ATTN_WARPS = 4;
constexpr int ATTN_QR = 16;       // query rows per block

template <typename KVT> __device__ __forceinline__ void load8(const KVT *p, float (&f)[8]);
template <> __device__ __forceinline__ void load8<float>(const float *p, float (&f)[8]) {
  float4 a = *reinterpret_cast<const float4 *>(p), b = *reinterpret_cast<const float4 *>(p + 4);
  f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}
template <> __device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16 *p, float (&f)[8]) {
  uint4 v = *reinterpret_cast<const uint4 *>(p);
  uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    f[2 * j] = bf16_bits_to_float(w[j] & 0xffffu);
    f[2 * j + 1] = bf16_bits_to_float(w[j] >> 16);
  }
}

template <> __device__ __forceinline__ void load8<__half>(const __half *p, float (&f)[8]) {
  uint4 v = *reinterpret_cast<const uint4 *>(p);
  const __half2 *h = reinterpret_cast<const __half2 *>(&v);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 x = __half22float2(h[j]);
    f[2 * j] = x.x;
    f[2 * j + 1] = x.y;
  }
}
template <int D, typename KVT>
__global__ void __launch_bounds__(ATTN_WARPS * 32)
attn_partial_kernel(const float *__restrict__ qkv, int ldq, const KVT *__restrict__ kc,
                    const KVT *__restrict__ vc, int max_seq, int nq, int nkv, int R, int RB, int CH,
                    const int *__restrict__ pos0_ptr, float *__restrict__ part_o,
                    float *__restrict__ part_ml, int nsplit) {
  constexpr int E = D / 32;
  const int G = nq / nkv;
  const int split = blockIdx.x, n_rb = (R + RB - 1) / RB;
  const int kvh = blockIdx.y / n_rb, rb = blockIdx.y % n_rb, b = blockIdx.z;
  const int r0 = rb * RB, r1 = min(R, r0 + RB), nQ = (r1 - r0) * G;
  const int pos0 = *pos0_ptr;
  const int j0 = split * CH, j1 = min(j0 + CH, pos0 + r1);      // keys [j0, j1); last row sees pos0+r1-1
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  __shared__ float q_s[ATTN_QR][D];
  __shared__ float p_s[ATTN_WARPS][ATTN_QR][32];
  __shared__ float red_m[ATTN_WARPS][ATTN_QR], red_l[ATTN_WARPS][ATTN_QR];
  extern __shared__ __align__(16) float o_s[];                   // [ATTN_WARPS][ATTN_QR][D]

  if (j0 >= j1) {                                                 // empty slice: mark and leave
    for (int qi = threadIdx.x; qi < nQ; qi += blockDim.x) {
      int r = r0 + qi / G, h = kvh * G + qi % G;
      size_t slot = ((size_t)(b * R + r) * nq + h) * nsplit + split;
      part_ml[slot * 2] = -INFINITY;
      part_ml[slot * 2 + 1] = 0.f;
    }
    return;
  }
  const float scale = rsqrtf((float)D);
  for (int idx = threadIdx.x; idx < ATTN_QR * D; idx += blockDim.x) {
    int qi = idx / D, dd = idx % D;
    float v = 0.f;
    if (qi < nQ) {
      int r = r0 + qi / G, h = kvh * G + qi % G;
      v = qkv[(size_t)(b * R + r) * ldq + (size_t)h * D + dd] * scale;
    }
    q_s[qi][dd] = v;
  }
  __syncthreads();

  const KVT *kbase = kc + ((size_t)b * nkv + kvh) * max_seq * D;
  const KVT *vbase = vc + ((size_t)b * nkv + kvh) * max_seq * D;
  float m_run[ATTN_QR], l_run[ATTN_QR], o_acc[ATTN_QR][E];
#pragma unroll
  for (int qi = 0; qi < ATTN_QR; ++qi) {
    m_run[qi] = -INFINITY; l_run[qi] = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) o_acc[qi][e] = 0.f;
  }

  for (int jb = j0 + warp * 32; jb < j1; jb += ATTN_WARPS * 32) {
    const int j = jb + lane;
    float s[ATTN_QR];
#pragma unroll
    for (int qi = 0; qi < ATTN_QR; ++qi) s[qi] = 0.f;
    if (j < j1) {
      const KVT *kr = kbase + (size_t)j * D;
      for (int c = 0; c < D / 8; ++c) {
        float kf[8];
        load8<KVT>(kr + c * 8, kf);
#pragma unroll
        for (int qi = 0; qi < ATTN_QR; ++qi) {
          const float4 qa = *reinterpret_cast<const float4 *>(&q_s[qi][c * 8]);
          const float4 qb = *reinterpret_cast<const float4 *>(&q_s[qi][c * 8 + 4]);
          s[qi] += kf[0] * qa.x + kf[1] * qa.y + kf[2] * qa.z + kf[3] * qa.w + kf[4] * qb.x +
                   kf[5] * qb.y + kf[6] * qb.z + kf[7] * qb.w;
        }
      }
    }
#pragma unroll
    for (int qi = 0; qi < ATTN_QR; ++qi) {
      if (qi < nQ) {                                  // uniform across the warp
        const int pos = pos0 + r0 + qi / G;
        const bool ok = (j < j1) && (j <= pos);
        const float sv = ok ? s[qi] : -INFINITY;
        const float m_new = fmaxf(m_run[qi], warp_max(sv));
        float p = 0.f, corr = 1.f;
        if (m_new > -INFINITY) {
          corr = __expf(m_run[qi] - m_new);           // exp(-inf) = 0 on the first block
          p = ok ? __expf(sv - m_new) : 0.f;
        }
        l_run[qi] = l_run[qi] * corr + warp_sum(p);
        m_run[qi] = m_new;
#pragma unroll
        for (int e = 0; e < E; ++e) o_acc[qi][e] *= corr;
        p_s[warp][qi][lane] = p;
      }
    }
    __syncwarp();
    const int n_here = min(32, j1 - jb);
    for (int jj = 0; jj < n_here; ++jj) {
      const KVT *vr = vbase + (size_t)(jb + jj) * D + lane * E;
      float vf[E];
#pragma unroll
      for (int e = 0; e < E; ++e) vf[e] = (float)vr[e];
#pragma unroll
      for (int qi = 0; qi < ATTN_QR; ++qi) {
        if (qi < nQ) {
          const float p = p_s[warp][qi][jj];
#pragma unroll
          for (int e = 0; e < E; ++e) o_acc[qi][e] += p * vf[e];
        }
      }
    }
    __syncwarp();
  }

  // combine the warps of the block
#pragma unroll
  for (int qi = 0; qi < ATTN_QR; ++qi) {
    if (lane == 0) { red_m[warp][qi] = m_run[qi]; red_l[warp][qi] = l_run[qi]; }
#pragma unroll
    for (int e = 0; e < E; ++e) o_s[((size_t)warp * ATTN_QR + qi) * D + lane * E + e] = o_acc[qi][e];
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < nQ * D; idx += blockDim.x) {
    int qi = idx / D, dd = idx % D;
    float m = -INFINITY;
#pragma unroll
    for (int w = 0; w < ATTN_WARPS; ++w) m = fmaxf(m, red_m[w][qi]);
    float l = 0.f, o = 0.f;
#pragma unroll
    for (int w = 0; w < ATTN_WARPS; ++w) {
      float f = red_m[w][qi] > -INFINITY ? __expf(red_m[w][qi] - m) : 0.f;
      l += red_l[w][qi] * f;
      o += o_s[((size_t)w * ATTN_QR + qi) * D + dd] * f;
    }
    int r = r0 + qi / G, h = kvh * G + qi % G;
    size_t slot = ((size_t)(b * R + r) * nq + h) * nsplit + split;
    part_o[slot * D + dd] = o;
    if (dd == 0) { part_ml[slot * 2] = m; part_ml[slot * 2 + 1] = l; }
  }
}

// One warp per (row, head): act[m][h*D + :] = sum_s w_s o_s / sum_s w_s l_s, w_s = exp(m_s - max m).
template <int D>
__global__ void attn_merge_kernel(const float *__restrict__ part_o, const float *__restrict__ part_ml,
                                  int nsplit, int n_rows_heads, int nq, float *__restrict__ act, int lda) {
  constexpr int E = D / 32;
  int lane = threadIdx.x & 31;
  int idx = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (idx >= n_rows_heads) return;
  int m = idx / nq, h = idx % nq;
  const float *ml = part_ml + (size_t)idx * nsplit * 2;
  float mx = -INFINITY;
  for (int s = 0; s < nsplit; ++s)
    if (ml[2 * s + 1] > 0.f) mx = fmaxf(mx, ml[2 * s]);
  float l = 0.f, o[E];
#pragma unroll
  for (int e = 0; e < E; ++e) o[e] = 0.f;
  for (int s = 0; s < nsplit; ++s) {
    float ls = ml[2 * s + 1];
    if (ls > 0.f) {
      float f = __expf(ml[2 * s] - mx);
      l += ls * f;
      const float *po = part_o + ((size_t)idx * nsplit + s) * D + lane * E;
#pragma unroll
      for (int e = 0; e < E; ++e) o[e] += po[e] * f;
    }
  }
  float inv = 1.f / l;
#pragma unroll
  for (int e = 0; e < E; ++e) act[(size_t)m * lda + (size_t)h * D + lane * E + e] = o[e] * inv;
}

// ------------------------------------------------------------------------------------
// a8: the lower->upper boundary of a full pass.  Only the newest row of each sequence goes
// on into the decoding layers (Section 2.2); the refill rows' outputs are dropped.
// ------------------------------------------------------------------------------------
__global__ void select_last_kernel(const float *__restrict__ x_lo, int R, int H, float *__restrict__ x_up) {
  int b = blockIdx.x;
  const float *src = x_lo + ((size_t)b * R + (R - 1)) * H;
  for (int k = threadIdx.x; k < H; k += blockDim.x) x_up[(size_t)b * H + k] = src[k];
}

// ------------------------------------------------------------------------------------
// The ExDy variant (Section 2.1, the paragraph after Eq. 4): the short passes also run the first
// L_e encoding layers, and the output of those layers, h_enc, stands where the default has the
// embedding.  h_enc of a position that has not been through the thinking layers yet is kept
// (pending row = position - lo_len) and fed to them at the next full pass.
// ------------------------------------------------------------------------------------
// pend[b][newest - lo_len][:] = x_up[b][:]
__global__ void save_pending_kernel(const float *__restrict__ x_up, float *__restrict__ pend, int pend_cap, int H,
                                    const DevState *st) {
  const int b = blockIdx.x, r = st->newest - st->lo_len;
  if (r < 0 || r >= pend_cap) return;
  float *dst = pend + ((size_t)b * pend_cap + r) * H;
  for (int k = threadIdx.x; k < H; k += blockDim.x) dst[k] = x_up[(size_t)b * H + k];
}

// x_lo[b][r][:] = pend[b][r][:] for r < R - 1, x_up[b][:] for the newest row r = R - 1
__global__ void gather_pending_kernel(const float *__restrict__ pend, int pend_cap, const float *__restrict__ x_up, int R, int H,
                                      float *__restrict__ x_lo) {
  const int b = blockIdx.x / R, r = blockIdx.x % R;
  const float *src = r < R - 1 ? pend + ((size_t)b * pend_cap + r) * H : x_up + (size_t)b * H;
  float *dst = x_lo + (size_t)blockIdx.x * H;
  for (int k = threadIdx.x; k < H; k += blockDim.x) dst[k] = src[k];
}

// dst[i] = src[i] / dst[i] += src[i], n floats (n a multiple of 4)
__global__ void copy_rows_kernel(const float *__restrict__ src, float *__restrict__ dst, size_t n4, int accumulate) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    float4 v = reinterpret_cast<const float4 *>(src)[i];
    if (accumulate) {
      const float4 d = reinterpret_cast<const float4 *>(dst)[i];
      v.x += d.x; v.y += d.y; v.z += d.z; v.w += d.w;
    }
    reinterpret_cast<float4 *>(dst)[i] = v;
  }
}

// Eq. 3-4 over a chunk of rows of the masked parallel forward: row (b, r) sits at position
// p0 + r; at a mask position (inside the prompt, or (p - (P-1)) mod tau == 0: the anchors of
// Section 2.2) the decoding layers read h_think (x), or base + h_think with the literal sum of
// Eq. 4; elsewhere they read base (h_emb, or h_enc when encoding layers are reused).
__global__ void masked_select_kernel(float *__restrict__ x, const float *__restrict__ base, int R, int H, int p0, int P,
                                     int tau, int literal_sum) {
  const int r = blockIdx.x % R, p = p0 + r;
  const bool m = p < P || (p - (P - 1)) % tau == 0;
  float *xr = x + (size_t)blockIdx.x * H;
  const float *br = base + (size_t)blockIdx.x * H;
  if (m && !literal_sum) return;
  for (int k = threadIdx.x; k < H; k += blockDim.x) xr[k] = m ? br[k] + xr[k] : br[k];
}

// x_up[b][:] = x[b][r][:]
__global__ void select_row_kernel(const float *__restrict__ x, int R, int r, int H, float *__restrict__ x_up) {
  const int b = blockIdx.x;
  const float *src = x + ((size_t)b * R + r) * H;
  for (int k = threadIdx.x; k < H; k += blockDim.x) x_up[(size_t)b * H + k] = src[k];
}

// ------------------------------------------------------------------------------------
// a9 (second half): greedy pick, lowest index on ties; a10: feed the token back.
// Two levels: ARGMAX_SLICES blocks per sequence each find the best of their slice of the
// vocabulary, then one block per sequence picks among them.  The token goes to position
// n_known of the token buffer unless a forced token already sits there (teacher forcing), and
// to out_argmax if given.
// ------------------------------------------------------------------------------------
constexpr int ARGMAX_SLICES = 16;

__device__ __forceinline__ void argmax_block_reduce(float best, int bi, float *sv, int *si) {
  sv[threadIdx.x] = best; si[threadIdx.x] = bi;
  __syncthreads();
  for (int s = blockDim.x >> 1; s > 0; s >>= 1) {
    if (threadIdx.x < s) {
      float v2 = sv[threadIdx.x + s]; int i2 = si[threadIdx.x + s];
      if (v2 > sv[threadIdx.x] || (v2 == sv[threadIdx.x] && i2 < si[threadIdx.x])) {
        sv[threadIdx.x] = v2; si[threadIdx.x] = i2;
      }
    }
    __syncthreads();
  }
}

// grid (sequences, ARGMAX_SLICES), 256 threads
__global__ void argmax_slices_kernel(const float *__restrict__ logits, int ldl, int V, float *__restrict__ part_val,
                                     int *__restrict__ part_idx, const DevState *__restrict__ st, SampleParams sp) {
  const int b = blockIdx.x, per = (V + gridDim.y - 1) / gridDim.y;
  const int i0 = blockIdx.y * per, i1 = min(V, i0 + per);
  const float *z = logits + (size_t)b * ldl;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  const int position = st->n_known;                  // where the picked token will sit
  if (per % 4 == 0 && ldl % 4 == 0) {
    // four logits per load (the slice starts on a 16-byte boundary); indices rise within a thread, so the
    // first of equal values stays
    for (int i = i0 + 4 * threadIdx.x; i < i1; i += 4 * blockDim.x) {
      if (i + 4 <= i1) {
        const float4 q = *reinterpret_cast<const float4 *>(z + i);
        const float e[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float v = pick_value(e[j], i + j, position, b, sp);
          if (v > best) { best = v; bi = i + j; }
        }
      } else {
        for (int j = i; j < i1; ++j) {
          const float v = pick_value(z[j], j, position, b, sp);
          if (v > best) { best = v; bi = j; }
        }
      }
    }
  } else {
    for (int i = i0 + threadIdx.x; i < i1; i += blockDim.x) {
      float v = pick_value(z[i], i, position, b, sp);
      if (v > best) { best = v; bi = i; }
    }
  }
  __shared__ float sv[256];
  __shared__ int si[256];
  argmax_block_reduce(best, bi, sv, si);
  if (threadIdx.x == 0) {
    part_val[b * gridDim.y + blockIdx.y] = sv[0];
    part_idx[b * gridDim.y + blockIdx.y] = si[0];
  }
}

// grid (sequences), 32 threads
__global__ void argmax_pick_kernel(const float *__restrict__ part_val, const int *__restrict__ part_idx, int n_slices,
                                   int *__restrict__ tokens, int max_seq, const DevState *__restrict__ st, int write_token,
                                   int *__restrict__ out_argmax) {
  const int b = blockIdx.x;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  for (int i = threadIdx.x; i < n_slices; i += blockDim.x) {
    float v = part_val[b * n_slices + i];
    int ix = part_idx[b * n_slices + i];
    if (v > best || (v == best && ix < bi)) { best = v; bi = ix; }
  }
  __shared__ float sv[32];
  __shared__ int si[32];
  argmax_block_reduce(best, bi, sv, si);
  if (threadIdx.x == 0) {
    int pick = si[0] == 0x7fffffff ? 0 : si[0];
    if (write_token) tokens[(size_t)b * max_seq + st->n_known] = pick;
    if (out_argmax) out_argmax[b] = pick;
  }
}

// a0: schedule counters after a pass (Section 2.2).  kind: 0 = prefill of P rows, 1 = full
// pass, 2 = decoding-layers-only pass.
__global__ void advance_state_kernel(DevState *st, int kind, int P) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  if (kind == 0) {
    st->n_known = P + 1; st->lo_len = P; st->up_len = P; st->cycle = 1;
    st->slot = 1 % st->tau; st->n_emitted = 1;
  } else {
    if (kind == 1) { st->lo_len = st->n_known; st->cycle += 1; }
    st->up_len = st->n_known;
    st->n_known += 1;
    st->slot = (st->slot + 1) % st->tau;
    st->n_emitted += 1;
  }
  st->newest = st->n_known - 1;
}

__global__ void set_int_kernel(int *p, int v) { *p = v; }

// out[b][i] = tokens[b][first + i], i < n  (the tokens a decode call produced)
__global__ void gather_tokens_kernel(const int *__restrict__ tokens, int max_seq, int first, int n,
                                     int ld_out, int *__restrict__ out) {
  int b = blockIdx.x;
  for (int i = threadIdx.x; i < n; i += blockDim.x) out[(size_t)b * ld_out + i] = tokens[(size_t)b * max_seq + first + i];
}

}  // namespace dmtd
