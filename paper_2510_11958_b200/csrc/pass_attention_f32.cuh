// Attention stage of the pass kernel for an fp32 KV cache: steps a3 (QK-norm, rotary embedding,
// KV append) and a4 (split-KV attention) in plain fp32 FMAs.
//
// With an fp32 cache the tensor-core form needs three mma.sync per product (bf16 hi/lo pairs),
// and mma.sync issues slowly on this GPU (measured: about 30 cycles per m16n8k16 per SM
// sub-partition, 2.2 us for one 64-key tile); the same tile is 0.26 M FMAs at most, the K and V
// tiles stay fp32 in shared memory (no splitting, so they arrive by asynchronous copies), and the
// result is exact fp32 arithmetic.
#pragma once

#include "pass_attention.cuh"

namespace dmtd {

constexpr int PK_F_KROW = 528;                                   // bytes per K row: 512 + 16, conflict-free 16-byte reads by 8 lanes on 8 rows
constexpr int PK_F_PARTS = 4;                                    // a score is the sum of 4 partial dot products over 32 dimensions each

// Map of the fp32 attention scratch for tiles of TK keys (at most 64: the score step maps a key to
// a lane of one of two warps).  The per-step kernel uses 64-key tiles; the pass kernel, whose
// scratch is what the weight rings leave of the SM's shared memory, 48-key tiles.
template <int TK>
struct AttnF32Map {
  static_assert(TK % 8 == 0 && TK <= 64, "tile size");
  static constexpr int TKEYS = TK;
  static constexpr int K = 0;                                    // K tile [TK][PK_F_KROW]
  static constexpr int V = K + TK * PK_F_KROW;                   // V tile [TK][128] floats
  static constexpr int Q = V + TK * PK_D * 4;                    // Q [PK_QR][128] floats, scaled by 1/sqrt(d)
  static constexpr int S = Q + PK_QR * PK_D * 4;                 // partial scores [part][TK][PK_QR]; part 0's area then holds the probabilities
  static constexpr int STAT = S + PK_F_PARTS * TK * PK_QR * 4;   // running max, running sum, rescale factor [3][PK_QR]
  static constexpr int NEW = STAT + 3 * PK_QR * 4;               // K rows of the pass [4][128], then V rows [4][128]
  static constexpr int W = NEW + 2 * PK_MAX_ROWS * PK_D * 4;     // q-norm weights, k-norm weights (floats), rotary frequencies (doubles)
  static constexpr int ROWS = W + 2 * PK_D * 4 + (PK_D / 2) * 8; // the pass's q | k | v vectors of one kv head, fp32, per row
  static constexpr int END = ROWS + PK_MAX_ROWS * PK_AT_ROW_FLOATS * 4;
  // the partial-output overlay of the combine step lies over K, V, Q and the scores (all consumed by then)
  static_assert(PK_WARPS * PK_QR * PK_OROW * 4 <= STAT, "partial-output overlay reaches the running statistics");
};
using PassF32Map = AttnF32Map<48>;
static_assert(PassF32Map::END <= PK_SCRATCH_BYTES, "fp32 attention scratch does not fit");

// QK-norm (Section 3.1's Qwen3 block) and the half-split rotary embedding of one head vector,
// one value per lane and quarter: v[j] is element lane + 32 j.
__device__ __forceinline__ void head_norm_rope(const float *w, const double *inv_freq, float eps, float scale, int pos,
                                               int lane, float (&v)[4]) {
  float ss = v[0] * v[0] + v[1] * v[1] + v[2] * v[2] + v[3] * v[3];
  ss = warp_sum(ss);
  const float inv = rsqrtf(ss / (float)PK_D + eps) * scale;
#pragma unroll
  for (int j = 0; j < 4; ++j) v[j] = v[j] * inv * w[lane + 32 * j];
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    // angle reduced to [-pi, pi] in double, then the fast sine and cosine
    double a = (double)pos * inv_freq[lane + 32 * j];
    a -= 6.283185307179586 * rint(a * 0.15915494309189535);
    float sn, cs;
    __sincosf((float)a, &sn, &cs);
    const float x0 = v[j], x1 = v[j + 2];
    v[j] = x0 * cs - x1 * sn;
    v[j + 2] = x1 * cs + x0 * sn;
  }
}

// Step a3 for one (sequence, kv head): one warp per head vector of the pass's rows.
template <class L>
__device__ __forceinline__ void attn_new_rows_f32(const PassParams &P, const PassLayer &Ly, unsigned char *sc, int b, int kvh,
                                                  int R, int pos0, bool write_cache) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = P.nq / P.nkv, nQ = R * G;
  const float *rows = reinterpret_cast<const float *>(sc + L::ROWS);
  const float *w_q = reinterpret_cast<const float *>(sc + L::W), *w_k = w_q + PK_D;
  const double *inv_freq = reinterpret_cast<const double *>(sc + L::W + 2 * PK_D * 4);
  const float scale = rsqrtf((float)PK_D);
#pragma unroll 1
  for (int task = warp; task < nQ + 2 * R; task += PK_WARPS) {
    int r, col, kind;                                   // kind 0 q, 1 k, 2 v
    if (task < nQ) { r = task / G; col = (task % G) * PK_D; kind = 0; }
    else if (task < nQ + R) { r = task - nQ; col = G * PK_D; kind = 1; }
    else { r = task - nQ - R; col = (G + 1) * PK_D; kind = 2; }
    const float *src = rows + r * PK_AT_ROW_FLOATS + col;
    float v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = src[lane + 32 * j];
    if (kind != 2) head_norm_rope(kind == 0 ? w_q : w_k, inv_freq, P.eps, kind == 0 ? scale : 1.f, pos0 + r, lane, v);
    float *dst;
    if (kind == 0) dst = reinterpret_cast<float *>(sc + L::Q) + task * PK_D;
    else dst = reinterpret_cast<float *>(sc + L::NEW) + ((kind == 2 ? PK_MAX_ROWS : 0) + r) * PK_D;
#pragma unroll
    for (int j = 0; j < 4; ++j) dst[lane + 32 * j] = v[j];
    if (kind != 0 && write_cache) {
      float *cache = reinterpret_cast<float *>(kind == 1 ? Ly.kc : Ly.vc) +
                     (((size_t)b * P.nkv + kvh) * P.max_seq + pos0 + r) * PK_D;
#pragma unroll
      for (int j = 0; j < 4; ++j) cache[lane + 32 * j] = v[j];
    }
  }
}

__device__ __forceinline__ float4 lds_f4(const unsigned char *p) { return *reinterpret_cast<const float4 *>(p); }

// One tile in shared memory, in three steps with a block sync between them: partial scores
// (reads K and Q), the softmax step (scores to probabilities, running max and sum), O += P V
// (reads V).  Key index i of the slice sits at position (i < n_cached ? j0 + i : pos_new + i -
// n_cached); query row q may see positions up to row_pos0 + q / G.
template <class L>
__device__ __forceinline__ void attn_f32_scores(unsigned char *sc, int nQ, int n_t) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float *const sm_s = reinterpret_cast<float *>(sc + L::S);
  {
    // partial scores: warp = (part, half of the tile's keys), lane = key.  Part p is dimensions
    // 32 p .. 32 p + 31; the lanes of a warp read the same Q values (one broadcast each) and
    // their own K rows (row stride 528 bytes: no bank conflicts); the four parts of a score meet
    // in the softmax step.
    const int part = warp & 3, key = (warp >> 2) * 32 + lane;
    if (key < n_t) {
      float4 kr[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) kr[j] = lds_f4(sc + L::K + key * PK_F_KROW + (part * 8 + j) * 16);
      // four query rows at a time: four independent chains of FMAs (rows beyond nQ hold whatever
      // the scratch held; nobody reads their sums)
#pragma unroll 1
      for (int q0 = 0; q0 < nQ; q0 += 4) {
        const unsigned char *qp = sc + L::Q + q0 * PK_D * 4 + part * 128;
        float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float4 qv = lds_f4(qp + e * PK_D * 4 + j * 16);
            s[e] += kr[j].x * qv.x + kr[j].y * qv.y + kr[j].z * qv.z + kr[j].w * qv.w;
          }
        }
        *reinterpret_cast<float4 *>(sm_s + (part * L::TKEYS + key) * PK_QR + q0) = make_float4(s[0], s[1], s[2], s[3]);
      }
    }
  }
}

template <class L>
__device__ __forceinline__ void attn_f32_softmax(unsigned char *sc, int nQ, int G, int n_t, int tile0, int n_cached, int j0,
                                                 int pos_new, int row_pos0) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float *const sm_s = reinterpret_cast<float *>(sc + L::S);
  float *const m_run = reinterpret_cast<float *>(sc + L::STAT), *const l_run = m_run + PK_QR, *const corr = l_run + PK_QR;
      // per query row: the tile's max joins the running max; scores become probabilities
#pragma unroll 2
      for (int q = warp; q < nQ; q += PK_WARPS) {
        float v[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int key = lane + 32 * h, idx = tile0 + key;
          const int key_pos = idx < n_cached ? j0 + idx : pos_new + (idx - n_cached);
          v[h] = -INFINITY;
          if (key < n_t && key_pos <= row_pos0 + q / G) {
            v[h] = 0.f;
#pragma unroll
            for (int p = 0; p < PK_F_PARTS; ++p) v[h] += sm_s[(p * L::TKEYS + key) * PK_QR + q];
          }
        }
        const float v0 = v[0], v1 = v[1];
        const float m_old = m_run[q];
        const float m_new = fmaxf(m_old, warp_max(fmaxf(v0, v1)));
        const float p0 = v0 > -INFINITY ? __expf(v0 - m_new) : 0.f;
        const float p1 = v1 > -INFINITY ? __expf(v1 - m_new) : 0.f;
        sm_s[lane * PK_QR + q] = p0;
        if (lane + 32 < L::TKEYS) sm_s[(lane + 32) * PK_QR + q] = p1;
        const float ps = warp_sum(p0 + p1);
        if (lane == 0) {
          const float f = m_old > -INFINITY ? __expf(m_old - m_new) : 0.f;
          corr[q] = f;
          l_run[q] = l_run[q] * f + ps;
          m_run[q] = m_new;
        }
      }
}

template <class L>
__device__ __forceinline__ void attn_f32_pv(unsigned char *sc, float (&acc)[PK_QR][4], int nQ, int n_t) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float *const corr = reinterpret_cast<const float *>(sc + L::STAT) + 2 * PK_QR;
      // O += P V: warp = key group (keys warp, warp + 8, ..), lane = 4 output dimensions
#pragma unroll
      for (int q = 0; q < PK_QR; ++q) {
        if (q < nQ) {
          const float f = corr[q];
          acc[q][0] *= f; acc[q][1] *= f; acc[q][2] *= f; acc[q][3] *= f;
        }
      }
#pragma unroll 2
      for (int key = warp; key < n_t; key += PK_WARPS) {
        const float4 vv = lds_f4(sc + L::V + (key * PK_D + lane * 4) * 4);
#pragma unroll
        for (int q4 = 0; q4 < PK_QR / 4; ++q4) {
          if (q4 * 4 < nQ) {
            const float4 pv = lds_f4(sc + L::S + (key * PK_QR + q4 * 4) * 4);
            const float pq[4] = {pv.x, pv.y, pv.z, pv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              acc[q4 * 4 + e][0] += pq[e] * vv.x; acc[q4 * 4 + e][1] += pq[e] * vv.y;
              acc[q4 * 4 + e][2] += pq[e] * vv.z; acc[q4 * 4 + e][3] += pq[e] * vv.w;
            }
          }
        }
      }
}

// The three steps on a tile that is complete in shared memory; the caller syncs before the tile's
// space is written again.
template <class L>
__device__ __forceinline__ void attn_f32_tile(unsigned char *sc, float (&acc)[PK_QR][4], int nQ, int G, int n_t, int tile0,
                                              int n_cached, int j0, int pos_new, int row_pos0) {
  attn_f32_scores<L>(sc, nQ, n_t);
  pk_sync();
  attn_f32_softmax<L>(sc, nQ, G, n_t, tile0, n_cached, j0, pos_new, row_pos0);
  pk_sync();
  attn_f32_pv<L>(sc, acc, nQ, n_t);
}

// The slice's partial result: the key groups' outputs summed, with the running max and sum, at
// slot (row0 + q / G, head0 + q % G, split), where a (row, head) owns `slot_stride` slots.
template <class L>
__device__ __forceinline__ void attn_f32_combine(unsigned char *sc, float (&acc)[PK_QR][4], int nQ, int G, int row0, int head0,
                                                 int nq, int slot_stride, int split, float *part_o, float *part_ml) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float *const m_run = reinterpret_cast<const float *>(sc + L::STAT), *const l_run = m_run + PK_QR;
    float *const o_s = reinterpret_cast<float *>(sc + PK_PA_OS);
    pk_sync();                                            // tiles consumed: their space becomes o_s
#pragma unroll
    for (int q = 0; q < PK_QR; ++q)
      if (q < nQ) *reinterpret_cast<float4 *>(o_s + (warp * PK_QR + q) * PK_OROW + lane * 4) = make_float4(acc[q][0], acc[q][1], acc[q][2], acc[q][3]);
    pk_sync();
    if ((int)threadIdx.x < nQ) {
      const int qi = threadIdx.x;
      const size_t slot = ((size_t)(row0 + qi / G) * nq + head0 + qi % G) * slot_stride + split;
      *reinterpret_cast<float2 *>(part_ml + slot * 2) = make_float2(m_run[qi], l_run[qi]);
    }
#pragma unroll 1
    for (int idx = threadIdx.x; idx < nQ * (PK_D / 4); idx += PK_THREADS) {
      const int qi = idx / (PK_D / 4), d4 = idx % (PK_D / 4);
      float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int w = 0; w < PK_WARPS; ++w) {
        const float4 v = *reinterpret_cast<const float4 *>(o_s + (w * PK_QR + qi) * PK_OROW + d4 * 4);
        sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
      }
      const size_t slot = ((size_t)(row0 + qi / G) * nq + head0 + qi % G) * slot_stride + split;
      *reinterpret_cast<float4 *>(part_o + slot * PK_D + d4 * 4) = sum;
    }
}

// Steps a3 + a4 for the items (sequence, kv head, key slice) of this block, fp32 cache.
// Per 64-key tile: scores by (key, quarter-of-d) threads with the K row in registers; softmax
// statistics by one warp per query row; P V by (key group = warp, 4 output dims = lane) threads.
__device__ __noinline__ void attention_stage_f32(const PassParams &P, const PassLayer &Ly, int R, int pos0, int nsplit, int CH) {
  const PassShared S = pass_shared();
  const int G = P.nq / P.nkv, nQ = R * G;
  const int items = P.B * P.nkv * nsplit;
  if ((int)blockIdx.x >= items) return;
  unsigned char *const sc = S.bstage;
  float *const m_run = reinterpret_cast<float *>(sc + PassF32Map::STAT), *const l_run = m_run + PK_QR;

#pragma unroll 1
  for (int item = blockIdx.x; item < items; item += gridDim.x) {
    const int split = item % nsplit, kvh = (item / nsplit) % P.nkv, b = item / (nsplit * P.nkv);
    // keys [j0, j1) of the cache, then (last slice) the R keys of the pass
    const int j0 = split * CH, j1 = min(j0 + CH, pos0);
    const int n_cached = max(0, j1 - j0);
    const int n_keys = n_cached + (split == nsplit - 1 ? R : 0);
    const float *kc = reinterpret_cast<const float *>(Ly.kc) + (((size_t)b * P.nkv + kvh) * P.max_seq + j0) * PK_D;
    const float *vc = reinterpret_cast<const float *>(Ly.vc) + (((size_t)b * P.nkv + kvh) * P.max_seq + j0) * PK_D;
    PK_SUBSTAMP(0);
    pk_sync();                                            // the previous item is done with the scratch
    // the pass's own q | k | v vectors of this kv head, the two norm weights and the rotary
    // frequencies: asynchronous 16-byte copies by all threads, a group of their own so that the
    // rows can be waited for while the cached tile is still on its way.  (Bulk copies by one
    // thread need a cross-proxy fence after the grid barrier first: 1 - 1.5 us before the request
    // was out, against 0.4 us this way.)
    {
      const int ldq = (P.nq + 2 * P.nkv) * PK_D, per_row = (G + 2) * (PK_D / 4), n_rows_units = R * per_row;
      const uint32_t sc_u32 = smem_u32(sc);
#pragma unroll 1
      for (int c = threadIdx.x; c < n_rows_units + 96; c += PK_THREADS) {
        if (c < n_rows_units) {
          const int r = c / per_row, u = c - r * per_row, hd = u >> 5, part = u & 31;
          const int col = hd < G ? (kvh * G + hd) * PK_D : hd == G ? (P.nq + kvh) * PK_D : (P.nq + P.nkv + kvh) * PK_D;
          cp_async16(sc_u32 + PassF32Map::ROWS + (r * PK_AT_ROW_FLOATS + hd * PK_D) * 4 + part * 16,
                     P.qkv + (size_t)(b * R + r) * ldq + col + part * 4);
        } else {
          const int w = c - n_rows_units;                     // 32 + 32 units of norm weights, 32 of frequencies
          const void *src = w < 32 ? (const void *)(Ly.w_qn + w * 4) : w < 64 ? (const void *)(Ly.w_kn + (w - 32) * 4)
                                                                              : (const void *)(P.inv_freq + (w - 64) * 2);
          cp_async16(sc_u32 + PassF32Map::W + w * 16, src);
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    PK_SUBSTAMP(1);
    // cached rows of a tile: asynchronous 16-byte copies, 32 of K and 32 of V per row
    auto fetch_cached = [&](int tile0) {
      const int n_c = min(PassF32Map::TKEYS, n_cached - tile0);
#pragma unroll 1
      for (int c = threadIdx.x; c < n_c * 64; c += PK_THREADS) {
        const int row = c >> 6, u = c & 63;
        const uint32_t dst = smem_u32(sc) + (u < 32 ? PassF32Map::K + row * PK_F_KROW + u * 16 : PassF32Map::V + row * PK_D * 4 + (u - 32) * 16);
        cp_async16(dst, (u < 32 ? kc : vc) + (size_t)(tile0 + row) * PK_D + (u & 31) * 4);
      }
    };
    fetch_cached(0);                                      // in flight while the pass's own rows arrive
    PK_SUBSTAMP(2);
    if ((int)threadIdx.x < PK_QR) { m_run[threadIdx.x] = -INFINITY; l_run[threadIdx.x] = 0.f; }
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 1;" ::: "memory");   // the rows' group; the tile's may still be open
    pk_sync();
    PK_SUBSTAMP(3);
    attn_new_rows_f32<PassF32Map>(P, Ly, sc, b, kvh, R, pos0, split == 0);
    PK_SUBSTAMP(4);

    float acc[PK_QR][4];
#pragma unroll
    for (int q = 0; q < PK_QR; ++q) acc[q][0] = acc[q][1] = acc[q][2] = acc[q][3] = 0.f;
#pragma unroll 1
    for (int tile0 = 0; tile0 < n_keys; tile0 += PassF32Map::TKEYS) {
      const int n_t = min(PassF32Map::TKEYS, n_keys - tile0);
      pk_sync();                                          // new rows written / previous tile consumed
      PK_SUBSTAMP(8);
      if (tile0 > 0) fetch_cached(tile0);
      // the pass's own rows that fall into this tile
#pragma unroll 1
      for (int c = threadIdx.x + max(0, n_cached - tile0) * 64; c < n_t * 64; c += PK_THREADS) {
        const int row = c >> 6, u = c & 63, r = tile0 + row - n_cached;
        const float4 val = lds_f4(sc + PassF32Map::NEW + (((u < 32 ? 0 : PK_MAX_ROWS) + r) * PK_D + (u & 31) * 4) * 4);
        *reinterpret_cast<float4 *>(sc + (u < 32 ? PassF32Map::K + row * PK_F_KROW + u * 16 : PassF32Map::V + row * PK_D * 4 + (u - 32) * 16)) = val;
      }
      PK_SUBSTAMP(9);
      cp_async_wait_all();
      pk_sync();
      PK_SUBSTAMP(10);
      attn_f32_tile<PassF32Map>(sc, acc, nQ, G, n_t, tile0, n_cached, j0, pos0, pos0);
    }
    PK_SUBSTAMP(5);
    attn_f32_combine<PassF32Map>(sc, acc, nQ, G, b * R, kvh * G, P.nq, PK_NSPLIT_CAP, split, P.part_o, P.part_ml);
    PK_SUBSTAMP(6);
  }
  pk_sync();
  PK_SUBSTAMP(7);
}

}  // namespace dmtd
