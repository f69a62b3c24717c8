// Step a4 as a kernel of its own, for the per-step path (prefill, batches the pass kernel does
// not take) and for dmtd_attention_decode: split-KV attention on the tensor cores.  One block
// per (key slice, kv head x row block, sequence); the G query heads of the kv head for up to
// 16 / G new positions form one m16 tile of query rows that share every key and value the block
// stages in shared memory.  Same tile arithmetic as the attention stage of the pass kernel;
// the slices are merged by attn_merge_kernel.
#pragma once

#include "pass_attention_f32.cuh"

namespace dmtd {

// Work layout of this kernel's tiles: each of the first four warps takes 16 keys of a 64-key tile
// against all 128 output dimensions, with the Q fragments in registers.  (The pass kernel's
// attention stage spreads one tile over all eight warps, two per key group, which halves the
// latency of its single tile but repeats the Q K^T products; here, where tiles follow one another
// and mma.sync issue is the limit, the repeated products cost 10 % of the throughput.)
// One 64-key tile against the 16 query rows: this warp's 16 keys.  acc holds the warp's running
// max, running sum (per lane, summed over the four lanes of a row at the end) and output.
struct AttnAccW {
  float m_run[2], l_part[2];
  float o[16][4];
};

// Keys of the tile are key_idx0 + row; key index i sits at position (i < n_cached ? j0 + i :
// pos_new + i - n_cached); query row q may see positions up to row_pos0 + q / G.
// k_off / v_off: where the tile's K and V (hi parts) sit in the scratch.
template <class Op>
// kg: which 16 keys of the tile this call takes (the decode kernel gives every warp its own group,
// the prefill kernel walks all four with every warp).
__device__ __forceinline__ void attn_tile_compute_w(AttnAccW &A, unsigned char *sc, const uint4 (&qh)[4][2], int n_t, int tile0,
                                                  int n_cached, int j0, int pos_new, int row_pos0, int G,
                                                  int k_off, int v_off, int kg) {
  const int warp = kg, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const uint32_t kh_tile = smem_u32(sc + k_off);
  const uint32_t vh_tile = smem_u32(sc + v_off);
  float (&m_run)[2] = A.m_run;
  float (&l_part)[2] = A.l_part;
  float (&o)[16][4] = A.o;
  if (warp * 16 < n_t) {
        float c[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f;
#pragma unroll
          for (int kb = 0; kb < 4; ++kb) {
            const uint32_t off = (warp * 16 + nt * 8 + g) * PK_KROW + kb * 64 + t * 16;
            const uint4 Kh = lds128(kh_tile + off);
            Op::mma(c[nt], qh[kb][0].x, qh[kb][1].x, qh[kb][0].y, qh[kb][1].y, Kh.x, Kh.y);
            Op::mma(c[nt], qh[kb][0].z, qh[kb][1].z, qh[kb][0].w, qh[kb][1].w, Kh.z, Kh.w);
          }
        }
        // causal / range mask: lane holds rows g (e = 0, 1) and g + 8 (e = 2, 3), keys 2t, 2t + 1 of each n-tile
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int kl = warp * 16 + nt * 8 + 2 * t + (e & 1), idx = tile0 + kl, row = g + (e >> 1) * 8;
            const int key_pos = idx < n_cached ? j0 + idx : pos_new + (idx - n_cached);
            const bool ok = kl < n_t && key_pos <= row_pos0 + row / G;
            c[nt][e] = ok ? c[nt][e] : -INFINITY;
            mx[e >> 1] = fmaxf(mx[e >> 1], c[nt][e]);
          }
        }
        float corr[2];
#pragma unroll
        for (int hr = 0; hr < 2; ++hr) {
          mx[hr] = fmaxf(mx[hr], __shfl_xor_sync(0xffffffffu, mx[hr], 1));
          mx[hr] = fmaxf(mx[hr], __shfl_xor_sync(0xffffffffu, mx[hr], 2));
          const float m_new = fmaxf(m_run[hr], mx[hr]);
          corr[hr] = m_new > -INFINITY ? __expf(m_run[hr] - m_new) : 1.f;
          m_run[hr] = m_new;
        }
        float psum[2] = {0.f, 0.f};
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float p = c[nt][e] > -INFINITY ? __expf(c[nt][e] - m_run[e >> 1]) : 0.f;
            c[nt][e] = p;
            psum[e >> 1] += p;
          }
        }
        l_part[0] = l_part[0] * corr[0] + psum[0];
        l_part[1] = l_part[1] * corr[1] + psum[1];
        // P as the A operand: hi parts and (fp32 cache) lo parts
        uint32_t ah[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float p0 = c[i >> 1][(i & 1) * 2], p1 = c[i >> 1][(i & 1) * 2 + 1];
          ah[i] = Op::pack2(p0, p1);
        }
        const int mi = lane >> 3, rr = lane & 7;
        const uint32_t v_off = (warp * 16 + (mi & 1) * 8 + rr) * PK_VROW + (mi >> 1) * 16;
#pragma unroll
        for (int d2 = 0; d2 < 8; ++d2) {
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4_trans(vh_tile + v_off + d2 * 32, b0, b1, b2, b3);
          o[2 * d2][0] *= corr[0]; o[2 * d2][1] *= corr[0]; o[2 * d2][2] *= corr[1]; o[2 * d2][3] *= corr[1];
          o[2 * d2 + 1][0] *= corr[0]; o[2 * d2 + 1][1] *= corr[0]; o[2 * d2 + 1][2] *= corr[1]; o[2 * d2 + 1][3] *= corr[1];
          Op::mma(o[2 * d2], ah[0], ah[1], ah[2], ah[3], b0, b1);
          Op::mma(o[2 * d2 + 1], ah[0], ah[1], ah[2], ah[3], b2, b3);
        }
      }
}

// The same tile with the operands swapped, for at most 8 query rows (one new position of up to 8
// query heads per KV head: every decode pass of a batch).  With the query rows on the M axis an
// m16 tile is three quarters padding at 4 rows, and mma.sync issue, not HBM, bounds the kernel
// (128 MMAs per 64-key tile).  Here the 16 keys of the warp are the M axis of S^T = K Q^T and the
// 128 output dimensions the M axis of O^T = V^T P^T, the query rows the 8 columns: 64 MMAs per tile.
// Accumulator layout: thread (g, t) holds columns (query rows) 2t, 2t + 1 of rows g and g + 8.
struct AttnAccS {
  float m_run[2], l_part[2];       // per query row 2t, 2t + 1: running max, this lane's share of the running sum
  float o[8][4];                   // O^T: m-tile dt = dimensions 16 dt .. + 15
};

template <class Op>
__device__ __forceinline__ void attn_tile_compute_swap(AttnAccS &A, unsigned char *sc, const uint4 (&qh)[4], int n_t, int tile0,
                                                       int j0, int row_pos0, int G, int k_off, int v_off) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const uint32_t kh_tile = smem_u32(sc + k_off);
  const uint32_t vh_tile = smem_u32(sc + v_off);
  if (warp * 16 >= n_t) return;
  // S^T = K Q^T: A = the warp's 16 key rows (the same permutation of the 32 dimensions of a k block
  // on both operands: a lane's 16 bytes are dimensions 8t .. 8t + 7), B = the query rows
  float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int kb = 0; kb < 4; ++kb) {
    const uint32_t off = (warp * 16 + g) * PK_KROW + kb * 64 + t * 16;
    const uint4 K0 = lds128(kh_tile + off), K1 = lds128(kh_tile + off + 8 * PK_KROW);
    Op::mma(c, K0.x, K1.x, K0.y, K1.y, qh[kb].x, qh[kb].y);
    Op::mma(c, K0.z, K1.z, K0.w, K1.w, qh[kb].z, qh[kb].w);
  }
  // mask: rows are keys g, g + 8 of the warp's 16, columns query rows 2t, 2t + 1
  float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const int kl = warp * 16 + g + (e >> 1) * 8, q = 2 * t + (e & 1);
    const bool ok = kl < n_t && j0 + tile0 + kl <= row_pos0 + q / G;
    c[e] = ok ? c[e] : -INFINITY;
    mx[e & 1] = fmaxf(mx[e & 1], c[e]);
  }
  float corr[2];
#pragma unroll
  for (int hq = 0; hq < 2; ++hq) {
    // over the warp's 16 keys: the 8 lanes that share t
    mx[hq] = fmaxf(mx[hq], __shfl_xor_sync(0xffffffffu, mx[hq], 4));
    mx[hq] = fmaxf(mx[hq], __shfl_xor_sync(0xffffffffu, mx[hq], 8));
    mx[hq] = fmaxf(mx[hq], __shfl_xor_sync(0xffffffffu, mx[hq], 16));
    const float m_new = fmaxf(A.m_run[hq], mx[hq]);
    corr[hq] = m_new > -INFINITY ? __expf(A.m_run[hq] - m_new) : 1.f;
    A.m_run[hq] = m_new;
  }
  float psum[2] = {0.f, 0.f};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float p = c[e] > -INFINITY ? __expf(c[e] - A.m_run[e & 1]) : 0.f;
    c[e] = p;
    psum[e & 1] += p;
  }
  A.l_part[0] = A.l_part[0] * corr[0] + psum[0];
  A.l_part[1] = A.l_part[1] * corr[1] + psum[1];
  // P^T as the B operand (k = key, n = query row): lane (g, t) needs keys 2t, 2t + 1 (and + 8) of query
  // row g; they sit in lanes (2t, g / 2) and (2t + 1, g / 2), element g & 1 of each pair
  const uint32_t x = Op::pack2(c[0], c[1]), y = Op::pack2(c[2], c[3]);
  const int src_a = (2 * t) * 4 + (g >> 1), src_b = (2 * t + 1) * 4 + (g >> 1);
  const uint32_t xa = __shfl_sync(0xffffffffu, x, src_a), xb = __shfl_sync(0xffffffffu, x, src_b);
  const uint32_t ya = __shfl_sync(0xffffffffu, y, src_a), yb = __shfl_sync(0xffffffffu, y, src_b);
  const uint32_t sel = (g & 1) ? 0x7632u : 0x5410u;       // high or low halves of the two words
  const uint32_t b0 = __byte_perm(xa, xb, sel), b1 = __byte_perm(ya, yb, sel);
  // O^T += V^T P^T: A = V^T (m = dimension, k = key) through ldmatrix.trans of the key rows
  const int mi = lane >> 3, rr = lane & 7;
  const uint32_t v_row = (warp * 16 + (mi >> 1) * 8 + rr) * PK_VROW + (mi & 1) * 16;
#pragma unroll
  for (int dt = 0; dt < 8; ++dt) {
    uint32_t a0, a1, a2, a3;
    ldmatrix_x4_trans(vh_tile + v_row + dt * 32, a0, a1, a2, a3);
    A.o[dt][0] *= corr[0]; A.o[dt][1] *= corr[1]; A.o[dt][2] *= corr[0]; A.o[dt][3] *= corr[1];
    Op::mma(A.o[dt], a0, a1, a2, a3, b0, b1);
  }
}

// Combine of the swapped layout: the warps' partial outputs O^T go to shared memory as [warp][query
// row][dimension], then as in attn_combine_store_w.
__device__ __forceinline__ void attn_combine_store_swap(AttnAccS &A, unsigned char *sc, int nQ, int G, int row0, int head0,
                                                        int nq, int slot_stride, int split, float *part_o, float *part_ml) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  float *const o_s = reinterpret_cast<float *>(sc + PK_AT_OS);
  float *const red_m = reinterpret_cast<float *>(sc + PK_AT_RED);
  float *const red_l = red_m + PK_WARPS * PK_QR;
  pk_sync();                                            // tiles consumed: their space becomes o_s
#pragma unroll
  for (int hq = 0; hq < 2; ++hq) {
    float l = A.l_part[hq];
    l += __shfl_xor_sync(0xffffffffu, l, 4);
    l += __shfl_xor_sync(0xffffffffu, l, 8);
    l += __shfl_xor_sync(0xffffffffu, l, 16);
    if (g == 0) { red_m[warp * PK_QR + 2 * t + hq] = A.m_run[hq]; red_l[warp * PK_QR + 2 * t + hq] = l; }
  }
  if (warp < 4) {
#pragma unroll
    for (int dt = 0; dt < 8; ++dt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int q = 2 * t + (e & 1), d = dt * 16 + g + (e >> 1) * 8;
        if (q < nQ) o_s[(warp * PK_QR + q) * PK_OROW + d] = A.o[dt][e];
      }
    }
  }
  pk_sync();
  // warps 4 - 7 took no keys: their running max stays -inf and their share is skipped
  if ((int)threadIdx.x < nQ) {
    const int qi = threadIdx.x;
    float m = -INFINITY;
#pragma unroll
    for (int w = 0; w < 4; ++w) m = fmaxf(m, red_m[w * PK_QR + qi]);
    float l = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float mw = red_m[w * PK_QR + qi];
      const float f = mw > -INFINITY ? __expf(mw - m) : 0.f;
      l += red_l[w * PK_QR + qi] * f;
      red_l[w * PK_QR + qi] = f;
    }
    const size_t slot = ((size_t)(row0 + qi / G) * nq + head0 + qi % G) * slot_stride + split;
    part_ml[slot * 2] = m;
    part_ml[slot * 2 + 1] = l;
  }
  pk_sync();
  for (int idx = threadIdx.x; idx < nQ * (PK_D / 4); idx += PK_THREADS) {
    const int qi = idx / (PK_D / 4), d4 = idx % (PK_D / 4);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float f = red_l[w * PK_QR + qi];
      if (f != 0.f) {
        const float4 v = *reinterpret_cast<const float4 *>(o_s + (w * PK_QR + qi) * PK_OROW + d4 * 4);
        acc.x += v.x * f; acc.y += v.y * f; acc.z += v.z * f; acc.w += v.w * f;
      }
    }
    const size_t slot = ((size_t)(row0 + qi / G) * nq + head0 + qi % G) * slot_stride + split;
    *reinterpret_cast<float4 *>(part_o + slot * PK_D + d4 * 4) = acc;
  }
}

// Combine the warps of the block into the slice's partial result: unnormalised output with its
// max and sum, written to part_o / part_ml at slot (row0 + q / G, head0 + q % G, split), where a
// (row, head) owns `slot_stride` consecutive slots.
__device__ __forceinline__ void attn_combine_store_w(AttnAccW &A, unsigned char *sc, int nQ, int G, int row0, int head0, int nq,
                                                   int slot_stride, int split, float *part_o, float *part_ml) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  float *const o_s = reinterpret_cast<float *>(sc + PK_AT_OS);
  float *const red_m = reinterpret_cast<float *>(sc + PK_AT_RED);
  float *const red_l = red_m + PK_WARPS * PK_QR;
  float (&m_run)[2] = A.m_run;
  float (&l_part)[2] = A.l_part;
  float (&o)[16][4] = A.o;
  // combine the warps into this slice's partial result
  pk_sync();                                            // tiles consumed: their space becomes o_s
#pragma unroll
  for (int hr = 0; hr < 2; ++hr) {
    l_part[hr] += __shfl_xor_sync(0xffffffffu, l_part[hr], 1);
    l_part[hr] += __shfl_xor_sync(0xffffffffu, l_part[hr], 2);
    if (t == 0) { red_m[warp * PK_QR + g + 8 * hr] = m_run[hr]; red_l[warp * PK_QR + g + 8 * hr] = l_part[hr]; }
  }
  if (g < nQ) {
#pragma unroll
    for (int dt = 0; dt < 16; ++dt)
      *reinterpret_cast<float2 *>(o_s + (warp * PK_QR + g) * PK_OROW + dt * 8 + 2 * t) = make_float2(o[dt][0], o[dt][1]);
  }
  if (g + 8 < nQ) {
#pragma unroll
    for (int dt = 0; dt < 16; ++dt)
      *reinterpret_cast<float2 *>(o_s + (warp * PK_QR + g + 8) * PK_OROW + dt * 8 + 2 * t) = make_float2(o[dt][2], o[dt][3]);
  }
  pk_sync();
  // per query row: the slice's max and sum, and the factor each warp's share is scaled by
  if ((int)threadIdx.x < nQ) {
    const int qi = threadIdx.x;
    float m = -INFINITY;
#pragma unroll
    for (int w = 0; w < PK_WARPS; ++w) m = fmaxf(m, red_m[w * PK_QR + qi]);
    float l = 0.f;
#pragma unroll
    for (int w = 0; w < PK_WARPS; ++w) {
      const float mw = red_m[w * PK_QR + qi];
      const float f = mw > -INFINITY ? __expf(mw - m) : 0.f;
      l += red_l[w * PK_QR + qi] * f;
      red_l[w * PK_QR + qi] = f;
    }
    const size_t slot = ((size_t)(row0 + qi / G) * nq + head0 + qi % G) * slot_stride + split;
    part_ml[slot * 2] = m;
    part_ml[slot * 2 + 1] = l;
  }
  pk_sync();
  for (int idx = threadIdx.x; idx < nQ * (PK_D / 4); idx += PK_THREADS) {
    const int qi = idx / (PK_D / 4), d4 = idx % (PK_D / 4);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int w = 0; w < PK_WARPS; ++w) {
      const float f = red_l[w * PK_QR + qi];
      const float4 v = *reinterpret_cast<const float4 *>(o_s + (w * PK_QR + qi) * PK_OROW + d4 * 4);
      acc.x += v.x * f; acc.y += v.y * f; acc.z += v.z * f; acc.w += v.w * f;
    }
    const size_t slot = ((size_t)(row0 + qi / G) * nq + head0 + qi % G) * slot_stride + split;
    *reinterpret_cast<float4 *>(part_o + slot * PK_D + d4 * 4) = acc;
  }
}


constexpr int ATTN_TC_NEW = PK_AT_ROWS;          // fused form: K rows of the pass [ATTN_TC_MAX_NEW][128] (cache type), then V rows
constexpr int ATTN_TC_MAX_NEW = 15;              // new positions per sequence the fused form takes (more: the prefill kernel)
constexpr int ATTN_TC_SMEM = ATTN_TC_NEW + 2 * ATTN_TC_MAX_NEW * PK_D * 2;   // tiles, Q, partial-output overlay, reduction arrays, new rows
static_assert(2 * (ATTN_TC_SMEM + 1024) <= 228 * 1024, "two blocks per SM");

// What the fused form of attn_tc_kernel needs for step a3 (QK-norm, rotary embedding, KV append): with these the
// kernel reads the raw q | k | v rows of the QKV projection itself; every block normalises and rotates its own
// query rows and the new K rows that fall into its key slice (a few rows, recomputed by the blocks that share
// them), and the block that owns a position appends its K and V rows to the cache.  w_qn == nullptr: the rows in
// qkv are finished already and the new K / V rows are in the cache (the stand-alone attention call).
struct AttnFuse {
  const float *w_qn, *w_kn;        // QK-norm weights [128]
  const float2 *table;             // (cos, sin) of the pass's positions [R][64]
  float eps;
};
// QK-norm and rotary embedding of one head vector, one value per lane and quarter (v[j] = element lane + 32 j).
__device__ __forceinline__ void head_norm_rope_table(const float *w, const float2 *cs_row, float eps, int lane, float (&v)[4]) {
  float ss = v[0] * v[0] + v[1] * v[1] + v[2] * v[2] + v[3] * v[3];
  ss = warp_sum(ss);
  const float inv = rsqrtf(ss / (float)PK_D + eps);
#pragma unroll
  for (int j = 0; j < 4; ++j) v[j] = v[j] * inv * w[lane + 32 * j];
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const float2 cs = cs_row[lane + 32 * j];
    const float a = v[j], bb = v[j + 2];
    v[j] = a * cs.x - bb * cs.y;
    v[j + 2] = bb * cs.x + a * cs.y;
  }
}

// qkv [B*R][ldq]: q heads already normalised and rotated (not scaled); K and V of the new rows
// already in the cache.  Cache [b][kv head][max_seq][128] bf16.
template <class Op, bool FUSED = false>
__global__ void __launch_bounds__(PK_THREADS, 2)      // 16-bit cache: two blocks per SM overlap load and math
attn_tc_kernel(const float *__restrict__ qkv, int ldq, const void *__restrict__ kc, const void *__restrict__ vc, int max_seq,
               int nq, int nkv, int R, int RB, int CH, const int *__restrict__ pos0_ptr, float *__restrict__ part_o,
               float *__restrict__ part_ml, int nsplit, AttnFuse F = AttnFuse{nullptr, nullptr, nullptr, 0.f}) {
  extern __shared__ __align__(1024) unsigned char sc[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int G = nq / nkv, n_rb = (R + RB - 1) / RB;
  const int split = blockIdx.x, kvh = blockIdx.y / n_rb, rb = blockIdx.y % n_rb, b = blockIdx.z;
  const int r0 = rb * RB, r1 = min(R, r0 + RB), nQ = (r1 - r0) * G;
  const int pos0 = *pos0_ptr;
  const int j0 = split * CH, j1 = min(j0 + CH, pos0 + r1);      // the last row of the block sees position pos0 + r1 - 1
  if (j0 >= j1) {                                                 // empty slice: mark and leave
    for (int qi = threadIdx.x; qi < nQ; qi += PK_THREADS) {
      const size_t slot = ((size_t)(b * R + r0 + qi / G) * nq + kvh * G + qi % G) * nsplit + split;
      part_ml[slot * 2] = -INFINITY;
      part_ml[slot * 2 + 1] = 0.f;
    }
    return;
  }
  const uint32_t kh_tile = smem_u32(sc + PK_AT_KH), vh_tile = smem_u32(sc + PK_AT_VH);
  const uint32_t qh_tile = smem_u32(sc + PK_AT_QH);
  // Q tile: rows beyond nQ zero; row qi = (position r0 + qi / G, head kvh*G + qi % G), scaled by 1/sqrt(d)
  for (int i = threadIdx.x; i < 2 * PK_QR * PK_QROW / 16; i += PK_THREADS) sts128(qh_tile + i * 16, make_uint4(0u, 0u, 0u, 0u));
  __syncthreads();
  const float scale = rsqrtf((float)PK_D);
  for (int qi = warp; qi < nQ; qi += PK_WARPS) {
    const float *src = qkv + (size_t)(b * R + r0 + qi / G) * ldq + (size_t)(kvh * G + qi % G) * PK_D;
    typename Op::T *qh = reinterpret_cast<typename Op::T *>(sc + PK_AT_QH + qi * PK_QROW);
    float v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = src[lane + 32 * j];
    if (FUSED) head_norm_rope_table(F.w_qn, F.table + (size_t)(r0 + qi / G) * (PK_D / 2), F.eps, lane, v);
#pragma unroll
    for (int j = 0; j < 4; ++j) qh[lane + 32 * j] = Op::from_float(v[j] * scale);
  }
  const size_t head_off = ((size_t)b * nkv + kvh) * max_seq * PK_D;
  const int n_keys = j1 - j0;
  // fused form: the pass's rows r_lo .. r_hi - 1 sit at positions inside this block's key slice; their K and V
  // come from the projection's output, not from the cache
  const int r_lo = FUSED ? max(0, j0 - pos0) : 0, r_hi = FUSED ? max(r_lo, min(r1, j1 - pos0)) : 0;
  if (FUSED) {
    typename Op::T *new_k = reinterpret_cast<typename Op::T *>(sc + ATTN_TC_NEW);
    typename Op::T *new_v = new_k + ATTN_TC_MAX_NEW * PK_D;
    for (int task = warp; task < 2 * (r_hi - r_lo); task += PK_WARPS) {
      const int r = r_lo + (task >> 1), is_v = task & 1;
      const float *src = qkv + (size_t)(b * R + r) * ldq + (size_t)(nq + (is_v ? nkv : 0) + kvh) * PK_D;
      float v[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) v[j] = src[lane + 32 * j];
      if (!is_v) head_norm_rope_table(F.w_kn, F.table + (size_t)r * (PK_D / 2), F.eps, lane, v);
      typename Op::T *row = (is_v ? new_v : new_k) + (r - r_lo) * PK_D;
      typename Op::T *cache = const_cast<typename Op::T *>(reinterpret_cast<const typename Op::T *>(is_v ? vc : kc)) + head_off +
                              (size_t)(pos0 + r) * PK_D;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const typename Op::T h = Op::from_float(v[j]);
        row[lane + 32 * j] = h;
        if (r >= r0) cache[lane + 32 * j] = h;           // the row block that owns the position appends it
      }
    }
  }
  // bf16 cache: two tile buffers (the lo-part areas are free here), tile i+1 in flight while
  // tile i is multiplied
  const typename Op::T *kb = reinterpret_cast<const typename Op::T *>(kc) + head_off;
  const typename Op::T *vb = reinterpret_cast<const typename Op::T *>(vc) + head_off;
  auto fetch = [&](int tile0, int buf) {
    const int n_t = min(PK_TK, n_keys - tile0);
    const int n_c = FUSED ? max(0, min(n_t, pos0 - (j0 + tile0))) : n_t;       // rows of the tile that come from the cache
    const uint32_t k_t = smem_u32(sc + (buf ? PK_AT_KL : PK_AT_KH)), v_t = smem_u32(sc + (buf ? PK_AT_VL : PK_AT_VH));
    for (int c = threadIdx.x; c < n_c * 32; c += PK_THREADS) {
      const int row = c >> 5, part = c & 31;
      const uint32_t dst = part < 16 ? k_t + row * PK_KROW + part * 16 : v_t + row * PK_VROW + (part - 16) * 16;
      cp_async16(dst, (part < 16 ? kb : vb) + (size_t)(j0 + tile0 + row) * PK_D + (part & 15) * 8);
    }
    const int n16 = min(PK_TK, (n_t + 15) & ~15);
    for (int c = threadIdx.x; c < (n16 - n_t) * 16; c += PK_THREADS)      // P = 0 times stale bits must stay 0
      sts128(v_t + (n_t + (c >> 4)) * PK_VROW + (c & 15) * 16, make_uint4(0u, 0u, 0u, 0u));
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  // fused form: the pass's own rows of a tile, from the new-row area (written before the barrier in front of the
  // tile's multiplication; the tile buffer is free: the tile two trips back has been consumed)
  auto place_new = [&](int tile0, int buf) {
    if (!FUSED) return;
    const int n_t = min(PK_TK, n_keys - tile0);
    const int first = max(0, pos0 - (j0 + tile0));                             // first row of the tile that is a new row
    const uint32_t k_t = smem_u32(sc + (buf ? PK_AT_KL : PK_AT_KH)), v_t = smem_u32(sc + (buf ? PK_AT_VL : PK_AT_VH));
    for (int c = threadIdx.x + first * 32; c < n_t * 32; c += PK_THREADS) {
      const int row = c >> 5, part = c & 31, r = j0 + tile0 + row - pos0 - r_lo;
      const uint4 val = *reinterpret_cast<const uint4 *>(sc + ATTN_TC_NEW + ((part < 16 ? 0 : ATTN_TC_MAX_NEW) + r) * PK_D * 2 + (part & 15) * 16);
      sts128(part < 16 ? k_t + row * PK_KROW + part * 16 : v_t + row * PK_VROW + (part - 16) * 16, val);
    }
  };
  fetch(0, 0);
  int buf = 0;
  if (nQ <= 8) {
    // at most 8 query rows (a decode pass): keys and output dimensions on the M axis of the MMAs
    AttnAccS A;
    A.m_run[0] = A.m_run[1] = -INFINITY;
    A.l_part[0] = A.l_part[1] = 0.f;
#pragma unroll
    for (int dt = 0; dt < 8; ++dt) A.o[dt][0] = A.o[dt][1] = A.o[dt][2] = A.o[dt][3] = 0.f;
    uint4 qs[4];
    for (int tile0 = 0; tile0 < n_keys; tile0 += PK_TK, buf ^= 1) {
      const int n_t = min(PK_TK, n_keys - tile0);
      if (tile0 + PK_TK < n_keys) {
        fetch(tile0 + PK_TK, buf ^ 1);
        asm volatile("cp.async.wait_group 1;" ::: "memory");
      } else {
        asm volatile("cp.async.wait_group 0;" ::: "memory");
      }
      if (FUSED && tile0 == 0) __syncthreads();         // the new-row area is written
      place_new(tile0, buf);
      __syncthreads();                                  // tile (and, the first time, Q) visible to all
      if (tile0 == 0) {
#pragma unroll
        for (int kbk = 0; kbk < 4; ++kbk) qs[kbk] = lds128(qh_tile + g * PK_QROW + kbk * 64 + t * 16);
      }
      attn_tile_compute_swap<Op>(A, sc, qs, n_t, tile0, j0, pos0 + r0, G, buf ? PK_AT_KL : PK_AT_KH, buf ? PK_AT_VL : PK_AT_VH);
      __syncthreads();                                  // done with this buffer before it is refilled
    }
    attn_combine_store_swap(A, sc, nQ, G, b * R + r0, kvh * G, nq, nsplit, split, part_o, part_ml);
    return;
  }
  AttnAccW A;
  A.m_run[0] = A.m_run[1] = -INFINITY;
  A.l_part[0] = A.l_part[1] = 0.f;
#pragma unroll
  for (int dt = 0; dt < 16; ++dt) A.o[dt][0] = A.o[dt][1] = A.o[dt][2] = A.o[dt][3] = 0.f;
  uint4 qh[4][2];
  for (int tile0 = 0; tile0 < n_keys; tile0 += PK_TK, buf ^= 1) {
    const int n_t = min(PK_TK, n_keys - tile0);
    if (tile0 + PK_TK < n_keys) {
      fetch(tile0 + PK_TK, buf ^ 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    if (FUSED && tile0 == 0) __syncthreads();           // the new-row area is written
    place_new(tile0, buf);
    __syncthreads();                                    // tile (and, the first time, Q) visible to all
    if (tile0 == 0) {
#pragma unroll
      for (int kbk = 0; kbk < 4; ++kbk) {
        qh[kbk][0] = lds128(qh_tile + g * PK_QROW + kbk * 64 + t * 16);
        qh[kbk][1] = lds128(qh_tile + (g + 8) * PK_QROW + kbk * 64 + t * 16);
      }
    }
    attn_tile_compute_w<Op>(A, sc, qh, n_t, tile0, 0x7fffffff, j0, 0, pos0 + r0, G, buf ? PK_AT_KL : PK_AT_KH,
                             buf ? PK_AT_VL : PK_AT_VH, warp);
    __syncthreads();                                    // done with this buffer before it is refilled
  }
  attn_combine_store_w(A, sc, nQ, G, b * R + r0, kvh * G, nq, nsplit, split, part_o, part_ml);
}

// Causal attention of a chunk of R new positions per sequence (the prefill, Section 2.2: all prompt
// rows through all layers) for a 16-bit cache, flash-attention style: a block takes 8 x (16 / G)
// consecutive positions of one (sequence, kv head), every warp owns 16 query rows (16 / G positions
// x G heads) with their running max, sum and output in registers, and all warps share the 64-key
// tiles of K and V that stream through shared memory once per block.  No key slices and no merge:
// the normalised rows go straight to out [B*R][ld].  (The decode kernel above, run over 4-position
// row blocks, re-read the keys before every row block: the prefill was bound by L2, not by HBM.)
constexpr int ATTN_PF_Q = PK_AT_QH;                                    // Q tiles [warp][16][PK_QROW] behind the two K / V buffers
constexpr int ATTN_PF_SMEM = ATTN_PF_Q + PK_WARPS * PK_QR * PK_QROW;

template <class Op>
__global__ void __launch_bounds__(PK_THREADS, 2)
attn_prefill_kernel(const float *__restrict__ qkv, int ldq, const void *__restrict__ kc, const void *__restrict__ vc, int max_seq,
                    int nq, int nkv, int R, const int *__restrict__ pos0_ptr, float *__restrict__ out, int ld) {
  extern __shared__ __align__(1024) unsigned char sc[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int G = nq / nkv, PW = PK_QR / G, QB = PK_WARPS * PW;         // positions per warp and per block
  const int kvh = blockIdx.y, b = blockIdx.z;
  const int r0 = blockIdx.x * QB, r1 = min(R, r0 + QB);
  const int pos0 = *pos0_ptr;
  const int wr0 = r0 + warp * PW, wr1 = min(R, wr0 + PW);             // this warp's positions [wr0, wr1) of the chunk
  // Q tile of the warp: row i = (position wr0 + i / G, head kvh * G + i % G), scaled by 1/sqrt(d); rows past the chunk zero
  const float scale = rsqrtf((float)PK_D);
  typename Op::T *qt = reinterpret_cast<typename Op::T *>(sc + ATTN_PF_Q + warp * PK_QR * PK_QROW);
  for (int i = 0; i < PK_QR; ++i) {
    const int r = wr0 + i / G;
    const float *src = qkv + (size_t)(b * R + min(r, R - 1)) * ldq + (size_t)(kvh * G + i % G) * PK_D;
#pragma unroll
    for (int j = 0; j < 4; ++j)
      qt[i * (PK_QROW / 2) + lane + 32 * j] = Op::from_float(r < R ? src[lane + 32 * j] * scale : 0.f);
  }
  __syncwarp();
  uint4 qh[4][2];
  const uint32_t q_u32 = smem_u32(qt);
#pragma unroll
  for (int kbk = 0; kbk < 4; ++kbk) {
    qh[kbk][0] = lds128(q_u32 + g * PK_QROW + kbk * 64 + t * 16);
    qh[kbk][1] = lds128(q_u32 + (g + 8) * PK_QROW + kbk * 64 + t * 16);
  }
  const size_t head_off = ((size_t)b * nkv + kvh) * max_seq * PK_D;
  const typename Op::T *kb = reinterpret_cast<const typename Op::T *>(kc) + head_off;
  const typename Op::T *vb = reinterpret_cast<const typename Op::T *>(vc) + head_off;
  const int n_keys = pos0 + r1;                                       // the block's last position sees keys [0, pos0 + r1)
  auto fetch = [&](int tile0, int buf) {
    const int n_t = min(PK_TK, n_keys - tile0);
    const uint32_t k_t = smem_u32(sc + (buf ? PK_AT_KL : PK_AT_KH)), v_t = smem_u32(sc + (buf ? PK_AT_VL : PK_AT_VH));
    for (int c = threadIdx.x; c < n_t * 32; c += PK_THREADS) {
      const int row = c >> 5, part = c & 31;
      const uint32_t dst = part < 16 ? k_t + row * PK_KROW + part * 16 : v_t + row * PK_VROW + (part - 16) * 16;
      cp_async16(dst, (part < 16 ? kb : vb) + (size_t)(tile0 + row) * PK_D + (part & 15) * 8);
    }
    const int n16 = min(PK_TK, (n_t + 15) & ~15);
    for (int c = threadIdx.x; c < (n16 - n_t) * 16; c += PK_THREADS)      // P = 0 times stale bits must stay 0
      sts128(v_t + (n_t + (c >> 4)) * PK_VROW + (c & 15) * 16, make_uint4(0u, 0u, 0u, 0u));
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  AttnAccW A;
  A.m_run[0] = A.m_run[1] = -INFINITY;
  A.l_part[0] = A.l_part[1] = 0.f;
#pragma unroll
  for (int dt = 0; dt < 16; ++dt) A.o[dt][0] = A.o[dt][1] = A.o[dt][2] = A.o[dt][3] = 0.f;
  fetch(0, 0);
  int buf = 0;
  const int last_pos = pos0 + wr1 - 1;                                // the warp's last row sees keys up to here
  for (int tile0 = 0; tile0 < n_keys; tile0 += PK_TK, buf ^= 1) {
    const int n_t = min(PK_TK, n_keys - tile0);
    if (tile0 + PK_TK < n_keys) {
      fetch(tile0 + PK_TK, buf ^ 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();                                    // the tile is visible to all
    if (wr0 < wr1) {
#pragma unroll 1
      for (int kg = 0; kg < 4; ++kg)
        if (tile0 + kg * 16 <= last_pos)
          attn_tile_compute_w<Op>(A, sc, qh, n_t, tile0, 0x7fffffff, 0, 0, pos0 + wr0, G, buf ? PK_AT_KL : PK_AT_KH,
                                  buf ? PK_AT_VL : PK_AT_VH, kg);
    }
    __syncthreads();                                    // done with this buffer before it is refilled
  }
  // normalise and store: lane (g, t) holds rows g and g + 8, columns 8 dt + 2t, + 1
#pragma unroll
  for (int hr = 0; hr < 2; ++hr) {
    float l = A.l_part[hr];
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    const int i = g + 8 * hr, r = wr0 + i / G;
    if (r < wr1) {
      const float inv = 1.f / l;
      float *dst = out + (size_t)(b * R + r) * ld + (size_t)(kvh * G + i % G) * PK_D + 2 * t;
#pragma unroll
      for (int dt = 0; dt < 16; ++dt)
        *reinterpret_cast<float2 *>(dst + dt * 8) = make_float2(A.o[dt][2 * hr] * inv, A.o[dt][2 * hr + 1] * inv);
    }
  }
}

// The same step for an fp32 cache in plain FMAs (three mma.sync per product would be needed for
// fp32 accuracy, and they issue too slowly): the tile arithmetic of the pass kernel's fp32
// attention stage, one 64-key tile in shared memory per block and two blocks per SM, so that one
// block's copies run under the other's arithmetic.
using StepF32Map = AttnF32Map<64>;
constexpr int ATTN_F32_SMEM = StepF32Map::NEW;           // K and V tile, Q, partial scores, running max / sum / rescale factor

__global__ void __launch_bounds__(PK_THREADS, 2)
attn_f32_kernel(const float *__restrict__ qkv, int ldq, const float *__restrict__ kc, const float *__restrict__ vc, int max_seq,
                int nq, int nkv, int R, int RB, int CH, const int *__restrict__ pos0_ptr, float *__restrict__ part_o,
                float *__restrict__ part_ml, int nsplit) {
  extern __shared__ __align__(1024) unsigned char sc[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = nq / nkv, n_rb = (R + RB - 1) / RB;
  const int split = blockIdx.x, kvh = blockIdx.y / n_rb, rb = blockIdx.y % n_rb, b = blockIdx.z;
  const int r0 = rb * RB, r1 = min(R, r0 + RB), nQ = (r1 - r0) * G;
  const int pos0 = *pos0_ptr;
  const int j0 = split * CH, j1 = min(j0 + CH, pos0 + r1);      // the last row of the block sees position pos0 + r1 - 1
  if (j0 >= j1) {                                                 // empty slice: mark and leave
    for (int qi = threadIdx.x; qi < nQ; qi += PK_THREADS) {
      const size_t slot = ((size_t)(b * R + r0 + qi / G) * nq + kvh * G + qi % G) * nsplit + split;
      part_ml[slot * 2] = -INFINITY;
      part_ml[slot * 2 + 1] = 0.f;
    }
    return;
  }
  // Q rows, scaled by 1/sqrt(d): row qi = (position r0 + qi / G, head kvh*G + qi % G)
  const float scale = rsqrtf((float)PK_D);
  for (int qi = warp; qi < nQ; qi += PK_WARPS) {
    const float *src = qkv + (size_t)(b * R + r0 + qi / G) * ldq + (size_t)(kvh * G + qi % G) * PK_D;
    float *dst = reinterpret_cast<float *>(sc + StepF32Map::Q) + qi * PK_D;
#pragma unroll
    for (int j = 0; j < 4; ++j) dst[lane + 32 * j] = src[lane + 32 * j] * scale;
  }
  float *const m_run = reinterpret_cast<float *>(sc + StepF32Map::STAT), *const l_run = m_run + PK_QR;
  if ((int)threadIdx.x < PK_QR) { m_run[threadIdx.x] = -INFINITY; l_run[threadIdx.x] = 0.f; }
  const float *kb = kc + (((size_t)b * nkv + kvh) * max_seq + j0) * PK_D;
  const float *vb = vc + (((size_t)b * nkv + kvh) * max_seq + j0) * PK_D;
  float acc[PK_QR][4];
#pragma unroll
  for (int q = 0; q < PK_QR; ++q) acc[q][0] = acc[q][1] = acc[q][2] = acc[q][3] = 0.f;
  const int n_keys = j1 - j0;
  // The K and the V tile are loaded as two groups of asynchronous copies, each re-issued for the
  // next tile as soon as the step that reads it is over: K of tile i + 1 arrives under the
  // softmax step and P V of tile i, V of tile i + 1 under the scores of tile i + 1.
  auto fetch = [&](const float *rows, int tile0, int dst_off, int row_bytes) {
    const int n_t = min(PK_TK, n_keys - tile0);
#pragma unroll 1
    for (int c = threadIdx.x; c < n_t * 32; c += PK_THREADS) {
      const int row = c >> 5, u = c & 31;
      if (tile0 < n_keys) cp_async16(smem_u32(sc) + dst_off + row * row_bytes + u * 16, rows + (size_t)(tile0 + row) * PK_D + u * 4);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");      // an empty group past the last tile keeps the counts uniform
  };
  fetch(kb, 0, StepF32Map::K, PK_F_KROW);
  fetch(vb, 0, StepF32Map::V, PK_D * 4);
#pragma unroll 1
  for (int tile0 = 0; tile0 < n_keys; tile0 += PK_TK) {
    const int n_t = min(PK_TK, n_keys - tile0);
    asm volatile("cp.async.wait_group 1;" ::: "memory");      // K of this tile (V may still be on its way)
    __syncthreads();                                      // ... from every thread; the first time also Q and the statistics
    attn_f32_scores<StepF32Map>(sc, nQ, n_t);
    __syncthreads();                                      // K consumed
    fetch(kb, tile0 + PK_TK, StepF32Map::K, PK_F_KROW);
    // every key comes from the cache: key index i sits at position j0 + i
    attn_f32_softmax<StepF32Map>(sc, nQ, G, n_t, tile0, 0x7fffffff, j0, 0, pos0 + r0);
    asm volatile("cp.async.wait_group 1;" ::: "memory");      // V of this tile (the next K may still be on its way)
    __syncthreads();                                      // probabilities and V from every thread
    attn_f32_pv<StepF32Map>(sc, acc, nQ, n_t);
    __syncthreads();                                      // V and the probabilities consumed
    fetch(vb, tile0 + PK_TK, StepF32Map::V, PK_D * 4);
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  attn_f32_combine<StepF32Map>(sc, acc, nQ, G, b * R + r0, kvh * G, nq, nsplit, split, part_o, part_ml);
}

}  // namespace dmtd
