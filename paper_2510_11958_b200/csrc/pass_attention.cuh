// Attention stage of the pass kernel: steps a3 (QK-norm, rotary embedding, KV append) and a4
// (split-KV attention on the tensor cores; the key slices are merged by the O projection's
// prologue).
//
// This file is the tensor-core form, used with a bf16 cache: Q, K, P and V enter the MMAs as
// single bf16 values.  fp32 caches run the FMA form (pass_attention_f32.cuh): fp32 accuracy on
// the tensor cores would take three mma.sync per product (bf16 hi + lo pairs), which issue too
// slowly here.  On the 36-layer model a bf16 cache alone moves the logits by up to 0.05, an fp32
// cache by 1e-4.
#pragma once

#include "pass_prologues.cuh"

namespace dmtd {

// Profiling builds: clock64() of thread 0 of the first block at points inside the attention
// stage (the last layer's values stay), in the 16 slots before the wall-clock slots.
#ifdef DMTD_PASS_TIMING
#define PK_SUBSTAMP(i)                                                                     \
  do {                                                                                     \
    if (threadIdx.x == 0 && blockIdx.x == 0 && P.timing) P.timing[4096 - 4 - 16 + (i)] = clock64(); \
  } while (0)
#else
#define PK_SUBSTAMP(i) do {} while (0)
#endif

constexpr int PK_TK = 64;                                     // keys per shared-memory tile
constexpr int PK_KROW = 320;                                  // bytes per K row: 256 + 64, conflict-free 16-byte operand loads
constexpr int PK_VROW = 272;                                  // bytes per V row: 256 + 16, conflict-free ldmatrix
constexpr int PK_QROW = 272;
constexpr int PK_OROW = PK_D + 8;                             // floats per partial-output row, padded against bank conflicts
// layout of the attention scratch (the activation staging area and the row staging area behind it)
constexpr int PK_AT_KH = 0;                                   // K tile, hi parts [PK_TK][PK_KROW]
constexpr int PK_AT_KL = PK_AT_KH + PK_TK * PK_KROW;          // second K tile (the standalone kernel's double buffer)
constexpr int PK_AT_VH = PK_AT_KL + PK_TK * PK_KROW;          // V tile, hi parts [PK_TK][PK_VROW]
constexpr int PK_AT_VL = PK_AT_VH + PK_TK * PK_VROW;          // second V tile
constexpr int PK_AT_QH = PK_AT_VL + PK_TK * PK_VROW;          // Q tile [PK_QR][PK_QROW], hi then lo
constexpr int PK_AT_QL = PK_AT_QH + PK_QR * PK_QROW;
constexpr int PK_AT_NEW = PK_AT_QL + PK_QR * PK_QROW;         // K rows of the pass [4][128] floats, then V rows [4][128]
constexpr int PK_AT_TILES_END = PK_AT_NEW + 2 * PK_MAX_ROWS * PK_D * 4;
constexpr int PK_AT_OS = 0;                                   // after the tiles are consumed: [warps][16][PK_OROW] floats
constexpr int PK_AT_RED = 90112;                              // running max [warps][16], then sum / merge factor [warps][16]
constexpr int PK_AT_ROWS = PK_AT_RED + 2 * PK_WARPS * PK_QR * 4;   // the pass's q | k | v vectors of one kv head, fp32, per row
constexpr int PK_AT_ROW_FLOATS = (PK_MAX_GROUP + 2) * PK_D;
constexpr int PK_AT_END = PK_AT_ROWS + PK_MAX_ROWS * PK_AT_ROW_FLOATS * 4;
static_assert(PK_AT_TILES_END <= PK_AT_RED && PK_WARPS * PK_QR * PK_OROW * 4 <= PK_AT_RED, "attention scratch overlaps");
// The pass kernel keeps one tile of each kind, so its map of the same pieces is more compact (its
// scratch is what the weight rings leave of the SM's shared memory):
constexpr int PK_PA_KH = 0;                                   // K tile [PK_TK][PK_KROW]
constexpr int PK_PA_VH = PK_PA_KH + PK_TK * PK_KROW;          // V tile [PK_TK][PK_VROW]
constexpr int PK_PA_QH = PK_PA_VH + PK_TK * PK_VROW;          // Q tile [PK_QR][PK_QROW], and a second one kept zero
constexpr int PK_PA_NEW = PK_PA_QH + 2 * PK_QR * PK_QROW;     // K rows of the pass [4][128] floats, then V rows [4][128]
constexpr int PK_PA_TILES_END = PK_PA_NEW + 2 * PK_MAX_ROWS * PK_D * 4;
constexpr int PK_PA_OS = 0;                                   // after the tiles are consumed: [warps][16][PK_OROW] floats
constexpr int PK_PA_RED = PK_WARPS * PK_QR * PK_OROW * 4;     // running max [warps][16], then sum / merge factor [warps][16]
constexpr int PK_PA_ROWS = PK_PA_RED + 2 * PK_WARPS * PK_QR * 4;   // the pass's q | k | v vectors of one kv head, fp32, per row
constexpr int PK_PA_W = PK_PA_ROWS + PK_MAX_ROWS * PK_AT_ROW_FLOATS * 4;   // q-norm, k-norm weights (floats), rotary frequencies (doubles)
constexpr int PK_PA_END = PK_PA_W + 2 * PK_D * 4 + (PK_D / 2) * 8;
static_assert(PK_PA_TILES_END <= PK_PA_RED, "attention scratch overlaps");
static_assert(PK_PA_END <= PK_SCRATCH_BYTES, "attention scratch does not fit");

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}

// Key slices of one (sequence, kv head): nsplit slices of CH cached keys; the last slice also
// takes the R keys of the pass itself.
__device__ __forceinline__ void attn_plan_device(const PassParams &P, int pos0, int &nsplit, int &CH) {
  int want = max(1, min(PK_NSPLIT_CAP, (int)gridDim.x / (P.B * P.nkv)));
  CH = max(1, (pos0 + want - 1) / want);
  CH = (CH + 7) & ~7;
  nsplit = max(1, (pos0 + CH - 1) / CH);
}

// 8 values -> 16 bytes of bf16.
template <class Op>
__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
  return make_uint4(Op::pack2(f[0], f[1]), Op::pack2(f[2], f[3]), Op::pack2(f[4], f[5]), Op::pack2(f[6], f[7]));
}

// Step a3 for one (sequence, kv head): one warp per head vector of the pass's rows (staged in
// shared memory as q heads | k | v per row).  Query rows go to the Q tile (scaled by 1/sqrt(d));
// K and V rows go to the new-row area as floats already rounded to the cache's type and, from
// the block that owns slice 0, into the cache.
template <class Op>
__device__ __forceinline__ void attn_new_rows(const PassParams &P, const PassLayer &Ly, unsigned char *sc, int b, int kvh,
                                              int R, int pos0, bool write_cache) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = P.nq / P.nkv, nQ = R * G;
  const float *rows = reinterpret_cast<const float *>(sc + PK_PA_ROWS);
  const float *w_q = reinterpret_cast<const float *>(sc + PK_PA_W), *w_k = w_q + PK_D;
  const double *inv_freq = reinterpret_cast<const double *>(sc + PK_PA_W + 2 * PK_D * 4);
  const float scale = rsqrtf((float)PK_D);
#pragma unroll 1
  for (int task = warp; task < nQ + 2 * R; task += PK_WARPS) {
    int r, col, kind;                                   // kind 0 q, 1 k, 2 v
    if (task < nQ) { r = task / G; col = (task % G) * PK_D; kind = 0; }
    else if (task < nQ + R) { r = task - nQ; col = G * PK_D; kind = 1; }
    else { r = task - nQ - R; col = (G + 1) * PK_D; kind = 2; }
    const float *src = rows + r * PK_AT_ROW_FLOATS + col;
    const int pos = pos0 + r;
    float v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = src[lane + 32 * j];
    if (kind != 2) {
      float ss = v[0] * v[0] + v[1] * v[1] + v[2] * v[2] + v[3] * v[3];
      ss = warp_sum(ss);
      const float inv = rsqrtf(ss / (float)PK_D + P.eps) * (kind == 0 ? scale : 1.f);
      const float *w = kind == 0 ? w_q : w_k;
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
    if (kind == 0) {
      typename Op::T *qh = reinterpret_cast<typename Op::T *>(sc + PK_PA_QH + task * PK_QROW);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        qh[lane + 32 * j] = Op::from_float(v[j]);
      }
    } else {
      float *row = reinterpret_cast<float *>(sc + PK_PA_NEW) + ((kind == 2 ? PK_MAX_ROWS : 0) + r) * PK_D;
      const size_t at = (((size_t)b * P.nkv + kvh) * P.max_seq + pos) * PK_D;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const typename Op::T h = Op::from_float(v[j]);
        row[lane + 32 * j] = Op::to_float(h);
        if (write_cache) reinterpret_cast<typename Op::T *>(kind == 1 ? Ly.kc : Ly.vc)[at + lane + 32 * j] = h;
      }
    }
  }
}

// One 64-key tile against the 16 query rows.  Warp w takes keys 16 (w & 3) .. + 15 of the tile
// and output dimensions 64 (w >> 2) .. + 63: the two warps of a key group compute the same
// scores and each multiplies them with its half of V.  acc holds the warp's running max, running
// sum (per lane, summed over the four lanes of a row at the end) and output.
struct AttnAcc {
  float m_run[2], l_part[2];
  float o[8][4];
};

// Keys of the tile are key_idx0 + row; key index i sits at position (i < n_cached ? j0 + i :
// pos_new + i - n_cached); query row q may see positions up to row_pos0 + q / G.
// k_off / v_off: where the tile's K and V (hi parts) sit in the scratch.  The Q fragments are
// read from shared memory in a rolled loop: the code stays short (instruction fetch, not
// arithmetic, bounds a stage that runs once per layer).
template <class Op>
__device__ __forceinline__ void attn_tile_compute(AttnAcc &A, unsigned char *sc, int n_t, int tile0, int n_cached, int j0,
                                                  int pos_new, int row_pos0, int G, int k_off = PK_PA_KH,
                                                  int v_off = PK_PA_VH) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int kg = warp & 3, dh = warp >> 2;
  const uint32_t kh_tile = smem_u32(sc + k_off);
  const uint32_t vh_tile = smem_u32(sc + v_off);
  const uint32_t qh_tile = smem_u32(sc + PK_PA_QH);
  float (&m_run)[2] = A.m_run;
  float (&l_part)[2] = A.l_part;
  float (&o)[8][4] = A.o;
  if (kg * 16 >= n_t) return;
  float c[2][4];
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f;
#pragma unroll 1
  for (int kb = 0; kb < 4; ++kb) {
    const uint32_t q_off = g * PK_QROW + kb * 64 + t * 16;
    const uint4 q0 = lds128(qh_tile + q_off), q1 = lds128(qh_tile + q_off + 8 * PK_QROW);
    #pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const uint32_t off = (kg * 16 + nt * 8 + g) * PK_KROW + kb * 64 + t * 16;
      const uint4 Kh = lds128(kh_tile + off);
      Op::mma(c[nt], q0.x, q1.x, q0.y, q1.y, Kh.x, Kh.y);
      Op::mma(c[nt], q0.z, q1.z, q0.w, q1.w, Kh.z, Kh.w);
    }
  }
  // causal / range mask: lane holds rows g (e = 0, 1) and g + 8 (e = 2, 3), keys 2t, 2t + 1 of each n-tile
  float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int kl = kg * 16 + nt * 8 + 2 * t + (e & 1), idx = tile0 + kl, row = g + (e >> 1) * 8;
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
  const uint32_t v_row = (kg * 16 + (mi & 1) * 8 + rr) * PK_VROW + (mi >> 1) * 16 + dh * 128;
#pragma unroll
  for (int d2 = 0; d2 < 4; ++d2) {
    uint32_t b0, b1, b2, b3;
    ldmatrix_x4_trans(vh_tile + v_row + d2 * 32, b0, b1, b2, b3);
    o[2 * d2][0] *= corr[0]; o[2 * d2][1] *= corr[0]; o[2 * d2][2] *= corr[1]; o[2 * d2][3] *= corr[1];
    o[2 * d2 + 1][0] *= corr[0]; o[2 * d2 + 1][1] *= corr[0]; o[2 * d2 + 1][2] *= corr[1]; o[2 * d2 + 1][3] *= corr[1];
    Op::mma(o[2 * d2], ah[0], ah[1], ah[2], ah[3], b0, b1);
    Op::mma(o[2 * d2 + 1], ah[0], ah[1], ah[2], ah[3], b2, b3);
  }
}

// Combine the key groups of the block into the slice's partial result: unnormalised output with
// its max and sum, written to part_o / part_ml at slot (row0 + q / G, head0 + q % G, split),
// where a (row, head) owns `slot_stride` consecutive slots.
constexpr int PK_KGROUPS = 4;
__device__ __forceinline__ void attn_combine_store(AttnAcc &A, unsigned char *sc, int nQ, int G, int row0, int head0, int nq,
                                                   int slot_stride, int split, float *part_o, float *part_ml) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int kg = warp & 3, dh = warp >> 2;
  float *const o_s = reinterpret_cast<float *>(sc + PK_PA_OS);
  float *const red_m = reinterpret_cast<float *>(sc + PK_PA_RED);
  float *const red_l = red_m + PK_WARPS * PK_QR;
  float (&m_run)[2] = A.m_run;
  float (&l_part)[2] = A.l_part;
  float (&o)[8][4] = A.o;
  pk_sync();                                            // tiles consumed: their space becomes o_s
#pragma unroll
  for (int hr = 0; hr < 2; ++hr) {
    l_part[hr] += __shfl_xor_sync(0xffffffffu, l_part[hr], 1);
    l_part[hr] += __shfl_xor_sync(0xffffffffu, l_part[hr], 2);
    if (t == 0 && dh == 0) { red_m[kg * PK_QR + g + 8 * hr] = m_run[hr]; red_l[kg * PK_QR + g + 8 * hr] = l_part[hr]; }
  }
#pragma unroll
  for (int hr = 0; hr < 2; ++hr) {
    if (g + 8 * hr < nQ) {
      float *dst = o_s + (kg * PK_QR + g + 8 * hr) * PK_OROW + dh * 64 + 2 * t;
#pragma unroll
      for (int dt = 0; dt < 8; ++dt) *reinterpret_cast<float2 *>(dst + dt * 8) = make_float2(o[dt][2 * hr], o[dt][2 * hr + 1]);
    }
  }
  pk_sync();
  // per query row: the slice's max and sum, and the factor each key group's share is scaled by
  if ((int)threadIdx.x < nQ) {
    const int qi = threadIdx.x;
    float m = -INFINITY;
#pragma unroll
    for (int w = 0; w < PK_KGROUPS; ++w) m = fmaxf(m, red_m[w * PK_QR + qi]);
    float l = 0.f;
#pragma unroll
    for (int w = 0; w < PK_KGROUPS; ++w) {
      const float mw = red_m[w * PK_QR + qi];
      const float f = mw > -INFINITY ? __expf(mw - m) : 0.f;
      l += red_l[w * PK_QR + qi] * f;
      red_l[w * PK_QR + qi] = f;
    }
    const size_t slot = ((size_t)(row0 + qi / G) * nq + head0 + qi % G) * slot_stride + split;
    *reinterpret_cast<float2 *>(part_ml + slot * 2) = make_float2(m, l);
  }
  pk_sync();
#pragma unroll 1
  for (int idx = threadIdx.x; idx < nQ * (PK_D / 4); idx += PK_THREADS) {
    const int qi = idx / (PK_D / 4), d4 = idx % (PK_D / 4);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int w = 0; w < PK_KGROUPS; ++w) {
      const float f = red_l[w * PK_QR + qi];
      const float4 v = *reinterpret_cast<const float4 *>(o_s + (w * PK_QR + qi) * PK_OROW + d4 * 4);
      acc.x += v.x * f; acc.y += v.y * f; acc.z += v.z * f; acc.w += v.w * f;
    }
    const size_t slot = ((size_t)(row0 + qi / G) * nq + head0 + qi % G) * slot_stride + split;
    *reinterpret_cast<float4 *>(part_o + slot * PK_D + d4 * 4) = acc;
  }
}

// Steps a3 + a4 for the items (sequence, kv head, key slice) of this block.  The R*G query rows
// of an item form one m16 tile; S = Q K^T and O = P V run as mma.m16n8k16 with K and V staged in
// shared memory, each warp taking 16 keys of a 64-key tile with its own running max and sum.
// The slice's unnormalised partial output goes to global memory with its max and sum; the
// prologue of the O projection merges the slices.
template <class Op>
__device__ __noinline__ void attention_stage(const PassParams &P, const PassLayer &Ly, int R, int pos0, int nsplit, int CH) {
  const PassShared S = pass_shared();
  const int G = P.nq / P.nkv, nQ = R * G;
  const int items = P.B * P.nkv * nsplit;
  if ((int)blockIdx.x >= items) return;

  unsigned char *const sc = S.bstage;
  const uint32_t kh_tile = smem_u32(sc + PK_PA_KH);
  const uint32_t vh_tile = smem_u32(sc + PK_PA_VH);
  const uint32_t qh_tile = smem_u32(sc + PK_PA_QH);
  // a 16-byte part (8 values) of a tile row: parts 0..15 are K, 16..31 are V
  auto put_part = [&](int row, int part, const float (&f)[8]) {
    const uint4 hi = pack8<Op>(f);
    const uint32_t off = part < 16 ? row * PK_KROW + part * 16 : row * PK_VROW + (part - 16) * 16;
    sts128((part < 16 ? kh_tile : vh_tile) + off, hi);
  };

#pragma unroll 1
  for (int item = blockIdx.x; item < items; item += gridDim.x) {
    const int split = item % nsplit, kvh = (item / nsplit) % P.nkv, b = item / (nsplit * P.nkv);
    // keys [j0, j1) of the cache, then (last slice) the R keys of the pass
    const int j0 = split * CH, j1 = min(j0 + CH, pos0);
    const int n_cached = max(0, j1 - j0);
    const int n_keys = n_cached + (split == nsplit - 1 ? R : 0);
    const size_t head_off = ((size_t)b * P.nkv + kvh) * P.max_seq * PK_D;
    // cached rows of a tile
    auto fetch_cached = [&](int tile0) {
      const int n_c = min(PK_TK, n_cached - tile0);
      // bf16 cache: asynchronous copies, 16 bytes each
      const typename Op::T *kb = reinterpret_cast<const typename Op::T *>(Ly.kc) + head_off;
      const typename Op::T *vb = reinterpret_cast<const typename Op::T *>(Ly.vc) + head_off;
#pragma unroll 1
      for (int c = threadIdx.x; c < n_c * 32; c += PK_THREADS) {
        const int row = c >> 5, part = c & 31;
        const uint32_t dst = part < 16 ? kh_tile + row * PK_KROW + part * 16 : vh_tile + row * PK_VROW + (part - 16) * 16;
        cp_async16(dst, (part < 16 ? kb : vb) + (size_t)(j0 + tile0 + row) * PK_D + (part & 15) * 8);
      }
    
    };
    PK_SUBSTAMP(0);
    pk_sync();                                            // the previous item is done with the scratch
    // the pass's own q | k | v vectors of this kv head, the two norm weights and the rotary frequencies:
    // asynchronous 16-byte copies by all threads, a group of their own so that the rows can be waited for while
    // the cached tile is still on its way.  (Bulk copies by one thread need a cross-proxy fence after the grid
    // barrier first and are issued one after the other: 0.9 us before the request was out.)
    {
      const int ldq = (P.nq + 2 * P.nkv) * PK_D, per_row = (G + 2) * (PK_D / 4), n_rows_units = R * per_row;
      const uint32_t sc_u32 = smem_u32(sc);
#pragma unroll 1
      for (int c = threadIdx.x; c < n_rows_units + 96; c += PK_THREADS) {
        if (c < n_rows_units) {
          const int r = c / per_row, u = c - r * per_row, hd = u >> 5, part = u & 31;
          const int col = hd < G ? (kvh * G + hd) * PK_D : hd == G ? (P.nq + kvh) * PK_D : (P.nq + P.nkv + kvh) * PK_D;
          cp_async16(sc_u32 + PK_PA_ROWS + (r * PK_AT_ROW_FLOATS + hd * PK_D) * 4 + part * 16,
                     P.qkv + (size_t)(b * R + r) * ldq + col + part * 4);
        } else {
          const int w = c - n_rows_units;                     // 32 + 32 units of norm weights, 32 of frequencies
          const void *src = w < 32 ? (const void *)(Ly.w_qn + w * 4) : w < 64 ? (const void *)(Ly.w_kn + (w - 32) * 4)
                                                                              : (const void *)(P.inv_freq + (w - 64) * 2);
          cp_async16(sc_u32 + PK_PA_W + w * 16, src);
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    PK_SUBSTAMP(1);
    fetch_cached(0);                                      // in flight while the pass's own rows arrive
    PK_SUBSTAMP(2);
    // query rows beyond nQ are zero (the previous item's partial outputs lay over the Q tiles)
#pragma unroll 1
    for (int i = threadIdx.x; i < 2 * PK_QR * PK_QROW / 16; i += PK_THREADS) sts128(qh_tile + i * 16, make_uint4(0u, 0u, 0u, 0u));
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 1;" ::: "memory");   // the rows' group; the tile's may still be open
    pk_sync();
    PK_SUBSTAMP(3);
    attn_new_rows<Op>(P, Ly, sc, b, kvh, R, pos0, split == 0);
    PK_SUBSTAMP(4);

    AttnAcc A;
    A.m_run[0] = A.m_run[1] = -INFINITY;
    A.l_part[0] = A.l_part[1] = 0.f;
#pragma unroll
    for (int dt = 0; dt < 8; ++dt) A.o[dt][0] = A.o[dt][1] = A.o[dt][2] = A.o[dt][3] = 0.f;
#pragma unroll 1
    for (int tile0 = 0; tile0 < n_keys; tile0 += PK_TK) {
      const int n_t = min(PK_TK, n_keys - tile0);
      pk_sync();                                          // new rows written / previous tile consumed
      PK_SUBSTAMP(8);
      if (tile0 > 0) fetch_cached(tile0);
#pragma unroll 1
      for (int c = threadIdx.x + max(0, n_cached - tile0) * 32; c < n_t * 32; c += PK_THREADS) {
        const int row = c >> 5, part = c & 31, r = tile0 + row - n_cached;
        const float *src = reinterpret_cast<const float *>(sc + PK_PA_NEW) + ((part < 16 ? 0 : PK_MAX_ROWS) + r) * PK_D + (part & 15) * 8;
        const float f[8] = {src[0], src[1], src[2], src[3], src[4], src[5], src[6], src[7]};
        put_part(row, part, f);
      }
      const int n16 = min(PK_TK, (n_t + 15) & ~15);
#pragma unroll 1
      for (int c = threadIdx.x; c < (n16 - n_t) * 16; c += PK_THREADS) {    // P = 0 times stale bits must stay 0
        const uint32_t off = (n_t + (c >> 4)) * PK_VROW + (c & 15) * 16;
        sts128(vh_tile + off, make_uint4(0u, 0u, 0u, 0u));
      }
      PK_SUBSTAMP(9);
      cp_async_wait_all();
      pk_sync();
      PK_SUBSTAMP(10);
      attn_tile_compute<Op>(A, sc, n_t, tile0, n_cached, j0, pos0, pos0, G);
    }
    PK_SUBSTAMP(5);
    attn_combine_store(A, sc, nQ, G, b * R, kvh * G, P.nq, PK_NSPLIT_CAP, split, P.part_o, P.part_ml);
    PK_SUBSTAMP(6);
  }
  pk_sync();
  PK_SUBSTAMP(7);
}

}  // namespace dmtd
