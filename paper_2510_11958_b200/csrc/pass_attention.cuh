// Attention stage of the pass kernel: steps a3 (QK-norm, rotary embedding, KV append) and a4
// (split-KV attention on the tensor cores, online-softmax merge of the key slices).
#pragma once

#include "pass_prologues.cuh"

namespace dmtd {

constexpr int PK_TK = 64;                                     // keys per shared-memory tile
constexpr int PK_KROW = 320;                                  // bytes per K row: 256 + 64, conflict-free 16-byte operand loads
constexpr int PK_VROW = 272;                                  // bytes per V row: 256 + 16, conflict-free ldmatrix
constexpr int PK_QROW = 272;
// layout of the attention scratch (the activation staging area and the row staging area behind it)
constexpr int PK_AT_K = 0;                                    // [PK_TK][PK_KROW]
constexpr int PK_AT_V = PK_AT_K + PK_TK * PK_KROW;            // [PK_TK][PK_VROW]
constexpr int PK_AT_Q = PK_AT_V + PK_TK * PK_VROW;            // [PK_QR][PK_QROW]
constexpr int PK_AT_NEW = PK_AT_Q + PK_QR * PK_QROW;          // K rows of the pass [4][256 B], then V rows [4][256 B]
constexpr int PK_AT_OS = 0;                                   // after the tiles are consumed: [warps][16][PK_OROW] floats
constexpr int PK_OROW = PK_D + 8;                             // padded: the 8 rows a warp stores at once hit different banks
constexpr int PK_AT_RED = PK_WARPS * PK_QR * PK_OROW * 4;     // running max [warps][16], then each warp's merge factor [warps][16]
constexpr int PK_AT_ROWS = PK_AT_RED + 2 * PK_WARPS * PK_QR * 4;   // the pass's q | k | v vectors of one kv head, fp32, per row
constexpr int PK_AT_ROW_FLOATS = (PK_QR + 2) * PK_D;
constexpr int PK_AT_END = PK_AT_ROWS + PK_MAX_ROWS * PK_AT_ROW_FLOATS * 4;
static_assert(PK_AT_NEW + 2 * PK_MAX_ROWS * 256 <= PK_AT_RED, "tiles overlap the reduction arrays");
static_assert(PK_AT_END <= PK_BSTAGE_BYTES + PK_XS_BYTES, "attention scratch does not fit");

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

// Step a3 for one (sequence, kv head): one warp per head vector of the pass's rows (staged in
// shared memory as q heads | k | v per row).  Query rows
// go to the Q tile (bf16, scaled by 1/sqrt(d)); K and V rows go to the new-row area and, from
// the block that owns slice 0, into the cache.
__device__ __forceinline__ void attn_new_rows(const PassParams &P, const PassLayer &Ly, unsigned char *sc, int b, int kvh,
                                              int R, int pos0, bool write_cache) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = P.nq / P.nkv, nQ = R * G;
  const float *rows = reinterpret_cast<const float *>(sc + PK_AT_ROWS);
  const float scale = rsqrtf((float)PK_D);
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
      const float *w = kind == 0 ? Ly.w_qn : Ly.w_kn;
#pragma unroll
      for (int j = 0; j < 4; ++j) v[j] = v[j] * inv * __ldg(w + lane + 32 * j);
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        // angle reduced to [-pi, pi] in double, then the fast sine and cosine
        double a = (double)pos * P.inv_freq[lane + 32 * j];
        a -= 6.283185307179586 * rint(a * 0.15915494309189535);
        float sn, cs;
        __sincosf((float)a, &sn, &cs);
        const float x0 = v[j], x1 = v[j + 2];
        v[j] = x0 * cs - x1 * sn;
        v[j + 2] = x1 * cs + x0 * sn;
      }
    }
    __nv_bfloat16 *row = reinterpret_cast<__nv_bfloat16 *>(
        kind == 0 ? sc + PK_AT_Q + task * PK_QROW : sc + PK_AT_NEW + ((kind == 2 ? PK_MAX_ROWS : 0) + r) * 256);
    __nv_bfloat16 *cache = (kind == 1 ? Ly.kc : Ly.vc) + (((size_t)b * P.nkv + kvh) * P.max_seq + pos) * PK_D;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const __nv_bfloat16 h = __float2bfloat16_rn(v[j]);
      row[lane + 32 * j] = h;
      if (kind != 0 && write_cache) cache[lane + 32 * j] = h;
    }
  }
}

// Steps a3 + a4 for the items (sequence, kv head, key slice) of this block.  The R*G query rows
// of an item form one m16 tile; S = Q K^T and O = P V run as mma.m16n8k16 with K and V staged in
// shared memory, each warp taking 16 keys of a 64-key tile with its own running max and sum.
// The slice's unnormalised partial output goes to global memory with its max and sum; the
// prologue of the O projection merges the slices.
__device__ __noinline__ void attention_stage(const PassParams &P, const PassLayer &Ly, int R, int pos0) {
  const PassShared S = pass_shared();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int G = P.nq / P.nkv, nQ = R * G;
  int nsplit, CH;
  attn_plan_device(P, pos0, nsplit, CH);
  const int items = P.B * P.nkv * nsplit;
  if ((int)blockIdx.x >= items) return;

  unsigned char *const sc = S.bstage;
  const uint32_t k_tile = smem_u32(sc + PK_AT_K), v_tile = smem_u32(sc + PK_AT_V), q_tile = smem_u32(sc + PK_AT_Q);
  float *const o_s = reinterpret_cast<float *>(sc + PK_AT_OS);
  float *const red_m = reinterpret_cast<float *>(sc + PK_AT_RED);
  float *const red_l = red_m + PK_WARPS * PK_QR;

  for (int item = blockIdx.x; item < items; item += gridDim.x) {
    const int split = item % nsplit, kvh = (item / nsplit) % P.nkv, b = item / (nsplit * P.nkv);
    // keys [j0, j1) of the cache, then (last slice) the R keys of the pass
    const int j0 = split * CH, j1 = min(j0 + CH, pos0);
    const int n_cached = max(0, j1 - j0);
    const int n_keys = n_cached + (split == nsplit - 1 ? R : 0);
    const __nv_bfloat16 *kbase = Ly.kc + ((size_t)b * P.nkv + kvh) * P.max_seq * PK_D;
    const __nv_bfloat16 *vbase = Ly.vc + ((size_t)b * P.nkv + kvh) * P.max_seq * PK_D;
    // cached rows of a tile: asynchronous copies, 16 bytes each (a row is 16 K parts and 16 V parts)
    auto fetch_cached = [&](int tile0) {
      const int n_c = min(PK_TK, n_cached - tile0);
      for (int c = threadIdx.x; c < n_c * 32; c += PK_THREADS) {
        const int row = c >> 5, part = c & 31;
        const uint32_t dst = part < 16 ? k_tile + row * PK_KROW + part * 16 : v_tile + row * PK_VROW + (part - 16) * 16;
        cp_async16(dst, (part < 16 ? kbase : vbase) + (size_t)(j0 + tile0 + row) * PK_D + (part & 15) * 8);
      }
    };
    pk_sync();                                            // the previous item is done with the scratch
    if (threadIdx.x == 0) {
      // the pass's own q | k | v vectors of this kv head: three bulk copies per row
      const int ldq = (P.nq + 2 * P.nkv) * PK_D;
      stage_begin(S, (uint32_t)(R * (G + 2) * PK_D * 4));
      for (int r = 0; r < R; ++r) {
        const float *src = P.qkv + (size_t)(b * R + r) * ldq;
        float *dst = reinterpret_cast<float *>(sc + PK_AT_ROWS) + r * PK_AT_ROW_FLOATS;
        stage_copy(S, dst, src + kvh * G * PK_D, (uint32_t)(G * PK_D * 4));
        stage_copy(S, dst + G * PK_D, src + (P.nq + kvh) * PK_D, PK_D * 4);
        stage_copy(S, dst + (G + 1) * PK_D, src + (P.nq + P.nkv + kvh) * PK_D, PK_D * 4);
      }
    }
    fetch_cached(0);                                      // in flight while the pass's own rows are prepared
    // query rows beyond nQ are zero (the previous item's partial outputs lay over the Q tile)
    for (int i = threadIdx.x; i < PK_QR * PK_QROW / 16; i += PK_THREADS) sts128(q_tile + i * 16, make_uint4(0u, 0u, 0u, 0u));
    stage_wait(P, S);
    attn_new_rows(P, Ly, sc, b, kvh, R, pos0, split == 0);

    float m_run[2] = {-INFINITY, -INFINITY}, l_part[2] = {0.f, 0.f};
    float o[16][4];
#pragma unroll
    for (int dt = 0; dt < 16; ++dt) o[dt][0] = o[dt][1] = o[dt][2] = o[dt][3] = 0.f;
    uint4 qf[4][2];
    for (int tile0 = 0; tile0 < n_keys; tile0 += PK_TK) {
      const int n_t = min(PK_TK, n_keys - tile0);
      pk_sync();                                          // new rows written / previous tile consumed
      if (tile0 > 0) fetch_cached(tile0);
      for (int c = threadIdx.x + max(0, n_cached - tile0) * 32; c < n_t * 32; c += PK_THREADS) {
        const int row = c >> 5, part = c & 31, idx = tile0 + row;
        const uint32_t dst = part < 16 ? k_tile + row * PK_KROW + part * 16 : v_tile + row * PK_VROW + (part - 16) * 16;
        const unsigned char *src = sc + PK_AT_NEW + ((part < 16 ? 0 : PK_MAX_ROWS) + (idx - n_cached)) * 256 + (part & 15) * 16;
        sts128(dst, *reinterpret_cast<const uint4 *>(src));
      }
      const int n16 = min(PK_TK, (n_t + 15) & ~15);
      for (int c = threadIdx.x; c < (n16 - n_t) * 16; c += PK_THREADS)      // P = 0 times stale bits must stay 0
        sts128(v_tile + (n_t + (c >> 4)) * PK_VROW + (c & 15) * 16, make_uint4(0u, 0u, 0u, 0u));
      cp_async_wait_all();
      pk_sync();
      if (tile0 == 0) {
#pragma unroll
        for (int kb = 0; kb < 4; ++kb) {
          qf[kb][0] = lds128(q_tile + g * PK_QROW + kb * 64 + t * 16);
          qf[kb][1] = lds128(q_tile + (g + 8) * PK_QROW + kb * 64 + t * 16);
        }
      }
      if (warp * 16 < n_t) {
        float c[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f;
#pragma unroll
          for (int kb = 0; kb < 4; ++kb) {
            const uint4 Kv = lds128(k_tile + (warp * 16 + nt * 8 + g) * PK_KROW + kb * 64 + t * 16);
            mma_bf16_16816(c[nt], qf[kb][0].x, qf[kb][1].x, qf[kb][0].y, qf[kb][1].y, Kv.x, Kv.y);
            mma_bf16_16816(c[nt], qf[kb][0].z, qf[kb][1].z, qf[kb][0].w, qf[kb][1].w, Kv.z, Kv.w);
          }
        }
        // causal / range mask: lane holds rows g (e = 0, 1) and g + 8 (e = 2, 3), keys 2t, 2t + 1 of each n-tile
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int kl = warp * 16 + nt * 8 + 2 * t + (e & 1), idx = tile0 + kl, row = g + (e >> 1) * 8;
            const int key_pos = idx < n_cached ? j0 + idx : pos0 + (idx - n_cached);
            const bool ok = kl < n_t && key_pos <= pos0 + row / G;
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
        const uint32_t a0 = pack_bf16x2(c[0][0], c[0][1]), a1 = pack_bf16x2(c[0][2], c[0][3]);
        const uint32_t a2 = pack_bf16x2(c[1][0], c[1][1]), a3 = pack_bf16x2(c[1][2], c[1][3]);
        const int mi = lane >> 3, rr = lane & 7;
        const uint32_t v_addr = v_tile + (warp * 16 + (mi & 1) * 8 + rr) * PK_VROW + (mi >> 1) * 16;
#pragma unroll
        for (int d2 = 0; d2 < 8; ++d2) {
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4_trans(v_addr + d2 * 32, b0, b1, b2, b3);
          o[2 * d2][0] *= corr[0]; o[2 * d2][1] *= corr[0]; o[2 * d2][2] *= corr[1]; o[2 * d2][3] *= corr[1];
          o[2 * d2 + 1][0] *= corr[0]; o[2 * d2 + 1][1] *= corr[0]; o[2 * d2 + 1][2] *= corr[1]; o[2 * d2 + 1][3] *= corr[1];
          mma_bf16_16816(o[2 * d2], a0, a1, a2, a3, b0, b1);
          mma_bf16_16816(o[2 * d2 + 1], a0, a1, a2, a3, b2, b3);
        }
      }
    }

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
      const size_t slot = ((size_t)(b * R + qi / G) * P.nq + kvh * G + qi % G) * PK_NSPLIT_CAP + split;
      P.part_ml[slot * 2] = m;
      P.part_ml[slot * 2 + 1] = l;
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
      const size_t slot = ((size_t)(b * R + qi / G) * P.nq + kvh * G + qi % G) * PK_NSPLIT_CAP + split;
      *reinterpret_cast<float4 *>(P.part_o + slot * PK_D + d4 * 4) = acc;
    }

  }
  pk_sync();
}

}  // namespace dmtd
