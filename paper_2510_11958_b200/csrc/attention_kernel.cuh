// Step a4 as a kernel of its own, for the per-step path (prefill, batches the pass kernel does
// not take) and for dmtd_attention_decode: split-KV attention on the tensor cores.  One block
// per (key slice, kv head x row block, sequence); the G query heads of the kv head for up to
// 16 / G new positions form one m16 tile of query rows that share every key and value the block
// stages in shared memory.  Same tile arithmetic as the attention stage of the pass kernel;
// the slices are merged by attn_merge_kernel.
#pragma once

#include "pass_attention.cuh"

namespace dmtd {

constexpr int ATTN_TC_SMEM = PK_AT_ROWS;         // tiles, Q, partial-output overlay, reduction arrays

// qkv [B*R][ldq]: q heads already normalised and rotated (not scaled); K and V of the new rows
// already in the cache.  Cache [b][kv head][max_seq][128] bf16 (PRECISE = false) or fp32.
template <bool PRECISE>
__global__ void __launch_bounds__(PK_THREADS, PRECISE ? 1 : 2)      // bf16 cache: two blocks per SM overlap load and math
attn_tc_kernel(const float *__restrict__ qkv, int ldq, const void *__restrict__ kc, const void *__restrict__ vc, int max_seq,
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
  const uint32_t kh_tile = smem_u32(sc + PK_AT_KH), vh_tile = smem_u32(sc + PK_AT_VH), vl_tile = smem_u32(sc + PK_AT_VL);
  const uint32_t qh_tile = smem_u32(sc + PK_AT_QH);
  // Q tile: rows beyond nQ zero; row qi = (position r0 + qi / G, head kvh*G + qi % G), scaled by 1/sqrt(d)
  for (int i = threadIdx.x; i < 2 * PK_QR * PK_QROW / 16; i += PK_THREADS) sts128(qh_tile + i * 16, make_uint4(0u, 0u, 0u, 0u));
  __syncthreads();
  const float scale = rsqrtf((float)PK_D);
  for (int qi = warp; qi < nQ; qi += PK_WARPS) {
    const float *src = qkv + (size_t)(b * R + r0 + qi / G) * ldq + (size_t)(kvh * G + qi % G) * PK_D;
    __nv_bfloat16 *qh = reinterpret_cast<__nv_bfloat16 *>(sc + PK_AT_QH + qi * PK_QROW);
    __nv_bfloat16 *ql = reinterpret_cast<__nv_bfloat16 *>(sc + PK_AT_QL + qi * PK_QROW);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float v = src[lane + 32 * j] * scale;
      const __nv_bfloat16 h = __float2bfloat16_rn(v);
      qh[lane + 32 * j] = h;
      if (PRECISE) ql[lane + 32 * j] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
  }
  const size_t head_off = ((size_t)b * nkv + kvh) * max_seq * PK_D;
  AttnAcc A;
  A.m_run[0] = A.m_run[1] = -INFINITY;
  A.l_part[0] = A.l_part[1] = 0.f;
#pragma unroll
  for (int dt = 0; dt < 8; ++dt) A.o[dt][0] = A.o[dt][1] = A.o[dt][2] = A.o[dt][3] = 0.f;
  const int n_keys = j1 - j0;
  if (!PRECISE) {
    // bf16 cache: two tile buffers (the lo-part areas are free here), tile i+1 in flight while
    // tile i is multiplied
    const __nv_bfloat16 *kb = reinterpret_cast<const __nv_bfloat16 *>(kc) + head_off;
    const __nv_bfloat16 *vb = reinterpret_cast<const __nv_bfloat16 *>(vc) + head_off;
    auto fetch = [&](int tile0, int buf) {
      const int n_t = min(PK_TK, n_keys - tile0);
      const uint32_t k_t = smem_u32(sc + (buf ? PK_AT_KL : PK_AT_KH)), v_t = smem_u32(sc + (buf ? PK_AT_VL : PK_AT_VH));
      for (int c = threadIdx.x; c < n_t * 32; c += PK_THREADS) {
        const int row = c >> 5, part = c & 31;
        const uint32_t dst = part < 16 ? k_t + row * PK_KROW + part * 16 : v_t + row * PK_VROW + (part - 16) * 16;
        cp_async16(dst, (part < 16 ? kb : vb) + (size_t)(j0 + tile0 + row) * PK_D + (part & 15) * 8);
      }
      const int n16 = min(PK_TK, (n_t + 15) & ~15);
      for (int c = threadIdx.x; c < (n16 - n_t) * 16; c += PK_THREADS)      // P = 0 times stale bits must stay 0
        sts128(v_t + (n_t + (c >> 4)) * PK_VROW + (c & 15) * 16, make_uint4(0u, 0u, 0u, 0u));
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    fetch(0, 0);
    int buf = 0;
    for (int tile0 = 0; tile0 < n_keys; tile0 += PK_TK, buf ^= 1) {
      const int n_t = min(PK_TK, n_keys - tile0);
      if (tile0 + PK_TK < n_keys) {
        fetch(tile0 + PK_TK, buf ^ 1);
        asm volatile("cp.async.wait_group 1;" ::: "memory");
      } else {
        asm volatile("cp.async.wait_group 0;" ::: "memory");
      }
      __syncthreads();                                    // tile (and, the first time, Q) visible to all
      attn_tile_compute<false>(A, sc, n_t, tile0, 0x7fffffff, j0, 0, pos0 + r0, G, buf ? PK_AT_KL : PK_AT_KH,
                               buf ? PK_AT_VL : PK_AT_VH);
      __syncthreads();                                    // done with this buffer before it is refilled
    }
  } else {
    for (int tile0 = 0; tile0 < n_keys; tile0 += PK_TK) {
      const int n_t = min(PK_TK, n_keys - tile0);
      __syncthreads();                                      // Q written / previous tile consumed
      if (!PRECISE) {
        const __nv_bfloat16 *kb = reinterpret_cast<const __nv_bfloat16 *>(kc) + head_off;
        const __nv_bfloat16 *vb = reinterpret_cast<const __nv_bfloat16 *>(vc) + head_off;
        for (int c = threadIdx.x; c < n_t * 32; c += PK_THREADS) {
          const int row = c >> 5, part = c & 31;
          const uint32_t dst = part < 16 ? kh_tile + row * PK_KROW + part * 16 : vh_tile + row * PK_VROW + (part - 16) * 16;
          cp_async16(dst, (part < 16 ? kb : vb) + (size_t)(j0 + tile0 + row) * PK_D + (part & 15) * 8);
        }
      } else {
        attn_fetch_f32(reinterpret_cast<const float *>(kc) + head_off + (size_t)(j0 + tile0) * PK_D,
                       reinterpret_cast<const float *>(vc) + head_off + (size_t)(j0 + tile0) * PK_D, n_t, sc);
      }
      const int n16 = min(PK_TK, (n_t + 15) & ~15);
      for (int c = threadIdx.x; c < (n16 - n_t) * 16; c += PK_THREADS) {      // P = 0 times stale bits must stay 0
        const uint32_t off = (n_t + (c >> 4)) * PK_VROW + (c & 15) * 16;
        sts128(vh_tile + off, make_uint4(0u, 0u, 0u, 0u));
        if (PRECISE) sts128(vl_tile + off, make_uint4(0u, 0u, 0u, 0u));
      }
      cp_async_wait_all();
      __syncthreads();
      // every key comes from the cache: key index i sits at position j0 + i
      attn_tile_compute<PRECISE>(A, sc, n_t, tile0, 0x7fffffff, j0, 0, pos0 + r0, G);
    }
  }
  attn_combine_store(A, sc, nQ, G, b * R + r0, kvh * G, nq, nsplit, split, part_o, part_ml);
}

}  // namespace dmtd
