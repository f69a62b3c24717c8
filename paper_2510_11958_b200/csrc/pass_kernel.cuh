// One decode pass of the DMTD schedule (Section 2.2 of the paper) as ONE persistent kernel.
//
// A pass is a fixed list of stages: per layer QKV -> ATTN -> OPROJ -> GATEUP -> DOWN, then the
// tied LM head, the greedy pick and the counter update.  One block per SM runs every stage;
// blocks meet at a grid-wide barrier between stages (cooperative launch, bounded spin).
//
// Decode at small batch is bound by streaming the weights from HBM, and a stage boundary
// would drain that stream.  Weights do not depend on activations, so every warp owns a fixed,
// contiguous share of every matrix of the pass and pulls it through a private ring of shared
// memory slots with bulk asynchronous copies that run ahead of the arithmetic - across stage
// boundaries and barriers - as far as the ring allows.
#pragma once

#include "pass_attention_f32.cuh"

namespace dmtd {

// Profiling builds (-DDMTD_PASS_TIMING) record clock64() of thread 0 of the first and the last
// block after every prologue, projection and barrier; the last four slots of each block hold
// clock64() and the nanosecond wall clock at kernel entry and at kernel exit, which give the
// SM clock rate of the launch and the time outside the stamped stages.
#ifdef DMTD_PASS_TIMING
constexpr int PK_TIMING_SLOTS = 4096;
#define PK_STAMP()                                                                                   \
  do {                                                                                               \
    if (threadIdx.x == 0 && P.timing && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1) &&          \
        stamp_n < PK_TIMING_SLOTS - 4)                                                               \
      P.timing[(blockIdx.x ? PK_TIMING_SLOTS : 0) + stamp_n++] = clock64();                          \
  } while (0)
#define PK_STAMP_WALL(i)                                                                             \
  do {                                                                                               \
    if (threadIdx.x == 0 && P.timing && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1)) {          \
      long long ns;                                                                                  \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));                                         \
      long long *t = P.timing + (blockIdx.x ? PK_TIMING_SLOTS : 0) + PK_TIMING_SLOTS - 4 + 2 * (i);  \
      t[0] = clock64();                                                                              \
      t[1] = ns;                                                                                     \
    }                                                                                                \
  } while (0)
// ... and, for the projections of the pass's last layer, when each chunk of the streams of warps 0 and 7 of
// the first block was there to be consumed: slots 2048 + 64 * projection + 32 * (warp == 7) hold the clock
// before and after the wait for every chunk, and at the end of the warp's share.
#define PK_CHUNK_STAMP(i)                                                                            \
  do {                                                                                               \
    if (chunk_log >= 0 && (i) < 32 && lane == 0 && (warp == 0 || warp == 7) && blockIdx.x == 0 && P.timing) \
      P.timing[chunk_log + (warp ? 32 : 0) + (i)] = clock64();                                       \
  } while (0)
#define PK_CHUNK_LOG_ARG , int chunk_log
#else
#define PK_STAMP() do {} while (0)
#define PK_STAMP_WALL(i) do {} while (0)
#define PK_CHUNK_STAMP(i) do {} while (0)
#define PK_CHUNK_LOG_ARG
#endif

#ifndef DMTD_PASS_NACC
#define DMTD_PASS_NACC 2
#endif
constexpr int PK_NACC = DMTD_PASS_NACC;

// out[m][n] += sum_k W[n][k] act[m][k] over this warp's share of W, streamed through its ring.
// Weights are the A operand of mma.m16n8k16 (register order, straight from the ring), the
// activation hi/lo columns the B operand.  One atom per trip of a loop that is not unrolled:
// the loop stays a few dozen instructions, holds everything in registers, and the other warps
// of the block hide the shared-memory latency.
__device__ __noinline__ bool gemv_consume(const PassParams &P, const PackedMat &W, int kind, int M, float *__restrict__ out,
                                          int ldo PK_CHUNK_LOG_ARG) {
  const PassShared S = pass_shared();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  WarpPipe pp = S.pipes[warp];
  const int aps = W.aps, n_tiles = W.n_tiles, N = W.N;
  const MatPlan &pl = S.plans[kind];
  const int w0 = pl.w0[warp], w1 = pl.w1[warp];
  if (w0 >= w1) return true;
  const int row_bytes = b_row_bytes(aps * 32);
  const int s_first = pl.s_first, s = pl.ws[warp];
  int T = pl.wT[warp], a = pl.wa[warp];
  uint32_t b_addr = smem_u32(S.bstage) + (s - s_first) * 8 * row_bytes + g * row_bytes + t * 16;
  const bool need_b = g < 2 * M;                          // columns beyond 2M belong to no activation row
  const int tile_mask = (PK_CHUNK_ATOMS % aps == 0 && (aps & (aps - 1)) == 0) ? aps - 1 : 0;
  // The loop is bound by the number of instructions a warp issues per atom (two warps per scheduler:
  // every instruction costs its full latency), not by the MMAs or by shared memory.  So: the
  // activation fragments of the slab's (at most 8) atoms live in registers, loaded once per slab; the
  // share is walked in segments (the atoms of one 16-row tile that lie in one chunk) whose body is
  // unrolled over the position inside the tile, so that nothing but two loads and two MMAs is left per
  // atom; the bookkeeping (chunk hand-over, the tile's reductions) is per segment.
  uint4 Bq[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    Bq[k] = make_uint4(0u, 0u, 0u, 0u);
    if (need_b && k < aps) Bq[k] = lds128(b_addr + k * 64);
  }
  // PK_NACC accumulators taken in turn (measured: 2, 4, 8 and 16 give 0.65, 0.74, 0.76 and 0.83 us per 8-atom
  // chunk: the loop is bound by the rate at which the SM takes mma.sync, about one m16n8k16 per 32 cycles and
  // scheduler, not by the chain through an accumulator)
  float acc[PK_NACC][4];
#pragma unroll
  for (int i = 0; i < PK_NACC; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
  int left = w1 - w0, slot_left = 0;
  uint32_t ptr = 0;
#ifdef DMTD_PASS_TIMING
  int chunk_i = 0;
#endif
  while (left > 0) {
    if (slot_left == 0) {
      PK_CHUNK_STAMP(chunk_i++);
      if (!pipe_wait(P, pp)) {
        if (lane == 0) S.pipes[warp] = pp;
        return false;
      }
      PK_CHUNK_STAMP(chunk_i++);
      ptr = pp.ring + (pp.consumed % PK_SLOTS) * PK_CHUNK_BYTES + lane * 16;
      slot_left = min(PK_CHUNK_ATOMS - (a & tile_mask), left);          // as pipe_issue cut it
    }
    const int a_hi = min(aps, a + min(left, slot_left));
    if (a == 0 && a_hi == 8) {
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const uint4 A0 = lds128(ptr + k * 1024), A1 = lds128(ptr + k * 1024 + 512);
        mma_bf16_16816(acc[(2 * k) % PK_NACC], A0.x, A1.x, A0.y, A1.y, Bq[k].x, Bq[k].y);
        mma_bf16_16816(acc[(2 * k + 1) % PK_NACC], A0.z, A1.z, A0.w, A1.w, Bq[k].z, Bq[k].w);
      }
      ptr += 8 * 1024;
    } else {
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (k >= a && k < a_hi) {
          const uint4 A0 = lds128(ptr), A1 = lds128(ptr + 512);
          mma_bf16_16816(acc[(2 * k) % PK_NACC], A0.x, A1.x, A0.y, A1.y, Bq[k].x, Bq[k].y);
          mma_bf16_16816(acc[(2 * k + 1) % PK_NACC], A0.z, A1.z, A0.w, A1.w, Bq[k].z, Bq[k].w);
          ptr += 1024;
        }
      }
    }
    left -= a_hi - a;
    slot_left -= a_hi - a;
    a = a_hi;
    if (slot_left == 0) {
      pp.consumed += 1;
      __syncwarp();
      if (lane == 0) {
        fence_proxy_async();
        pipe_issue(P, pp);
      }
    }
    if (a == aps || left == 0) {
      // accumulator columns 2t (hi) and 2t+1 (lo) belong to activation row t
      const int n_lo = T * 16 + g;
      float lo = 0.f, hi = 0.f;
#pragma unroll
      for (int i = 0; i < PK_NACC; ++i) {
        lo += acc[i][0] + acc[i][1];
        hi += acc[i][2] + acc[i][3];
        acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
      }
      if (t < M) {
        if (n_lo < N) atomicAdd(out + (size_t)t * ldo + n_lo, lo);
        if (n_lo + 8 < N) atomicAdd(out + (size_t)t * ldo + n_lo + 8, hi);
      }
      a = 0;
      if (++T == n_tiles && left > 0) {
        T = 0;
        b_addr += 8 * row_bytes;
#pragma unroll
        for (int k = 0; k < 8; ++k)
          if (need_b && k < aps) Bq[k] = lds128(b_addr + k * 64);
      }
    }
  }
  PK_CHUNK_STAMP(chunk_i++);
  if (lane == 0) S.pipes[warp] = pp;
  __syncwarp();
  return true;
}

// Greedy pick, first level: this block's slice of the vocabulary, lowest index on ties.
__device__ __noinline__ void argmax_partial(const PassParams &P) {
  const PassShared S = pass_shared();
  const int per = (P.vocab + gridDim.x - 1) / gridDim.x;
  const int i0 = blockIdx.x * per, i1 = min(P.vocab, i0 + per);
  float *sv = reinterpret_cast<float *>(S.bstage);
  int *si = reinterpret_cast<int *>(S.bstage) + PK_THREADS;
  const int position = P.st->n_known;                 // where the picked token will sit
  for (int b = 0; b < P.B; ++b) {
    float best = -INFINITY;
    int bi = 0x7fffffff;
    for (int i = i0 + threadIdx.x; i < i1; i += PK_THREADS) {
      const float v = pick_value(__ldcg(P.logits + (size_t)b * P.ldl + i), i, position, b, P.sample);
      if (v > best) { best = v; bi = i; }
    }
    pk_sync();
    sv[threadIdx.x] = best; si[threadIdx.x] = bi;
    pk_sync();
    for (int s = PK_THREADS >> 1; s > 0; s >>= 1) {
      if (threadIdx.x < s) {
        const float v2 = sv[threadIdx.x + s];
        const int i2 = si[threadIdx.x + s];
        if (v2 > sv[threadIdx.x] || (v2 == sv[threadIdx.x] && i2 < si[threadIdx.x])) {
          sv[threadIdx.x] = v2; si[threadIdx.x] = i2;
        }
      }
      pk_sync();
    }
    if (threadIdx.x == 0) {
      P.amax_val[b * gridDim.x + blockIdx.x] = sv[0];
      P.amax_idx[b * gridDim.x + blockIdx.x] = si[0];
    }
  }
}

// Greedy pick, second level; a10 token feedback; a0 counters.  Block 0 only.
__device__ __noinline__ void argmax_final(const PassParams &P) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_known = P.st->n_known;
  if (warp < P.B) {
    const int b = warp;
    float best = -INFINITY;
    int bi = 0x7fffffff;
    for (int c = lane; c < (int)gridDim.x; c += 32) {
      const float v = __ldcg(P.amax_val + b * gridDim.x + c);
      const int i = __ldcg(P.amax_idx + b * gridDim.x + c);
      if (v > best || (v == best && i < bi)) { best = v; bi = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float v2 = __shfl_xor_sync(0xffffffffu, best, o);
      const int i2 = __shfl_xor_sync(0xffffffffu, bi, o);
      if (v2 > best || (v2 == best && i2 < bi)) { best = v2; bi = i2; }
    }
    if (lane == 0) {
      const int pick = bi == 0x7fffffff ? 0 : bi;
      if (P.write_token) P.tokens[(size_t)b * P.max_seq + n_known] = pick;
      if (P.out_argmax) P.out_argmax[b] = pick;
    }
  }
  pk_sync();
  if (threadIdx.x == 0) {
    DevState *st = P.st;
    if (P.kind == 1) { st->lo_len = st->n_known; st->cycle += 1; }
    st->up_len = st->n_known;
    st->n_known += 1;
    st->slot = (st->slot + 1) % st->tau;
    st->n_emitted += 1;
    st->newest = st->n_known - 1;
  }
}

__global__ void __launch_bounds__(PK_THREADS, 1) dmtd_pass_kernel(const __grid_constant__ PassParams P) {
  PK_STAMP_WALL(0);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const PassShared S = pass_shared();
  const int nL = P.l_end - P.l_begin;
  {
    const int *src = reinterpret_cast<const int *>(P.layers + P.l_begin);
    int *dst = reinterpret_cast<int *>(S.layers);
    for (int i = threadIdx.x; i < nL * (int)(sizeof(PassLayer) / 4); i += PK_THREADS) dst[i] = src[i];
  }
  if (threadIdx.x == 0) {
    *S.abort_flag = 0;
    *S.stage_uses = 0u;
    mbar_init(smem_u32(S.stage_bar), 1);
  }
  if (lane == 0) {
    for (int s = 0; s < PK_SLOTS; ++s) mbar_init(smem_u32(S.bars + warp * PK_SLOTS + s), 1);
    fence_mbar_init();
  }
  pk_sync();
  plans_fill(P, S);
  pk_sync();

  const int lo_len = P.st->lo_len, newest = P.st->newest;
  {
    WarpPipe pp;
    pp.ring = smem_u32(S.ring) + warp * PK_SLOTS * PK_CHUNK_BYTES;
    pp.bars = smem_u32(S.bars + warp * PK_SLOTS);
    pp.issued = pp.consumed = 0;
    cursor_init(pp.cur, P, warp);
    if (lane == 0) {
      for (int s = 0; s < PK_SLOTS; ++s) pipe_issue(P, pp);
      S.pipes[warp] = pp;
    }
    __syncwarp();
  }

  unsigned bar_target = 0;
#ifdef DMTD_PASS_TIMING
  int stamp_n = 0;
#endif
  PK_STAMP();
  const int ldqkv = (P.nq + 2 * P.nkv) * PK_D, ldgu = 2 * P.I;
  const bool has_lower = P.l_begin < P.l_split;
  const int M_max = P.B * (has_lower ? P.R_lo : 1);

  // buffers the projections accumulate into start at zero; a1: the first layer's rows
  grid_zero(P.qkv, M_max * ldqkv);
  grid_zero(P.gu, M_max * ldgu);
  grid_zero(P.logits, P.B * P.ldl);
  if (has_lower) embed_rows(P, P.x_lo, M_max, P.R_lo, lo_len);
  else embed_rows(P, P.x_up, P.B, 1, newest);
  bool ok = grid_barrier(P, bar_target);

  // Stage list: five stages per layer, then the LM head.  Every stage is a prologue that puts
  // the activations this block needs into shared memory, the block's share of one projection,
  // and a grid barrier.  The attention stage has no projection.
  // the key slices of the attention stages depend on the context length only: worked out once per pass
  int nsplit_lo, CH_lo, nsplit_up, CH_up;
  attn_plan_device(P, lo_len, nsplit_lo, CH_lo);
  attn_plan_device(P, newest, nsplit_up, CH_up);
  const int n_stages = nL * 5 + 1;
  for (int stage = 0, li = 0, ph = 0; stage < n_stages && ok; ++stage, ph = ph == 4 ? 0 : ph + 1, li += ph == 0) {
    const bool head = li == nL;
    const int l = P.l_begin + li;
    const bool lower = !head && l < P.l_split;
    const int R = lower ? P.R_lo : 1, M = P.B * R, pos0 = lower ? lo_len : newest;
    float *x = lower ? P.x_lo : P.x_up;
    const int nsplit = lower ? nsplit_lo : nsplit_up, CH = lower ? CH_lo : CH_up;      // key slices of the attention stage
    const PassLayer &Ly = S.layers[head ? 0 : li];
    const PackedMat *W = nullptr;
    float *out = nullptr;
    int ldo = 0;
    if (head) {
      // a9: final norm, tied head
      norm_prologue(P, P.x_up, (size_t)P.H, M, P.w_final, P.embed, PK_MAT_HEAD);
      W = &P.embed; out = P.logits; ldo = P.ldl;
    } else if (ph == 0) {
      // a2: RMSNorm, QKV projection; a8 at the first decoding layer of a full pass: the newest
      // row of each sequence is read straight from the lower stack's rows and copied to x_up
      if (has_lower && l == P.l_split) {
        select_rows(P);
        norm_prologue(P, P.x_lo + (size_t)(P.R_lo - 1) * P.H, (size_t)P.R_lo * P.H, M, Ly.w_in, Ly.qkv, PK_MAT_QKV);
      } else {
        norm_prologue(P, x, (size_t)P.H, M, Ly.w_in, Ly.qkv, PK_MAT_QKV);
      }
      W = &Ly.qkv; out = P.qkv; ldo = ldqkv;
    } else if (ph == 1) {
      // a3 + a4: QK-norm, RoPE, KV append, attention over the key slices
      if (P.kv_f32) attention_stage_f32(P, Ly, R, pos0, nsplit, CH);
      else if (P.kv_f16) attention_stage<OpF16>(P, Ly, R, pos0, nsplit, CH);
      else attention_stage<OpBf16>(P, Ly, R, pos0, nsplit, CH);
      if (PK_ATTN_PF_ATOMS > 0) {
        const int items = P.B * P.nkv * nsplit;
        if ((int)blockIdx.x >= items) prefetch_matrix_part(Ly.gu, (int)blockIdx.x - items, (int)gridDim.x - items);
      }
    } else if (ph == 2) {
      // a4 merge of the key slices + a5: O projection into the residual rows
      grid_zero(P.gu, M_max * ldgu);
      merge_prologue(P, M, nsplit, Ly.o);
      W = &Ly.o; out = x; ldo = P.H;
    } else if (ph == 3) {
      // a6: RMSNorm, gate and up projections
      norm_prologue(P, x, (size_t)P.H, M, Ly.w_post, Ly.gu, PK_MAT_GU);
      W = &Ly.gu; out = P.gu; ldo = ldgu;
    } else {
      // a6 gate + a7: down projection into the residual rows
      grid_zero(P.qkv, M_max * ldqkv);
      swiglu_prologue(P, M, Ly.down);
      W = &Ly.down; out = x; ldo = P.H;
    }
    // the prologue's own loads are done: ask L2 for the next atoms of the warp's stream (HBM is idle until the
    // projection has drained the ring)
    if (PK_PRO_PF_ATOMS > 0 && lane == 0 && ph != 1 && ph != 2)
      prefetch_own_stream(S.pipes[warp].cur, (!head && ph == 3) ? PK_ATTN_PF_ATOMS : 0);
    PK_STAMP();
#ifdef DMTD_PASS_TIMING
    const int chunk_log = (!head && li == nL - 1 && ph != 1) ? 2048 + 64 * (ph - (ph > 1)) : -1;
    if (W && !gemv_consume(P, *W, head ? PK_MAT_HEAD : ph - (ph > 1), M, out, ldo, chunk_log)) *S.abort_flag = 1;
#else
    if (W && !gemv_consume(P, *W, head ? PK_MAT_HEAD : ph - (ph > 1), M, out, ldo)) *S.abort_flag = 1;
#endif
    PK_STAMP();
#ifdef DMTD_PASS_TIMING
    // every block's wall clock at the end of its share of the last layer's projections (slots 3200 + 160 * projection + block)
    if (threadIdx.x == 0 && P.timing && !head && li == nL - 1 && gridDim.x <= 160) {
      long long ns;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));
      P.timing[3200 + 160 * (ph == 1 ? 4 : ph - (ph > 1)) + blockIdx.x] = ns;
    }
#endif
    ok = grid_barrier(P, bar_target);
    PK_STAMP();
  }

  if (ok) {
    argmax_partial(P);
    ok = grid_barrier(P, bar_target);
  }
  if (ok && blockIdx.x == 0) argmax_final(P);

  // leave no copy in flight: a slot this warp still waits for gets a bounded wait
  WarpPipe pp = S.pipes[warp];
  while (pp.consumed < pp.issued) {
    const unsigned slot = pp.consumed % PK_SLOTS;
    const uint32_t parity = (pp.consumed / PK_SLOTS) & 1u;
    const long long t0 = clock64();
    while (!mbar_try_wait(pp.bars + slot * 8, parity))
      if (clock64() - t0 > P.wait_limit) break;
    pp.consumed += 1;
  }
  PK_STAMP_WALL(1);
}

}  // namespace dmtd
