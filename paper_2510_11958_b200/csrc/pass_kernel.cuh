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
// boundaries and barriers - as far as the ring allows.  The barrier and the short
// activation prologue of each stage then cost latency on the consumer side only; the HBM
// stream keeps running underneath.
#pragma once

#include "common.cuh"

namespace dmtd {

constexpr int PK_WARPS = 8;
constexpr int PK_THREADS = PK_WARPS * 32;
constexpr int PK_CHUNK_ATOMS = 4;                          // atoms per bulk copy
constexpr int PK_CHUNK_BYTES = PK_CHUNK_ATOMS * 1024;
constexpr int PK_SLOTS = 5;                                // ring slots per warp
constexpr int PK_MAX_ROWS = 4;                             // activation rows (B*R) per stage
constexpr int PK_MAX_KS = 1280;                            // largest k-slab of a packed matrix
constexpr int PK_MAX_LAYERS = 48;
constexpr int PK_NSPLIT_CAP = 32;                          // key slices per (sequence, kv head)
constexpr int PK_MERGE_HEADS = 16;                         // heads one block merges for its O-proj share
constexpr int PK_D = 128;                                  // head_dim
constexpr int PK_QR = 16;                                  // query rows per attention item

// shared memory map (bytes)
constexpr int PK_RING_BYTES = PK_WARPS * PK_SLOTS * PK_CHUNK_BYTES;           // 163840
constexpr int PK_BROW_MAX = PK_MAX_KS * 2 + 64;                               // 2624
constexpr int PK_BSTAGE_BYTES = 2 * 8 * PK_BROW_MAX;                          // 41984: two slabs of 8 columns
constexpr int PK_MISC_BYTES = PK_MAX_ROWS * PK_MERGE_HEADS * PK_NSPLIT_CAP * 4;   // 8192
constexpr int PK_OFF_RING = 0;
constexpr int PK_OFF_BSTAGE = PK_OFF_RING + PK_RING_BYTES;
constexpr int PK_OFF_MISC = PK_OFF_BSTAGE + PK_BSTAGE_BYTES;
constexpr int PK_OFF_BARS = PK_OFF_MISC + PK_MISC_BYTES;
constexpr int PK_OFF_SMALL = PK_OFF_BARS + PK_WARPS * PK_SLOTS * 8;
constexpr int PK_SMALL_BYTES = 256;
constexpr int PK_OFF_LAYERS = PK_OFF_SMALL + PK_SMALL_BYTES;

enum { PK_ERR_NONE = 0, PK_ERR_TOKEN = 1, PK_ERR_COPY_WAIT = 2, PK_ERR_BARRIER_WAIT = 3 };

struct PassLayer {
  PackedMat qkv, o, gu, down;
  const float *w_in, *w_post, *w_qn, *w_kn;
  __nv_bfloat16 *kc, *vc;                 // this layer's cache [sequence][kv head][max_seq][128]
};

struct PassParams {
  const PassLayer *layers;                // device array, all layers of the model
  PackedMat embed;
  const float *w_final;
  const double *inv_freq;
  int l_begin, l_split, l_end;            // layers [l_begin, l_split): R_lo rows at lo_len..; [l_split, l_end): newest row
  int R_lo, B;
  int H, I, nq, nkv, vocab, max_seq, ldl;
  float eps;
  int kind;                               // 1 full pass, 2 decoding layers only (counter update)
  int write_token, literal_sum;
  int *tokens;
  DevState *st;
  float *x_lo, *x_up, *qkv, *gu, *logits, *part_o, *part_ml;
  float *amax_val;
  int *amax_idx;
  int *out_argmax;
  unsigned int *barrier;                  // zero at launch
  int *error;                             // sticky, 0 = fine
  long long wait_limit;                   // clock ticks a device-side wait may take
};

constexpr int PK_SMEM_BYTES = PK_OFF_LAYERS + PK_MAX_LAYERS * (int)sizeof(PassLayer);

// ---------------------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// global -> this block's shared memory, completion counted in bytes on an mbarrier
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

// ---------------------------------------------------------------------------- block state

struct PassShared {
  unsigned char *ring;      // [warp][slot][PK_CHUNK_BYTES]
  unsigned char *bstage;    // activation columns of up to two k-slabs; attention scratch
  float *misc;              // merge weights / attention small arrays
  uint64_t *bars;           // [warp][slot]
  volatile int *abort_flag;
  float *red;               // [PK_WARPS][PK_MAX_ROWS]
  PassLayer *layers;        // layers [l_begin, l_end) of this pass
};

// A warp's view of its weight stream: the chunks of its share of every matrix of the pass, in
// pass order.  Lane 0 runs the producer cursor; all lanes agree on `consumed`.
struct WarpPipe {
  uint32_t ring, bars;      // shared addresses of this warp's slots and barriers
  unsigned issued, consumed;
  int p_mat, n_mats;
  long long p_pos, p_end;
  const uint4 *p_base;
};

__device__ __forceinline__ const PackedMat &pass_matrix(const PassParams &P, const PassShared &S, int q) {
  int n_layer_mats = 4 * (P.l_end - P.l_begin);
  if (q >= n_layer_mats) return P.embed;
  const PassLayer &L = S.layers[q >> 2];
  switch (q & 3) {
    case 0: return L.qkv;
    case 1: return L.o;
    case 2: return L.gu;
    default: return L.down;
  }
}

// Atoms [c0, c1) of the block and [w0, w1) of the warp: equal contiguous cuts of the stream.
__device__ __forceinline__ void stream_ranges(const PackedMat &W, int warp, long long &c0, long long &c1,
                                              long long &w0, long long &w1) {
  const long long A = packed_atoms(W);
  c0 = A * blockIdx.x / gridDim.x;
  c1 = A * (blockIdx.x + 1) / gridDim.x;
  w0 = c0 + (c1 - c0) * warp / PK_WARPS;
  w1 = c0 + (c1 - c0) * (warp + 1) / PK_WARPS;
}

// Lane 0: issue the next chunk of the warp's stream, if any is left in the pass.
__device__ __forceinline__ void pipe_issue(const PassParams &P, const PassShared &S, WarpPipe &pp, int warp) {
  while (pp.p_pos >= pp.p_end) {
    if (++pp.p_mat >= pp.n_mats) { pp.p_mat = pp.n_mats; return; }
    const PackedMat &W = pass_matrix(P, S, pp.p_mat);
    long long c0, c1, w0, w1;
    stream_ranges(W, warp, c0, c1, w0, w1);
    pp.p_pos = w0; pp.p_end = w1; pp.p_base = W.w;
  }
  const int n = (int)min((long long)PK_CHUNK_ATOMS, pp.p_end - pp.p_pos);
  const unsigned slot = pp.issued % PK_SLOTS;
  const uint32_t bar = pp.bars + slot * 8;
  mbar_expect_tx(bar, (uint32_t)n * 1024u);
  bulk_g2s(pp.ring + slot * PK_CHUNK_BYTES, pp.p_base + pp.p_pos * 64, (uint32_t)n * 1024u, bar);
  pp.p_pos += n;
  pp.issued += 1;
}

// All lanes: wait until chunk `consumed` has landed.  Bounded; false = gave up.
__device__ __forceinline__ bool pipe_wait(const PassParams &P, const PassShared &S, const WarpPipe &pp) {
  const unsigned slot = pp.consumed % PK_SLOTS;
  const uint32_t parity = (pp.consumed / PK_SLOTS) & 1u;
  const uint32_t bar = pp.bars + slot * 8;
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > P.wait_limit || *S.abort_flag) {
      *S.abort_flag = 1;
      atomicMax(P.error, PK_ERR_COPY_WAIT);
      return false;
    }
  }
  return true;
}

// Grid-wide barrier: every block arrives once per stage; `target` counts arrivals so far.
__device__ __forceinline__ bool grid_barrier(const PassParams &P, const PassShared &S, unsigned &target) {
  __syncthreads();
  if (threadIdx.x == 0) {
    target += gridDim.x;
    if (*S.abort_flag) {
      atomicMax(P.error, PK_ERR_BARRIER_WAIT);
    } else {
      __threadfence();
      atomicAdd(P.barrier, 1u);
      const long long t0 = clock64();
      unsigned spins = 0;
      while (ld_acquire_u32(P.barrier) < target) {
        if ((++spins & 63u) == 0u &&
            (clock64() - t0 > P.wait_limit || *reinterpret_cast<volatile int *>(P.error) > PK_ERR_TOKEN)) {
          atomicMax(P.error, PK_ERR_BARRIER_WAIT);
          *S.abort_flag = 1;
          break;
        }
      }
      __threadfence();
    }
  }
  __syncthreads();
  return *S.abort_flag == 0;
}

// ---------------------------------------------------------------------------- small helpers

__device__ __forceinline__ void unpack8(uint4 v, float (&f)[8]) {
  uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    f[2 * j] = bf16_bits_to_float(w[j] & 0xffffu);
    f[2 * j + 1] = bf16_bits_to_float(w[j] >> 16);
  }
}

__device__ __forceinline__ void ldcg8(const float *p, float (&f)[8]) {
  float4 a = __ldcg(reinterpret_cast<const float4 *>(p)), b = __ldcg(reinterpret_cast<const float4 *>(p) + 1);
  f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}

// Values k = 8u .. 8u+7 of row `tok` of the packed embedding matrix.
__device__ __forceinline__ void embed8(const PackedMat &E, int tok, int u, float (&f)[8]) {
  const int k = u * 8, atom = k >> 5, t = (k >> 3) & 3;
  const int s = atom / E.aps, a = atom % E.aps;
  const int T = tok >> 4, half = (tok >> 3) & 1, g = tok & 7;
  unpack8(__ldg(E.w + (((long long)s * E.n_tiles + T) * E.aps + a) * 64 + half * 32 + g * 4 + t), f);
}

__device__ __forceinline__ int b_row_bytes(int KS) { return ((KS * 2) % 128 == 64) ? KS * 2 : KS * 2 + 64; }

// Write 8 activation values (k_local .. k_local+7 of a slab) of row m as the hi and lo bf16 columns.
__device__ __forceinline__ void store_act8(unsigned char *slab_base, int row_bytes, int m, int k_local,
                                           const float (&v)[8]) {
  __align__(16) __nv_bfloat16 h[8], l[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) split_bf16(v[j], h[j], l[j]);
  *reinterpret_cast<uint4 *>(slab_base + (size_t)(2 * m) * row_bytes + k_local * 2) = *reinterpret_cast<uint4 *>(h);
  *reinterpret_cast<uint4 *>(slab_base + (size_t)(2 * m + 1) * row_bytes + k_local * 2) = *reinterpret_cast<uint4 *>(l);
}

// Which k-slabs this block's share of W touches.
struct SlabSpan { int first, count, KS, row_bytes; };
__device__ __forceinline__ SlabSpan slab_span(const PackedMat &W) {
  long long c0, c1, w0, w1;
  stream_ranges(W, 0, c0, c1, w0, w1);
  SlabSpan sp;
  sp.KS = W.aps * 32;
  sp.row_bytes = b_row_bytes(sp.KS);
  const long long slab_atoms = (long long)W.n_tiles * W.aps;
  if (c0 >= c1) { sp.first = 0; sp.count = 0; return sp; }
  sp.first = (int)(c0 / slab_atoms);
  sp.count = (int)((c1 - 1) / slab_atoms) - sp.first + 1;
  return sp;
}

// ---------------------------------------------------------------------------- stage prologues

// Where the rows entering a norm come from.
enum { SRC_X = 0, SRC_EMBED = 1, SRC_BOUNDARY = 2 };

struct RowSource {
  int mode;
  const float *x;        // SRC_X: rows [M][H]; SRC_BOUNDARY: x_lo
  float *x_out;          // SRC_EMBED / SRC_BOUNDARY: the residual rows to initialise
  int R, pos0;           // row m = b*R + r sits at position pos0 + r
  int R_lo;              // SRC_BOUNDARY: rows per sequence in x_lo
  int add_embed;         // SRC_BOUNDARY: literal sum of Eq. 4
};

__device__ __forceinline__ int checked_token(const PassParams &P, int b, int pos) {
  int tok = P.tokens[(size_t)b * P.max_seq + pos];
  if (tok < 0 || tok >= P.embed.N) {
    atomicMax(P.error, PK_ERR_TOKEN);
    tok = min(max(tok, 0), P.embed.N - 1);
  }
  return tok;
}

__device__ __forceinline__ void source8(const PassParams &P, const RowSource &rs, int m, int tok, int u, float (&f)[8]) {
  if (rs.mode == SRC_X) {
    ldcg8(rs.x + (size_t)m * P.H + u * 8, f);
  } else if (rs.mode == SRC_EMBED) {
    embed8(P.embed, tok, u, f);
  } else {
    ldcg8(rs.x + ((size_t)m * rs.R_lo + rs.R_lo - 1) * P.H + u * 8, f);
    if (rs.add_embed) {
      float e[8];
      embed8(P.embed, tok, u, e);
#pragma unroll
      for (int j = 0; j < 8; ++j) f[j] += e[j];
    }
  }
}

// RMSNorm of the M source rows, written as bf16 hi/lo columns for the k-slabs this block needs
// of matrix W (steps a2 / a6 / a9, first half).  Also initialises the residual rows when they
// come from the embedding or from the lower stack (steps a1, a8).
__device__ void norm_prologue(const PassParams &P, const PassShared &S, const RowSource &rs, int M,
                              const float *w_norm, const PackedMat &W) {
  const int units = P.H / 8;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float ss[PK_MAX_ROWS];
  int toks[PK_MAX_ROWS];
#pragma unroll
  for (int m = 0; m < PK_MAX_ROWS; ++m) {
    ss[m] = 0.f;
    toks[m] = 0;
    if (m < M && rs.mode != SRC_X) toks[m] = checked_token(P, m / rs.R, rs.pos0 + m % rs.R);
  }
#pragma unroll
  for (int m = 0; m < PK_MAX_ROWS; ++m) {
    if (m < M) {
      for (int u = threadIdx.x; u < units; u += PK_THREADS) {
        float f[8];
        source8(P, rs, m, toks[m], u, f);
#pragma unroll
        for (int j = 0; j < 8; ++j) ss[m] += f[j] * f[j];
        if (rs.mode != SRC_X && ((m * units + u) % gridDim.x) == blockIdx.x) {
          float *dst = rs.x_out + (size_t)m * P.H + u * 8;
          *reinterpret_cast<float4 *>(dst) = make_float4(f[0], f[1], f[2], f[3]);
          *reinterpret_cast<float4 *>(dst + 4) = make_float4(f[4], f[5], f[6], f[7]);
        }
      }
    }
  }
#pragma unroll
  for (int m = 0; m < PK_MAX_ROWS; ++m) {
    float v = warp_sum(ss[m]);
    if (lane == 0) S.red[warp * PK_MAX_ROWS + m] = v;
  }
  __syncthreads();
  float inv[PK_MAX_ROWS];
#pragma unroll
  for (int m = 0; m < PK_MAX_ROWS; ++m) {
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < PK_WARPS; ++w) v += S.red[w * PK_MAX_ROWS + m];
    inv[m] = rsqrtf(v / (float)P.H + P.eps);
  }
  const SlabSpan sp = slab_span(W);
  const int slab_units = sp.KS / 8;
  for (int sl = 0; sl < sp.count; ++sl) {
    unsigned char *base = S.bstage + (size_t)sl * 8 * sp.row_bytes;
    const int u0 = (sp.first + sl) * slab_units;
#pragma unroll
    for (int m = 0; m < PK_MAX_ROWS; ++m) {
      if (m < M) {
        for (int uu = threadIdx.x; uu < slab_units; uu += PK_THREADS) {
          float f[8];
          source8(P, rs, m, toks[m], u0 + uu, f);
          const float4 wa = __ldg(reinterpret_cast<const float4 *>(w_norm + (u0 + uu) * 8));
          const float4 wb = __ldg(reinterpret_cast<const float4 *>(w_norm + (u0 + uu) * 8) + 1);
          f[0] *= inv[m] * wa.x; f[1] *= inv[m] * wa.y; f[2] *= inv[m] * wa.z; f[3] *= inv[m] * wa.w;
          f[4] *= inv[m] * wb.x; f[5] *= inv[m] * wb.y; f[6] *= inv[m] * wb.z; f[7] *= inv[m] * wb.w;
          store_act8(base, sp.row_bytes, m, uu * 8, f);
        }
      }
    }
  }
  __syncthreads();
}

// SwiGLU gate (step a6, second half) for the k-slabs this block needs of the down projection.
__device__ void swiglu_prologue(const PassParams &P, const PassShared &S, int M, const PackedMat &W) {
  const SlabSpan sp = slab_span(W);
  const int slab_units = sp.KS / 8, ldgu = 2 * P.I;
  for (int sl = 0; sl < sp.count; ++sl) {
    unsigned char *base = S.bstage + (size_t)sl * 8 * sp.row_bytes;
    const int k0 = (sp.first + sl) * sp.KS;
    for (int idx = threadIdx.x; idx < M * slab_units; idx += PK_THREADS) {
      const int m = idx / slab_units, uu = idx % slab_units;
      float g[8], u[8], f[8];
      ldcg8(P.gu + (size_t)m * ldgu + k0 + uu * 8, g);
      ldcg8(P.gu + (size_t)m * ldgu + P.I + k0 + uu * 8, u);
#pragma unroll
      for (int j = 0; j < 8; ++j) f[j] = g[j] / (1.f + expf(-g[j])) * u[j];
      store_act8(base, sp.row_bytes, m, uu * 8, f);
    }
  }
  __syncthreads();
}

// Key slices of one (sequence, kv head): nsplit slices of CH cached keys; the last slice also
// takes the R keys of the pass itself.
__device__ __forceinline__ void attn_plan_device(const PassParams &P, int pos0, int &nsplit, int &CH) {
  int want = max(1, min(PK_NSPLIT_CAP, (int)gridDim.x / (P.B * P.nkv)));
  CH = max(1, (pos0 + want - 1) / want);
  CH = (CH + 7) & ~7;
  nsplit = max(1, (pos0 + CH - 1) / CH);
}

// Online-softmax merge of the key slices (step a4, second half) for the heads this block's
// share of the O projection multiplies, written as bf16 hi/lo columns.
__device__ void merge_prologue(const PassParams &P, const PassShared &S, int M, int pos0, const PackedMat &W) {
  int nsplit, CH;
  attn_plan_device(P, pos0, nsplit, CH);
  const SlabSpan sp = slab_span(W);
  if (sp.count > 0) {
    const int k_first = sp.first * sp.KS, k_end = (sp.first + sp.count) * sp.KS;
    const int h_first = k_first / PK_D, n_heads = (k_end - 1) / PK_D - h_first + 1;
    // weights of every slice, normalised by the merged sum
    for (int idx = threadIdx.x; idx < M * n_heads; idx += PK_THREADS) {
      const int m = idx / n_heads, hh = idx % n_heads;
      const float *ml = P.part_ml + ((size_t)m * P.nq + h_first + hh) * PK_NSPLIT_CAP * 2;
      float mx = -INFINITY;
      for (int s = 0; s < nsplit; ++s) {
        const float2 v = __ldcg(reinterpret_cast<const float2 *>(ml) + s);
        if (v.y > 0.f) mx = fmaxf(mx, v.x);
      }
      float l = 0.f;
      float *wt = S.misc + (size_t)idx * PK_NSPLIT_CAP;
      for (int s = 0; s < nsplit; ++s) {
        const float2 v = __ldcg(reinterpret_cast<const float2 *>(ml) + s);
        const float f = v.y > 0.f ? __expf(v.x - mx) : 0.f;
        wt[s] = f;
        l += v.y * f;
      }
      const float inv = 1.f / l;
      for (int s = 0; s < nsplit; ++s) wt[s] *= inv;
    }
    __syncthreads();
    const int slab_units = sp.KS / 8;
    for (int idx = threadIdx.x; idx < sp.count * M * slab_units; idx += PK_THREADS) {
      const int uu = idx % slab_units, m = (idx / slab_units) % M, sl = idx / (slab_units * M);
      const int k = (sp.first + sl) * sp.KS + uu * 8, h = k / PK_D, dd = k % PK_D;
      const float *wt = S.misc + (size_t)(m * n_heads + h - h_first) * PK_NSPLIT_CAP;
      const float *po = P.part_o + (((size_t)m * P.nq + h) * PK_NSPLIT_CAP) * PK_D + dd;
      float f[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      for (int s = 0; s < nsplit; ++s) {
        float v[8];
        ldcg8(po + (size_t)s * PK_D, v);
        const float w = wt[s];
#pragma unroll
        for (int j = 0; j < 8; ++j) f[j] += w * v[j];
      }
      store_act8(S.bstage + (size_t)sl * 8 * sp.row_bytes, sp.row_bytes, m, uu * 8, f);
    }
  }
  __syncthreads();
}

// ---------------------------------------------------------------------------- projection

// out[m][n] += sum_k W[n][k] act[m][k] over this warp's share of W, streamed through its ring.
// Weights are the A operand of mma.m16n8k16 (register order, straight from the ring), the
// activation hi/lo columns the B operand.
__device__ bool gemv_consume(const PassParams &P, const PassShared &S, WarpPipe &pp, const PackedMat &W, int M,
                             float *__restrict__ out, int ldo) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  long long c0, c1, w0, w1;
  stream_ranges(W, warp, c0, c1, w0, w1);
  if (w0 >= w1) return true;
  const long long slab_atoms = (long long)W.n_tiles * W.aps;
  const int KS = W.aps * 32, row_bytes = b_row_bytes(KS);
  const int s_first = (int)(c0 / slab_atoms);
  int s = (int)(w0 / slab_atoms);
  long long in_slab = w0 - (long long)s * slab_atoms;
  int T = (int)(in_slab / W.aps), a = (int)(in_slab % W.aps);
  const uint32_t bst = smem_u32(S.bstage) + g * row_bytes + t * 16;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  long long idx = w0;
  while (idx < w1) {
    const int n = (int)min((long long)PK_CHUNK_ATOMS, w1 - idx);
    if (!pipe_wait(P, S, pp)) return false;
    const uint32_t slot_addr = pp.ring + (pp.consumed % PK_SLOTS) * PK_CHUNK_BYTES + lane * 16;
    uint4 A0[PK_CHUNK_ATOMS], A1[PK_CHUNK_ATOMS];
#pragma unroll
    for (int u = 0; u < PK_CHUNK_ATOMS; ++u) {
      if (u < n) {
        A0[u] = lds128(slot_addr + u * 1024);
        A1[u] = lds128(slot_addr + u * 1024 + 512);
      }
    }
#pragma unroll
    for (int u = 0; u < PK_CHUNK_ATOMS; ++u) {
      if (u < n) {
        const uint4 Bv = lds128(bst + (s - s_first) * 8 * row_bytes + a * 64);
        mma_bf16_16816(acc, A0[u].x, A1[u].x, A0[u].y, A1[u].y, Bv.x, Bv.y);
        mma_bf16_16816(acc, A0[u].z, A1[u].z, A0[u].w, A1[u].w, Bv.z, Bv.w);
        ++a;
        ++idx;
        if (a == W.aps || idx == w1) {
          // accumulator columns 2t (hi) and 2t+1 (lo) belong to activation row t
          const int n_lo = T * 16 + g;
          if (t < M) {
            if (n_lo < W.N) atomicAdd(out + (size_t)t * ldo + n_lo, acc[0] + acc[1]);
            if (n_lo + 8 < W.N) atomicAdd(out + (size_t)t * ldo + n_lo + 8, acc[2] + acc[3]);
          }
          acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
          a = 0;
          if (++T == W.n_tiles) { T = 0; ++s; }
        }
      }
    }
    pp.consumed += 1;
    __syncwarp();
    if (lane == 0) {
      fence_proxy_async();
      pipe_issue(P, S, pp, warp);
    }
  }
  return true;
}

// Clear `n` floats, the work spread over the grid.
__device__ __forceinline__ void grid_zero(float *p, int n) {
  for (int i = (blockIdx.x * PK_THREADS + threadIdx.x) * 4; i < n; i += gridDim.x * PK_THREADS * 4) {
    if (i + 4 <= n) {
      *reinterpret_cast<float4 *>(p + i) = make_float4(0.f, 0.f, 0.f, 0.f);
    } else {
      for (int j = i; j < n; ++j) p[j] = 0.f;
    }
  }
}

// ---------------------------------------------------------------------------- attention

__device__ __forceinline__ void load_bf16x8(const __nv_bfloat16 *p, float (&f)[8]) {
  unpack8(*reinterpret_cast<const uint4 *>(p), f);
}

// Steps a3 + a4 (first half) for the items (sequence, kv head, key slice) of this block: per-head
// QK-norm, rotary embedding, KV append, then attention of the R*G query rows against the slice,
// leaving unnormalised partial outputs with their running max and sum.
__device__ void attention_stage(const PassParams &P, const PassShared &S, const PassLayer &Ly, int R, int pos0) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = P.nq / P.nkv, nQ = R * G, ldq = (P.nq + 2 * P.nkv) * PK_D;
  int nsplit, CH;
  attn_plan_device(P, pos0, nsplit, CH);
  const int items = P.B * P.nkv * nsplit;

  float *q_s = reinterpret_cast<float *>(S.bstage);                               // [PK_QR][128]
  float *p_s = q_s + PK_QR * PK_D;                                                 // [PK_WARPS][PK_QR][32], later o_s
  float *o_s = p_s;                                                                // [PK_WARPS][4][128]
  __nv_bfloat16 *knew_s = reinterpret_cast<__nv_bfloat16 *>(p_s + PK_WARPS * PK_QR * 32);   // [4][128]
  __nv_bfloat16 *vnew_s = knew_s + PK_MAX_ROWS * PK_D;
  float *red_m = reinterpret_cast<float *>(vnew_s + PK_MAX_ROWS * PK_D);           // [PK_WARPS][PK_QR]
  float *red_l = red_m + PK_WARPS * PK_QR;
  const float scale = rsqrtf((float)PK_D);

  for (int item = blockIdx.x; item < items; item += gridDim.x) {
    const int split = item % nsplit, kvh = (item / nsplit) % P.nkv, b = item / (nsplit * P.nkv);
    __syncthreads();
    // a3: one warp per head vector of the new rows
    for (int task = warp; task < nQ + 2 * R; task += PK_WARPS) {
      int r, col, kind;                                   // kind 0 q, 1 k, 2 v
      if (task < nQ) { r = task / G; col = (kvh * G + task % G) * PK_D; kind = 0; }
      else if (task < nQ + R) { r = task - nQ; col = (P.nq + kvh) * PK_D; kind = 1; }
      else { r = task - nQ - R; col = (P.nq + P.nkv + kvh) * PK_D; kind = 2; }
      const float *src = P.qkv + (size_t)(b * R + r) * ldq + col;
      const int pos = pos0 + r;
      float v[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) v[j] = __ldcg(src + lane + 32 * j);
      if (kind == 2) {
        __nv_bfloat16 *dst = Ly.vc + (((size_t)b * P.nkv + kvh) * P.max_seq + pos) * PK_D;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const __nv_bfloat16 h = __float2bfloat16_rn(v[j]);
          vnew_s[r * PK_D + lane + 32 * j] = h;
          if (split == 0) dst[lane + 32 * j] = h;
        }
        continue;
      }
      float ss = v[0] * v[0] + v[1] * v[1] + v[2] * v[2] + v[3] * v[3];
      ss = warp_sum(ss);
      const float inv = rsqrtf(ss / (float)PK_D + P.eps);
      const float *w = kind == 0 ? Ly.w_qn : Ly.w_kn;
#pragma unroll
      for (int j = 0; j < 4; ++j) v[j] = v[j] * inv * __ldg(w + lane + 32 * j);
      float o[4];
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        double sn, cs;
        sincos((double)pos * P.inv_freq[lane + 32 * j], &sn, &cs);
        const float c = (float)cs, s_ = (float)sn;
        o[j] = v[j] * c - v[j + 2] * s_;
        o[j + 2] = v[j + 2] * c + v[j] * s_;
      }
      if (kind == 0) {
#pragma unroll
        for (int j = 0; j < 4; ++j) q_s[task * PK_D + lane + 32 * j] = o[j] * scale;
      } else {
        __nv_bfloat16 *dst = Ly.kc + (((size_t)b * P.nkv + kvh) * P.max_seq + pos) * PK_D;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const __nv_bfloat16 h = __float2bfloat16_rn(o[j]);
          knew_s[r * PK_D + lane + 32 * j] = h;
          if (split == 0) dst[lane + 32 * j] = h;
        }
      }
    }
    __syncthreads();

    // a4: keys [j0, j1) of the cache, then (last slice) the R new keys
    const int j0 = split * CH, j1 = min(j0 + CH, pos0);
    const int n_cached = max(0, j1 - j0);
    const int n_keys = n_cached + (split == nsplit - 1 ? R : 0);
    const __nv_bfloat16 *kbase = Ly.kc + ((size_t)b * P.nkv + kvh) * P.max_seq * PK_D;
    const __nv_bfloat16 *vbase = Ly.vc + ((size_t)b * P.nkv + kvh) * P.max_seq * PK_D;
    float m_run[PK_QR], l_run[PK_QR], o_acc[PK_QR][4];
#pragma unroll
    for (int qi = 0; qi < PK_QR; ++qi) {
      m_run[qi] = -INFINITY; l_run[qi] = 0.f;
      o_acc[qi][0] = o_acc[qi][1] = o_acc[qi][2] = o_acc[qi][3] = 0.f;
    }
    for (int base = warp * 32; base < n_keys; base += PK_WARPS * 32) {
      const int jj = base + lane;
      const bool valid = jj < n_keys;
      const bool fresh = jj >= n_cached;
      const int key_pos = fresh ? pos0 + (jj - n_cached) : j0 + jj;
      float s[PK_QR];
#pragma unroll
      for (int qi = 0; qi < PK_QR; ++qi) s[qi] = 0.f;
      if (valid) {
        const __nv_bfloat16 *kr = fresh ? knew_s + (jj - n_cached) * PK_D : kbase + (size_t)key_pos * PK_D;
        for (int c = 0; c < PK_D / 8; ++c) {
          float kf[8];
          load_bf16x8(kr + c * 8, kf);
#pragma unroll
          for (int qi = 0; qi < PK_QR; ++qi) {
            if (qi < nQ) {
              const float4 qa = *reinterpret_cast<const float4 *>(q_s + qi * PK_D + c * 8);
              const float4 qb = *reinterpret_cast<const float4 *>(q_s + qi * PK_D + c * 8 + 4);
              s[qi] += kf[0] * qa.x + kf[1] * qa.y + kf[2] * qa.z + kf[3] * qa.w + kf[4] * qb.x + kf[5] * qb.y +
                       kf[6] * qb.z + kf[7] * qb.w;
            }
          }
        }
      }
#pragma unroll
      for (int qi = 0; qi < PK_QR; ++qi) {
        if (qi < nQ) {
          const bool ok = valid && key_pos <= pos0 + qi / G;
          const float sv = ok ? s[qi] : -INFINITY;
          const float m_new = fmaxf(m_run[qi], warp_max(sv));
          float p = 0.f, corr = 1.f;
          if (m_new > -INFINITY) {
            corr = __expf(m_run[qi] - m_new);
            p = ok ? __expf(sv - m_new) : 0.f;
          }
          l_run[qi] = l_run[qi] * corr + warp_sum(p);
          m_run[qi] = m_new;
#pragma unroll
          for (int e = 0; e < 4; ++e) o_acc[qi][e] *= corr;
          p_s[(warp * PK_QR + qi) * 32 + lane] = p;
        }
      }
      __syncwarp();
      const int n_here = min(32, n_keys - base);
      for (int x = 0; x < n_here; ++x) {
        const int jx = base + x;
        const __nv_bfloat16 *vr =
            (jx >= n_cached ? vnew_s + (jx - n_cached) * PK_D : vbase + (size_t)(j0 + jx) * PK_D) + lane * 4;
        const uint2 raw = *reinterpret_cast<const uint2 *>(vr);
        const float v0 = bf16_bits_to_float(raw.x & 0xffffu), v1 = bf16_bits_to_float(raw.x >> 16);
        const float v2 = bf16_bits_to_float(raw.y & 0xffffu), v3 = bf16_bits_to_float(raw.y >> 16);
#pragma unroll
        for (int qi = 0; qi < PK_QR; ++qi) {
          if (qi < nQ) {
            const float p = p_s[(warp * PK_QR + qi) * 32 + x];
            o_acc[qi][0] += p * v0; o_acc[qi][1] += p * v1; o_acc[qi][2] += p * v2; o_acc[qi][3] += p * v3;
          }
        }
      }
      __syncwarp();
    }

    // combine the warps, four query rows at a time
#pragma unroll
    for (int qi = 0; qi < PK_QR; ++qi)
      if (lane == 0) { red_m[warp * PK_QR + qi] = m_run[qi]; red_l[warp * PK_QR + qi] = l_run[qi]; }
#pragma unroll
    for (int bt = 0; bt < PK_QR / 4; ++bt) {
      if (bt * 4 < nQ) {
        __syncthreads();
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4)
          *reinterpret_cast<float4 *>(o_s + ((warp * 4 + q4) * PK_D) + lane * 4) =
              make_float4(o_acc[bt * 4 + q4][0], o_acc[bt * 4 + q4][1], o_acc[bt * 4 + q4][2], o_acc[bt * 4 + q4][3]);
        __syncthreads();
        for (int idx = threadIdx.x; idx < 4 * PK_D; idx += PK_THREADS) {
          const int q4 = idx / PK_D, dd = idx % PK_D, qi = bt * 4 + q4;
          if (qi < nQ) {
            float m = -INFINITY;
#pragma unroll
            for (int w = 0; w < PK_WARPS; ++w) m = fmaxf(m, red_m[w * PK_QR + qi]);
            float l = 0.f, o = 0.f;
#pragma unroll
            for (int w = 0; w < PK_WARPS; ++w) {
              const float mw = red_m[w * PK_QR + qi];
              const float f = mw > -INFINITY ? __expf(mw - m) : 0.f;
              l += red_l[w * PK_QR + qi] * f;
              o += o_s[(w * 4 + q4) * PK_D + dd] * f;
            }
            const int r = qi / G, h = kvh * G + qi % G;
            const size_t slot = ((size_t)(b * R + r) * P.nq + h) * PK_NSPLIT_CAP + split;
            P.part_o[slot * PK_D + dd] = o;
            if (dd == 0) { P.part_ml[slot * 2] = m; P.part_ml[slot * 2 + 1] = l; }
          }
        }
      }
    }
  }
  __syncthreads();
}

// ---------------------------------------------------------------------------- the pass

__global__ void __launch_bounds__(PK_THREADS, 1) dmtd_pass_kernel(const PassParams P) {
  extern __shared__ __align__(1024) unsigned char smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  PassShared S;
  S.ring = smem + PK_OFF_RING;
  S.bstage = smem + PK_OFF_BSTAGE;
  S.misc = reinterpret_cast<float *>(smem + PK_OFF_MISC);
  S.bars = reinterpret_cast<uint64_t *>(smem + PK_OFF_BARS);
  S.abort_flag = reinterpret_cast<volatile int *>(smem + PK_OFF_SMALL);
  S.red = reinterpret_cast<float *>(smem + PK_OFF_SMALL + 16);
  S.layers = reinterpret_cast<PassLayer *>(smem + PK_OFF_LAYERS);

  const int nL = P.l_end - P.l_begin;
  {
    const int *src = reinterpret_cast<const int *>(P.layers + P.l_begin);
    int *dst = reinterpret_cast<int *>(S.layers);
    for (int i = threadIdx.x; i < nL * (int)(sizeof(PassLayer) / 4); i += PK_THREADS) dst[i] = src[i];
  }
  if (threadIdx.x == 0) *S.abort_flag = 0;
  if (lane == 0) {
    for (int s = 0; s < PK_SLOTS; ++s) mbar_init(smem_u32(S.bars + warp * PK_SLOTS + s), 1);
    fence_mbar_init();
  }
  __syncthreads();

  const int lo_len = P.st->lo_len, newest = P.st->newest;
  WarpPipe pp;
  pp.ring = smem_u32(S.ring) + warp * PK_SLOTS * PK_CHUNK_BYTES;
  pp.bars = smem_u32(S.bars + warp * PK_SLOTS);
  pp.issued = pp.consumed = 0;
  pp.p_mat = -1; pp.n_mats = 4 * nL + 1;
  pp.p_pos = pp.p_end = 0; pp.p_base = nullptr;
  if (lane == 0)
    for (int s = 0; s < PK_SLOTS; ++s) pipe_issue(P, S, pp, warp);

  unsigned bar_target = 0;
  bool ok = true;
  const int ldqkv = (P.nq + 2 * P.nkv) * PK_D, ldgu = 2 * P.I;
  const int M_max = P.B * ((P.l_begin < P.l_split) ? P.R_lo : 1);

  // buffers the projections accumulate into start at zero
  grid_zero(P.qkv, M_max * ldqkv);
  grid_zero(P.gu, M_max * ldgu);
  grid_zero(P.logits, P.B * P.ldl);
  ok = grid_barrier(P, S, bar_target);

  for (int li = 0; li < nL && ok; ++li) {
    const int l = P.l_begin + li;
    const bool lower = l < P.l_split;
    const int R = lower ? P.R_lo : 1, M = P.B * R, pos0 = lower ? lo_len : newest;
    float *x = lower ? P.x_lo : P.x_up;
    const PassLayer &Ly = S.layers[li];

    // ---- a1/a8 + a2: rows in, RMSNorm, QKV projection
    RowSource rs;
    rs.R = R; rs.pos0 = pos0; rs.R_lo = P.R_lo; rs.add_embed = P.literal_sum; rs.x_out = x;
    if (li == 0) { rs.mode = SRC_EMBED; rs.x = nullptr; }
    else if (l == P.l_split && P.l_begin < P.l_split) { rs.mode = SRC_BOUNDARY; rs.x = P.x_lo; }
    else { rs.mode = SRC_X; rs.x = x; }
    norm_prologue(P, S, rs, M, Ly.w_in, Ly.qkv);
    ok = gemv_consume(P, S, pp, Ly.qkv, M, P.qkv, ldqkv);
    if (!ok) *S.abort_flag = 1;
    if (!(ok = grid_barrier(P, S, bar_target))) break;

    // ---- a3 + a4: QK-norm, RoPE, KV append, attention over the key slices
    attention_stage(P, S, Ly, R, pos0);
    if (!(ok = grid_barrier(P, S, bar_target))) break;

    // ---- a4 merge + a5: O projection into the residual rows
    grid_zero(P.gu, M_max * ldgu);
    merge_prologue(P, S, M, pos0, Ly.o);
    ok = gemv_consume(P, S, pp, Ly.o, M, x, P.H);
    if (!ok) *S.abort_flag = 1;
    if (!(ok = grid_barrier(P, S, bar_target))) break;

    // ---- a6: RMSNorm, gate and up projections
    rs.mode = SRC_X; rs.x = x;
    norm_prologue(P, S, rs, M, Ly.w_post, Ly.gu);
    ok = gemv_consume(P, S, pp, Ly.gu, M, P.gu, ldgu);
    if (!ok) *S.abort_flag = 1;
    if (!(ok = grid_barrier(P, S, bar_target))) break;

    // ---- a6 gate + a7: down projection into the residual rows
    grid_zero(P.qkv, M_max * ldqkv);
    swiglu_prologue(P, S, M, Ly.down);
    ok = gemv_consume(P, S, pp, Ly.down, M, x, P.H);
    if (!ok) *S.abort_flag = 1;
    if (!(ok = grid_barrier(P, S, bar_target))) break;
  }

  if (ok) {
    // ---- a9: final norm, tied head
    RowSource rs;
    rs.mode = SRC_X; rs.x = P.x_up; rs.x_out = nullptr; rs.R = 1; rs.pos0 = newest; rs.R_lo = P.R_lo; rs.add_embed = 0;
    norm_prologue(P, S, rs, P.B, P.w_final, P.embed);
    ok = gemv_consume(P, S, pp, P.embed, P.B, P.logits, P.ldl);
    if (!ok) *S.abort_flag = 1;
    ok = grid_barrier(P, S, bar_target);
  }
  if (ok) {
    // ---- greedy pick, first level: this block's slice of the vocabulary
    const int per = (P.vocab + gridDim.x - 1) / gridDim.x;
    const int i0 = blockIdx.x * per, i1 = min(P.vocab, i0 + per);
    float *sv = reinterpret_cast<float *>(S.bstage);
    int *si = reinterpret_cast<int *>(S.bstage) + PK_THREADS;
    for (int b = 0; b < P.B; ++b) {
      float best = -INFINITY;
      int bi = 0x7fffffff;
      for (int i = i0 + threadIdx.x; i < i1; i += PK_THREADS) {
        const float v = __ldcg(P.logits + (size_t)b * P.ldl + i);
        if (v > best) { best = v; bi = i; }
      }
      __syncthreads();
      sv[threadIdx.x] = best; si[threadIdx.x] = bi;
      __syncthreads();
      for (int s = PK_THREADS >> 1; s > 0; s >>= 1) {
        if (threadIdx.x < s) {
          const float v2 = sv[threadIdx.x + s];
          const int i2 = si[threadIdx.x + s];
          if (v2 > sv[threadIdx.x] || (v2 == sv[threadIdx.x] && i2 < si[threadIdx.x])) {
            sv[threadIdx.x] = v2; si[threadIdx.x] = i2;
          }
        }
        __syncthreads();
      }
      if (threadIdx.x == 0) {
        P.amax_val[b * gridDim.x + blockIdx.x] = sv[0];
        P.amax_idx[b * gridDim.x + blockIdx.x] = si[0];
      }
    }
    ok = grid_barrier(P, S, bar_target);
  }
  if (ok && blockIdx.x == 0) {
    // ---- greedy pick, second level (lowest index on ties); a10 token feedback; a0 counters
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
    __syncthreads();
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

  // leave no copy in flight: a slot this warp still waits for gets a bounded wait
  while (pp.consumed < __shfl_sync(0xffffffffu, pp.issued, 0)) {
    const unsigned slot = pp.consumed % PK_SLOTS;
    const uint32_t parity = (pp.consumed / PK_SLOTS) & 1u;
    const long long t0 = clock64();
    while (!mbar_try_wait(pp.bars + slot * 8, parity))
      if (clock64() - t0 > P.wait_limit) break;
    pp.consumed += 1;
  }
}

}  // namespace dmtd
