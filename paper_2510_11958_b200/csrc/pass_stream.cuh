// The per-warp weight stream of the pass kernel, the grid barrier, and small load/store helpers.
#pragma once

#include "pass_common.cuh"

namespace dmtd {

// Profiling builds: clock64() of thread 0 of the first block at points inside a norm prologue (slots 3072 ..)
// and the grid barrier (3088 ..); the values of the last call stay.
#ifdef DMTD_PASS_TIMING
#define PK_PROSTAMP(i)                                                                 \
  do {                                                                                 \
    if (threadIdx.x == 0 && blockIdx.x == 0 && P.timing) P.timing[3072 + (i)] = clock64(); \
  } while (0)
#else
#define PK_PROSTAMP(i) do {} while (0)
#endif

// Position in one warp's weight stream: its share of every matrix of the pass, in pass order.
// Atom counts are 32-bit: the host checks atoms * blocks < 2^31 for every matrix.
struct StreamCursor {
  int mat, n_mats, warp;
  int pos, end;
  int tile_mask;            // atoms per 16-row tile - 1 where chunks can be cut at tile boundaries, else 0
  const uint4 *base;
};

// A warp's ring: lane 0 runs the producer cursor; all lanes agree on `consumed`.  Lives in
// shared memory between stages and in registers inside a projection.
struct WarpPipe {
  uint32_t ring, bars;      // shared addresses of this warp's slots and barriers
  unsigned issued, consumed;
  StreamCursor cur;
};
static_assert(sizeof(WarpPipe) * PK_WARPS <= 1024 - 256, "pipe state does not fit");

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
__device__ __forceinline__ void stream_ranges(const PackedMat &W, int warp, int &c0, int &c1, int &w0, int &w1) {
  const unsigned A = (unsigned)(W.n_slabs * W.n_tiles * W.aps);
  c0 = (int)(A * blockIdx.x / gridDim.x);
  c1 = (int)(A * (blockIdx.x + 1) / gridDim.x);
  w0 = c0 + (c1 - c0) * warp / PK_WARPS;
  w1 = c0 + (c1 - c0) * (warp + 1) / PK_WARPS;
}

// While the attention stage runs, HBM is idle (the rings are full) and the blocks without an attention item wait
// in its barrier.  They ask L2 for a part of the layer's gate+up matrix: for every warp of the grid the atoms
// [skip, skip + atoms) of its share (the first `skip` the ring requests by itself during the O projection).
// The requests compete with nothing that a barrier waits for.  idle_rank: this block's index among the n_idle
// blocks without an item.  Requests of one chunk each, spread evenly over the idle blocks: the copy engine of
// an SM works them off at about 30 GB/s, and a block that is still issuing is late at the barrier (whole 32 KiB
// requests from a few threads: the attention barrier took 23 us; all requests on the first idle blocks: 10 us).
// 32 KiB per warp (38 MB, what HBM delivers in the 6 us it is idle) is the measured optimum: the gate+up
// projection 13.5 -> 10.5 us.
#ifndef DMTD_PASS_ATTN_PF
#define DMTD_PASS_ATTN_PF 32
#endif
constexpr int PK_ATTN_PF_ATOMS = DMTD_PASS_ATTN_PF;
constexpr int PK_ATTN_PF_SKIP = PK_SLOTS * PK_CHUNK_ATOMS;
__device__ __forceinline__ void prefetch_matrix_part(const PackedMat &W, int idle_rank, int n_idle) {
  constexpr int REQ = (PK_ATTN_PF_ATOMS + PK_CHUNK_ATOMS - 1) / PK_CHUNK_ATOMS;      // requests per warp
  const unsigned A = (unsigned)(W.n_slabs * W.n_tiles * W.aps);
  const int total = (int)gridDim.x * PK_WARPS * REQ;
#pragma unroll 1
  for (int j = (int)threadIdx.x * n_idle + idle_rank; j < total; j += n_idle * PK_THREADS) {     // spread evenly over the idle blocks
    const int k = j % REQ, wg = j / REQ, warp = wg % PK_WARPS, blk = wg / PK_WARPS;
    const int c0 = (int)(A * (unsigned)blk / gridDim.x), c1 = (int)(A * (unsigned)(blk + 1) / gridDim.x);
    const int w0 = c0 + (c1 - c0) * warp / PK_WARPS, w1 = c0 + (c1 - c0) * (warp + 1) / PK_WARPS;
    const int start = w0 + PK_ATTN_PF_SKIP + k * PK_CHUNK_ATOMS;
    const int n = min(min(PK_CHUNK_ATOMS, PK_ATTN_PF_ATOMS - k * PK_CHUNK_ATOMS), w1 - start);
    if (n > 0)
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(W.w + (size_t)start * 64), "r"(n * 1024) : "memory");
  }
}

// At the end of a prologue (every block is past the barrier, the rings have been refilled, the prologue's own
// loads have landed, HBM is idle until the projection has drained the rings): lane 0 of every warp asks L2 for
// the next atoms of its own stream behind what the ring holds, `skip` atoms further on where an earlier request
// covered those already.  Measured with the request below (Qwen3-4B shape, batch 1): 880 -> 910 tokens/s; the
// same requests issued at the end of a projection, before the barrier, cost 4-10 % (they queue in front of
// the slowest block's last chunks, for which the barrier waits).
#ifndef DMTD_PASS_PRO_PF
#define DMTD_PASS_PRO_PF 16
#endif
constexpr int PK_PRO_PF_ATOMS = DMTD_PASS_PRO_PF;
__device__ __forceinline__ void prefetch_own_stream(const StreamCursor &cur, int skip) {
#pragma unroll 1
  for (int k = 0; k < PK_PRO_PF_ATOMS; k += PK_CHUNK_ATOMS) {
    const int start = cur.pos + skip + k;
    const int n = min(min(PK_CHUNK_ATOMS, PK_PRO_PF_ATOMS - k), cur.end - start);
    if (n > 0)
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(cur.base + (size_t)start * 64), "r"(n * 1024) : "memory");
  }
}

__device__ __forceinline__ const PackedMat &matrix_of_kind(const PassParams &P, const PassShared &S, int kind) {
  if (kind == PK_MAT_HEAD) return P.embed;
  const PassLayer &L = S.layers[0];
  return kind == PK_MAT_QKV ? L.qkv : kind == PK_MAT_O ? L.o : kind == PK_MAT_GU ? L.gu : L.down;
}
// Kernel entry: one thread per (matrix kind, warp) fills the plans (S.layers must be in place).
__device__ __forceinline__ void plans_fill(const PassParams &P, const PassShared &S) {
  const int kind = threadIdx.x / PK_WARPS, warp = threadIdx.x % PK_WARPS;
  if (kind >= PK_MAT_KINDS) return;
  if (kind != PK_MAT_HEAD && P.l_end == P.l_begin) return;
  const PackedMat &W = matrix_of_kind(P, S, kind);
  MatPlan &pl = S.plans[kind];
  int c0, c1, w0, w1;
  stream_ranges(W, warp, c0, c1, w0, w1);
  const int slab_atoms = W.n_tiles * W.aps;
  pl.w0[warp] = w0; pl.w1[warp] = w1;
  const int s = w0 / slab_atoms, in_slab = w0 - s * slab_atoms;
  pl.ws[warp] = s; pl.wT[warp] = in_slab / W.aps; pl.wa[warp] = in_slab % W.aps;
  if (warp == 0) {
    pl.c0 = c0; pl.c1 = c1;
    pl.s_first = c0 < c1 ? c0 / slab_atoms : 0;
    pl.s_count = c0 < c1 ? (c1 - 1) / slab_atoms - pl.s_first + 1 : 0;
  }
}

__device__ __forceinline__ void cursor_init(StreamCursor &c, const PassParams &P, int warp) {
  c.mat = -1; c.n_mats = 4 * (P.l_end - P.l_begin) + 1; c.warp = warp;
  c.pos = c.end = 0; c.tile_mask = 0; c.base = nullptr;
}

// Move the cursor to the warp's share of the next matrix that has one (once per matrix).
__device__ __noinline__ bool cursor_next_matrix(StreamCursor &c, const PassParams &P) {
  const PassShared S = pass_shared();
  while (c.pos >= c.end) {
    if (++c.mat >= c.n_mats) { c.mat = c.n_mats; return false; }
    const PackedMat &W = pass_matrix(P, S, c.mat);
    const MatPlan &pl = S.plans[c.mat >= 4 * (P.l_end - P.l_begin) ? PK_MAT_HEAD : (c.mat & 3)];
    c.pos = pl.w0[c.warp]; c.end = pl.w1[c.warp]; c.base = W.w;
    c.tile_mask = (PK_CHUNK_ATOMS % W.aps == 0 && (W.aps & (W.aps - 1)) == 0) ? W.aps - 1 : 0;
  }
  return true;
}

// Lane 0: issue the next chunk of the warp's stream, if any is left in the pass.
__device__ __forceinline__ void pipe_issue(const PassParams &P, WarpPipe &pp) {
  if (pp.cur.pos >= pp.cur.end) {
    // once per matrix; the copy keeps the ring state itself in registers (only an object whose address
    // is taken has to live in memory)
    StreamCursor next = pp.cur;
    const bool more = cursor_next_matrix(next, P);
    pp.cur = next;
    if (!more) return;
  }
  // a chunk ends where a tile ends (the first chunk of a share is the short one): the consumer then
  // meets whole tiles, which it multiplies without a test per atom
  const int n = min(PK_CHUNK_ATOMS - (pp.cur.pos & pp.cur.tile_mask), pp.cur.end - pp.cur.pos);
  const unsigned slot = pp.issued % PK_SLOTS;
  const uint32_t bar = pp.bars + slot * 8;
  mbar_expect_tx(bar, (uint32_t)n * 1024u);
  // read once: lowest priority in L2 (measured: +2.4 % tokens/s; the stages' shared data stays in L2)
  bulk_g2s_hint(pp.ring + slot * PK_CHUNK_BYTES, pp.cur.base + (size_t)pp.cur.pos * 64, (uint32_t)n * 1024u, bar,
                l2_policy_evict_first());
  pp.cur.pos += n;
  pp.issued += 1;
}

__device__ __noinline__ bool pipe_wait_slow(const PassParams &P, uint32_t bar, uint32_t parity) {
  const PassShared S = pass_shared();
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

// All lanes: wait until chunk `consumed` has landed.  Bounded; false = gave up.
__device__ __forceinline__ bool pipe_wait(const PassParams &P, const WarpPipe &pp) {
  const unsigned slot = pp.consumed % PK_SLOTS;
  const uint32_t parity = (pp.consumed / PK_SLOTS) & 1u;
  const uint32_t bar = pp.bars + slot * 8;
  if (mbar_try_wait(bar, parity)) return true;
  return pipe_wait_slow(P, bar, parity);
}

// Grid-wide barrier: every block arrives once per stage; `target` counts arrivals so far.
__device__ __noinline__ bool grid_barrier(const PassParams &P, unsigned &target) {
  const PassShared S = pass_shared();
  PK_PROSTAMP(16);
  pk_sync();
  PK_PROSTAMP(17);
  if (threadIdx.x == 0) {
    target += gridDim.x;
    if (*S.abort_flag) {
      atomicMax(P.error, PK_ERR_BARRIER_WAIT);
    } else {
      red_release_add(P.barrier, 1u);
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
    }
  }
  PK_PROSTAMP(18);
  pk_sync();
  PK_PROSTAMP(19);
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

// Values k = 8u .. 8u+7 of row `tok` of the packed embedding matrix.
__device__ __forceinline__ void embed8(const PackedMat &E, int tok, int u, float (&f)[8]) {
  const int k = u * 8, atom = k >> 5, t = (k >> 3) & 3;
  const int s = atom / E.aps, a = atom % E.aps;
  const int T = tok >> 4, half = (tok >> 3) & 1, g = tok & 7;
  unpack8(__ldg(E.w + (((long long)s * E.n_tiles + T) * E.aps + a) * 64 + half * 32 + g * 4 + t), f);
}

__device__ __forceinline__ int b_row_bytes(int KS) { return ((KS * 2) % 128 == 64) ? KS * 2 : KS * 2 + 64; }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

// Write 4 activation values (k_local .. k_local+3 of a slab) of row m as the hi and lo bf16
// columns: x = hi + lo with |error| <= 2^-17 |x|.
__device__ __forceinline__ void store_act4(unsigned char *slab_base, int row_bytes, int m, int k_local, float4 v) {
  const uint32_t h0 = pack_bf16x2(v.x, v.y), h1 = pack_bf16x2(v.z, v.w);
  const float r0 = v.x - __uint_as_float(h0 << 16), r1 = v.y - __uint_as_float(h0 & 0xffff0000u);
  const float r2 = v.z - __uint_as_float(h1 << 16), r3 = v.w - __uint_as_float(h1 & 0xffff0000u);
  *reinterpret_cast<uint2 *>(slab_base + (size_t)(2 * m) * row_bytes + k_local * 2) = make_uint2(h0, h1);
  *reinterpret_cast<uint2 *>(slab_base + (size_t)(2 * m + 1) * row_bytes + k_local * 2) =
      make_uint2(pack_bf16x2(r0, r1), pack_bf16x2(r2, r3));
}

// Which k-slabs this block's share of W touches.
struct SlabSpan { int first, count, KS, row_bytes; };
__device__ __forceinline__ SlabSpan slab_span(const PassShared &S, const PackedMat &W, int kind) {
  SlabSpan sp;
  sp.KS = W.aps * 32;
  sp.row_bytes = b_row_bytes(sp.KS);
  sp.first = S.plans[kind].s_first;
  sp.count = S.plans[kind].s_count;
  return sp;
}

// Clear `n` floats, the work spread over the grid.
__device__ __forceinline__ void grid_zero(float *p, int n) {
#pragma unroll 1
  for (int i = (blockIdx.x * PK_THREADS + threadIdx.x) * 4; i < n; i += gridDim.x * PK_THREADS * 4) {
    if (i + 4 <= n) {
      *reinterpret_cast<float4 *>(p + i) = make_float4(0.f, 0.f, 0.f, 0.f);
    } else {
      for (int j = i; j < n; ++j) p[j] = 0.f;
    }
  }
}

}  // namespace dmtd
