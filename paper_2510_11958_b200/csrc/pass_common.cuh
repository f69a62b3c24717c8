// Shared definitions of the persistent pass kernel: sizes, parameters, PTX wrappers, the
// shared-memory map, the per-warp weight stream and the grid barrier.
//
// Lessons the layout encodes (measured on B200, Qwen3-4B shape, batch 1):
//  * every stage runs once per layer and the stages of a layer are different code, so the code
//    of one layer must stay resident in the instruction cache: stage functions are separate,
//    small, and loop instead of unrolling;
//  * any load that crosses the chip costs a microsecond or more while the weight stream is
//    running, so a stage issues all of its loads before it uses any, and nothing in the weight
//    loop touches local or global memory;
//  * more bulk copies in flight than bandwidth x latency only lengthen every other round trip:
//    with 16 KiB per warp in flight a barrier poll or an activation load waited 3-4 us behind
//    the block's own weight traffic, with 8 KiB about half of that, at the same stream rate;
//    asking for the next projection's weights to be prefetched into L2 at a stage boundary made
//    the following projection slower, not faster, so nothing is requested beyond the ring;
//  * the grid barrier is one counter (release-add, acquire-poll by one thread per block): 2-3 us.
//    A flag per block polled by a warp (no atomic serialisation) took 5-6 us.
//  * handing a stage's outputs over without barriers was tried: every partial sum added with one
//    64-bit reduction to a word that carries a fixed-point sum and a count of the atoms summed in,
//    the next stage polling the words it needs.  It ran at the speed of the barrier version (what
//    a stage waits for is the slowest block's share, 1 - 2.5 us behind the median and a different
//    block every time, not the barrier's own 1.2 us), and a block's inputs come from only some of
//    the blocks, so nothing tells it when a buffer may be cleared or reused: one run in ten had a
//    pass with logits off by 1e-2.  Dropped.  (atomicAdd on unsigned long long compiled to the
//    returning form and slowed the weight loop by 15 %; red.global.add.u64 in PTX did not.)
//  * handing the block's chunks to its warps from one shared counter (so that the warps of a
//    block finish a projection together instead of 1-2 us apart) was tried: the bookkeeping per
//    4 KiB chunk (shared-memory atomic, table look-ups, two divisions, slot records) sits
//    between a slot becoming free and its next request, and the stream ran at half speed.
//    Fixed per-warp shares keep that path to a few dozen instructions.
//  * mma.sync issues once per 32 cycles per SM sub-partition here (the hmma sub-pipe counter of ncu):
//    with two warps per sub-partition and two MMAs per atom that is 128 of the 150 cycles the weight
//    loop takes per atom and warp - 2.3 times the SM's share of HBM, so the loop keeps up, and a ring
//    filled during a barrier is drained at that rate.  It is too slow for attention with bf16 hi/lo
//    pairs, which is why the fp32-cache attention stage uses FMAs.
//  * the weight loop must stay short: with one atom per trip and the tile bookkeeping inside it
//    (about 45 instructions per atom, each at its full latency with two warps per sub-partition) a
//    warp took 260 cycles per atom, exactly the SM's share of HBM, and never waited for a chunk.
#pragma once

#include "common.cuh"

namespace dmtd {

// Ring geometry (overridable at build time for sweeps).  Measured on the Qwen3-4B shape, batch 1,
// with a consumer loop that took one atom per trip, us per layer of a full pass: chunks of 4 / 5 / 6 /
// 7 / 8 atoms in 2 slots 66.9 / 64.9 / 63.6 / 63.5 / 64.8; 3 slots of 5 atoms 64.6, 4 slots of 4 atoms
// 64.7.  The loop that multiplies a whole 16-row tile (8 atoms at 256-wide k-slabs) in straight-line
// code wants a chunk to be a tile: 8 atoms (861 against 850 tokens/s with 7).  Two things pull one way: the copy
// engine of an SM spends ~100 cycles per bulk copy whatever its size (a plain stream of 4 KiB copies
// tops out at 60 GB/s per SM, of 8 KiB copies at 100 GB/s; the SM's share of HBM is 44 GB/s), and
// what the rings hold is what HBM delivers while the stage threads sit in a barrier.  The other
// way: every other load of the SM waits behind the copies in flight.
#ifndef DMTD_PASS_CHUNK
#define DMTD_PASS_CHUNK 8
#endif
#ifndef DMTD_PASS_SLOTS
#define DMTD_PASS_SLOTS 2
#endif
constexpr int PK_WARPS = 8;
constexpr int PK_THREADS = PK_WARPS * 32;
constexpr int PK_CHUNK_ATOMS = DMTD_PASS_CHUNK;            // atoms (1 KiB each) per bulk copy
constexpr int PK_CHUNK_BYTES = PK_CHUNK_ATOMS * 1024;

constexpr int PK_SLOTS = DMTD_PASS_SLOTS;                  // ring slots per warp
constexpr int PK_MAX_ROWS = 4;                             // activation rows (B*R) per stage
constexpr int PK_MAX_KS = 256;                             // largest k-slab of a packed matrix the kernel streams
constexpr int PK_MAX_LAYERS = 40;
constexpr int PK_NSPLIT_CAP = 16;                          // key slices per (sequence, kv head)
constexpr int PK_D = 128;                                  // head_dim
constexpr int PK_QR = 16;                                  // query rows per attention item
constexpr int PK_MAX_GROUP = 4;                            // query heads per kv head

// shared memory map (bytes)
constexpr int PK_RING_BYTES = PK_WARPS * PK_SLOTS * PK_CHUNK_BYTES;           // 114688
constexpr int PK_BROW_MAX = PK_MAX_KS * 2 + 64;                               // 576
constexpr int PK_BSTAGE_BYTES = 2 * 8 * PK_BROW_MAX;                          // 9216: two slabs of 8 columns
constexpr int PK_SCRATCH_BYTES = 88576;                                       // bstage + xs; the attention stages lay their own map over both
constexpr int PK_XS_BYTES = PK_SCRATCH_BYTES - PK_BSTAGE_BYTES;
constexpr int PK_XS_FLOATS = PK_XS_BYTES / 4;                                 // 19840: staged activation rows
constexpr int PK_OFF_RING = 0;
constexpr int PK_OFF_BSTAGE = PK_OFF_RING + PK_RING_BYTES;
constexpr int PK_OFF_XS = PK_OFF_BSTAGE + PK_BSTAGE_BYTES;                    // directly behind bstage
constexpr int PK_OFF_BARS = PK_OFF_XS + PK_XS_BYTES;
constexpr int PK_OFF_SMALL = PK_OFF_BARS + PK_WARPS * PK_SLOTS * 8;
constexpr int PK_SMALL_BYTES = 2048;
constexpr int PK_OFF_LAYERS = PK_OFF_SMALL + PK_SMALL_BYTES;

enum { PK_ERR_NONE = 0, PK_ERR_TOKEN = 1, PK_ERR_COPY_WAIT = 2, PK_ERR_BARRIER_WAIT = 3 };

struct PassLayer {
  PackedMat qkv, o, gu, down;
  const float *w_in, *w_post, *w_qn, *w_kn;
  void *kc, *vc;                          // this layer's cache [sequence][kv head][max_seq][128], bf16 or fp32
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
  int kv_f32;                             // the KV cache holds fp32 (else a 16-bit type)
  int kv_f16;                             // ... fp16 (else bf16)
  int write_token;
  int *tokens;
  DevState *st;
  float *x_lo, *x_up, *qkv, *gu, *logits, *part_o, *part_ml;
  float *amax_val;
  int *amax_idx;
  int *out_argmax;
  unsigned int *barrier;                  // zero at launch
  int *error;                             // sticky, 0 = fine
  long long wait_limit;                   // clock ticks a device-side wait may take
  SampleParams sample;                    // greedy pick, or a draw from softmax(logits / T)
  long long *timing;                      // stage time stamps (profiling builds), or NULL
};

constexpr int PK_SMEM_BYTES = PK_OFF_LAYERS + PK_MAX_LAYERS * (int)sizeof(PassLayer);
static_assert(PK_SMEM_BYTES <= 227 * 1024, "shared memory map too large");

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
// the same question without waiting: try_wait may suspend the thread for a while before it answers no
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
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
// the same with an L2 eviction priority: a stream that is read once should not push what the stages share
// through L2 (activations, partial sums, KV rows, the kernel's own instructions) out of it
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar, uint64_t pol) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar), "l"(pol)
               : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// orders this thread's earlier generic-proxy accesses to global memory before its later bulk copies
// (the unqualified fence also waits for shared-memory traffic and costs hundreds of cycles)
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release_add(unsigned *p, unsigned v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint4 v) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void pk_sync() { __syncthreads(); }

// ---------------------------------------------------------------------------- block state

struct WarpPipe;

// Where this block's and its warps' shares of a matrix begin and end (atoms of the stream), which k-slabs the
// block's share touches, and where in its slab a warp's share starts.  Every layer has the same five matrix shapes
// (QKV, O, gate+up, down; the tied head), so the plans are worked out once per launch: between two grid barriers
// everything is serial latency, and the divisions of these index computations were a measurable part of it.
enum { PK_MAT_QKV = 0, PK_MAT_O = 1, PK_MAT_GU = 2, PK_MAT_DOWN = 3, PK_MAT_HEAD = 4, PK_MAT_KINDS = 5 };
struct MatPlan {
  int c0, c1;                     // the block's atoms [c0, c1)
  int s_first, s_count;           // k-slabs the block's share touches
  int w0[PK_WARPS], w1[PK_WARPS]; // the warps' atoms
  int ws[PK_WARPS], wT[PK_WARPS], wa[PK_WARPS];   // slab, 16-row tile and atom in the tile where a warp's share starts
};

static_assert(PK_MAT_KINDS * sizeof(MatPlan) <= 1024, "matrix plans do not fit the small area");

struct PassShared {
  unsigned char *ring;      // [warp][slot][PK_CHUNK_BYTES]
  unsigned char *bstage;    // activation columns of up to two k-slabs; attention scratch (with xs)
  float *xs;                // staged activation rows
  uint64_t *bars;           // [warp][slot]
  volatile int *abort_flag;
  volatile unsigned *stage_uses;        // completed uses of stage_bar (its parity)
  uint64_t *stage_bar;      // completion of the bulk copies that stage a prologue's inputs
  float *red;               // [PK_WARPS][PK_MAX_ROWS]
  WarpPipe *pipes;          // [PK_WARPS] ring state of every warp between stages
  MatPlan *plans;           // [PK_MAT_KINDS]
  PassLayer *layers;        // layers [l_begin, l_end) of this pass
};

extern __shared__ __align__(1024) unsigned char pk_smem[];

// The block's shared memory map: constant offsets, so building it costs nothing.
__device__ __forceinline__ PassShared pass_shared() {
  PassShared S;
  S.ring = pk_smem + PK_OFF_RING;
  S.bstage = pk_smem + PK_OFF_BSTAGE;
  S.xs = reinterpret_cast<float *>(pk_smem + PK_OFF_XS);
  S.bars = reinterpret_cast<uint64_t *>(pk_smem + PK_OFF_BARS);
  S.abort_flag = reinterpret_cast<volatile int *>(pk_smem + PK_OFF_SMALL);
  S.stage_uses = reinterpret_cast<volatile unsigned *>(pk_smem + PK_OFF_SMALL + 4);
  S.stage_bar = reinterpret_cast<uint64_t *>(pk_smem + PK_OFF_SMALL + 8);
  S.red = reinterpret_cast<float *>(pk_smem + PK_OFF_SMALL + 64);
  S.pipes = reinterpret_cast<WarpPipe *>(pk_smem + PK_OFF_SMALL + 256);
  S.plans = reinterpret_cast<MatPlan *>(pk_smem + PK_OFF_SMALL + 1024);
  S.layers = reinterpret_cast<PassLayer *>(pk_smem + PK_OFF_LAYERS);
  return S;
}

}  // namespace dmtd
