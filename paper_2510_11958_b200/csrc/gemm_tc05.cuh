// Skinny GEMM on the 5th-generation tensor cores (tcgen05, sm_100a) for projections with many
// activation rows: out[m][n] += sum_k W[n][k] act[m][k] for 5..128 rows m.
//
// Operands are swapped against the usual orientation: the 128 weight rows of a tile are the M
// axis of the MMA, the activation rows its N axis (each row as two columns, the bf16 hi and lo
// parts of the fp32 activation, summed in the epilogue), so that every weight byte is read from
// HBM once whatever the batch is.  Both operands are K-major in shared memory in the interleaved
// (no swizzle) canonical form: 8 rows x 16 bytes per core matrix, core matrices of a 64-k block
// ordered [k chunk of 8][row group of 8].  The weights are stored in global memory in exactly
// that order (one 16 KiB block per (row tile, k block)), the activations are written that way by
// act_blocks_kernel, so a pipeline stage is two bulk copies.  Accumulators live in tensor memory
// (128 lanes x N columns of fp32), read back with tcgen05.ld for the epilogue.
//
// Warp roles: warp 0 issues the bulk copies, warp 1 owns the tensor memory and issues the MMAs,
// warps 2-5 run the epilogue (each reads the 32 lanes of its quarter).  Every wait is bounded and
// reports through an error word; tensor memory is freed on every path.
#pragma once

#include "pass_stream.cuh"

namespace dmtd {

constexpr int TG_THREADS = 192;
constexpr int TG_STAGES = 6;                 // most pipeline stages a block may be given
constexpr int TG_ROWS = 128;                 // weight rows per tile (MMA M)
constexpr int TG_KB = 64;                    // k per pipeline stage: four MMAs of K = 16
constexpr int TG_WBLOCK = TG_ROWS * TG_KB * 2;      // 16384 bytes
constexpr int TG_MAX_COLS = 256;             // MMA N: two columns per activation row
constexpr int TG_MAX_SWEEPS = 8;             // sweeps of 128 activation rows in one launch
enum { TG_ERR_WAIT = 4 };

// A weight matrix [N][K] as 16 KiB blocks [row tile][k block][k chunk 8][row group 16][row 8][8 values].
struct UmmaMat {
  const uint4 *w;
  int N, K;
  int n_tiles;       // ceil(N / 128)
  int n_kb;          // K / 64
};

struct GemmTcParams {
  UmmaMat W;
  const uint4 *act_blocks;   // [k block][N_cols * 128 bytes], see act_blocks_kernel
  int n_cols;                // MMA N: multiple of 16, >= 2 * rows
  int rows;                  // activation rows of this launch
  float *out;                // [rows][ldo], accumulated into
  int ldo;
  int ksplit;                // blocks per row tile, each taking a share of the k blocks
  int stages;                // pipeline stages of a block, 2 .. TG_STAGES
  int n_sweeps;              // sets of up to 128 activation rows in this launch (prefill chunks); set s has its
                             // activation blocks s * n_kb blocks further and its output rows 128 s further.
                             // Consecutive blocks of the grid are the sweeps of one (row tile, k share): they
                             // run together, and all but the first find the weight blocks in L2.
  int *error;
  long long wait_limit;
};

__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  // start address, leading (between the two k chunks of an MMA) and stride (between 8-row groups)
  // byte offsets, all without their 4 low bits; descriptor version 1; no swizzle
  return (uint64_t)((smem_addr & 0x3ffff) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46);
}

// kind::f16 instruction descriptor: fp32 accumulate, bf16 A and B, both K-major, M = 128, N = n_cols
__device__ __forceinline__ uint32_t umma_instr_desc(int n_cols) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n_cols >> 3) << 17) | ((uint32_t)(TG_ROWS >> 4) << 24);
}

__device__ __forceinline__ bool tg_wait(uint32_t bar, uint32_t parity, const GemmTcParams &P) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > P.wait_limit || *reinterpret_cast<volatile int *>(P.error) >= TG_ERR_WAIT) {
      atomicMax(P.error, TG_ERR_WAIT);
      return false;
    }
  }
  return true;
}

__global__ void __launch_bounds__(TG_THREADS, 1) gemm_tc05_kernel(const __grid_constant__ GemmTcParams P) {
  extern __shared__ __align__(1024) unsigned char tg_smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int act_block = P.n_cols * 128, stage_bytes = TG_WBLOCK + act_block;
  const int S = P.stages;
  uint64_t *bars = reinterpret_cast<uint64_t *>(tg_smem + S * stage_bytes);    // full[S], empty[S], done
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * S + 1);
  volatile int *gave_up = reinterpret_cast<volatile int *>(tmem_slot + 1);   // a wait of this block ran out: no epilogue
  const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + S), done = smem_u32(bars + 2 * S);

  const int sweep = blockIdx.x % P.n_sweeps, unit = blockIdx.x / P.n_sweeps;
  const int tile = unit / P.ksplit, ks = unit % P.ksplit;
  const int rows = min(TG_MAX_COLS / 2, P.rows - sweep * (TG_MAX_COLS / 2));        // rows of this sweep
  const uint4 *act_blocks = P.act_blocks + (size_t)sweep * P.W.n_kb * (P.n_cols * 8);
  float *out = P.out + (size_t)sweep * (TG_MAX_COLS / 2) * P.ldo;
  const int kb0 = P.W.n_kb * ks / P.ksplit, kb1 = P.W.n_kb * (ks + 1) / P.ksplit, n_it = kb1 - kb0;
  int tmem_cols = 32;
  while (tmem_cols < P.n_cols) tmem_cols <<= 1;

  // the kernel after this one (the next projection's activation-block kernel, launched the same way) may become
  // resident now; it waits for this grid's completion before it reads or writes anything, and the GEMM behind it
  // can then request its first weight blocks while this grid's last blocks finish
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x == 0) {
    for (int s = 0; s < 2 * S + 1; ++s) mbar_init(smem_u32(bars + s), 1);
    *gave_up = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *tmem_slot;

  if (warp == 0 && lane == 0) {
    // ---- producer: two bulk copies per k block.  The kernel is launched so that it may start
    // while the kernel before it (which writes the activation blocks) is still running: the
    // weight blocks of the first stages are requested at once, the activation blocks only after
    // that kernel has completed and its writes are visible.
    const int n_first = min(S, n_it);
    for (int i = 0; i < n_first; ++i) {
      mbar_expect_tx(full0 + i * 8, (uint32_t)stage_bytes);
      bulk_g2s(smem_u32(tg_smem + i * stage_bytes), P.W.w + ((size_t)tile * P.W.n_kb + kb0 + i) * (TG_WBLOCK / 16), TG_WBLOCK,
               full0 + i * 8);
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int i = 0; i < n_first; ++i)
      bulk_g2s(smem_u32(tg_smem + i * stage_bytes) + TG_WBLOCK, act_blocks + (size_t)(kb0 + i) * (act_block / 16),
               (uint32_t)act_block, full0 + i * 8);
    for (int i = n_first; i < n_it; ++i) {
      const int st = i % S;
      if (!tg_wait(empty0 + st * 8, ((i / S) - 1) & 1, P)) break;
      const uint32_t dst = smem_u32(tg_smem + st * stage_bytes);
      mbar_expect_tx(full0 + st * 8, (uint32_t)stage_bytes);
      bulk_g2s(dst, P.W.w + ((size_t)tile * P.W.n_kb + kb0 + i) * (TG_WBLOCK / 16), TG_WBLOCK, full0 + st * 8);
      bulk_g2s(dst + TG_WBLOCK, act_blocks + (size_t)(kb0 + i) * (act_block / 16), (uint32_t)act_block, full0 + st * 8);
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer: four K = 16 MMAs per k block, then release the stage
    const uint32_t idesc = umma_instr_desc(P.n_cols);
    const uint32_t b_lbo = (uint32_t)(P.n_cols / 8) * 128;
    bool ok = true;
    for (int i = 0; i < n_it && ok; ++i) {
      const int st = i % S;
      ok = tg_wait(full0 + st * 8, (i / S) & 1, P);
      if (!ok) { *gave_up = 1; __threadfence_block(); break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t a_base = smem_u32(tg_smem + st * stage_bytes), b_base = a_base + TG_WBLOCK;
#pragma unroll
      for (int kk = 0; kk < TG_KB / 16; ++kk) {
        const uint64_t da = umma_smem_desc(a_base + kk * 2 * (TG_ROWS / 8) * 128, (TG_ROWS / 8) * 128, 128);
        const uint64_t db = umma_smem_desc(b_base + kk * 2 * b_lbo, b_lbo, 128);
        const uint32_t accumulate = (i > 0 || kk > 0) ? 1u : 0u;
        asm volatile(
            "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
            " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n}\n" ::"r"(tmem),
            "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u)
            : "memory");
      }
      // arrives on the stage's empty barrier once the MMAs issued so far have read shared memory
      asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(empty0 + st * 8) : "memory");
    }
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(done) : "memory");
  } else if (warp >= 2) {
    // ---- epilogue: thread = weight row (lane of tensor memory), registers = columns
    const int quarter = warp & 3;
    const int n = tile * TG_ROWS + quarter * 32 + lane;
    // the accumulators are complete only if no wait of this block ran out
    if (tg_wait(done, 0, P) && !*gave_up) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      for (int c0 = 0; c0 < P.n_cols && c0 < 2 * rows; c0 += 16) {
        uint32_t r[16];
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
            : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
              "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
            : "r"(tmem + ((uint32_t)(quarter * 32) << 16) + c0));
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int m = (c0 >> 1) + j;                  // columns 2m (hi) and 2m + 1 (lo) belong to activation row m
          if (m < rows && n < P.W.N) atomicAdd(out + (size_t)m * P.ldo + n, __uint_as_float(r[2 * j]) + __uint_as_float(r[2 * j + 1]));
        }
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
  }
}

// Activations [rows][lda] fp32 -> bf16 hi/lo columns in the canonical K-major block order:
// block kb holds k = 64 kb .. 64 kb + 63 as [k chunk 8][column group n_cols/8][column 8][8 values];
// column 2m is the hi part of row m, column 2m + 1 its lo part; columns beyond 2 * rows are zero.
// blockIdx.y = set of up to 128 rows (a sweep of the GEMM): its rows start 128 y further, its
// blocks n_kb blocks further.
// With gate_up_I > 0 the source rows hold gate | up values (gate at k, up at gate_up_I + k) and the
// activation is the SwiGLU gate silu(gate) * up (step a6, second half), computed on the way.
__global__ void act_blocks_kernel(const float *__restrict__ act_all, int lda, int rows_all, int K, int n_cols,
                                  uint4 *__restrict__ blocks_all, int gate_up_I) {
  const int rows = min(TG_MAX_COLS / 2, rows_all - (int)blockIdx.y * (TG_MAX_COLS / 2));
  const float *act = act_all + (size_t)blockIdx.y * (TG_MAX_COLS / 2) * lda;
  uint4 *blocks = blocks_all + (size_t)blockIdx.y * (K / TG_KB) * (n_cols * 8);
  // the GEMM that follows may be scheduled already: it waits for this grid before it reads the blocks
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // ... and this grid may itself have started before the kernel before it has finished (the GEMM of the previous
  // projection lets its dependents in at once): nothing is read or written before that kernel is complete
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int n_kb = K / TG_KB;
  const long long total = (long long)n_kb * 8 * n_cols;            // 16-byte units
  for (long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x; u < total; u += (long long)gridDim.x * blockDim.x) {
    const int col = (int)(u % n_cols), c = (int)((u / n_cols) % 8), kb = (int)(u / n_cols / 8);
    const int m = col >> 1, k = kb * TG_KB + c * 8;
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    if (m < rows) {
      const float4 a = *reinterpret_cast<const float4 *>(act + (size_t)m * lda + k);
      const float4 b = *reinterpret_cast<const float4 *>(act + (size_t)m * lda + k + 4);
      float f[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
      if (gate_up_I > 0) {
        const float4 ua = *reinterpret_cast<const float4 *>(act + (size_t)m * lda + gate_up_I + k);
        const float4 ub = *reinterpret_cast<const float4 *>(act + (size_t)m * lda + gate_up_I + k + 4);
        const float u[8] = {ua.x, ua.y, ua.z, ua.w, ub.x, ub.y, ub.z, ub.w};
#pragma unroll
        for (int j = 0; j < 8; ++j) f[j] = f[j] / (1.f + expf(-f[j])) * u[j];
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t h = pack_bf16x2(f[2 * j], f[2 * j + 1]);
        w[j] = (col & 1) ? pack_bf16x2(f[2 * j] - __uint_as_float(h << 16), f[2 * j + 1] - __uint_as_float(h & 0xffff0000u)) : h;
      }
    }
    // column group = col / 8, column in group = col % 8
    blocks[((size_t)kb * 8 + c) * n_cols + col] = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// RMSNorm and the activation blocks in one kernel (steps a2 / a6 / a9, first half, on the tcgen05
// path): block g < n_groups takes 4 rows (a sweep of the GEMM is n_cols / 2 rows, padded with zero
// rows), sums their squares, and writes their hi and lo columns of every k block; the blocks
// behind them clear the buffer the GEMM accumulates into.  x [rows][ldx] fp32; K values per row.
constexpr int NAB_ROWS = 4;
__global__ void __launch_bounds__(256) norm_act_blocks_kernel(const float *__restrict__ x, int ldx, const float *__restrict__ w,
                                                              float eps, int rows_all, int K, int n_cols,
                                                              uint4 *__restrict__ blocks_all, int n_groups,
                                                              float4 *__restrict__ zero, size_t zero_n4) {
  // the GEMM that follows may be scheduled already: it waits for this grid before it reads the blocks
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // ... and this grid may itself have started before the kernel before it has finished (the GEMM of the previous
  // projection lets its dependents in at once): nothing is read or written before that kernel is complete
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if ((int)blockIdx.x >= n_groups) {
    const size_t n_z = (size_t)(gridDim.x - n_groups) * gridDim.y;
    for (size_t i = ((size_t)(blockIdx.x - n_groups) * gridDim.y + blockIdx.y) * blockDim.x + threadIdx.x; i < zero_n4;
         i += n_z * blockDim.x)
      zero[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    return;
  }
  const int sweep_rows = n_cols / 2, groups_per_sweep = sweep_rows / NAB_ROWS;
  const int sweep = blockIdx.x / groups_per_sweep, m_in0 = (blockIdx.x % groups_per_sweep) * NAB_ROWS;
  const int m0 = sweep * (TG_MAX_COLS / 2) + m_in0;                 // first row of the group (sweeps are 128 rows apart)
  const int n_kb = K / TG_KB;
  uint4 *blocks = blocks_all + (size_t)sweep * n_kb * (n_cols * 8);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __shared__ float part[8], inv[NAB_ROWS];
  {
    // two warps per row
    const int r = warp >> 1, m = m0 + r;
    float ss = 0.f;
    if (m < rows_all) {
      const float4 *xr = reinterpret_cast<const float4 *>(x + (size_t)m * ldx);
      for (int k4 = (warp & 1) * 32 + lane; k4 < K / 4; k4 += 64) {
        const float4 v = xr[k4];
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
      }
    }
    ss = warp_sum(ss);
    if (lane == 0) part[warp] = ss;
  }
  __syncthreads();
  if (threadIdx.x < NAB_ROWS) inv[threadIdx.x] = rsqrtf((part[2 * threadIdx.x] + part[2 * threadIdx.x + 1]) / (float)K + eps);
  __syncthreads();
  // unit = (k block, k chunk of 8, row of the group): this thread writes the row's hi and lo columns;
  // blockIdx.y takes a share of the k blocks (every share needs the whole row's sum of squares)
  const int kb_lo = n_kb * blockIdx.y / gridDim.y, kb_hi = n_kb * (blockIdx.y + 1) / gridDim.y;
  const int total = (kb_hi - kb_lo) * 8 * NAB_ROWS;
  for (int u = threadIdx.x; u < total; u += blockDim.x) {
    const int r = u % NAB_ROWS, c = (u / NAB_ROWS) % 8, kb = kb_lo + u / (NAB_ROWS * 8);
    const int m = m0 + r, k = kb * TG_KB + c * 8;
    uint32_t hi[4] = {0u, 0u, 0u, 0u}, lo[4] = {0u, 0u, 0u, 0u};
    if (m < rows_all) {
      const float4 a = *reinterpret_cast<const float4 *>(x + (size_t)m * ldx + k);
      const float4 b = *reinterpret_cast<const float4 *>(x + (size_t)m * ldx + k + 4);
      const float4 wa = __ldg(reinterpret_cast<const float4 *>(w + k)), wb = __ldg(reinterpret_cast<const float4 *>(w + k + 4));
      const float s = inv[r];
      const float f[8] = {a.x * s * wa.x, a.y * s * wa.y, a.z * s * wa.z, a.w * s * wa.w,
                          b.x * s * wb.x, b.y * s * wb.y, b.z * s * wb.z, b.w * s * wb.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        hi[j] = pack_bf16x2(f[2 * j], f[2 * j + 1]);
        lo[j] = pack_bf16x2(f[2 * j] - __uint_as_float(hi[j] << 16), f[2 * j + 1] - __uint_as_float(hi[j] & 0xffff0000u));
      }
    }
    uint4 *dst = blocks + ((size_t)kb * 8 + c) * n_cols + 2 * (m_in0 + r);
    dst[0] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    dst[1] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
  }
}

// The merge of the attention's key slices (step a4, second half) and the activation blocks of the O
// projection in one kernel: block g takes 4 rows, works out the weight of every (row, head, slice)
// from the slices' running max and sum, and writes the merged head outputs as hi and lo columns.
// part_o [(row * nq + head) * nsplit + slice][D], part_ml the same with (max, sum); K = nq * D.
constexpr int MAB_MAX_SLOTS = 2048;            // (rows of a group) x heads x slices the weights of a group may take
__global__ void __launch_bounds__(256) merge_act_blocks_kernel(const float *__restrict__ part_o, const float *__restrict__ part_ml,
                                                               int nsplit, int nq, int D, int rows_all, int n_cols,
                                                               uint4 *__restrict__ blocks_all) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // ... and this grid may itself have started before the kernel before it has finished (the GEMM of the previous
  // projection lets its dependents in at once): nothing is read or written before that kernel is complete
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int K = nq * D, n_kb = K / TG_KB;
  const int sweep_rows = n_cols / 2, groups_per_sweep = sweep_rows / NAB_ROWS;
  const int sweep = blockIdx.x / groups_per_sweep, m_in0 = (blockIdx.x % groups_per_sweep) * NAB_ROWS;
  const int m0 = sweep * (TG_MAX_COLS / 2) + m_in0;
  uint4 *blocks = blocks_all + (size_t)sweep * n_kb * (n_cols * 8);
  __shared__ float wgt[MAB_MAX_SLOTS];
  // weights: one thread per (row, head)
  for (int i = threadIdx.x; i < NAB_ROWS * nq; i += blockDim.x) {
    const int r = i / nq, h = i % nq, m = m0 + r;
    float *wr = wgt + (size_t)i * nsplit;
    if (m >= rows_all) { for (int s = 0; s < nsplit; ++s) wr[s] = 0.f; continue; }
    const float *ml = part_ml + ((size_t)m * nq + h) * nsplit * 2;
    float mx = -INFINITY;
    for (int s = 0; s < nsplit; ++s)
      if (ml[2 * s + 1] > 0.f) mx = fmaxf(mx, ml[2 * s]);
    float l = 0.f;
    for (int s = 0; s < nsplit; ++s) {
      const float ls = ml[2 * s + 1];
      const float f = ls > 0.f ? __expf(ml[2 * s] - mx) : 0.f;
      wr[s] = f;
      l += ls * f;
    }
    const float inv = 1.f / l;
    for (int s = 0; s < nsplit; ++s) wr[s] *= inv;
  }
  __syncthreads();
  const int kb_lo = n_kb * blockIdx.y / gridDim.y, kb_hi = n_kb * (blockIdx.y + 1) / gridDim.y;   // this block's share of the k blocks
  const int total = (kb_hi - kb_lo) * 8 * NAB_ROWS;
  for (int u = threadIdx.x; u < total; u += blockDim.x) {
    const int r = u % NAB_ROWS, c = (u / NAB_ROWS) % 8, kb = kb_lo + u / (NAB_ROWS * 8);
    const int m = m0 + r, k = kb * TG_KB + c * 8, h = k / D, d0 = k - h * D;
    uint32_t hi[4] = {0u, 0u, 0u, 0u}, lo[4] = {0u, 0u, 0u, 0u};
    if (m < rows_all) {
      float f[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      const float *wr = wgt + (size_t)(r * nq + h) * nsplit;
      const float *po = part_o + ((size_t)m * nq + h) * nsplit * D + d0;
      for (int s = 0; s < nsplit; ++s) {
        const float ws = wr[s];
        if (ws != 0.f) {                                   // empty slices hold nothing that may be read
          const float4 a = *reinterpret_cast<const float4 *>(po + (size_t)s * D);
          const float4 b = *reinterpret_cast<const float4 *>(po + (size_t)s * D + 4);
          f[0] += ws * a.x; f[1] += ws * a.y; f[2] += ws * a.z; f[3] += ws * a.w;
          f[4] += ws * b.x; f[5] += ws * b.y; f[6] += ws * b.z; f[7] += ws * b.w;
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        hi[j] = pack_bf16x2(f[2 * j], f[2 * j + 1]);
        lo[j] = pack_bf16x2(f[2 * j] - __uint_as_float(hi[j] << 16), f[2 * j + 1] - __uint_as_float(hi[j] & 0xffff0000u));
      }
    }
    uint4 *dst = blocks + ((size_t)kb * 8 + c) * n_cols + 2 * (m_in0 + r);
    dst[0] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    dst[1] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
  }
}

// Weights [N][K] bf16 row-major (rows [row0, row0 + N_src) of the fused matrix) -> 16 KiB blocks.
__global__ void pack_umma_kernel(const __nv_bfloat16 *__restrict__ src, int N_src, int K, int row0, int n_kb,
                                 uint4 *__restrict__ dst) {
  const long long total = (long long)N_src * (K / 8);              // 16-byte units of the source
  for (long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x; u < total; u += (long long)gridDim.x * blockDim.x) {
    const int kc = (int)(u % (K / 8)), row = row0 + (int)(u / (K / 8));
    const int tile = row / TG_ROWS, rg = (row % TG_ROWS) / 8, j = row % 8, kb = kc / 8, c = kc % 8;
    dst[(((size_t)tile * n_kb + kb) * 8 + c) * TG_ROWS + rg * 8 + j] =
        *reinterpret_cast<const uint4 *>(src + (size_t)(row - row0) * K + kc * 8);
  }
}

}  // namespace dmtd
