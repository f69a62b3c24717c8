// Shared device-side definitions of the DMTD decode library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace dmtd {

// Device-resident schedule counters (Section 2.2 of the paper); kernels read their row
// positions from here so that a captured CUDA graph stays valid as the context grows.
struct DevState {
  int n_known;    // tokens whose id is known
  int lo_len;     // positions with KV in the lower layers; first row of a full pass's refill
  int up_len;     // positions with KV in the decoding layers
  int cycle;
  int slot;
  int n_emitted;
  int newest;     // n_known - 1: position fed to the decoding layers
  int scratch;    // row origin for prefill chunks and dmtd_step_layers
  int error;      // sticky: 1 = token id out of range
  int tau;
  int pad[6];
};

// A weight matrix [N][K] as the kernels read it.
//  bf16: a stream of 1 KiB "atoms".  An atom holds 16 rows x 32 k in the register order of
//        the A operand of mma.m16n8k16: two halves (rows g and g+8) of 32 lanes x 16 bytes,
//        lane (g = lane/4, t = lane%4) owning k = 8t..8t+7 of the atom.  Atoms are ordered
//        [k-slab][row tile][atom in slab]; a slab is `aps` atoms (KS = 32*aps values of k).
//  fp32: plain row-major [N][K].
struct PackedMat {
  const uint4 *w;     // bf16 atom stream
  const float *wf;    // fp32 row-major
  int N, K;
  int n_tiles;        // ceil(N / 16)
  int aps;            // atoms per slab
  int n_slabs;        // K / (32 * aps)
};

__host__ __device__ inline long long packed_atoms(const PackedMat &m) {
  return (long long)m.n_slabs * m.n_tiles * m.aps;
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t bits16) {
  return __uint_as_float(bits16 << 16);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Split an fp32 value into two bf16 terms hi + lo (|error| <= 2^-17 |x|): tensor-core
// operands must be bf16, and a single rounding of the activations would exceed the logit
// tolerance after 36 layers.
__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16 &hi, __nv_bfloat16 &lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// D += A * B, m16n8k16, bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Sampling beside the greedy rule: the token is argmax_i (z_i / T + g_i) with standard Gumbel
// noise g_i = -log(-log(u_i)), a draw from softmax(z / T) that keeps the vocabulary-parallel
// two-level pick of the greedy path.  u_i comes from Philox4x32-10 (Salmon et al., SC'11), a
// counter-based generator: counter (i / 4, position, sequence, 0), key = seed, word i mod 4, its
// top 24 bits + 1/2 over 2^24.  on == 0: greedy.
struct SampleParams {
  float inv_temperature;
  unsigned key0, key1;
  int on;
};

__device__ __forceinline__ uint4 philox4x32_10(uint4 c, unsigned k0, unsigned k1) {
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const unsigned hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const unsigned hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return c;
}

// The value the pick compares for vocabulary entry i: the logit itself, or logit / T + noise.
__device__ __forceinline__ float pick_value(float z, int i, int position, int sequence, const SampleParams &sp) {
  if (!sp.on) return z;
  const uint4 r = philox4x32_10(make_uint4((unsigned)i >> 2, (unsigned)position, (unsigned)sequence, 0u), sp.key0, sp.key1);
  const unsigned w = (i & 3) == 0 ? r.x : (i & 3) == 1 ? r.y : (i & 3) == 2 ? r.z : r.w;
  const float u = ((float)(w >> 8) + 0.5f) * (1.0f / 16777216.0f);
  return z * sp.inv_temperature - logf(-logf(u));
}

// The same with fp16 inputs (an fp16 KV cache: 11 significant bits against bf16's 8).
__device__ __forceinline__ void mma_f16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                              uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// 16-bit operand types of the tensor-core attention kernel.
struct OpBf16 {
  using T = __nv_bfloat16;
  static __device__ __forceinline__ T from_float(float v) { return __float2bfloat16_rn(v); }
  static __device__ __forceinline__ float to_float(T v) { return __bfloat162float(v); }
  static __device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
  }
  static __device__ __forceinline__ void mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1) { mma_bf16_16816(d, a0, a1, a2, a3, b0, b1); }
};
struct OpF16 {
  using T = __half;
  static __device__ __forceinline__ T from_float(float v) { return __float2half_rn(v); }
  static __device__ __forceinline__ float to_float(T v) { return __half2float(v); }
  static __device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
  }
  static __device__ __forceinline__ void mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1) { mma_f16_16816(d, a0, a1, a2, a3, b0, b1); }
};

__device__ __forceinline__ uint4 ldg_stream(const uint4 *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

}  // namespace dmtd
