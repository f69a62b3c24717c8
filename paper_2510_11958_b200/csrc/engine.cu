// Host side of the DMTD decode library: context, weight repacking, the cycle scheduler of
// Section 2.2 of the paper, and the C ABI declared in include/dmtd.h.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <numeric>
#include <string>
#include <type_traits>
#include <vector>

#include "../../include/dmtd.h"
#include "kernels.cuh"
#include "pass_kernel.cuh"
#include "attention_kernel.cuh"
#include "gemm_tc05.cuh"

using namespace dmtd;

namespace {

thread_local std::string g_create_error;

// Clock ticks a device-side wait (grid barrier, bulk-copy or tensor-core barrier) may spin before
// it gives up and reports through the context's error word: about a second of SM clock.
constexpr long long kDeviceWaitLimitTicks = 2000000000ll;

struct LayerDev {
  PackedMat qkv, o, gu, down;
  UmmaMat qkv_u{}, o_u{}, gu_u{}, down_u{};     // second copy for the tcgen05 GEMM (contexts with many rows)
  float *w_in, *w_post, *w_qn, *w_kn;
};

}  // namespace

struct dmtd_ctx {
  dmtd_model_shape s{};
  int L_d = 0, tau = 0, max_batch = 0, max_seq = 0;
  int L_e = 0;                              // encoding layers the short passes reuse as well (ExDy); 0 = none
  int device = 0, n_sms = 0;
  cudaStream_t stream = nullptr;
  cudaStream_t capture_stream = nullptr;    // graphs are recorded here (the caller's stream may be the legacy one)
  std::string err;
  std::vector<void *> allocs;
  size_t mem[4] = {0, 0, 0, 0};             // device bytes held: atom-stream weights, tcgen05 block weights, KV cache, the rest
  int mem_kind = 3;                         // category the next allocations count towards

  // model
  std::vector<LayerDev> layers;
  PackedMat embed{};
  UmmaMat embed_u{};
  bool umma_ok = false, use_umma = true;    // tcgen05 GEMM for projections of more than 4 rows
  int gemm_stages = 0;                      // pipeline stages of its blocks; 0: chosen per launch
  uint4 *act_blocks = nullptr;
  float *w_final = nullptr;
  double *inv_freq = nullptr;

  // sequence state
  void *kc = nullptr, *vc = nullptr;        // [L][max_batch][nkv][max_seq][D]
  size_t kv_layer_elems = 0;
  int *tokens = nullptr;                    // [max_batch][max_seq]
  DevState *dstate = nullptr;
  int *h_error = nullptr;                   // pinned host copy of the device error word, refreshed by calls that synchronise
  dmtd_status device_failure = DMTD_OK;     // sticky until dmtd_reset: a device-side check or wait reported an error
  dmtd_state h{};                           // host mirror
  bool prefilled = false;
  int B = 0;

  // workspace
  int ws_rows = 0, lda = 0, ldqkv = 0, ldgu = 0, ldl = 0, CH = 0, nsplit_max = 0;
  float *x_lo = nullptr, *x_up = nullptr, *act = nullptr, *qkv = nullptr, *gu = nullptr,
        *logits = nullptr, *part_o = nullptr, *part_ml = nullptr;
  float2 *rope_tab = nullptr;
  float *h_pend = nullptr;                  // [max_batch][pend_cap][hidden]: h_enc of positions the thinking layers have not seen
  float *h_base = nullptr;                  // [ws_rows][hidden]: h_emb / h_enc of a chunk of rows (literal sum, masked forward)
  int pend_cap = 0;

  // options
  bool use_graph = true, literal_sum = false, use_fused = true, use_tc_attention = true;
  bool fuse_qk_rope = true;                 // QK-norm, RoPE and the KV append inside the tensor-core attention kernel
  float temperature = 0.f;                  // > 0: tokens are drawn from softmax(logits / temperature); 0: greedy
  uint64_t sample_seed = 0;

  // fused pass kernel: one persistent launch per pass
  bool fused_ok = false;
  PassLayer *pass_layers = nullptr;         // device [n_layers]
  float *f_part_o = nullptr, *f_part_ml = nullptr, *amax_val = nullptr;
  int *amax_idx = nullptr;
  unsigned int *grid_bar = nullptr;
  float *pick_val = nullptr;                // per-step greedy pick: best of every vocabulary slice, [max_batch][ARGMAX_SLICES]
  int *pick_idx = nullptr;
  long long *pass_timing = nullptr;         // profiling builds only

  // graphs: [kind 1 = full, 2 = upper-only]
  cudaGraphExec_t graph_exec[3] = {nullptr, nullptr, nullptr};
  int graph_nodes[3] = {0, 0, 0};
  int graph_B = 0, graph_tau = 0;
  bool capturing = false;

  int64_t launches = 0;
};

namespace {

dmtd_status fail(dmtd_ctx *c, dmtd_status st, const char *fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (c) c->err = buf; else g_create_error = buf;
  return st;
}

#define CUDA_TRY(c, expr)                                                                   \
  do {                                                                                      \
    cudaError_t e_ = (expr);                                                                \
    if (e_ != cudaSuccess)                                                                  \
      return fail((c), DMTD_ERR_CUDA, "%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e_), \
                  __FILE__, __LINE__);                                                      \
  } while (0)

template <typename T>
dmtd_status dev_alloc(dmtd_ctx *c, T **p, size_t n) {
  void *q = nullptr;
  CUDA_TRY(c, cudaMalloc(&q, std::max<size_t>(n, 1) * sizeof(T)));
  c->allocs.push_back(q);
  c->mem[c->mem_kind] += std::max<size_t>(n, 1) * sizeof(T);
  *p = static_cast<T *>(q);
  return DMTD_OK;
}

dmtd_status check_launch(dmtd_ctx *c, const char *what) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(c, DMTD_ERR_CUDA, "launch of %s failed: %s", what, cudaGetErrorString(e));
  c->launches += 1;
  return DMTD_OK;
}
#define LAUNCH_OK(c, what)                          \
  do {                                              \
    dmtd_status s_ = check_launch((c), (what));     \
    if (s_ != DMTD_OK) return s_;                   \
  } while (0)
#define TRY(expr)                                   \
  do {                                              \
    dmtd_status s_ = (expr);                        \
    if (s_ != DMTD_OK) return s_;                   \
  } while (0)

bool is_bf16(const dmtd_ctx *c) { return c->s.weight_dtype == DMTD_BF16; }
size_t wbytes(const dmtd_ctx *c) { return is_bf16(c) ? 2 : 4; }

// Largest divisor of the atom count per row that keeps a k-slab at or below `cap` atoms.
int choose_aps(int K, int cap) {
  int atoms = K / 32, best = 1;
  for (int d = 1; d <= std::min(atoms, cap); ++d)
    if (atoms % d == 0) best = d;
  return best;
}

// Build one packed matrix from up to three row blocks (e.g. q, k, v) of equal K.
dmtd_status pack_matrix(dmtd_ctx *c, PackedMat *out, int K, const void *const *srcs, const int *Ns, int n_src,
                        int aps_cap) {
  int N = 0;
  for (int i = 0; i < n_src; ++i) N += Ns[i];
  PackedMat m{};
  m.N = N; m.K = K; m.n_tiles = (N + 15) / 16;
  if (is_bf16(c)) {
    m.aps = choose_aps(K, aps_cap);
    m.n_slabs = K / 32 / m.aps;
    uint4 *dst = nullptr;
    c->mem_kind = 0;
    TRY(dev_alloc(c, &dst, (size_t)packed_atoms(m) * 64));
    c->mem_kind = 3;
    int tile0 = 0;
    for (int i = 0; i < n_src; ++i) {
      if (tile0 * 16 != (int)std::accumulate(Ns, Ns + i, 0))
        return fail(c, DMTD_ERR_SHAPE, "row blocks of a fused matrix must be multiples of 16 rows");
      long long chunks = (long long)m.n_slabs * ((Ns[i] + 15) / 16) * m.aps * 64;
      int grid = (int)std::min<long long>((chunks + 255) / 256, 65535);
      pack_bf16_kernel<<<grid, 256, 0, c->stream>>>(static_cast<const __nv_bfloat16 *>(srcs[i]), Ns[i], K, dst,
                                                    tile0, m.n_tiles, m.aps, m.n_slabs);
      LAUNCH_OK(c, "pack_bf16_kernel");
      tile0 += (Ns[i] + 15) / 16;
    }
    m.w = dst;
  } else {
    float *dst = nullptr;
    c->mem_kind = 0;
    TRY(dev_alloc(c, &dst, (size_t)N * K));
    c->mem_kind = 3;
    size_t off = 0;
    for (int i = 0; i < n_src; ++i) {
      CUDA_TRY(c, cudaMemcpyAsync(dst + off, srcs[i], (size_t)Ns[i] * K * 4, cudaMemcpyDeviceToDevice, c->stream));
      off += (size_t)Ns[i] * K;
    }
    m.wf = dst;
  }
  *out = m;
  return DMTD_OK;
}

dmtd_status vec_to_float(dmtd_ctx *c, float **out, const void *src, int n) {
  TRY(dev_alloc(c, out, (size_t)n));
  if (is_bf16(c))
    to_float_kernel<__nv_bfloat16><<<(n + 255) / 256, 256, 0, c->stream>>>(static_cast<const __nv_bfloat16 *>(src), *out, n);
  else
    to_float_kernel<float><<<(n + 255) / 256, 256, 0, c->stream>>>(static_cast<const float *>(src), *out, n);
  LAUNCH_OK(c, "to_float_kernel");
  return DMTD_OK;
}

// Second copy of a (fused) matrix in the block order of the tcgen05 GEMM.
dmtd_status pack_umma(dmtd_ctx *c, UmmaMat *out, int K, const void *const *srcs, const int *Ns, int n_src) {
  int N = 0;
  for (int i = 0; i < n_src; ++i) N += Ns[i];
  UmmaMat m{};
  m.N = N; m.K = K; m.n_tiles = (N + TG_ROWS - 1) / TG_ROWS; m.n_kb = K / TG_KB;
  uint4 *dst = nullptr;
  size_t units = (size_t)m.n_tiles * m.n_kb * (TG_WBLOCK / 16);
  c->mem_kind = 1;
  TRY(dev_alloc(c, &dst, units));
  c->mem_kind = 3;
  CUDA_TRY(c, cudaMemsetAsync(dst, 0, units * 16, c->stream));
  int row0 = 0;
  for (int i = 0; i < n_src; ++i) {
    long long total = (long long)Ns[i] * (K / 8);
    int grid = (int)std::min<long long>((total + 255) / 256, 65535);
    pack_umma_kernel<<<grid, 256, 0, c->stream>>>(static_cast<const __nv_bfloat16 *>(srcs[i]), Ns[i], K, row0, m.n_kb, dst);
    LAUNCH_OK(c, "pack_umma_kernel");
    row0 += Ns[i];
  }
  m.w = dst;
  *out = m;
  return DMTD_OK;
}

// ---------------------------------------------------------------------------- launches

int gemv_smem_bytes(const PackedMat &W, int NT) {
  int KS = W.aps * 32;
  int row_bytes = ((KS * 2) % 128 == 64) ? KS * 2 : KS * 2 + 64;
  return 8 * NT * row_bytes;
}

template <int NT>
dmtd_status launch_gemv_nt(dmtd_ctx *c, const PackedMat &W, const float *act, int lda, int M, float *out, int ldo) {
  int smem = gemv_smem_bytes(W, NT);
  gemv_bf16_kernel<NT><<<2 * c->n_sms, GEMV_THREADS, smem, c->stream>>>(W, act, lda, M, out, ldo);
  LAUNCH_OK(c, "gemv_bf16_kernel");
  return DMTD_OK;
}

// out[m][n] += sum_k W[n][k] act[m][k] on the tcgen05 tensor cores.  A block multiplies a 128-row
// weight tile with up to 128 activation rows (a sweep); prefill chunks of more rows are several
// sweeps in one launch (up to TG_MAX_SWEEPS), ordered so that the sweeps of one weight tile run
// together and share it through L2.
// Launch with programmatic stream serialisation: the kernel's blocks may become resident while the
// kernel before it in the stream is still running; it calls griddepcontrol.wait before it touches
// anything that kernel (or one before it) writes.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// With `norm_w` the activations are RMSNorm(act rows) * norm_w, computed while the blocks are written, and
// the output rows are cleared first (the projections after a norm write a fresh buffer).
dmtd_status launch_gemm_tc05(dmtd_ctx *c, const UmmaMat &W, const float *act, int lda, int M, float *out, int ldo,
                             int gate_up_I = 0, const float *norm_w = nullptr, int merge_nsplit = 0) {
  const int SET = TG_MAX_COLS / 2;                       // rows per sweep
  for (int m0 = 0; m0 < M; m0 += TG_MAX_SWEEPS * SET) {
    GemmTcParams P{};
    P.W = W; P.act_blocks = c->act_blocks;
    P.rows = std::min(TG_MAX_SWEEPS * SET, M - m0);
    P.n_sweeps = (P.rows + SET - 1) / SET;
    P.n_cols = P.n_sweeps > 1 ? TG_MAX_COLS : (2 * P.rows + 15) / 16 * 16;
    P.out = out + (size_t)m0 * ldo; P.ldo = ldo;
    P.error = &c->dstate->error; P.wait_limit = kDeviceWaitLimitTicks;
    // Every block of a launch should be resident at once (a block streams at the rate its own
    // stages allow, so a second round of blocks doubles the time): blocks per SM follow from
    // shared memory and tensor memory; with more row tiles than that, two-stage blocks make room
    // for two per SM.  Row tiles are then split along k over as many blocks as still fit.
    // (Several sweeps fill the SMs by themselves: no k split then.)
    int tmem_cols = 32;
    while (tmem_cols < P.n_cols) tmem_cols <<= 1;
    auto smem_of = [&](int st) { return st * (TG_WBLOCK + P.n_cols * 128) + 128; };
    auto per_sm_of = [&](int st) { return std::max(1, std::min((227 * 1024) / (smem_of(st) + 1024), 512 / tmem_cols)); };
    // stages: what keeps the most weight blocks in flight per SM (stages x resident blocks: a block streams at the
    // rate its bytes in flight allow), more resident blocks on a tie (their fill and epilogue overlap)
    const int max_stages = std::min(TG_STAGES, (227 * 1024 - 1024 - 128) / (TG_WBLOCK + P.n_cols * 128));
    P.stages = 2;
    for (int st = 2; st <= max_stages; ++st)
      if (st * per_sm_of(st) > P.stages * per_sm_of(P.stages)) P.stages = st;
    if (c->gemm_stages >= 2) P.stages = std::min(c->gemm_stages, max_stages);
    if (P.n_sweeps == 1 && W.n_tiles > c->n_sms * per_sm_of(P.stages) && W.n_tiles <= c->n_sms * per_sm_of(2)) P.stages = 2;
    const int slots = c->n_sms * per_sm_of(P.stages);
    P.ksplit = std::max(1, std::min(W.n_kb, slots / (W.n_tiles * P.n_sweeps)));
    if (merge_nsplit > 0) {
      // `act` is unused: the activations are the attention's key slices, merged on the way
      const int n_groups = P.n_sweeps * (P.n_cols / 2 / NAB_ROWS);
      const int ky = std::max(1, std::min(W.n_kb, 4 * c->n_sms / std::max(1, n_groups)));
      CUDA_TRY(c, launch_pdl(merge_act_blocks_kernel, dim3(n_groups, ky), dim3(256), 0, c->stream,
                             c->part_o + (size_t)m0 * c->s.n_q_heads * merge_nsplit * c->s.head_dim,
                             c->part_ml + (size_t)m0 * c->s.n_q_heads * merge_nsplit * 2, merge_nsplit, c->s.n_q_heads,
                             c->s.head_dim, P.rows, P.n_cols, c->act_blocks));
      LAUNCH_OK(c, "merge_act_blocks_kernel");
    } else if (norm_w) {
      const int n_groups = P.n_sweeps * (P.n_cols / 2 / NAB_ROWS);
      const size_t zero_n4 = (size_t)P.rows * ldo / 4;                  // ldo is a multiple of 4 (checked by the caller)
      const int n_zero = (int)std::min<size_t>((zero_n4 + 1023) / 1024, 2 * c->n_sms);
      const int ky = std::max(1, std::min(W.n_kb, 4 * c->n_sms / std::max(1, n_groups)));
      CUDA_TRY(c, launch_pdl(norm_act_blocks_kernel, dim3(n_groups + (n_zero + ky - 1) / ky, ky), dim3(256), 0, c->stream,
                             act + (size_t)m0 * lda, lda, norm_w, c->s.rms_eps, P.rows, W.K, P.n_cols, c->act_blocks, n_groups,
                             reinterpret_cast<float4 *>(out + (size_t)m0 * ldo), zero_n4));
      LAUNCH_OK(c, "norm_act_blocks_kernel");
    } else {
      long long units = (long long)W.n_kb * 8 * P.n_cols;
      CUDA_TRY(c, launch_pdl(act_blocks_kernel, dim3((int)std::min<long long>((units + 255) / 256, 4096), P.n_sweeps), dim3(256), 0,
                             c->stream, act + (size_t)m0 * lda, lda, P.rows, W.K, P.n_cols, c->act_blocks, gate_up_I));
      LAUNCH_OK(c, "act_blocks_kernel");
    }
    int smem = smem_of(P.stages);
    // launched with programmatic stream serialisation: its blocks may start (allocate tensor
    // memory, request their first weight blocks) while act_blocks_kernel is still running
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(W.n_tiles * P.ksplit * P.n_sweeps); cfg.blockDim = dim3(TG_THREADS);
    cfg.dynamicSmemBytes = (size_t)smem; cfg.stream = c->stream;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr; cfg.numAttrs = 1;
    CUDA_TRY(c, cudaLaunchKernelEx(&cfg, gemm_tc05_kernel, P));
    LAUNCH_OK(c, "gemm_tc05_kernel");
  }
  return DMTD_OK;
}

// out[m][n] += sum_k W[n][k] act[m][k]
dmtd_status launch_gemv(dmtd_ctx *c, const PackedMat &W, const UmmaMat &U, const float *act, int lda, int M, float *out,
                        int ldo) {
  if (U.w && c->use_umma && M > 4) return launch_gemm_tc05(c, U, act, lda, M, out, ldo);
  if (W.wf) {
    gemv_f32_kernel<<<2 * c->n_sms, 256, 0, c->stream>>>(W, act, lda, M, out, ldo);
    LAUNCH_OK(c, "gemv_f32_kernel");
    return DMTD_OK;
  }
  if (M <= 4) return launch_gemv_nt<1>(c, W, act, lda, M, out, ldo);
  if (M <= 8) return launch_gemv_nt<2>(c, W, act, lda, M, out, ldo);
  return launch_gemv_nt<4>(c, W, act, lda, M, out, ldo);
}

template <int D, typename KVT>
dmtd_status launch_attention_t(dmtd_ctx *c, int layer, int B, int R, const int *pos0, int nsplit, bool merge, bool flash) {
  const dmtd_model_shape &s = c->s;
  int M = B * R, heads = s.n_q_heads + 2 * s.n_kv_heads, G = s.n_q_heads / s.n_kv_heads;
  KVT *kc = static_cast<KVT *>(c->kc) + (size_t)layer * c->kv_layer_elems;
  KVT *vc = static_cast<KVT *>(c->vc) + (size_t)layer * c->kv_layer_elems;
  const LayerDev &lw = c->layers[layer];
  // a3 inside the attention kernel (16-bit cache, head_dim 128, decode-sized chunks): one launch less per layer
  const bool fused_a3 = D == PK_D && !std::is_same<KVT, float>::value && c->use_tc_attention && c->fuse_qk_rope && !flash &&
                        R <= ATTN_TC_MAX_NEW;
  if (!fused_a3) {
    qk_norm_rope_append_kernel<D, KVT><<<dim3(M, (heads + 3) / 4), 128, 0, c->stream>>>(
        c->qkv, c->ldqkv, s.n_q_heads, s.n_kv_heads, R, lw.w_qn, lw.w_kn, s.rms_eps, c->rope_tab, pos0, kc, vc,
        c->max_seq);
    LAUNCH_OK(c, "qk_norm_rope_append_kernel");
  }
  if constexpr (D == PK_D && !std::is_same<KVT, float>::value) {
    if (flash) {
      // a chunk of many positions per sequence (the prefill): the causal kernel, rows straight into `act`
      using Op = typename std::conditional<std::is_same<KVT, __half>::value, OpF16, OpBf16>::type;
      const int QB = PK_WARPS * (PK_QR / G);
      attn_prefill_kernel<Op><<<dim3((R + QB - 1) / QB, s.n_kv_heads, B), PK_THREADS, ATTN_PF_SMEM, c->stream>>>(
          c->qkv, c->ldqkv, kc, vc, c->max_seq, s.n_q_heads, s.n_kv_heads, R, pos0, c->act, c->lda);
      LAUNCH_OK(c, "attn_prefill_kernel");
      return DMTD_OK;
    }
  }
  int RB = std::max(1, ATTN_QR / G), n_rb = (R + RB - 1) / RB;
  if (D == PK_D && c->use_tc_attention) {
    // head_dim 128: the tensor-core kernel with a bf16 cache, the FMA kernel with an fp32 cache
    if constexpr (std::is_same<KVT, float>::value) {
      attn_f32_kernel<<<dim3(nsplit, s.n_kv_heads * n_rb, B), PK_THREADS, ATTN_F32_SMEM, c->stream>>>(
          c->qkv, c->ldqkv, kc, vc, c->max_seq, s.n_q_heads, s.n_kv_heads, R, RB, c->CH, pos0, c->part_o, c->part_ml, nsplit);
    } else {
      using Op = typename std::conditional<std::is_same<KVT, __half>::value, OpF16, OpBf16>::type;
      if (fused_a3)
        attn_tc_kernel<Op, true><<<dim3(nsplit, s.n_kv_heads * n_rb, B), PK_THREADS, ATTN_TC_SMEM, c->stream>>>(
            c->qkv, c->ldqkv, kc, vc, c->max_seq, s.n_q_heads, s.n_kv_heads, R, RB, c->CH, pos0, c->part_o, c->part_ml, nsplit,
            AttnFuse{lw.w_qn, lw.w_kn, c->rope_tab, s.rms_eps});
      else
        attn_tc_kernel<Op><<<dim3(nsplit, s.n_kv_heads * n_rb, B), PK_THREADS, ATTN_TC_SMEM, c->stream>>>(
            c->qkv, c->ldqkv, kc, vc, c->max_seq, s.n_q_heads, s.n_kv_heads, R, RB, c->CH, pos0, c->part_o, c->part_ml, nsplit);
    }
  } else {
  size_t smem = (size_t)ATTN_WARPS * ATTN_QR * D * sizeof(float);
  attn_partial_kernel<D, KVT><<<dim3(nsplit, s.n_kv_heads * n_rb, B), ATTN_WARPS * 32, smem, c->stream>>>(
      c->qkv, c->ldqkv, kc, vc, c->max_seq, s.n_q_heads, s.n_kv_heads, R, RB, c->CH, pos0, c->part_o, c->part_ml,
      nsplit);
  }
  LAUNCH_OK(c, "attn_partial_kernel");
  if (!merge) return DMTD_OK;               // the O projection's activation-block kernel merges the slices
  int n_rh = M * s.n_q_heads;
  attn_merge_kernel<D><<<(n_rh + 3) / 4, 128, 0, c->stream>>>(c->part_o, c->part_ml, nsplit, n_rh, s.n_q_heads,
                                                             c->act, c->lda);
  LAUNCH_OK(c, "attn_merge_kernel");
  return DMTD_OK;
}

// Chunks of at least this many positions per sequence run the causal prefill kernel (16-bit cache, head_dim 128).
constexpr int kFlashMinRows = 16;
bool flash_attention_ok(const dmtd_ctx *c, int R) {
  const int G = c->s.n_q_heads / c->s.n_kv_heads;
  return c->use_tc_attention && c->s.head_dim == PK_D && c->s.kv_dtype != DMTD_F32 && R >= kFlashMinRows && PK_QR % G == 0;
}

dmtd_status launch_attention(dmtd_ctx *c, int layer, int B, int R, const int *pos0, int nsplit, bool merge = true,
                             bool flash = false) {
  const int kv = c->s.kv_dtype;
  if (c->s.head_dim == 128)
    return kv == DMTD_BF16 ? launch_attention_t<128, __nv_bfloat16>(c, layer, B, R, pos0, nsplit, merge, flash)
         : kv == DMTD_F16 ? launch_attention_t<128, __half>(c, layer, B, R, pos0, nsplit, merge, flash)
                          : launch_attention_t<128, float>(c, layer, B, R, pos0, nsplit, merge, flash);
  return kv == DMTD_BF16 ? launch_attention_t<64, __nv_bfloat16>(c, layer, B, R, pos0, nsplit, merge, flash)
       : kv == DMTD_F16 ? launch_attention_t<64, __half>(c, layer, B, R, pos0, nsplit, merge, flash)
                        : launch_attention_t<64, float>(c, layer, B, R, pos0, nsplit, merge, flash);
}

dmtd_status launch_rope_table(dmtd_ctx *c, const int *pos0, int R) {
  int half = c->s.head_dim / 2, n = R * half;
  rope_table_kernel<<<(n + 127) / 128, 128, 0, c->stream>>>(pos0, R, half, c->inv_freq, c->rope_tab);
  LAUNCH_OK(c, "rope_table_kernel");
  return DMTD_OK;
}

dmtd_status launch_embed(dmtd_ctx *c, const int *pos0, int B, int R, float *x, bool accumulate) {
  embed_kernel<<<B * R, 128, 0, c->stream>>>(c->embed, c->tokens, c->max_seq, pos0, R, x, c->s.hidden,
                                             accumulate ? 1 : 0, c->dstate);
  LAUNCH_OK(c, "embed_kernel");
  return DMTD_OK;
}

// Number of key slices to launch: all of them while capturing a graph (the graph must stay
// valid as the context grows), else just enough for keys [0, pos_end).
int splits_for(const dmtd_ctx *c, int pos_end) {
  if (c->capturing) return c->nsplit_max;
  return std::max(1, std::min(c->nsplit_max, (pos_end + c->CH - 1) / c->CH));
}

// One decoder layer (steps a2-a7) on x [B*R][hidden]; rows of sequence b sit at positions
// *pos0 .. *pos0+R-1.  pos_end = host's value of *pos0 + R.
dmtd_status run_layer(dmtd_ctx *c, int l, float *x, int B, int R, const int *pos0, int pos_end) {
  const dmtd_model_shape &s = c->s;
  const LayerDev &lw = c->layers[l];
  int M = B * R, H = s.hidden, I = s.intermediate, QD = s.n_q_heads * s.head_dim;
  // the tcgen05 path normalises while it writes its activation blocks
  const bool tc = lw.qkv_u.w && c->use_umma && M > 4 && c->ldqkv % 4 == 0 && c->ldgu % 4 == 0;
  if (tc) {
    TRY(launch_gemm_tc05(c, lw.qkv_u, x, H, M, c->qkv, c->ldqkv, 0, lw.w_in));
  } else {
    prep_norm_kernel<<<dim3(M, (c->ldqkv + PREP_ZERO_COLS - 1) / PREP_ZERO_COLS), 256, 0, c->stream>>>(
        x, H, lw.w_in, H, s.rms_eps, c->act, c->lda, c->qkv, c->ldqkv, c->ldqkv);
    LAUNCH_OK(c, "prep_norm_kernel");
    TRY(launch_gemv(c, lw.qkv, lw.qkv_u, c->act, c->lda, M, c->qkv, c->ldqkv));
  }
  const int nsplit = splits_for(c, pos_end);
  const bool flash = flash_attention_ok(c, R);
  const bool fuse_merge = tc && !flash && NAB_ROWS * s.n_q_heads * nsplit <= MAB_MAX_SLOTS;
  TRY(launch_attention(c, l, B, R, pos0, nsplit, !fuse_merge, flash));
  (void)QD;
  if (fuse_merge) TRY(launch_gemm_tc05(c, lw.o_u, nullptr, 0, M, x, H, 0, nullptr, nsplit));
  else TRY(launch_gemv(c, lw.o, lw.o_u, c->act, c->lda, M, x, H));
  if (tc) {
    TRY(launch_gemm_tc05(c, lw.gu_u, x, H, M, c->gu, c->ldgu, 0, lw.w_post));
  } else {
    prep_norm_kernel<<<dim3(M, (c->ldgu + PREP_ZERO_COLS - 1) / PREP_ZERO_COLS), 256, 0, c->stream>>>(
        x, H, lw.w_post, H, s.rms_eps, c->act, c->lda, c->gu, c->ldgu, c->ldgu);
    LAUNCH_OK(c, "prep_norm_kernel");
    TRY(launch_gemv(c, lw.gu, lw.gu_u, c->act, c->lda, M, c->gu, c->ldgu));
  }
  if (lw.down_u.w && c->use_umma && M > 4) {
    // the tcgen05 path gates while it writes its activation blocks
    TRY(launch_gemm_tc05(c, lw.down_u, c->gu, c->ldgu, M, x, H, I));
  } else {
    prep_swiglu_kernel<<<dim3((I + 255) / 256, M), 256, 0, c->stream>>>(c->gu, c->ldgu, I, c->act, c->lda);
    LAUNCH_OK(c, "prep_swiglu_kernel");
    TRY(launch_gemv(c, lw.down, lw.down_u, c->act, c->lda, M, x, H));
  }
  return DMTD_OK;
}

SampleParams sample_params(const dmtd_ctx *c) {
  SampleParams sp{};
  sp.on = c->temperature > 0.f ? 1 : 0;
  sp.inv_temperature = sp.on ? 1.f / c->temperature : 1.f;
  sp.key0 = (unsigned)c->sample_seed; sp.key1 = (unsigned)(c->sample_seed >> 32);
  return sp;
}

// Step a9/a10: final norm, tied LM head, greedy pick, token feedback.
dmtd_status run_head(dmtd_ctx *c, int B, bool write_token, int *out_argmax, float *out_logits, size_t out_pitch_floats = 0) {
  const dmtd_model_shape &s = c->s;
  if (c->embed_u.w && c->use_umma && B > 4 && c->ldl % 4 == 0) {
    TRY(launch_gemm_tc05(c, c->embed_u, c->x_up, s.hidden, B, c->logits, c->ldl, 0, c->w_final));
  } else {
    prep_norm_kernel<<<dim3(B, (c->ldl + PREP_ZERO_COLS - 1) / PREP_ZERO_COLS), 256, 0, c->stream>>>(
        c->x_up, s.hidden, c->w_final, s.hidden, s.rms_eps, c->act, c->lda,
                                               c->logits, c->ldl, c->ldl);
    LAUNCH_OK(c, "prep_norm_kernel");
    TRY(launch_gemv(c, c->embed, c->embed_u, c->act, c->lda, B, c->logits, c->ldl));
  }
  if (out_logits)
    CUDA_TRY(c, cudaMemcpy2DAsync(out_logits, (out_pitch_floats ? out_pitch_floats : (size_t)s.vocab) * 4, c->logits,
                                  (size_t)c->ldl * 4, (size_t)s.vocab * 4, B, cudaMemcpyDeviceToDevice, c->stream));
  argmax_slices_kernel<<<dim3(B, ARGMAX_SLICES), 256, 0, c->stream>>>(c->logits, c->ldl, s.vocab, c->pick_val, c->pick_idx,
                                                                      c->dstate, sample_params(c));
  LAUNCH_OK(c, "argmax_slices_kernel");
  argmax_pick_kernel<<<B, 32, 0, c->stream>>>(c->pick_val, c->pick_idx, ARGMAX_SLICES, c->tokens, c->max_seq, c->dstate,
                                              write_token ? 1 : 0, out_argmax);
  LAUNCH_OK(c, "argmax_pick_kernel");
  return DMTD_OK;
}

// Kernels that need more than 48 KiB of dynamic shared memory must be told so once per device
// (the attribute belongs to the device's copy of the kernel, not to the process): done at create,
// with the context's device current.
dmtd_status configure_kernels(dmtd_ctx *c) {
  const auto dyn = cudaFuncAttributeMaxDynamicSharedMemorySize;
  CUDA_TRY(c, cudaFuncSetAttribute(gemv_bf16_kernel<1>, dyn, 100 * 1024));
  CUDA_TRY(c, cudaFuncSetAttribute(gemv_bf16_kernel<2>, dyn, 100 * 1024));
  CUDA_TRY(c, cudaFuncSetAttribute(gemv_bf16_kernel<4>, dyn, 100 * 1024));
  CUDA_TRY(c, cudaFuncSetAttribute(gemm_tc05_kernel, dyn, 227 * 1024 - 1024));
  CUDA_TRY(c, cudaFuncSetAttribute(attn_f32_kernel, dyn, ATTN_F32_SMEM));
  CUDA_TRY(c, cudaFuncSetAttribute(attn_tc_kernel<OpBf16>, dyn, ATTN_TC_SMEM));
  CUDA_TRY(c, cudaFuncSetAttribute(attn_tc_kernel<OpF16>, dyn, ATTN_TC_SMEM));
  CUDA_TRY(c, cudaFuncSetAttribute(attn_tc_kernel<OpBf16, true>, dyn, ATTN_TC_SMEM));
  CUDA_TRY(c, cudaFuncSetAttribute(attn_tc_kernel<OpF16, true>, dyn, ATTN_TC_SMEM));
  CUDA_TRY(c, cudaFuncSetAttribute(attn_prefill_kernel<OpBf16>, dyn, ATTN_PF_SMEM));
  CUDA_TRY(c, cudaFuncSetAttribute(attn_prefill_kernel<OpF16>, dyn, ATTN_PF_SMEM));
  CUDA_TRY(c, cudaFuncSetAttribute(attn_partial_kernel<64, __half>, dyn, 64 * 1024));
  CUDA_TRY(c, cudaFuncSetAttribute(attn_partial_kernel<128, __half>, dyn, 64 * 1024));
  CUDA_TRY(c, cudaFuncSetAttribute(attn_partial_kernel<64, float>, dyn, 64 * 1024));
  CUDA_TRY(c, cudaFuncSetAttribute(attn_partial_kernel<64, __nv_bfloat16>, dyn, 64 * 1024));
  CUDA_TRY(c, cudaFuncSetAttribute(attn_partial_kernel<128, float>, dyn, 64 * 1024));
  CUDA_TRY(c, cudaFuncSetAttribute(attn_partial_kernel<128, __nv_bfloat16>, dyn, 64 * 1024));
  return DMTD_OK;
}

// ---------------------------------------------------------------------------- fused pass

// Can the block-per-SM pass kernel stream this matrix?  Its k-slab must fit the staging area
// and one block's share must not reach over more than two slabs.
bool fused_matrix_ok(const PackedMat &m, int grid) {
  if (!m.w) return false;
  long long slab_atoms = (long long)m.n_tiles * m.aps, per_block = (packed_atoms(m) + grid - 1) / grid;
  // 32-bit stream arithmetic in the kernel: atoms * blocks must fit
  return m.aps * 32 <= PK_MAX_KS && per_block <= slab_atoms && packed_atoms(m) * (grid + 1) < (1ll << 31);
}

// Set up what the fused pass kernel needs; leaves fused_ok false when the model or the device
// does not fit it (the per-step kernels then run every pass).
dmtd_status setup_fused(dmtd_ctx *c) {
  const dmtd_model_shape &s = c->s;
  c->fused_ok = false;
  if (!is_bf16(c) || s.head_dim != PK_D || s.n_layers > PK_MAX_LAYERS) return DMTD_OK;
  if (s.n_q_heads / s.n_kv_heads > PK_MAX_GROUP || s.hidden % 8 || s.hidden > PK_XS_FLOATS) return DMTD_OK;
  int coop = 0;
  CUDA_TRY(c, cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device));
  if (!coop) return DMTD_OK;
  if (cudaFuncSetAttribute(dmtd_pass_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PK_SMEM_BYTES) != cudaSuccess) {
    cudaGetLastError();
    return DMTD_OK;
  }
  int per_sm = 0;
  CUDA_TRY(c, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, dmtd_pass_kernel, PK_THREADS, PK_SMEM_BYTES));
  if (per_sm < 1) return DMTD_OK;
  if (!fused_matrix_ok(c->embed, c->n_sms)) return DMTD_OK;
  for (const LayerDev &ld : c->layers) {
    if (!fused_matrix_ok(ld.qkv, c->n_sms) || !fused_matrix_ok(ld.o, c->n_sms) || !fused_matrix_ok(ld.gu, c->n_sms) ||
        !fused_matrix_ok(ld.down, c->n_sms))
      return DMTD_OK;
    if ((ld.o.aps * 32) % PK_D) return DMTD_OK;
    // the kernel works out every block's share of a matrix once per launch, from the first layer of the pass:
    // all layers must have the same four shapes (they do: one hidden and one intermediate size per model)
    const LayerDev &l0 = c->layers[0];
    auto same = [](const PackedMat &a, const PackedMat &b) {
      return a.N == b.N && a.K == b.K && a.n_tiles == b.n_tiles && a.aps == b.aps && a.n_slabs == b.n_slabs;
    };
    if (!same(ld.qkv, l0.qkv) || !same(ld.o, l0.o) || !same(ld.gu, l0.gu) || !same(ld.down, l0.down)) return DMTD_OK;
  }
  std::vector<PassLayer> h(s.n_layers);
  for (int l = 0; l < s.n_layers; ++l) {
    const LayerDev &ld = c->layers[l];
    h[l].qkv = ld.qkv; h[l].o = ld.o; h[l].gu = ld.gu; h[l].down = ld.down;
    h[l].w_in = ld.w_in; h[l].w_post = ld.w_post; h[l].w_qn = ld.w_qn; h[l].w_kn = ld.w_kn;
    const size_t kvb = s.kv_dtype == DMTD_F32 ? 4 : 2;
    h[l].kc = static_cast<unsigned char *>(c->kc) + (size_t)l * c->kv_layer_elems * kvb;
    h[l].vc = static_cast<unsigned char *>(c->vc) + (size_t)l * c->kv_layer_elems * kvb;
  }
  TRY(dev_alloc(c, &c->pass_layers, h.size()));
  CUDA_TRY(c, cudaMemcpyAsync(c->pass_layers, h.data(), h.size() * sizeof(PassLayer), cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  size_t slots = (size_t)PK_MAX_ROWS * s.n_q_heads * PK_NSPLIT_CAP;
  TRY(dev_alloc(c, &c->f_part_o, slots * PK_D));
  TRY(dev_alloc(c, &c->f_part_ml, slots * 2));
  TRY(dev_alloc(c, &c->amax_val, (size_t)PK_MAX_ROWS * c->n_sms));
  TRY(dev_alloc(c, &c->amax_idx, (size_t)PK_MAX_ROWS * c->n_sms));
  TRY(dev_alloc(c, &c->grid_bar, 1));
#ifdef DMTD_PASS_TIMING
  TRY(dev_alloc(c, &c->pass_timing, (size_t)2 * PK_TIMING_SLOTS));
#endif
  c->fused_ok = true;
  return DMTD_OK;
}

bool fused_pass_ok(const dmtd_ctx *c, int kind, int R_lower) {
  if (!c->fused_ok || !c->use_fused || c->literal_sum || c->L_e > 0) return false;
  const int lo = c->s.n_layers - c->L_d;
  const int R = (kind == 1 && lo > 0) ? R_lower : 1;
  return c->B * R <= PK_MAX_ROWS && R * (c->s.n_q_heads / c->s.n_kv_heads) <= PK_QR &&
         c->B * R * c->s.hidden <= PK_XS_FLOATS;
}

// One pass (Section 2.2) as a single cooperative launch of the persistent pass kernel.
dmtd_status enqueue_pass_fused(dmtd_ctx *c, int kind, int R_lower, bool write_token, int *out_argmax, float *out_logits) {
  const dmtd_model_shape &s = c->s;
  const int L = s.n_layers, lo = L - c->L_d;
  PassParams P{};
  P.layers = c->pass_layers; P.embed = c->embed; P.w_final = c->w_final; P.inv_freq = c->inv_freq;
  P.l_begin = (kind == 1 && lo > 0) ? 0 : lo; P.l_split = lo; P.l_end = L;
  P.R_lo = (kind == 1 && lo > 0) ? R_lower : 1; P.B = c->B;
  P.H = s.hidden; P.I = s.intermediate; P.nq = s.n_q_heads; P.nkv = s.n_kv_heads; P.vocab = s.vocab;
  P.max_seq = c->max_seq; P.ldl = c->ldl; P.eps = s.rms_eps;
  P.kind = kind; P.write_token = write_token ? 1 : 0; P.kv_f32 = s.kv_dtype == DMTD_F32 ? 1 : 0; P.kv_f16 = s.kv_dtype == DMTD_F16 ? 1 : 0;
  P.tokens = c->tokens; P.st = c->dstate;
  P.x_lo = c->x_lo; P.x_up = c->x_up; P.qkv = c->qkv; P.gu = c->gu; P.logits = c->logits;
  P.timing = c->pass_timing;
  P.part_o = c->f_part_o; P.part_ml = c->f_part_ml; P.amax_val = c->amax_val; P.amax_idx = c->amax_idx;
  P.out_argmax = out_argmax; P.barrier = c->grid_bar; P.error = &c->dstate->error;
  P.wait_limit = kDeviceWaitLimitTicks;
  P.sample = sample_params(c);
  CUDA_TRY(c, cudaMemsetAsync(c->grid_bar, 0, sizeof(unsigned int), c->stream));
  void *args[] = {&P};
  CUDA_TRY(c, cudaLaunchCooperativeKernel((const void *)dmtd_pass_kernel, dim3(c->n_sms), dim3(PK_THREADS), args,
                                          (size_t)PK_SMEM_BYTES, c->stream));
  c->launches += 1;
  if (out_logits)
    CUDA_TRY(c, cudaMemcpy2DAsync(out_logits, (size_t)s.vocab * 4, c->logits, (size_t)c->ldl * 4, (size_t)s.vocab * 4, c->B,
                                  cudaMemcpyDeviceToDevice, c->stream));
  return DMTD_OK;
}

// One pass of the decode stage (Section 2.2).  kind 1: full pass - the R = n_known - lo_len
// pending rows through the lower layers (refill), the newest row through the decoding
// layers.  kind 2: the newest token's embedding through the decoding layers only.
dmtd_status enqueue_pass(dmtd_ctx *c, int kind, int R_lower, bool write_token, int *out_argmax, float *out_logits) {
  const int B = c->B, L = c->s.n_layers, lo = L - c->L_d, H = c->s.hidden;
  const int newest = c->h.n_known - 1;
  if (!c->capturing && fused_pass_ok(c, kind, R_lower))
    return enqueue_pass_fused(c, kind, R_lower, write_token, out_argmax, out_logits);
  if (c->L_e > 0) {
    // ExDy: the newest token's embedding goes through the encoding layers in every pass; their
    // output h_enc is kept until the thinking layers have seen the position
    const int Le = c->L_e;
    TRY(launch_embed(c, &c->dstate->newest, B, 1, c->x_up, false));
    TRY(launch_rope_table(c, &c->dstate->newest, 1));
    for (int l = 0; l < Le; ++l) TRY(run_layer(c, l, c->x_up, B, 1, &c->dstate->newest, newest + 1));
    if (kind == 1) {
      // full pass: the pending rows' h_enc and the newest row's through the thinking layers
      gather_pending_kernel<<<B * R_lower, 256, 0, c->stream>>>(c->h_pend, c->pend_cap, c->x_up, R_lower, H, c->x_lo);
      LAUNCH_OK(c, "gather_pending_kernel");
      TRY(launch_rope_table(c, &c->dstate->lo_len, R_lower));
      for (int l = Le; l < lo; ++l) TRY(run_layer(c, l, c->x_lo, B, R_lower, &c->dstate->lo_len, c->h.n_known));
      if (c->literal_sum) {
        select_last_kernel<<<B, 256, 0, c->stream>>>(c->x_lo, R_lower, H, c->h_base);
        LAUNCH_OK(c, "select_last_kernel");
        copy_rows_kernel<<<64, 256, 0, c->stream>>>(c->h_base, c->x_up, (size_t)B * H / 4, 1);
        LAUNCH_OK(c, "copy_rows_kernel");
      } else {
        select_last_kernel<<<B, 256, 0, c->stream>>>(c->x_lo, R_lower, H, c->x_up);
        LAUNCH_OK(c, "select_last_kernel");
      }
    } else if (kind == 2) {
      save_pending_kernel<<<B, 256, 0, c->stream>>>(c->x_up, c->h_pend, c->pend_cap, H, c->dstate);
      LAUNCH_OK(c, "save_pending_kernel");
    }
  } else if (kind == 1 && lo > 0) {
    TRY(launch_embed(c, &c->dstate->lo_len, B, R_lower, c->x_lo, false));
    TRY(launch_rope_table(c, &c->dstate->lo_len, R_lower));
    for (int l = 0; l < lo; ++l) TRY(run_layer(c, l, c->x_lo, B, R_lower, &c->dstate->lo_len, c->h.n_known));
    select_last_kernel<<<B, 256, 0, c->stream>>>(c->x_lo, R_lower, H, c->x_up);
    LAUNCH_OK(c, "select_last_kernel");
    if (c->literal_sum) TRY(launch_embed(c, &c->dstate->newest, B, 1, c->x_up, true));
  } else {
    TRY(launch_embed(c, &c->dstate->newest, B, 1, c->x_up, false));
  }
  TRY(launch_rope_table(c, &c->dstate->newest, 1));
  for (int l = lo; l < L; ++l) TRY(run_layer(c, l, c->x_up, B, 1, &c->dstate->newest, newest + 1));
  TRY(run_head(c, B, write_token, out_argmax, out_logits));
  advance_state_kernel<<<1, 1, 0, c->stream>>>(c->dstate, kind, 0);
  LAUNCH_OK(c, "advance_state_kernel");
  return DMTD_OK;
}

void host_advance(dmtd_ctx *c, int kind) {
  dmtd_state &h = c->h;
  if (kind == 1) { h.lo_len = h.n_known; h.cycle += 1; }
  h.up_len = h.n_known;
  h.n_known += 1;
  h.slot = (h.slot + 1) % h.tau;
  h.n_emitted += 1;
}

// Calls that return results to the host synchronise the stream anyway: they bring the device's
// error word along (4 bytes into pinned memory, queued before the synchronise) and turn it into a
// status.  The word is sticky on the device and the failure is sticky here until dmtd_reset.
dmtd_status queue_error_read(dmtd_ctx *c) {
  CUDA_TRY(c, cudaMemcpyAsync(c->h_error, &c->dstate->error, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  return DMTD_OK;
}
dmtd_status device_error_status(dmtd_ctx *c, int word) {
  if (word == 0) return DMTD_OK;
  if (word == PK_ERR_TOKEN) {
    c->device_failure = DMTD_ERR_INVALID_ARG;
    return fail(c, DMTD_ERR_INVALID_ARG, "a token id outside [0, vocab) reached the embedding gather; "
                "the results since then are invalid, call dmtd_reset");
  }
  c->device_failure = DMTD_ERR_TIMEOUT;
  return fail(c, DMTD_ERR_TIMEOUT, "a device-side wait gave up (%s); the results since then are invalid, call dmtd_reset",
              word == PK_ERR_COPY_WAIT ? "weight copy" : word == PK_ERR_BARRIER_WAIT ? "grid barrier" : "tensor-core pipeline");
}
#define CHECK_NOT_FAILED(c)                                                                          \
  do {                                                                                               \
    if ((c)->device_failure != DMTD_OK)                                                              \
      return fail((c), (c)->device_failure, "the context reported a device-side error earlier; call dmtd_reset"); \
  } while (0)

void drop_graphs(dmtd_ctx *c) {
  for (int k = 0; k < 3; ++k)
    if (c->graph_exec[k]) { cudaGraphExecDestroy(c->graph_exec[k]); c->graph_exec[k] = nullptr; }
}

// Capture a steady-state pass (R_lower = tau) into a graph.  Positions come from the device
// counters and the attention grid covers max_seq, so one graph serves the whole generation.
dmtd_status capture_pass(dmtd_ctx *c, int kind) {
  cudaGraph_t graph = nullptr;
  int64_t before = c->launches;
  if (!c->capture_stream) CUDA_TRY(c, cudaStreamCreateWithFlags(&c->capture_stream, cudaStreamNonBlocking));
  cudaError_t e = cudaStreamBeginCapture(c->capture_stream, cudaStreamCaptureModeThreadLocal);
  if (e != cudaSuccess) return fail(c, DMTD_ERR_CUDA, "begin capture: %s", cudaGetErrorString(e));
  cudaStream_t user_stream = c->stream;
  c->stream = c->capture_stream;
  c->capturing = true;
  dmtd_status st = enqueue_pass(c, kind, c->tau, true, nullptr, nullptr);
  e = cudaStreamEndCapture(c->capture_stream, &graph);
  c->capturing = false;
  c->stream = user_stream;
  int nodes = (int)(c->launches - before);
  c->launches = before;
  if (st != DMTD_OK) { if (graph) cudaGraphDestroy(graph); return st; }
  if (e != cudaSuccess) return fail(c, DMTD_ERR_CUDA, "end capture: %s", cudaGetErrorString(e));
  e = cudaGraphInstantiate(&c->graph_exec[kind], graph, 0);
  cudaGraphDestroy(graph);
  if (e != cudaSuccess) return fail(c, DMTD_ERR_CUDA, "graph instantiate: %s", cudaGetErrorString(e));
  c->graph_nodes[kind] = nodes;
  return DMTD_OK;
}

// Run the next pass of the schedule in greedy mode.
dmtd_status run_greedy_pass(dmtd_ctx *c) {
  int kind = c->h.slot == 0 ? 1 : 2;
  int R_lower = c->h.n_known - c->h.lo_len;
  bool steady = (kind == 2) || (R_lower == c->tau);
  if (fused_pass_ok(c, kind, R_lower)) {
    TRY(enqueue_pass_fused(c, kind, R_lower, true, nullptr, nullptr));
  } else if (c->use_graph && steady) {
    if (c->graph_B != c->B || c->graph_tau != c->tau) { drop_graphs(c); c->graph_B = c->B; c->graph_tau = c->tau; }
    if (!c->graph_exec[kind]) TRY(capture_pass(c, kind));
    CUDA_TRY(c, cudaGraphLaunch(c->graph_exec[kind], c->stream));
    c->launches += c->graph_nodes[kind];
  } else {
    TRY(enqueue_pass(c, kind, R_lower, true, nullptr, nullptr));
  }
  host_advance(c, kind);
  return DMTD_OK;
}

dmtd_status validate_shape(const dmtd_model_shape *s, int L_d, int tau, int max_batch, int max_seq) {
  if (s->n_layers < 1 || s->hidden < 1 || s->n_q_heads < 1 || s->n_kv_heads < 1 || s->intermediate < 1 || s->vocab < 1)
    return fail(nullptr, DMTD_ERR_SHAPE, "model dimensions must be positive");
  if (L_d < 1 || L_d > s->n_layers) return fail(nullptr, DMTD_ERR_SHAPE, "L_d must be in [1, n_layers]");
  if (tau < 1) return fail(nullptr, DMTD_ERR_SHAPE, "tau must be >= 1");
  if (max_batch < 1 || max_seq < 2) return fail(nullptr, DMTD_ERR_INVALID_ARG, "max_batch >= 1 and max_seq >= 2 required");
  if (s->n_q_heads % s->n_kv_heads) return fail(nullptr, DMTD_ERR_SHAPE, "n_q_heads must be a multiple of n_kv_heads");
  if (s->n_q_heads / s->n_kv_heads > ATTN_QR) return fail(nullptr, DMTD_ERR_SHAPE, "at most 16 query heads per kv head");
  if (s->head_dim != 64 && s->head_dim != 128) return fail(nullptr, DMTD_ERR_SHAPE, "head_dim must be 64 or 128");
  if (s->weight_dtype != DMTD_F32 && s->weight_dtype != DMTD_BF16) return fail(nullptr, DMTD_ERR_SHAPE, "weight_dtype");
  if (s->kv_dtype != DMTD_F32 && s->kv_dtype != DMTD_BF16 && s->kv_dtype != DMTD_F16) return fail(nullptr, DMTD_ERR_SHAPE, "kv_dtype");
  int mult = s->weight_dtype == DMTD_BF16 ? 32 : 4;
  if (s->hidden % mult || s->intermediate % mult)
    return fail(nullptr, DMTD_ERR_SHAPE, "hidden and intermediate must be multiples of %d", mult);
  if (s->weight_dtype == DMTD_BF16 && ((s->n_q_heads * s->head_dim) % 16 || s->intermediate % 16))
    return fail(nullptr, DMTD_ERR_SHAPE, "fused row blocks must be multiples of 16");
  if (!s->tied_lm_head) return fail(nullptr, DMTD_ERR_UNSUPPORTED, "only a tied LM head is supported");
  if (!(s->rope_theta > 0.f) || !(s->rms_eps >= 0.f)) return fail(nullptr, DMTD_ERR_SHAPE, "rope_theta / rms_eps");
  return DMTD_OK;
}

}  // namespace

// ================================================================================ C ABI

extern "C" {

dmtd_status dmtd_create(const dmtd_model_shape *shape, int32_t L_d, int32_t tau, int32_t max_batch,
                        int32_t max_seq, const dmtd_weights *w, void *cuda_stream, dmtd_ctx **out) {
  if (!shape || !w || !out || !w->embed || !w->final_norm || !w->layers)
    return fail(nullptr, DMTD_ERR_INVALID_ARG, "null argument");
  if (w->lm_head) return fail(nullptr, DMTD_ERR_UNSUPPORTED, "only a tied LM head is supported (lm_head must be NULL)");
  dmtd_status vs = validate_shape(shape, L_d, tau, max_batch, max_seq);
  if (vs != DMTD_OK) return vs;

  dmtd_ctx *c = new dmtd_ctx();
  auto bail = [&](dmtd_status st) { g_create_error = c->err; dmtd_destroy(c); return st; };
#define CTRY(expr) do { dmtd_status s__ = (expr); if (s__ != DMTD_OK) return bail(s__); } while (0)
#define CCUDA(expr) do { cudaError_t e__ = (expr); if (e__ != cudaSuccess) { \
    fail(c, DMTD_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e__)); return bail(DMTD_ERR_CUDA); } } while (0)

  c->s = *shape; c->L_d = L_d; c->tau = tau; c->max_batch = max_batch; c->max_seq = max_seq;
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  CCUDA(cudaGetDevice(&c->device));
  CCUDA(cudaDeviceGetAttribute(&c->n_sms, cudaDevAttrMultiProcessorCount, c->device));
  const dmtd_model_shape &s = c->s;
  const int H = s.hidden, D = s.head_dim, QD = s.n_q_heads * D, KVD = s.n_kv_heads * D, I = s.intermediate;

  // weights; every bf16 context whose dimensions fit also gets the copy the tcgen05 GEMM reads:
  // passes of more than 4 rows (batch x cycle length) and the prefill of every context use it
  c->umma_ok = s.weight_dtype == DMTD_BF16 && H % TG_KB == 0 && QD % TG_KB == 0 && I % TG_KB == 0;
  // DMTD_WEIGHT_COPIES=1 in the environment keeps only the atom stream (half the weight memory):
  // every projection then runs on the mma.sync kernels, the prefill included (slower from 5 rows up)
  if (const char *e = getenv("DMTD_WEIGHT_COPIES")) if (atoi(e) == 1) c->umma_ok = false;
  c->layers.resize(s.n_layers);
  // k-slab width of the packed matrices: contexts small enough for the pass kernel (which stages
  // only the slabs a block's share touches, and gains from short ones) get 256-wide slabs;
  // larger batches run the per-step GEMV, which is faster with 1280-wide slabs
  const int aps = max_batch <= PK_MAX_ROWS ? 8 : 40;
  for (int l = 0; l < s.n_layers; ++l) {
    const dmtd_layer_weights &lw = w->layers[l];
    const void *ptrs[] = {lw.input_norm, lw.q_proj, lw.k_proj, lw.v_proj, lw.q_norm, lw.k_norm, lw.o_proj,
                          lw.post_norm, lw.gate_proj, lw.up_proj, lw.down_proj};
    for (const void *p : ptrs)
      if (!p) { fail(c, DMTD_ERR_INVALID_ARG, "null weight pointer in layer %d", l); return bail(DMTD_ERR_INVALID_ARG); }
    LayerDev &ld = c->layers[l];
    const void *qkv_src[3] = {lw.q_proj, lw.k_proj, lw.v_proj};
    int qkv_n[3] = {QD, KVD, KVD};
    CTRY(pack_matrix(c, &ld.qkv, H, qkv_src, qkv_n, 3, aps));
    const void *o_src[1] = {lw.o_proj}; int o_n[1] = {H};
    // k-slabs of two heads: a block of the pass kernel then merges the attention slices of few heads
    CTRY(pack_matrix(c, &ld.o, QD, o_src, o_n, 1, D == 128 ? 8 : 40));
    const void *gu_src[2] = {lw.gate_proj, lw.up_proj}; int gu_n[2] = {I, I};
    CTRY(pack_matrix(c, &ld.gu, H, gu_src, gu_n, 2, aps));
    const void *d_src[1] = {lw.down_proj}; int d_n[1] = {H};
    CTRY(pack_matrix(c, &ld.down, I, d_src, d_n, 1, aps));
    if (c->umma_ok) {
      CTRY(pack_umma(c, &ld.qkv_u, H, qkv_src, qkv_n, 3));
      CTRY(pack_umma(c, &ld.o_u, QD, o_src, o_n, 1));
      CTRY(pack_umma(c, &ld.gu_u, H, gu_src, gu_n, 2));
      CTRY(pack_umma(c, &ld.down_u, I, d_src, d_n, 1));
    }
    CTRY(vec_to_float(c, &ld.w_in, lw.input_norm, H));
    CTRY(vec_to_float(c, &ld.w_post, lw.post_norm, H));
    CTRY(vec_to_float(c, &ld.w_qn, lw.q_norm, D));
    CTRY(vec_to_float(c, &ld.w_kn, lw.k_norm, D));
  }
  {
    const void *e_src[1] = {w->embed}; int e_n[1] = {s.vocab};
    CTRY(pack_matrix(c, &c->embed, H, e_src, e_n, 1, aps));
    if (c->umma_ok) CTRY(pack_umma(c, &c->embed_u, H, e_src, e_n, 1));
    CTRY(vec_to_float(c, &c->w_final, w->final_norm, H));
  }
  {
    std::vector<double> f(D / 2);
    for (int i = 0; i < D / 2; ++i) f[i] = std::pow((double)s.rope_theta, -2.0 * i / (double)D);
    CTRY(dev_alloc(c, &c->inv_freq, f.size()));
    CCUDA(cudaMemcpyAsync(c->inv_freq, f.data(), f.size() * sizeof(double), cudaMemcpyHostToDevice, c->stream));
    CCUDA(cudaStreamSynchronize(c->stream));
  }

  // sequence state
  size_t kvb = s.kv_dtype == DMTD_F32 ? 4 : 2;
  c->kv_layer_elems = (size_t)max_batch * s.n_kv_heads * max_seq * D;
  {
    unsigned char *p = nullptr;
    c->mem_kind = 2;
    CTRY(dev_alloc(c, &p, c->kv_layer_elems * s.n_layers * kvb)); c->kc = p;
    CTRY(dev_alloc(c, &p, c->kv_layer_elems * s.n_layers * kvb)); c->vc = p;
    c->mem_kind = 3;
  }
  CTRY(dev_alloc(c, &c->tokens, (size_t)max_batch * max_seq));
  CTRY(dev_alloc(c, &c->dstate, 1));
  CCUDA(cudaHostAlloc(reinterpret_cast<void **>(&c->h_error), sizeof(int), cudaHostAllocDefault));
  *c->h_error = 0;

  // workspace
  c->lda = std::max(H, std::max(QD, I));
  c->ldqkv = QD + 2 * KVD; c->ldgu = 2 * I; c->ldl = (s.vocab + 15) / 16 * 16;
  // Keys per slice of the split-KV attention: enough slices that a decode step of max_batch
  // sequences fills the SMs about four times over, and no more (every slice costs a block its
  // set-up, a partial result and a share of the merge); whole 64-key tiles.
  {
    const int want = std::max(1, std::min(64, 4 * c->n_sms / std::max(1, max_batch * s.n_kv_heads)));
    c->CH = std::max(64, ((max_seq + want - 1) / want + 63) / 64 * 64);
  }
  c->nsplit_max = (max_seq + c->CH - 1) / c->CH;
  // Rows of the workspace = rows of one prefill chunk: up to 1024 (fewer, larger launches, and the
  // row blocks of one sequence find its K and V in L2), less where many key slices would make
  // the slices' partial results large; never fewer than a decode pass needs.
  c->ws_rows = std::max(std::max(256, max_batch * std::max(tau, 8)), std::min(1024, 16384 / std::max(1, c->nsplit_max)));
  CTRY(dev_alloc(c, &c->x_lo, (size_t)c->ws_rows * H));
  CTRY(dev_alloc(c, &c->x_up, (size_t)max_batch * H));
  CTRY(dev_alloc(c, &c->act, (size_t)c->ws_rows * c->lda));
  CTRY(dev_alloc(c, &c->qkv, (size_t)c->ws_rows * c->ldqkv));
  CTRY(dev_alloc(c, &c->gu, (size_t)c->ws_rows * c->ldgu));
  CTRY(dev_alloc(c, &c->logits, (size_t)max_batch * c->ldl));
  CTRY(dev_alloc(c, &c->pick_val, (size_t)max_batch * ARGMAX_SLICES));
  CTRY(dev_alloc(c, &c->pick_idx, (size_t)max_batch * ARGMAX_SLICES));
  CTRY(dev_alloc(c, &c->part_o, (size_t)c->ws_rows * s.n_q_heads * c->nsplit_max * D));
  CTRY(dev_alloc(c, &c->part_ml, (size_t)c->ws_rows * s.n_q_heads * c->nsplit_max * 2));
  CTRY(dev_alloc(c, &c->rope_tab, (size_t)c->ws_rows * (D / 2)));
  c->pend_cap = std::max(1, c->ws_rows / max_batch);
  CTRY(dev_alloc(c, &c->h_pend, (size_t)max_batch * c->pend_cap * H));
  CTRY(dev_alloc(c, &c->h_base, (size_t)c->ws_rows * H));
  if (c->umma_ok) CTRY(dev_alloc(c, &c->act_blocks, (size_t)TG_MAX_SWEEPS * (c->lda / TG_KB) * 8 * TG_MAX_COLS));
  CTRY(configure_kernels(c));
  CTRY(setup_fused(c));
  CTRY(dmtd_reset(c));
  CCUDA(cudaStreamSynchronize(c->stream));   // repacking done: the caller may free its weights
#undef CTRY
#undef CCUDA
  *out = c;
  return DMTD_OK;
}

void dmtd_destroy(dmtd_ctx *c) {
  if (!c) return;
  if (c->stream || true) cudaStreamSynchronize(c->stream);
  drop_graphs(c);
  if (c->capture_stream) cudaStreamDestroy(c->capture_stream);
  for (void *p : c->allocs) cudaFree(p);
  if (c->h_error) cudaFreeHost(c->h_error);
  delete c;
}

dmtd_status dmtd_reset(dmtd_ctx *c) {
  if (!c) return DMTD_ERR_INVALID_ARG;
  DevState z{};
  z.tau = c->tau;
  CUDA_TRY(c, cudaMemcpyAsync(c->dstate, &z, sizeof z, cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  c->h = dmtd_state{};
  c->h.tau = c->tau; c->h.L_d = c->L_d;
  c->prefilled = false; c->B = 0;
  c->device_failure = DMTD_OK;
  if (c->h_error) *c->h_error = 0;
  return DMTD_OK;
}

dmtd_status dmtd_prefill(dmtd_ctx *c, const int32_t *prompt, int32_t B, int32_t P, const int32_t *forced_first,
                         int32_t *out_token, float *out_logits) {
  if (!c) return DMTD_ERR_INVALID_ARG;
  if (!prompt || B < 1 || P < 1) return fail(c, DMTD_ERR_INVALID_ARG, "prefill: null prompt or non-positive size");
  CHECK_NOT_FAILED(c);
  if (c->prefilled) return fail(c, DMTD_ERR_STATE, "prefill: context already holds a sequence; call dmtd_reset first");
  if (B > c->max_batch || P + 1 > c->max_seq) return fail(c, DMTD_ERR_CAPACITY, "prefill: B=%d P=%d exceed max_batch=%d max_seq=%d", B, P, c->max_batch, c->max_seq);
  const int L = c->s.n_layers, lo = L - c->L_d;
  c->B = B;
  CUDA_TRY(c, cudaMemcpy2DAsync(c->tokens, (size_t)c->max_seq * 4, prompt, (size_t)P * 4, (size_t)P * 4, B,
                                cudaMemcpyDeviceToDevice, c->stream));
  // All prompt rows through all layers (Section 2.2: the prefill is pass 1 of cycle 1), in
  // causal chunks of rows that fit the workspace.
  const int Rc_max = std::max(1, c->ws_rows / B);
  int last_R = 0;
  for (int p0 = 0; p0 < P; p0 += Rc_max) {
    int R = std::min(Rc_max, P - p0);
    set_int_kernel<<<1, 1, 0, c->stream>>>(&c->dstate->scratch, p0);
    LAUNCH_OK(c, "set_int_kernel");
    TRY(launch_embed(c, &c->dstate->scratch, B, R, c->x_lo, false));
    TRY(launch_rope_table(c, &c->dstate->scratch, R));
    for (int l = 0; l < L; ++l) {
      if (c->literal_sum && c->L_e > 0) {
        // Eq. 4's sum with h_enc in h_emb's place: keep the encoding layers' output, add it at the boundary
        if (l == c->L_e) {
          copy_rows_kernel<<<256, 256, 0, c->stream>>>(c->x_lo, c->h_base, (size_t)B * R * c->s.hidden / 4, 0);
          LAUNCH_OK(c, "copy_rows_kernel");
        }
        if (l == lo) {
          copy_rows_kernel<<<256, 256, 0, c->stream>>>(c->h_base, c->x_lo, (size_t)B * R * c->s.hidden / 4, 1);
          LAUNCH_OK(c, "copy_rows_kernel");
        }
      } else if (l == lo && c->literal_sum && lo > 0) {
        TRY(launch_embed(c, &c->dstate->scratch, B, R, c->x_lo, true));
      }
      TRY(run_layer(c, l, c->x_lo, B, R, &c->dstate->scratch, p0 + R));
    }
    last_R = R;
  }
  select_last_kernel<<<B, 256, 0, c->stream>>>(c->x_lo, last_R, c->s.hidden, c->x_up);
  LAUNCH_OK(c, "select_last_kernel");
  // n_known must read P when the head writes the token
  set_int_kernel<<<1, 1, 0, c->stream>>>(&c->dstate->n_known, P);
  LAUNCH_OK(c, "set_int_kernel");
  TRY(run_head(c, B, forced_first == nullptr, out_token, out_logits));
  if (forced_first)
    CUDA_TRY(c, cudaMemcpy2DAsync(c->tokens + P, (size_t)c->max_seq * 4, forced_first, 4, 4, B,
                                  cudaMemcpyDeviceToDevice, c->stream));
  advance_state_kernel<<<1, 1, 0, c->stream>>>(c->dstate, 0, P);
  LAUNCH_OK(c, "advance_state_kernel");
  c->h.n_known = P + 1; c->h.lo_len = P; c->h.up_len = P; c->h.cycle = 1;
  c->h.slot = 1 % c->tau; c->h.n_emitted = 1;
  c->prefilled = true;
  return DMTD_OK;
}

dmtd_status dmtd_decode_cycle(dmtd_ctx *c, int32_t max_new, int32_t *out_tokens, int32_t *n_out) {
  if (!c) return DMTD_ERR_INVALID_ARG;
  if (!n_out || max_new < 0) return fail(c, DMTD_ERR_INVALID_ARG, "decode_cycle: n_out is null or max_new < 0");
  *n_out = 0;
  CHECK_NOT_FAILED(c);
  if (!c->prefilled) return fail(c, DMTD_ERR_STATE, "decode_cycle: no prefill yet");
  const int first = c->h.n_known;
  int n = 0;
  dmtd_status rc = DMTD_OK;
  while (n < max_new) {
    if (c->h.n_known + 1 > c->max_seq) { rc = fail(c, DMTD_ERR_CAPACITY, "decode_cycle: position %d does not fit max_seq=%d", c->h.n_known, c->max_seq); break; }
    rc = run_greedy_pass(c);
    if (rc != DMTD_OK) break;                // the passes that were enqueued still count
    ++n;
    if (c->h.slot == 0) break;     // the cycle is complete
  }
  if (out_tokens && n > 0) {
    gather_tokens_kernel<<<c->B, 32, 0, c->stream>>>(c->tokens, c->max_seq, first, n, c->tau, out_tokens);
    LAUNCH_OK(c, "gather_tokens_kernel");
  }
  *n_out = n;
  return rc;
}

dmtd_status dmtd_decode_forced(dmtd_ctx *c, const int32_t *forced, int32_t n, float *out_logits, int32_t *out_argmax) {
  if (!c) return DMTD_ERR_INVALID_ARG;
  if (!forced || n < 0) return fail(c, DMTD_ERR_INVALID_ARG, "decode_forced: null forced tokens or n < 0");
  CHECK_NOT_FAILED(c);
  if (!c->prefilled) return fail(c, DMTD_ERR_STATE, "decode_forced: no prefill yet");
  if (c->h.n_known + n > c->max_seq) return fail(c, DMTD_ERR_CAPACITY, "decode_forced: %d more positions do not fit max_seq=%d", n, c->max_seq);
  if (n == 0) return DMTD_OK;
  // the forced tokens are the sequence's next n tokens: place them, then run the schedule
  // without letting the head overwrite them
  CUDA_TRY(c, cudaMemcpy2DAsync(c->tokens + c->h.n_known, (size_t)c->max_seq * 4, forced, (size_t)n * 4, (size_t)n * 4,
                                c->B, cudaMemcpyDeviceToDevice, c->stream));
  const size_t BV = (size_t)c->B * c->s.vocab;
  for (int i = 0; i < n; ++i) {
    int kind = c->h.slot == 0 ? 1 : 2;
    TRY(enqueue_pass(c, kind, c->h.n_known - c->h.lo_len, false, out_argmax ? out_argmax + (size_t)i * c->B : nullptr,
                     out_logits ? out_logits + (size_t)i * BV : nullptr));
    host_advance(c, kind);
  }
  return DMTD_OK;
}

dmtd_status dmtd_step_layers(dmtd_ctx *c, int32_t l0, int32_t l1, float *hidden, int32_t B, int32_t R, int32_t pos0) {
  if (!c) return DMTD_ERR_INVALID_ARG;
  if (!hidden || l0 < 0 || l1 > c->s.n_layers || l0 > l1 || B < 1 || R < 1 || pos0 < 0)
    return fail(c, DMTD_ERR_INVALID_ARG, "step_layers: bad layer range, sizes or null hidden");
  CHECK_NOT_FAILED(c);
  if (B > c->max_batch || R > c->max_seq || pos0 > c->max_seq - R || (long long)B * R > c->ws_rows)
    return fail(c, DMTD_ERR_CAPACITY, "step_layers: B=%d R=%d pos0=%d exceed max_batch=%d max_seq=%d rows=%d", B, R, pos0, c->max_batch, c->max_seq, c->ws_rows);
  set_int_kernel<<<1, 1, 0, c->stream>>>(&c->dstate->scratch, pos0);
  LAUNCH_OK(c, "set_int_kernel");
  TRY(launch_rope_table(c, &c->dstate->scratch, R));
  for (int l = l0; l < l1; ++l) TRY(run_layer(c, l, hidden, B, R, &c->dstate->scratch, pos0 + R));
  return DMTD_OK;
}

dmtd_status dmtd_masked_forward(dmtd_ctx *c, const int32_t *tokens, int32_t B, int32_t n, int32_t P, float *out_logits) {
  if (!c) return DMTD_ERR_INVALID_ARG;
  if (!tokens || !out_logits || B < 1 || P < 1 || n < P) return fail(c, DMTD_ERR_INVALID_ARG, "masked_forward: null pointer, or not 1 <= P <= n");
  CHECK_NOT_FAILED(c);
  if (c->prefilled) return fail(c, DMTD_ERR_STATE, "masked_forward: the context holds a sequence; call dmtd_reset first");
  if (B > c->max_batch || n > c->max_seq) return fail(c, DMTD_ERR_CAPACITY, "masked_forward: B=%d n=%d exceed max_batch=%d max_seq=%d", B, n, c->max_batch, c->max_seq);
  const int L = c->s.n_layers, lo = L - c->L_d, Le = c->L_e, H = c->s.hidden;
  c->B = B;
  CUDA_TRY(c, cudaMemcpy2DAsync(c->tokens, (size_t)c->max_seq * 4, tokens, (size_t)n * 4, (size_t)n * 4, B,
                                cudaMemcpyDeviceToDevice, c->stream));
  // Eq. 1-5 chunk by chunk: a chunk of rows goes through every layer before the next one starts
  // (each layer is causal and the earlier chunks' K and V are in the cache by then).
  const int Rc_max = std::max(1, c->ws_rows / B);
  const size_t n_out = (size_t)(n - (P - 1));
  for (int p0 = 0; p0 < n; p0 += Rc_max) {
    const int R = std::min(Rc_max, n - p0);
    const size_t n4 = (size_t)B * R * H / 4;
    set_int_kernel<<<1, 1, 0, c->stream>>>(&c->dstate->scratch, p0);
    LAUNCH_OK(c, "set_int_kernel");
    TRY(launch_embed(c, &c->dstate->scratch, B, R, c->x_lo, false));                 // h_emb
    TRY(launch_rope_table(c, &c->dstate->scratch, R));
    for (int l = 0; l < Le; ++l) TRY(run_layer(c, l, c->x_lo, B, R, &c->dstate->scratch, p0 + R));   // Eq. 1: h_enc
    copy_rows_kernel<<<256, 256, 0, c->stream>>>(c->x_lo, c->h_base, n4, 0);
    LAUNCH_OK(c, "copy_rows_kernel");
    for (int l = Le; l < lo; ++l) TRY(run_layer(c, l, c->x_lo, B, R, &c->dstate->scratch, p0 + R));  // Eq. 2: h_think
    masked_select_kernel<<<B * R, 256, 0, c->stream>>>(c->x_lo, c->h_base, R, H, p0, P, c->tau, c->literal_sum ? 1 : 0);   // Eq. 3-4
    LAUNCH_OK(c, "masked_select_kernel");
    for (int l = lo; l < L; ++l) TRY(run_layer(c, l, c->x_lo, B, R, &c->dstate->scratch, p0 + R));   // Eq. 5: decoding layers
    for (int r = std::max(0, P - 1 - p0); r < R; ++r) {                                                // ... and the LM head
      select_row_kernel<<<B, 256, 0, c->stream>>>(c->x_lo, R, r, H, c->x_up);
      LAUNCH_OK(c, "select_row_kernel");
      TRY(run_head(c, B, false, nullptr, out_logits + (size_t)(p0 + r - (P - 1)) * c->s.vocab, n_out * c->s.vocab));
    }
  }
  // the cache now holds this forward's K and V; the schedule state is untouched (still "no sequence")
  c->B = 0;
  return DMTD_OK;
}

dmtd_status dmtd_prefill_host(dmtd_ctx *c, const int32_t *prompt_host, int32_t B, int32_t P, int32_t *out_token_host) {
  if (!c) return DMTD_ERR_INVALID_ARG;
  if (!prompt_host || B < 1 || P < 1) return fail(c, DMTD_ERR_INVALID_ARG, "prefill_host: null prompt or non-positive size");
  if (c->prefilled) return fail(c, DMTD_ERR_STATE, "prefill_host: context already holds a sequence; call dmtd_reset first");
  if (B > c->max_batch || P + 1 > c->max_seq) return fail(c, DMTD_ERR_CAPACITY, "prefill_host: sizes exceed capacity");
  // stage the prompt at the tail of the act workspace (unused until the first layer runs)
  int *stage = reinterpret_cast<int *>(c->gu);
  if ((size_t)B * P > (size_t)c->ws_rows * c->ldgu) return fail(c, DMTD_ERR_CAPACITY, "prefill_host: prompt larger than staging space");
  CUDA_TRY(c, cudaMemcpyAsync(stage, prompt_host, (size_t)B * P * 4, cudaMemcpyHostToDevice, c->stream));
  // the token buffer copy inside dmtd_prefill reads `stage` before any layer writes gu
  TRY(dmtd_prefill(c, stage, B, P, nullptr, nullptr, nullptr));
  if (out_token_host)
    CUDA_TRY(c, cudaMemcpy2DAsync(out_token_host, 4, c->tokens + P, (size_t)c->max_seq * 4, 4, B, cudaMemcpyDeviceToHost, c->stream));
  TRY(queue_error_read(c));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  return device_error_status(c, *c->h_error);
}

dmtd_status dmtd_decode_cycle_host(dmtd_ctx *c, int32_t max_new, int32_t *out_tokens_host, int32_t *n_out) {
  if (!c) return DMTD_ERR_INVALID_ARG;
  if (!n_out) return fail(c, DMTD_ERR_INVALID_ARG, "decode_cycle_host: n_out is null");
  const int first = c->h.n_known;
  dmtd_status rc = dmtd_decode_cycle(c, max_new, nullptr, n_out);
  if (rc != DMTD_OK && rc != DMTD_ERR_CAPACITY) return rc;
  if (out_tokens_host && *n_out > 0)
    CUDA_TRY(c, cudaMemcpy2DAsync(out_tokens_host, (size_t)c->tau * 4, c->tokens + first, (size_t)c->max_seq * 4,
                                  (size_t)*n_out * 4, c->B, cudaMemcpyDeviceToHost, c->stream));
  TRY(queue_error_read(c));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  dmtd_status dev = device_error_status(c, *c->h_error);
  return dev != DMTD_OK ? dev : rc;
}

dmtd_status dmtd_get_state(const dmtd_ctx *c, dmtd_state *out) {
  if (!c || !out) return DMTD_ERR_INVALID_ARG;
  *out = c->h;
  return DMTD_OK;
}

dmtd_status dmtd_get_device_state(dmtd_ctx *c, dmtd_state *out) {
  if (!c || !out) return DMTD_ERR_INVALID_ARG;
  DevState d{};
  CUDA_TRY(c, cudaMemcpyAsync(&d, c->dstate, sizeof d, cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  TRY(device_error_status(c, d.error));
  out->n_known = d.n_known; out->lo_len = d.lo_len; out->up_len = d.up_len; out->cycle = d.cycle;
  out->slot = d.slot; out->n_emitted = d.n_emitted; out->tau = d.tau; out->L_d = c->L_d;
  return DMTD_OK;
}

dmtd_status dmtd_set_tau(dmtd_ctx *c, int32_t tau) {
  if (!c) return DMTD_ERR_INVALID_ARG;
  if (tau < 1) return fail(c, DMTD_ERR_SHAPE, "set_tau: tau must be >= 1");
  if (c->prefilled && c->h.slot != 0) return fail(c, DMTD_ERR_STATE, "set_tau: only at a cycle boundary");
  if (c->max_batch * tau > c->ws_rows) return fail(c, DMTD_ERR_CAPACITY, "set_tau: workspace too small for tau=%d", tau);
  c->tau = tau; c->h.tau = tau;
  CUDA_TRY(c, cudaMemcpyAsync(&c->dstate->tau, &c->tau, sizeof(int), cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  return DMTD_OK;
}

dmtd_status dmtd_set_sampling(dmtd_ctx *c, float temperature, uint64_t seed) {
  if (!c) return DMTD_ERR_INVALID_ARG;
  if (!(temperature >= 0.f) || std::isinf(temperature)) return fail(c, DMTD_ERR_INVALID_ARG, "set_sampling: temperature must be finite and >= 0");
  c->temperature = temperature; c->sample_seed = seed;
  drop_graphs(c);                           // the captured passes carry the old parameters
  return DMTD_OK;
}

dmtd_status dmtd_set_option(dmtd_ctx *c, const char *name, int64_t value) {
  if (!c || !name) return DMTD_ERR_INVALID_ARG;
  if (!strcmp(name, "encoding_layers")) {
    if (c->prefilled) return fail(c, DMTD_ERR_STATE, "encoding_layers can only change before the prefill (call dmtd_reset first)");
    if (value < 0 || value + c->L_d > c->s.n_layers)
      return fail(c, DMTD_ERR_SHAPE, "encoding_layers must be in [0, n_layers - L_d]");
    c->L_e = (int)value; drop_graphs(c); return DMTD_OK;
  }
  if (!strcmp(name, "tcgen05_gemm_stages")) {
    if (value != 0 && (value < 2 || value > TG_STAGES)) return fail(c, DMTD_ERR_INVALID_ARG, "tcgen05_gemm_stages takes 0 (chosen per launch) or 2..%d", TG_STAGES);
    c->gemm_stages = (int)value; drop_graphs(c); return DMTD_OK;
  }
  if (value != 0 && value != 1) return fail(c, DMTD_ERR_INVALID_ARG, "option %s takes 0 or 1", name);
  if (!strcmp(name, "cuda_graph")) { c->use_graph = value != 0; return DMTD_OK; }
  if (!strcmp(name, "literal_sum")) { c->literal_sum = value != 0; drop_graphs(c); return DMTD_OK; }
  if (!strcmp(name, "fused_pass")) { c->use_fused = value != 0; return DMTD_OK; }
  if (!strcmp(name, "fused_qk_rope")) { c->fuse_qk_rope = value != 0; drop_graphs(c); return DMTD_OK; }
  if (!strcmp(name, "tcgen05_gemm")) { c->use_umma = value != 0; drop_graphs(c); return DMTD_OK; }
  if (!strcmp(name, "tc_attention")) { c->use_tc_attention = value != 0; drop_graphs(c); return DMTD_OK; }
  return fail(c, DMTD_ERR_INVALID_ARG, "unknown option %s", name);
}

dmtd_status dmtd_get_kv(dmtd_ctx *c, int32_t layer, void **k, void **v) {
  if (!c || layer < 0 || layer >= c->s.n_layers) return DMTD_ERR_INVALID_ARG;
  size_t kvb = c->s.kv_dtype == DMTD_F32 ? 4 : 2;
  if (k) *k = static_cast<unsigned char *>(c->kc) + (size_t)layer * c->kv_layer_elems * kvb;
  if (v) *v = static_cast<unsigned char *>(c->vc) + (size_t)layer * c->kv_layer_elems * kvb;
  return DMTD_OK;
}

dmtd_status dmtd_debug_set_error_word(dmtd_ctx *c, int32_t word) {
  if (!c || word < 0) return DMTD_ERR_INVALID_ARG;
  CUDA_TRY(c, cudaMemcpyAsync(&c->dstate->error, &word, sizeof(int), cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  return DMTD_OK;
}

dmtd_status dmtd_get_memory_info(const dmtd_ctx *c, dmtd_memory_info *out) {
  if (!c || !out) return DMTD_ERR_INVALID_ARG;
  out->weight_stream_bytes = c->mem[0]; out->weight_block_bytes = c->mem[1];
  out->kv_cache_bytes = c->mem[2]; out->workspace_bytes = c->mem[3];
  return DMTD_OK;
}

dmtd_status dmtd_get_launch_count(const dmtd_ctx *c, int64_t *out) {
  if (!c || !out) return DMTD_ERR_INVALID_ARG;
  *out = c->launches;
  return DMTD_OK;
}

const char *dmtd_status_str(dmtd_status s) {
  switch (s) {
    case DMTD_OK: return "ok";
    case DMTD_ERR_INVALID_ARG: return "invalid argument";
    case DMTD_ERR_SHAPE: return "unsupported shape";
    case DMTD_ERR_STATE: return "call out of order";
    case DMTD_ERR_CAPACITY: return "capacity exceeded";
    case DMTD_ERR_CUDA: return "CUDA error";
    case DMTD_ERR_TIMEOUT: return "device wait timed out";
    case DMTD_ERR_UNSUPPORTED: return "unsupported";
  }
  return "unknown status";
}

const char *dmtd_last_error(const dmtd_ctx *c) { return c ? c->err.c_str() : g_create_error.c_str(); }

}  // extern "C"

// ---- step a4 as a context-free call ------------------------------------------------------

namespace {

struct AttnPlan { int CH, nsplit; size_t ml_off, o_off, bytes; };

// Scratch layout: [0, 256) the first position as a device int, then the running (max, sum)
// pairs, then the unnormalised partial outputs, one set per (row, head, key slice).
AttnPlan attn_plan(int B, int R, int nq, int D, int n_keys) {
  AttnPlan p{};
  // slices enough to fill a GPU of about 150 SMs four times over (the call does not know the
  // number of kv heads: a quarter of the query heads is assumed), each of whole 64-key tiles
  const int want = std::max(1, std::min(64, 600 / std::max(1, B * std::max(1, nq / 4))));
  p.CH = std::max(64, ((n_keys + want - 1) / want + 63) / 64 * 64);
  p.nsplit = std::max(1, (n_keys + p.CH - 1) / p.CH);
  size_t slots = (size_t)B * R * nq * p.nsplit;
  p.ml_off = 256;
  p.o_off = p.ml_off + (slots * 2 * sizeof(float) + 255) / 256 * 256;
  p.bytes = p.o_off + slots * D * sizeof(float);
  return p;
}

dmtd_status attention_check(const float *q, const void *k, const void *v, int kv_dtype, int B, int R, int nq, int nkv,
                            int D, int max_seq, int pos0, const float *out) {
  if (!q || !k || !v || !out || B < 1 || R < 1 || pos0 < 0 || max_seq < 1)
    return fail(nullptr, DMTD_ERR_INVALID_ARG, "attention: null pointer or non-positive size");
  if (kv_dtype != DMTD_F32 && kv_dtype != DMTD_BF16 && kv_dtype != DMTD_F16) return fail(nullptr, DMTD_ERR_SHAPE, "attention: kv_dtype");
  if (D != 64 && D != 128) return fail(nullptr, DMTD_ERR_SHAPE, "attention: head_dim must be 64 or 128");
  if (nq < 1 || nkv < 1 || nq % nkv || nq / nkv > ATTN_QR)
    return fail(nullptr, DMTD_ERR_SHAPE, "attention: n_q_heads must be a multiple of n_kv_heads, at most 16 per kv head");
  if (R > max_seq || pos0 > max_seq - R) return fail(nullptr, DMTD_ERR_CAPACITY, "attention: pos0 = %d with R = %d rows exceeds max_seq = %d", pos0, R, max_seq);
  return DMTD_OK;
}

template <int D, typename KVT>
dmtd_status attention_launch_t(const float *q, const void *k, const void *v, int B, int R, int nq, int nkv, int max_seq,
                               int pos0, unsigned char *scratch, const AttnPlan &p, float *out, cudaStream_t stream) {
  int *pos_dev = reinterpret_cast<int *>(scratch);
  float *part_ml = reinterpret_cast<float *>(scratch + p.ml_off);
  float *part_o = reinterpret_cast<float *>(scratch + p.o_off);
  const int G = nq / nkv, RB = std::max(1, ATTN_QR / G), n_rb = (R + RB - 1) / RB, ld = nq * D;
  set_int_kernel<<<1, 1, 0, stream>>>(pos_dev, pos0);
  cudaError_t e;
  if (D == PK_D) {
    if constexpr (std::is_same<KVT, float>::value) {
      e = cudaFuncSetAttribute(attn_f32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ATTN_F32_SMEM);
      if (e != cudaSuccess) return fail(nullptr, DMTD_ERR_CUDA, "attention: %s", cudaGetErrorString(e));
      attn_f32_kernel<<<dim3(p.nsplit, nkv * n_rb, B), PK_THREADS, ATTN_F32_SMEM, stream>>>(
          q, ld, static_cast<const float *>(k), static_cast<const float *>(v), max_seq, nq, nkv, R, RB, p.CH, pos_dev, part_o,
          part_ml, p.nsplit);
    } else {
      using Op = typename std::conditional<std::is_same<KVT, __half>::value, OpF16, OpBf16>::type;
      e = cudaFuncSetAttribute(attn_tc_kernel<Op>, cudaFuncAttributeMaxDynamicSharedMemorySize, ATTN_TC_SMEM);
      if (e != cudaSuccess) return fail(nullptr, DMTD_ERR_CUDA, "attention: %s", cudaGetErrorString(e));
      attn_tc_kernel<Op><<<dim3(p.nsplit, nkv * n_rb, B), PK_THREADS, ATTN_TC_SMEM, stream>>>(
          q, ld, k, v, max_seq, nq, nkv, R, RB, p.CH, pos_dev, part_o, part_ml, p.nsplit);
    }
  } else {
    size_t smem = (size_t)ATTN_WARPS * ATTN_QR * D * sizeof(float);
    e = cudaFuncSetAttribute(attn_partial_kernel<D, KVT>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
    if (e != cudaSuccess) return fail(nullptr, DMTD_ERR_CUDA, "attention: %s", cudaGetErrorString(e));
    attn_partial_kernel<D, KVT><<<dim3(p.nsplit, nkv * n_rb, B), ATTN_WARPS * 32, smem, stream>>>(
        q, ld, static_cast<const KVT *>(k), static_cast<const KVT *>(v), max_seq, nq, nkv, R, RB, p.CH, pos_dev, part_o,
        part_ml, p.nsplit);
  }
  int n_rh = B * R * nq;
  attn_merge_kernel<D><<<(n_rh + 3) / 4, 128, 0, stream>>>(part_o, part_ml, p.nsplit, n_rh, nq, out, ld);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(nullptr, DMTD_ERR_CUDA, "attention: launch failed: %s", cudaGetErrorString(e));
  return DMTD_OK;
}

dmtd_status attention_launch(const float *q, const void *k, const void *v, int kv_dtype, int B, int R, int nq, int nkv,
                             int D, int max_seq, int pos0, unsigned char *scratch, const AttnPlan &p, float *out,
                             cudaStream_t stream) {
  if (D == 128) {
    if (kv_dtype == DMTD_BF16) return attention_launch_t<128, __nv_bfloat16>(q, k, v, B, R, nq, nkv, max_seq, pos0, scratch, p, out, stream);
    if (kv_dtype == DMTD_F16) return attention_launch_t<128, __half>(q, k, v, B, R, nq, nkv, max_seq, pos0, scratch, p, out, stream);
    return attention_launch_t<128, float>(q, k, v, B, R, nq, nkv, max_seq, pos0, scratch, p, out, stream);
  }
  if (kv_dtype == DMTD_BF16) return attention_launch_t<64, __nv_bfloat16>(q, k, v, B, R, nq, nkv, max_seq, pos0, scratch, p, out, stream);
  if (kv_dtype == DMTD_F16) return attention_launch_t<64, __half>(q, k, v, B, R, nq, nkv, max_seq, pos0, scratch, p, out, stream);
  return attention_launch_t<64, float>(q, k, v, B, R, nq, nkv, max_seq, pos0, scratch, p, out, stream);
}

}  // namespace

extern "C" {

size_t dmtd_attention_scratch_bytes(int32_t B, int32_t R, int32_t nq, int32_t D, int32_t n_keys) {
  if (B < 1 || R < 1 || nq < 1 || D < 1 || n_keys < 1) return 0;
  return attn_plan(B, R, nq, D, n_keys).bytes;
}

dmtd_status dmtd_attention_decode(const float *q, const void *k, const void *v, int32_t kv_dtype, int32_t B, int32_t R,
                                  int32_t nq, int32_t nkv, int32_t D, int32_t max_seq, int32_t pos0, void *scratch,
                                  size_t scratch_bytes, float *out, void *cuda_stream) {
  dmtd_status st = attention_check(q, k, v, kv_dtype, B, R, nq, nkv, D, max_seq, pos0, out);
  if (st != DMTD_OK) return st;
  AttnPlan p = attn_plan(B, R, nq, D, pos0 + R);
  if (!scratch) return fail(nullptr, DMTD_ERR_INVALID_ARG, "attention: null scratch");
  if (scratch_bytes < p.bytes)
    return fail(nullptr, DMTD_ERR_CAPACITY, "attention: scratch of %zu bytes is smaller than the %zu needed", scratch_bytes, p.bytes);
  return attention_launch(q, k, v, kv_dtype, B, R, nq, nkv, D, max_seq, pos0, static_cast<unsigned char *>(scratch), p, out,
                          static_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"

// ---- the same call with its scratch inside the library ------------------------------------
//
// For callers that must not allocate: the partial results go to a fixed array in the device
// image.  In host code the array's name is only a handle; the device address is looked up
// once per device (with that device current) and passed to the kernels like any pointer.

static __device__ __align__(256) unsigned char g_attention_static_scratch[DMTD_ATTENTION_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
unsigned char *g_static_scratch_addr[kMaxDevices] = {};
std::mutex g_static_scratch_mu;

// Device address of the fixed scratch on the current device.
dmtd_status static_scratch_address(unsigned char **out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(nullptr, DMTD_ERR_CUDA, "attention_static: cudaGetDevice: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return fail(nullptr, DMTD_ERR_UNSUPPORTED, "attention_static: device index %d", dev);
  std::lock_guard<std::mutex> lock(g_static_scratch_mu);
  if (!g_static_scratch_addr[dev]) {
    void *p = nullptr;
    e = cudaGetSymbolAddress(&p, g_attention_static_scratch);
    if (e != cudaSuccess || !p)
      return fail(nullptr, DMTD_ERR_CUDA, "attention_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
    g_static_scratch_addr[dev] = static_cast<unsigned char *>(p);
  }
  *out = g_static_scratch_addr[dev];
  return DMTD_OK;
}

}  // namespace

extern "C" dmtd_status dmtd_attention_decode_static(const float *q, const void *k, const void *v, int32_t kv_dtype,
                                                    int32_t B, int32_t R, int32_t nq, int32_t nkv, int32_t D,
                                                    int32_t max_seq, int32_t pos0, float *out, void *cuda_stream) {
  dmtd_status st = attention_check(q, k, v, kv_dtype, B, R, nq, nkv, D, max_seq, pos0, out);
  if (st != DMTD_OK) return st;
  AttnPlan p = attn_plan(B, R, nq, D, pos0 + R);
  if (p.bytes > (size_t)DMTD_ATTENTION_STATIC_SCRATCH_BYTES)
    return fail(nullptr, DMTD_ERR_CAPACITY,
                "attention_static: this problem needs %zu bytes of scratch, the built-in array holds %zu; "
                "use dmtd_attention_decode with caller-owned scratch", p.bytes, (size_t)DMTD_ATTENTION_STATIC_SCRATCH_BYTES);
  unsigned char *scratch = nullptr;
  st = static_scratch_address(&scratch);
  if (st != DMTD_OK) return st;
  // nothing to clear: every (row, head, slice) entry the merge reads is written by this call
  return attention_launch(q, k, v, kv_dtype, B, R, nq, nkv, D, max_seq, pos0, scratch, p, out,
                          static_cast<cudaStream_t>(cuda_stream));
}

#ifdef DMTD_PASS_TIMING
// Profiling builds: copy out the stage time stamps of the last pass (2 x PK_TIMING_SLOTS ticks).
extern "C" int dmtd_debug_pass_timing(dmtd_ctx *c, long long *host_out) {
  if (!c || !c->pass_timing) return -1;
  cudaStreamSynchronize(c->stream);
  return (int)cudaMemcpy(host_out, c->pass_timing, sizeof(long long) * 2 * PK_TIMING_SLOTS, cudaMemcpyDeviceToHost);
}
#endif
