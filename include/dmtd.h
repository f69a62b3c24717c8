/*
 * dmtd.h - C ABI of the B200 (sm_100a) decode path of Direct Multi-Token Decoding (DMTD).
 *
 * DMTD (Section 2.2 of the paper) generates in fixed cycles of tau tokens.  The first pass
 * of a cycle runs all L layers; the other tau-1 passes run only the last L_d "decoding"
 * layers on the embedding of the newest token.  Tokens produced by such short passes have
 * no KV entries in the lower L-L_d layers; the next cycle's full pass feeds all of them
 * through the lower layers together with the newest token ("cyclical refilling"), and only
 * the newest row continues into the decoding layers.  The model is the Qwen3-style decoder
 * the paper fine-tunes (Section 3.1): RMSNorm, grouped-query attention with per-head QK-norm
 * and rotary position embedding, SwiGLU MLP, LM head tied to the embedding.
 *
 * Conventions
 *   - Every call returns a dmtd_status; nothing throws, aborts or exits.  On failure
 *     dmtd_last_error() gives a message.  A context is not thread-safe.
 *   - "device" pointers are CUDA device pointers on the context's device, "host" pointers
 *     are ordinary host memory.  All work is enqueued on the stream given at create; calls
 *     with host outputs synchronise that stream before returning, the others do not.
 *   - Weight matrices are [out_features, in_features] row-major, no biases.  dmtd_create
 *     copies and repacks them; the caller may free its buffers afterwards.  The library
 *     owns the packed weights, KV cache, token buffer, workspace and CUDA graphs.
 *   - Sequences of a batch advance in lock-step and have equal prompt length; there is no
 *     end-of-sequence handling (generation stops after the requested number of tokens).
 *   - Greedy decoding: argmax of the logits, lowest index on ties.
 *   - Device-side checks (a token id outside [0, vocab), which is clamped; a bounded wait of a
 *     kernel that ran out) set a sticky error word in device memory; no kernel traps.  Every
 *     call that synchronises the stream (dmtd_prefill_host, dmtd_decode_cycle_host,
 *     dmtd_get_device_state) reads the word and returns INVALID_ARG (token id) or TIMEOUT
 *     (wait).  From then on every call that would run kernels returns that status until
 *     dmtd_reset; the asynchronous calls made between the fault and its discovery have
 *     returned OK and advanced the host's copy of the schedule state, and what they produced
 *     is invalid.
 */
#ifndef DMTD_H
#define DMTD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dmtd_ctx dmtd_ctx;   /* opaque, library-owned */

typedef enum {
  DMTD_OK = 0,
  DMTD_ERR_INVALID_ARG = -1,   /* null pointer, negative size, ...                         */
  DMTD_ERR_SHAPE = -2,         /* model shape / L_d / tau the kernels cannot run           */
  DMTD_ERR_STATE = -3,         /* call out of order (decode before prefill, ...)           */
  DMTD_ERR_CAPACITY = -4,      /* batch > max_batch or positions > max_seq                 */
  DMTD_ERR_CUDA = -5,          /* a CUDA call failed; see dmtd_last_error                  */
  DMTD_ERR_TIMEOUT = -6,       /* a bounded device-side wait gave up                       */
  DMTD_ERR_UNSUPPORTED = -7
} dmtd_status;

enum { DMTD_F32 = 0, DMTD_BF16 = 1, DMTD_F16 = 2 };   /* DMTD_F16: KV cache only */

typedef struct {
  int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, intermediate, vocab;
  float rope_theta, rms_eps;
  int32_t weight_dtype;        /* DMTD_F32 or DMTD_BF16: storage type of every weight      */
  int32_t kv_dtype;            /* DMTD_F32, DMTD_BF16 or DMTD_F16: storage type of the KV    */
                               /* cache.  bf16 (8 significant bits) moves the logits of the  */
                               /* 36-layer model by more than 2e-2; fp16 (11 bits, K and V   */
                               /* are bounded by the QK-norm and the residual scale) by less */
                               /* than half of that at half of fp32's bytes; fp32 by 1e-4.   */
  int32_t tied_lm_head;        /* must be 1: the LM head is the embedding matrix           */
} dmtd_model_shape;

/* Device pointers in weight_dtype.  Norm vectors: input_norm/post_norm [hidden],
 * q_norm/k_norm [head_dim] (shared by all heads). */
typedef struct {
  const void *input_norm, *q_proj, *k_proj, *v_proj, *q_norm, *k_norm, *o_proj,
             *post_norm, *gate_proj, *up_proj, *down_proj;
} dmtd_layer_weights;

typedef struct {
  const void *embed;                  /* device [vocab, hidden]                             */
  const void *final_norm;             /* device [hidden]                                    */
  const void *lm_head;                /* must be NULL (tied)                                */
  const dmtd_layer_weights *layers;   /* HOST array [n_layers] of device pointers           */
} dmtd_weights;

/* Integer bookkeeping of the schedule (Section 2.2). */
typedef struct {
  int32_t n_known;    /* tokens whose id is known: prompt + emitted                         */
  int32_t lo_len;     /* positions with KV in the lower layers [0, L-L_d)                   */
  int32_t up_len;     /* positions with KV in the decoding layers [L-L_d, L)                */
  int32_t cycle;      /* 1 during the cycle the prefill starts; +1 per later full pass      */
  int32_t slot;       /* passes done in the current cycle, mod tau; 0 => next pass is full  */
  int32_t n_emitted;  /* tokens emitted so far, the prefill's included                      */
  int32_t tau, L_d;
} dmtd_state;

/* Create a context for one model and one (L_d, tau) split (Sections 2.2, 3.1: the last L_d
 * layers are the decoding layers, tau is the cycle length; tau = 1 is ordinary decoding).
 * max_batch / max_seq size the KV cache ([layer][sequence][kv head][max_seq][head_dim] for K
 * and for V) and the workspace.  `cuda_stream` is a cudaStream_t (NULL = default stream).
 * Errors: SHAPE if L_d not in [1, L], tau < 1, n_q_heads % n_kv_heads != 0, head_dim not 64
 * or 128, n_q_heads/n_kv_heads > 16, hidden or intermediate not a multiple of 32 (bf16) or
 * 4 (fp32); UNSUPPORTED if the LM head is not tied (tied_lm_head == 0 or lm_head != NULL);
 * CUDA if an allocation fails. */
dmtd_status dmtd_create(const dmtd_model_shape *shape, int32_t L_d, int32_t tau,
                        int32_t max_batch, int32_t max_seq, const dmtd_weights *weights,
                        void *cuda_stream, dmtd_ctx **out);
void dmtd_destroy(dmtd_ctx *ctx);

/* Forget the sequence state (KV contents become stale); the next call must be a prefill. */
dmtd_status dmtd_reset(dmtd_ctx *ctx);

/* Pass 1 of cycle 1 (Section 2.2): all P prompt positions of B sequences through all L
 * layers, KV written in every layer; emits the first token from the last row's logits.
 *   prompt        device int32 [B][P], ids in [0, vocab)
 *   forced_first  device int32 [B] or NULL; if given, it (not the argmax) becomes position P
 *   out_token     device int32 [B] or NULL: the argmax
 *   out_logits    device float [B][vocab] or NULL
 * Errors: STATE if already prefilled; CAPACITY if B > max_batch or P + 1 > max_seq. */
dmtd_status dmtd_prefill(dmtd_ctx *ctx, const int32_t *prompt, int32_t B, int32_t P,
                         const int32_t *forced_first, int32_t *out_token, float *out_logits);

/* Finish the current cycle, or run a whole one if at a cycle boundary (Section 2.2): the
 * first call after a prefill runs the tau-1 short passes of cycle 1; later calls run one full
 * pass (refill of the lower layers + newest row through all layers) and tau-1 short passes.
 * At most max_new tokens are produced (the cycle is cut short if needed).
 *   out_tokens  device int32 [B][tau] or NULL; columns [0, *n_out) are written
 *   n_out       host: tokens produced per sequence by this call
 * Errors: STATE before prefill; CAPACITY when the next position does not fit max_seq (the
 * passes that did fit have run and *n_out counts them). */
dmtd_status dmtd_decode_cycle(dmtd_ctx *ctx, int32_t max_new, int32_t *out_tokens,
                              int32_t *n_out);

/* Verification mode: n passes of the same schedule with teacher forcing.  After pass i the
 * token appended to sequence b is forced[b][i] instead of the model's choice.
 *   forced      device int32 [B][n]
 *   out_logits  device float [n][B][vocab] or NULL
 *   out_argmax  device int32 [n][B] or NULL: the model's own choice at each pass */
dmtd_status dmtd_decode_forced(dmtd_ctx *ctx, const int32_t *forced, int32_t n,
                               float *out_logits, int32_t *out_argmax);

/* The primitive both kinds of pass are made of (Section 2.2: a pass is a contiguous range
 * of layers applied to some rows): layers [l0, l1) on hidden [B][R][hidden] fp32 (device,
 * in place), rows of each sequence at positions pos0 .. pos0+R-1, attending causally to the
 * context's KV cache (positions < pos0 must have been written in those layers) and writing
 * the rows' K and V into it.  Does not touch the schedule state.
 * Errors: CAPACITY if pos0 + R > max_seq or B > max_batch. */
dmtd_status dmtd_step_layers(dmtd_ctx *ctx, int32_t l0, int32_t l1, float *hidden, int32_t B,
                             int32_t R, int32_t pos0);

/* Eq. 1-5 as one scoring pass over given token sequences (Section 2.1: the cyclical-masking
 * forward the decode schedule is the cached, incremental form of): every position through the
 * lower layers, the decoding layers reading the lower-stack output at mask positions (inside
 * the prompt and at the anchors P-1 + k tau, Section 2.2) and the embedding - or, with
 * encoding layers reused, their output - elsewhere; logits of positions P-1 .. n-1.
 *   tokens      device int32 [B][n]: prompt (P tokens) and continuation
 *   out_logits  device float [B][n - (P-1)][vocab]
 * Uses the context's cycle length, decoding-layer count and options (literal_sum,
 * encoding_layers).  Overwrites the KV cache from position 0 and leaves the context without a
 * sequence.  Errors: STATE if the context holds a sequence; CAPACITY if B > max_batch or
 * n > max_seq. */
dmtd_status dmtd_masked_forward(dmtd_ctx *ctx, const int32_t *tokens, int32_t B, int32_t n,
                                int32_t P, float *out_logits);

/* Step a4 on its own: split-KV attention of R new rows per sequence against a KV cache (the
 * attention of Section 2.2's passes needs the cached K and V of every earlier token), with the
 * online-softmax merge of the key slices.  No context is needed.
 *   q        device float [B][R][n_q_heads][head_dim], already normalised, rotated (not scaled)
 *   k, v     device [B][n_kv_heads][max_seq][head_dim] in kv_dtype; row r of a sequence sits at
 *            position pos0 + r and attends to positions [0, pos0 + r]; K and V of the R new
 *            positions must already be in the cache
 *   scratch  device memory of at least dmtd_attention_scratch_bytes(...) bytes, 256-byte
 *            aligned, owned by the caller; holds the per-slice partial results while the call's
 *            kernels run on `cuda_stream` (calls sharing one scratch must be stream-ordered)
 *   out      device float [B][R][n_q_heads][head_dim]
 * Errors: SHAPE for head_dim not 64/128, n_q_heads % n_kv_heads != 0 or more than 16 query
 * heads per KV head; CAPACITY if pos0 + R > max_seq or scratch_bytes is too small. */
size_t dmtd_attention_scratch_bytes(int32_t B, int32_t R, int32_t n_q_heads, int32_t head_dim,
                                    int32_t n_keys);
dmtd_status dmtd_attention_decode(const float *q, const void *k, const void *v, int32_t kv_dtype,
                                  int32_t B, int32_t R, int32_t n_q_heads, int32_t n_kv_heads,
                                  int32_t head_dim, int32_t max_seq, int32_t pos0, void *scratch,
                                  size_t scratch_bytes, float *out, void *cuda_stream);

/* dmtd_attention_decode for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of the call above, not a step of the method.)  It is
 * meant for a serving process that has handed every free byte of the GPU to its own memory pool,
 * so a cudaMalloc for the scratch would fail or fragment that pool, and for a latency-critical
 * decode loop where cudaMalloc / cudaFree would stall the whole device.  Arguments and results
 * are those of dmtd_attention_decode, minus the scratch: the per-slice partial results live in a
 * fixed array of DMTD_ATTENTION_STATIC_SCRATCH_BYTES bytes inside the library's device image
 * (every GPU that loads the library holds that much until the process exits).  The call makes no
 * cudaMalloc, cudaFree or other allocating call.
 *   - A problem whose dmtd_attention_scratch_bytes(...) exceeds that size is rejected with
 *     CAPACITY and nothing runs.
 *   - The first call on a device looks up the array's device address (once per device, with
 *     that device current); make that first call outside any stream capture.
 *   - All calls in the process share the one array.  It keeps the previous call's partials; the
 *     kernels overwrite every entry they later read, so nothing has to be cleared, but two calls
 *     whose kernels overlap on the GPU (different streams, different threads) race on it. */
#define DMTD_ATTENTION_STATIC_SCRATCH_BYTES (4u << 20)
dmtd_status dmtd_attention_decode_static(const float *q, const void *k, const void *v,
                                         int32_t kv_dtype, int32_t B, int32_t R, int32_t n_q_heads,
                                         int32_t n_kv_heads, int32_t head_dim, int32_t max_seq,
                                         int32_t pos0, float *out, void *cuda_stream);

/* Host-buffer forms of prefill and decode_cycle (same semantics; the copies to and from the
 * device are part of the call, which returns after the stream has drained).
 *   prompt_host [B][P], out_token_host [B], out_tokens_host [B][tau] */
dmtd_status dmtd_prefill_host(dmtd_ctx *ctx, const int32_t *prompt_host, int32_t B, int32_t P,
                              int32_t *out_token_host);
dmtd_status dmtd_decode_cycle_host(dmtd_ctx *ctx, int32_t max_new, int32_t *out_tokens_host,
                                   int32_t *n_out);

/* The schedule state as the host tracks it / as the device counters hold it (the second
 * synchronises the stream).  The two agree unless a device-side error was reported (see
 * Conventions); tests compare both with the oracle. */
dmtd_status dmtd_get_state(const dmtd_ctx *ctx, dmtd_state *out);
dmtd_status dmtd_get_device_state(dmtd_ctx *ctx, dmtd_state *out);

/* Change the cycle length (the paper evaluates inference cycle lengths other than the
 * training one, Section 3.7).  Only at a cycle boundary (slot == 0) or before prefill. */
dmtd_status dmtd_set_tau(dmtd_ctx *ctx, int32_t tau);

/* How the next token is picked from the logits.  temperature == 0 (the default): greedy, as in
 * the paper's experiments.  temperature > 0: a draw from softmax(logits / temperature) by the
 * Gumbel-max rule, argmax_i (logit_i / temperature - log(-log(u_i))), inside the same
 * vocabulary-parallel pick as the greedy rule (the paper has no sampling rule; this is what a
 * serving stack needs next to Section 3.7's runtime cycle lengths).  u_i in (0, 1) is made from
 * the top 24 bits of word i mod 4 of Philox4x32-10 with counter (i / 4, position of the token,
 * sequence index, 0) and key `seed`: a run is reproducible and independent of batch layout.
 * May be changed between any two calls.  Errors: INVALID_ARG for a negative or non-finite
 * temperature. */
dmtd_status dmtd_set_sampling(dmtd_ctx *ctx, float temperature, uint64_t seed);

/* Options, by name:
 *   "cuda_graph"   0/1  replay captured CUDA graphs for whole passes (default 1)
 *   "literal_sum"  0/1  upper-layer input of a full pass = embedding + lower-stack output, the
 *                       literal sum of Eq. 4, instead of the lower-stack output alone (default 0)
 *   "fused_pass"   0/1  run each decode pass as one persistent kernel where the model and batch
 *                       allow it (bf16 weights, head_dim 128, at most 4 rows per pass);
 *                       0 = always the per-step kernels (default 1)
 *   "encoding_layers" x  the ExDy variant (Section 2.1, the paragraph after Eq. 4; Section 3.3): the
 *                       short passes run the first x encoding layers as well as the last L_d
 *                       decoding layers, the decoding layers read the encoding layers' output
 *                       where the default reads the embedding, and a full pass refills only the
 *                       thinking layers [x, L - L_d).  0 <= x <= L - L_d; only before the prefill;
 *                       such contexts run the per-step kernels (default 0, the paper's E0Dy)
 *   "tc_attention" 0/1  attention of the per-step kernels by the tiled split-KV kernels for
 *                       head_dim 128 (tensor cores with a bf16 cache, FMAs with an fp32 cache)
 *                       instead of the one-warp-per-key-group kernel (default 1)
 *   "tcgen05_gemm" 0/1  projections of more than 4 rows (prefill chunks included) on the tcgen05
 *                       tensor cores; bf16 contexts whose hidden, query and intermediate sizes
 *                       are multiples of 64 hold the second weight copy it reads, which doubles
 *                       the weight memory of the context (default 1)
 *   "tcgen05_gemm_stages" n  pipeline stages of a block of that GEMM, 2..6; 0 = chosen per launch as
 *                       what keeps the most weight blocks in flight per SM (default 0)
 *   "fused_qk_rope" 0/1 QK-norm, rotary embedding and the KV append (Section 3.1's Qwen3 block) inside
 *                       the tensor-core attention kernel of the per-step path (16-bit cache, head_dim
 *                       128, chunks of fewer than 16 positions) instead of a launch of their own (default 1)
 * Errors: INVALID_ARG for an unknown name or value; SHAPE / STATE for encoding_layers as above. */
dmtd_status dmtd_set_option(dmtd_ctx *ctx, const char *name, int64_t value);

/* KV cache of one layer for inspection or for filling with test data: device pointers to
 * [max_batch][n_kv_heads][max_seq][head_dim] in kv_dtype. */
dmtd_status dmtd_get_kv(dmtd_ctx *ctx, int32_t layer, void **k, void **v);

/* Diagnostics: write the context's device error word from the host, as a device-side check
 * would (1 = token id out of range, 2 = weight-copy wait, 3 = grid-barrier wait, 4 =
 * tensor-core pipeline wait; 0 clears it).  Lets the error path of the synchronising calls be
 * exercised without making a GPU wait run out.  Synchronises the stream. */
dmtd_status dmtd_debug_set_error_word(dmtd_ctx *ctx, int32_t word);

/* Device memory the context holds, by purpose.  A bf16 context whose hidden, query and
 * intermediate sizes are multiples of 64 keeps its weights twice: as the atom stream the
 * mma.sync kernels and the pass kernel read (passes of up to 4 rows) and as the 16 KiB blocks
 * the tcgen05 GEMM reads (more rows, and every prefill): 2 x 8.04 GB for the Qwen3-4B shape.
 * With DMTD_WEIGHT_COPIES=1 in the environment at create only the first is kept. */
typedef struct {
  size_t weight_stream_bytes, weight_block_bytes, kv_cache_bytes, workspace_bytes;
} dmtd_memory_info;
dmtd_status dmtd_get_memory_info(const dmtd_ctx *ctx, dmtd_memory_info *out);

/* Number of this library's kernels launched on the stream since create (graph replays count
 * their kernel nodes). */
dmtd_status dmtd_get_launch_count(const dmtd_ctx *ctx, int64_t *out);

const char *dmtd_status_str(dmtd_status s);
const char *dmtd_last_error(const dmtd_ctx *ctx);   /* NULL: last error of a call without a context, on this thread */

#ifdef __cplusplus
}
#endif
#endif
