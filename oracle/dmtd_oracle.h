/*
 * CPU oracle for the decode path of Direct Multi-Token Decoding (DMTD).
 *
 * TEST INFRASTRUCTURE, NOT PRODUCT.  A plain, slow implementation used to check the
 * CUDA library and to report a CPU baseline.  It shares no code with the CUDA path and
 * the product never calls it.
 *
 * Arithmetic: every floating-point value is a C `double`; weights are read from their
 * storage type (fp32, or bf16 bit patterns) and widened exactly.  All pointers are host
 * pointers.  Functions return 0 on success and a negative code on bad arguments.
 *
 * What each function follows:
 *   model block      - the Qwen3-style decoder the paper fine-tunes (Section 3.1): RMSNorm,
 *                      grouped-query attention with per-head QK-norm and rotary embedding,
 *                      SwiGLU MLP, tied LM head.  The paper only names the model; the block
 *                      formulae are this build's reading and are pinned against a library
 *                      implementation of that architecture in the tests.
 *   schedule         - Section 2.2 (cycles of tau passes, cyclical refilling, Fig. 3 example).
 *   masked forward   - Section 2.1, Eq. 1-5, with the mask anchored as in Section 2.2.
 *   PLT              - Eq. 7.
 *
 * Parity pins: the unit functions are pinned to library routines and brute force, the
 * schedule to the worked example of Section 2.2 and to Eq. 7, the whole to the tau=1 and
 * L_d=L special cases.  The absolute logit values of a random-weight model are not printed
 * anywhere in the paper: for those, parity unpinned beyond the pins listed above.
 */
#ifndef DMTD_ORACLE_H
#define DMTD_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };

typedef struct {
  int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, intermediate, vocab;
  double rope_theta, rms_eps;
  int32_t weight_dtype;            /* ORACLE_F32 or ORACLE_BF16 (uint16 bit patterns) */
} oracle_shape;

/* Host pointers; matrices are [out_features, in_features] row-major, no biases. */
typedef struct {
  const void *input_norm, *q_proj, *k_proj, *v_proj, *q_norm, *k_norm, *o_proj,
             *post_norm, *gate_proj, *up_proj, *down_proj;
} oracle_layer_weights;

typedef struct {
  const void *embed;               /* [vocab, hidden]; also the LM head (tied) */
  const void *final_norm;          /* [hidden] */
  const oracle_layer_weights *layers;
} oracle_weights;

/* Integer bookkeeping of the schedule (Section 2.2). */
typedef struct {
  int32_t n_known;    /* tokens whose id is known: prompt + emitted                      */
  int32_t lo_len;     /* positions with KV in the lower layers [0, L-L_d)                */
  int32_t up_len;     /* positions with KV in the upper (decoding) layers [L-L_d, L)     */
  int32_t cycle;      /* 1 during the cycle the prefill starts; +1 per later full pass   */
  int32_t slot;       /* passes done in the current cycle, mod tau; 0 => next is full    */
  int32_t n_emitted;  /* tokens emitted so far, the prefill's included                   */
  int32_t tau, L_d;
} oracle_state;

/* One record per forward pass, in order (pass 0 is the prefill). */
typedef struct {
  int32_t kind;       /* 0 prefill, 1 full pass, 2 upper-only pass                       */
  int32_t lo_begin, lo_end;   /* positions fed to the lower layers: [lo_begin, lo_end)   */
  int32_t up_begin, up_end;   /* positions fed to the upper layers: [up_begin, up_end)   */
  int32_t cycle;
} oracle_pass_record;

typedef struct oracle_ctx oracle_ctx;

/* ---- unit functions (the exact routines the layer function is built from) ---------- */
/* y[r][i] = x[r][i] / sqrt(mean_i x[r][i]^2 + eps) * w[i]                                */
void oracle_rmsnorm(const double *x, const double *w, double eps, int rows, int n, double *y);
/* Rotary embedding, half-split pairing (i, i+d/2), angle pos * theta^(-2i/d). In place. */
void oracle_rope(double *v, int head_dim, int pos, double theta);
/* Causal grouped-query attention of R new rows at positions pos0..pos0+R-1 against keys
 * 0..pos0+R-1.  q [R][nq][d]; k, v [pos0+R][nkv][d]; out [R][nq][d]; scale 1/sqrt(d).   */
void oracle_attention(const double *q, const double *k, const double *v, int R, int pos0,
                      int nq, int nkv, int d, double *out);
/* y[r][o] = sum_k x[r][k] * W[o][k];  W in storage type `dtype`.                         */
void oracle_linear(const void *W, int dtype, int n_out, int n_in, const double *x, int rows,
                   double *y);
double oracle_silu(double t);
/* Philox4x32-10, the counter-based generator of Salmon et al. (SC'11). */
void oracle_philox4x32(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);
/* One draw from softmax(z / temperature) by the Gumbel-max rule with Philox noise keyed by
 * (seed; vocabulary index, position, sequence); temperature <= 0: greedy argmax.         */
int32_t oracle_sample_token(const double *z, int n, double temperature, uint64_t seed,
                            int32_t position, int32_t sequence);
/* Eq. 7. */
double oracle_plt(int L, int L_d, int tau);

/* ---- DMTD decode (Section 2.2) -------------------------------------------------------- */
int oracle_create(const oracle_shape *shape, int32_t L_d, int32_t tau, int32_t max_batch,
                  int32_t max_seq, const oracle_weights *w, oracle_ctx **out);
void oracle_destroy(oracle_ctx *c);
int oracle_reset(oracle_ctx *c);
int oracle_set_tau(oracle_ctx *c, int32_t tau);
/* full_pass_add_emb = 1 switches the upper-layer input at full-pass positions to
 * embedding + lower-stack output (the literal sum of Eq. 4); default 0 (select).        */
int oracle_set_literal_sum(oracle_ctx *c, int32_t on);
/* temperature > 0: every emitted token is drawn from softmax(logits / temperature) (the paper
 * decodes greedily; sampling is this build's extension, see oracle_sample_token); 0: greedy. */
int oracle_set_sampling(oracle_ctx *c, double temperature, uint64_t seed);
/* The ExDy variant (Section 2.1, the paragraph after Eq. 4; Section 3.3): the short passes reuse
 * the first L_e encoding layers as well as the last L_d decoding layers, and the decoding layers
 * read the encoding layers' output where the default reads the embedding.  Before prefill only;
 * L_e + L_d <= n_layers.  Default 0 (the paper's E0Dy setting).                            */
int oracle_set_encoding_layers(oracle_ctx *c, int32_t L_e);

/* Pass 1 of cycle 1: all P prompt rows through all layers.  out_token[B] = argmax of the
 * last row's logits (lowest index wins ties); out_logits [B][vocab] may be NULL.  If
 * forced_first is not NULL, that token (not the argmax) becomes position P.             */
int oracle_prefill(oracle_ctx *c, const int32_t *prompt, int32_t B, int32_t P,
                   const int32_t *forced_first, int32_t *out_token, double *out_logits);
/* Finish the current cycle (or run a whole one if at a boundary), at most max_new tokens.
 * out_tokens [B][tau] (first *n_out columns valid); out_logits [n_out][B][vocab] or NULL.*/
int oracle_decode_cycle(oracle_ctx *c, int32_t max_new, int32_t *out_tokens, int32_t *n_out,
                        double *out_logits);
/* n passes with teacher forcing: after pass i the token appended is forced[b][i].
 * out_logits [n][B][vocab] (may be NULL), out_argmax [n][B] = the model's own choice.   */
int oracle_decode_forced(oracle_ctx *c, const int32_t *forced, int32_t n, double *out_logits,
                         int32_t *out_argmax);
/* Layers [l0, l1) on hidden [B][R][hidden] (in place), rows at positions pos0..pos0+R-1,
 * reading and writing the context's KV cache.                                           */
int oracle_step_layers(oracle_ctx *c, int32_t l0, int32_t l1, double *hidden, int32_t B,
                       int32_t R, int32_t pos0);
int oracle_get_state(const oracle_ctx *c, oracle_state *s);
/* Copies up to max_records pass records; returns the number of passes run so far.       */
int oracle_get_trace(const oracle_ctx *c, oracle_pass_record *rec, int32_t max_records);
/* calls[l] = times layer l ran, rows[l] = rows (per sequence) it processed, since create
 * or reset.                                                                              */
int oracle_get_layer_counters(const oracle_ctx *c, int64_t *calls, int64_t *rows);
/* Direct access to the cache for tests: K and V of (layer, sequence b) as [max_seq][nkv][d]. */
double *oracle_k_cache(oracle_ctx *c, int32_t layer, int32_t b);
double *oracle_v_cache(oracle_ctx *c, int32_t layer, int32_t b);

/* ---- independent formulations used as pins ------------------------------------------ */
/* Plain autoregressive decoding: every step recomputes the whole sequence through all
 * layers with no cache reuse between steps.  tokens [P+n_new] holds the prompt on entry
 * and the full sequence on exit; if forced != NULL the appended tokens are forced[i].
 * out_logits [n_new][vocab] (may be NULL); out_argmax [n_new] (may be NULL).            */
int oracle_vanilla_generate(const oracle_shape *shape, const oracle_weights *w, int32_t *tokens,
                            int32_t P, int32_t n_new, const int32_t *forced,
                            double *out_logits, int32_t *out_argmax);
/* One masked parallel forward (Eq. 1-5) over tokens[0..n): lower stack causal over all
 * positions; upper-stack input at position p is the lower-stack output if p < P or
 * (p-(P-1)) mod tau == 0, else the token embedding; out_logits [n-(P-1)][vocab] are the
 * logits at positions P-1 .. n-1.                                                        */
int oracle_anchor_mask(int32_t p, int32_t P, int32_t tau);   /* the mask m_p of Eq. 3 */
int oracle_masked_parallel_forward(const oracle_shape *shape, const oracle_weights *w,
                                   int32_t L_d, int32_t tau, const int32_t *tokens, int32_t n,
                                   int32_t P, int32_t literal_sum, double *out_logits);

/* The same with L_e encoding layers reused (ExDy): h_enc = EncodingLayers(h_emb) is computed for
 * every position, h_think = ThinkingLayers(h_enc), and the decoding layers read h_think at mask
 * positions (h_enc + h_think with literal_sum) and h_enc elsewhere.                         */
int oracle_masked_parallel_forward_exdy(const oracle_shape *shape, const oracle_weights *w,
                                        int32_t L_e, int32_t L_d, int32_t tau,
                                        const int32_t *tokens, int32_t n, int32_t P,
                                        int32_t literal_sum, double *out_logits);

#ifdef __cplusplus
}
#endif
#endif
